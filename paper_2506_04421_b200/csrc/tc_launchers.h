// Launchers of the tensor-core (tcgen05 / TMA) kernels for bf16 tensors (internal).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "hmar_common.h"

namespace hmar {

int tc_fwd(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, __nv_bfloat16* out,
           float* lse, int BH, const ScaleTable& st, float scale, int* status, cudaStream_t stream);
int tc_fwd_packed(const __nv_bfloat16* qkv, __nv_bfloat16* out, float* lse, int B, int H, const ScaleTable& st,
                  float scale, int* status, cudaStream_t stream);
int tc_bwd(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, const __nv_bfloat16* out,
           const float* lse, const __nv_bfloat16* dout, __nv_bfloat16* dq, __nv_bfloat16* dk,
           __nv_bfloat16* dv, float* delta, float* dq_acc, int BH, const ScaleTable& st, float scale,
           int* status, cudaStream_t stream);
int tc_scale_step(const __nv_bfloat16* q, const __nv_bfloat16* k_prev, const __nv_bfloat16* v_prev,
                  const __nv_bfloat16* k_cur, const __nv_bfloat16* v_cur, __nv_bfloat16* out, float* lse,
                  int BH, int n_prev, int n_cur, float scale, int* status, cudaStream_t stream);
void tc_release_plans();

}  // namespace hmar
