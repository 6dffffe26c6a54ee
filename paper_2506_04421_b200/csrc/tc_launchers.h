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
// Share (thousandths) of a head's backward steps that lie in full tiles; picks the main kernel's instantiation.  Host only.
int tc_bwd_full_tile_permille(const ScaleTable& st);
int tc_bwd_packed(const __nv_bfloat16* qkv, const __nv_bfloat16* out, const float* lse, const __nv_bfloat16* dout,
                  __nv_bfloat16* dqkv, float* delta, float* dq_acc, int B, int H, const ScaleTable& st, float scale,
                  int* status, cudaStream_t stream);
// Inference step.  Rows are 64 contiguous elements; consecutive heads of a tensor are `*_head_stride` elements apart
// (n_rows * 64 for a dense [B,H,n,64] tensor, the ring's rows * 64 when prev and cur sit in one K/V ring buffer).
struct StepStrides {
    long long q, kv_prev, kv_cur, out;
};
int tc_scale_step(const __nv_bfloat16* q, const __nv_bfloat16* k_prev, const __nv_bfloat16* v_prev,
                  const __nv_bfloat16* k_cur, const __nv_bfloat16* v_cur, __nv_bfloat16* out, float* lse,
                  int BH, int n_prev, int n_cur, const StepStrides& strides, float scale, int* status, cudaStream_t stream);
// Small windows (at most kSmallMaxKeys keys, kSmallMaxQueries queries): one block per head, warp-level products.
// Measured on B200 at 1536 heads: the warp-level products run at about 130 TFLOP/s, so the small kernel is 2x
// faster than the 128-row tcgen05 tiles up to 52 keys (launch latency), level at 81 queries x 117 keys and
// 1.4x slower at 169 x 250, where the tensor-core kernel takes over.
constexpr int kSmallMaxKeys = 128;
constexpr int kSmallMaxQueries = 96;
bool step_small_applies(int n_prev, int n_cur);
int step_small(const __nv_bfloat16* q, const __nv_bfloat16* k_prev, const __nv_bfloat16* v_prev,
               const __nv_bfloat16* k_cur, const __nv_bfloat16* v_cur, __nv_bfloat16* out, float* lse, int BH, int n_prev,
               int n_cur, long long q_head_stride, long long kv_prev_head_stride, long long kv_cur_head_stride,
               long long out_head_stride, float scale, int* status, cudaStream_t stream);
void tc_release_plans();

}  // namespace hmar
