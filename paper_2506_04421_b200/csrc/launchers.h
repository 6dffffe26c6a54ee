// Internal launcher prototypes shared between the C-ABI layer and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include "hmar_common.h"

namespace hmar {

void count_launch(int n);

// Per-kernel timing (diagnostics): when profiling is on, a kernel launch wrapped in KernelTimer is
// bracketed by two events on its stream; hmar_profile_end() sums them per kernel name.
bool profile_enabled();
struct KernelTimer {
    KernelTimer(const char* name, cudaStream_t stream);
    ~KernelTimer();
    const char* name_;
    cudaStream_t stream_;
    cudaEvent_t begin_;
    bool on_;
};

template <typename T>
cudaError_t simt_fwd(const T* q, const T* k, const T* v, T* out, float* lse, int BH, int D,
                     const ScaleTable& st, float scale, cudaStream_t stream);
template <typename T>
cudaError_t simt_scale_step(const T* q, const T* k_prev, const T* v_prev, const T* k_cur, const T* v_cur,
                            T* out, float* lse, int BH, int D, int n_prev, int n_cur, float scale,
                            cudaStream_t stream);
template <typename T>
cudaError_t simt_bwd(const T* q, const T* k, const T* v, const T* out, const float* lse, const T* dout,
                     T* dq, T* dk, T* dv, float* delta, int BH, int D, const ScaleTable& st, float scale,
                     cudaStream_t stream);

cudaError_t launch_recon_accumulate(float* xhat, const float* codebook, const int* tokens_old, const int* tokens_new,
                                    const unsigned char* mask, int* tokens_out, int B, int C, int V, int side, int out_side,
                                    cudaStream_t stream);
cudaError_t launch_recon_downsample(const float* xhat, float* out, int B, int C, int in_side, int out_side,
                                    cudaStream_t stream);

}  // namespace hmar
