// Plain SIMT kernels for HMAR's Markovian masked attention: the fp32 debug build, and the bf16
// fall-back used while debugging the tensor-core kernels.  All arithmetic is fp32 FMA; inputs and
// outputs are float or bf16.  Two threads share one row, each owning half of the head dimensions.  These
// kernels are templated on the head dimension (32, 64, 128); the tensor-core kernels exist for 64 only.
//
// Mask (paper Sec. 4.1, Fig. attn-mask): a query of scale k sees keys [start[k-1], start[k+1]).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "hmar_common.h"
#include "launchers.h"

namespace hmar {
namespace {

constexpr int ROWS = 64;           // rows per block (128 threads)
constexpr int KT = 32;             // partner rows staged in shared memory per step

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f(float* p, float x) { *p = x; }
__device__ __forceinline__ void from_f(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Key/value rows of one head may come in two segments (previous scale, then current scale) for the
// inference step; the training kernels use a single segment.
template <typename T, int D>
struct KvView {
    const T* k0; const T* v0; int n0;
    const T* k1; const T* v1;
    __device__ __forceinline__ const T* krow(int j) const {
        return j < n0 ? k0 + (size_t)j * D : k1 + (size_t)(j - n0) * D;
    }
    __device__ __forceinline__ const T* vrow(int j) const {
        return j < n0 ? v0 + (size_t)j * D : v1 + (size_t)(j - n0) * D;
    }
};

template <typename T, int D>
__device__ __forceinline__ void stage_rows(float (*dst)[D], const T* src_base, int first, int count) {
    // dst[r][:] = row (first + r) for r < count; 128 threads, coalesced along D
    for (int idx = threadIdx.x; idx < count * D; idx += blockDim.x) {
        int r = idx / D, d = idx % D;
        dst[r][d] = to_f(src_base[(size_t)(first + r) * D + d]);
    }
}

// ---------------------------------------------------------------------------------------------
// Forward and inference step.  dense != 0: every query row sees all n_kv keys (inference step).
template <typename T, int D>
__global__ void __launch_bounds__(128)
simt_fwd_kernel(const T* __restrict__ q, const T* __restrict__ k0, const T* __restrict__ v0,
                const T* __restrict__ k1, const T* __restrict__ v1,
                T* __restrict__ out, float* __restrict__ lse,
                ScaleTable st, int n_q, int n0, int n1, int dense, float scale) {
    constexpr int DH = D / 2;          // dimensions per thread
    __shared__ float sK[KT][D];
    __shared__ float sV[KT][D];
    const int bh = blockIdx.y;
    const int row0 = blockIdx.x * ROWS;
    const int half = threadIdx.x & 1;
    const int row_raw = row0 + (threadIdx.x >> 1);
    const bool row_ok = row_raw < n_q;
    const int row = row_ok ? row_raw : n_q - 1;
    const int last_row = min(row0 + ROWS, n_q) - 1;

    KvView<T, D> kv{k0 + (size_t)bh * n0 * D, v0 + (size_t)bh * n0 * D, n0,
                 k1 ? k1 + (size_t)bh * n1 * D : nullptr, v1 ? v1 + (size_t)bh * n1 * D : nullptr};

    int lo, hi, blk_lo, blk_hi;
    if (dense) {
        lo = blk_lo = 0;
        hi = blk_hi = n0 + n1;
    } else {
        int s = scale_of_row(st, row);
        lo = st.start[first_key_scale(st.window, s)];
        hi = st.start[last_key_scale(st.window, s) + 1];
        int sf = scale_of_row(st, row0), sl = scale_of_row(st, last_row);
        blk_lo = st.start[first_key_scale(st.window, sf)];
        blk_hi = st.start[last_key_scale(st.window, sl) + 1];
    }

    float qr[DH], o[DH];
    const T* qp = q + ((size_t)bh * n_q + row) * D + half * DH;
#pragma unroll
    for (int d = 0; d < DH; ++d) { qr[d] = to_f(qp[d]); o[d] = 0.f; }
    float m = -INFINITY, l = 0.f;

    for (int t = blk_lo; t < blk_hi; t += KT) {
        const int cnt = min(KT, blk_hi - t);
        __syncthreads();
        for (int idx = threadIdx.x; idx < cnt * D; idx += blockDim.x) {
            int r = idx / D, d = idx % D;
            sK[r][d] = to_f(kv.krow(t + r)[d]);
            sV[r][d] = to_f(kv.vrow(t + r)[d]);
        }
        __syncthreads();
        for (int r = 0; r < cnt; ++r) {
            float s = 0.f;
#pragma unroll
            for (int d = 0; d < DH; ++d) s = fmaf(qr[d], sK[r][half * DH + d], s);
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s *= scale;
            const int j = t + r;
            if (j >= lo && j < hi) {
                float m_new = fmaxf(m, s);
                float corr = expf(m - m_new);      // exp(-inf) = 0 on the first key
                float p = expf(s - m_new);
                l = l * corr + p;
#pragma unroll
                for (int d = 0; d < DH; ++d) o[d] = fmaf(o[d], corr, p * sV[r][half * DH + d]);
                m = m_new;
            }
        }
    }
    if (row_ok) {
        const float inv = 1.f / l;
        T* op = out + ((size_t)bh * n_q + row) * D + half * DH;
#pragma unroll
        for (int d = 0; d < DH; ++d) from_f(op + d, o[d] * inv);
        if (lse != nullptr && half == 0) lse[(size_t)bh * n_q + row] = m + logf(l);
    }
}

// ---------------------------------------------------------------------------------------------
// delta_i = sum_d dO_id * O_id
template <typename T, int D>
__global__ void __launch_bounds__(128)
simt_delta_kernel(const T* __restrict__ out, const T* __restrict__ dout, float* __restrict__ delta,
                  size_t n_rows) {
    constexpr int DH = D / 2;          // dimensions per thread
    const size_t row = (size_t)blockIdx.x * ROWS + (threadIdx.x >> 1);
    const int half = threadIdx.x & 1;
    float acc = 0.f;
    if (row < n_rows) {
        const T* a = out + row * D + half * DH;
        const T* b = dout + row * D + half * DH;
#pragma unroll
        for (int d = 0; d < DH; ++d) acc = fmaf(to_f(a[d]), to_f(b[d]), acc);
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    if (row < n_rows && half == 0) delta[row] = acc;
}

// ---------------------------------------------------------------------------------------------
// dQ: one thread pair per query row, loop over the row's keys.
template <typename T, int D>
__global__ void __launch_bounds__(128)
simt_dq_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
               const T* __restrict__ dout, const float* __restrict__ lse,
               const float* __restrict__ delta, T* __restrict__ dq,
               ScaleTable st, int L, float scale) {
    constexpr int DH = D / 2;          // dimensions per thread
    __shared__ float sK[KT][D];
    __shared__ float sV[KT][D];
    const int bh = blockIdx.y;
    const int row0 = blockIdx.x * ROWS;
    const int half = threadIdx.x & 1;
    const int row_raw = row0 + (threadIdx.x >> 1);
    const bool row_ok = row_raw < L;
    const int row = row_ok ? row_raw : L - 1;
    const int last_row = min(row0 + ROWS, L) - 1;
    const int s_row = scale_of_row(st, row);
    const int lo = st.start[first_key_scale(st.window, s_row)], hi = st.start[last_key_scale(st.window, s_row) + 1];
    const int sf = scale_of_row(st, row0), sl = scale_of_row(st, last_row);
    const int blk_lo = st.start[first_key_scale(st.window, sf)], blk_hi = st.start[last_key_scale(st.window, sl) + 1];
    const size_t head = (size_t)bh * L;

    float qr[DH], gr[DH], acc[DH];
#pragma unroll
    for (int d = 0; d < DH; ++d) {
        qr[d] = to_f(q[(head + row) * D + half * DH + d]);
        gr[d] = to_f(dout[(head + row) * D + half * DH + d]);
        acc[d] = 0.f;
    }
    const float lse_i = lse[head + row], delta_i = delta[head + row];

    for (int t = blk_lo; t < blk_hi; t += KT) {
        const int cnt = min(KT, blk_hi - t);
        __syncthreads();
        stage_rows(sK, k + head * D, t, cnt);
        stage_rows(sV, v + head * D, t, cnt);
        __syncthreads();
        for (int r = 0; r < cnt; ++r) {
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int d = 0; d < DH; ++d) {
                s = fmaf(qr[d], sK[r][half * DH + d], s);
                dp = fmaf(gr[d], sV[r][half * DH + d], dp);
            }
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            dp += __shfl_xor_sync(0xffffffffu, dp, 1);
            const int j = t + r;
            if (j >= lo && j < hi) {
                float p = expf(s * scale - lse_i);
                float ds = p * (dp - delta_i);
#pragma unroll
                for (int d = 0; d < DH; ++d) acc[d] = fmaf(ds, sK[r][half * DH + d], acc[d]);
            }
        }
    }
    if (row_ok) {
        T* op = dq + (head + row) * D + half * DH;
#pragma unroll
        for (int d = 0; d < DH; ++d) from_f(op + d, acc[d] * scale);
    }
}

// ---------------------------------------------------------------------------------------------
// dK, dV: one thread pair per key row, loop over the queries that see it.
template <typename T, int D>
__global__ void __launch_bounds__(128)
simt_dkdv_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                 const T* __restrict__ dout, const float* __restrict__ lse,
                 const float* __restrict__ delta, T* __restrict__ dk, T* __restrict__ dv,
                 ScaleTable st, int L, float scale) {
    constexpr int DH = D / 2;          // dimensions per thread
    __shared__ float sQ[KT][D];
    __shared__ float sG[KT][D];
    __shared__ float sLse[KT];
    __shared__ float sDelta[KT];
    const int bh = blockIdx.y;
    const int row0 = blockIdx.x * ROWS;
    const int half = threadIdx.x & 1;
    const int row_raw = row0 + (threadIdx.x >> 1);
    const bool row_ok = row_raw < L;
    const int row = row_ok ? row_raw : L - 1;
    const int last_row = min(row0 + ROWS, L) - 1;
    const int K = st.n_scales;
    const int s_row = scale_of_row(st, row);
    // (under HMAR_WINDOW_PREV the keys of the last scale have no queries: lo = hi = L, and dK = dV = 0 is stored)
    const int lo = st.start[first_query_scale(st.window, s_row)], hi = max(lo, st.start[last_query_scale(st.window, s_row, K) + 1]);
    const int blk_lo = st.start[first_query_scale(st.window, scale_of_row(st, row0))];
    const int blk_hi = max(blk_lo, st.start[last_query_scale(st.window, scale_of_row(st, last_row), K) + 1]);
    const size_t head = (size_t)bh * L;

    float kr[DH], vr[DH], ak[DH], av[DH];
#pragma unroll
    for (int d = 0; d < DH; ++d) {
        kr[d] = to_f(k[(head + row) * D + half * DH + d]);
        vr[d] = to_f(v[(head + row) * D + half * DH + d]);
        ak[d] = 0.f;
        av[d] = 0.f;
    }

    for (int t = blk_lo; t < blk_hi; t += KT) {
        const int cnt = min(KT, blk_hi - t);
        __syncthreads();
        stage_rows(sQ, q + head * D, t, cnt);
        stage_rows(sG, dout + head * D, t, cnt);
        if (threadIdx.x < cnt) {
            sLse[threadIdx.x] = lse[head + t + threadIdx.x];
            sDelta[threadIdx.x] = delta[head + t + threadIdx.x];
        }
        __syncthreads();
        for (int r = 0; r < cnt; ++r) {
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int d = 0; d < DH; ++d) {
                s = fmaf(kr[d], sQ[r][half * DH + d], s);
                dp = fmaf(vr[d], sG[r][half * DH + d], dp);
            }
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            dp += __shfl_xor_sync(0xffffffffu, dp, 1);
            const int i = t + r;
            if (i >= lo && i < hi) {
                float p = expf(s * scale - sLse[r]);
                float ds = p * (dp - sDelta[r]);
#pragma unroll
                for (int d = 0; d < DH; ++d) {
                    av[d] = fmaf(p, sG[r][half * DH + d], av[d]);
                    ak[d] = fmaf(ds, sQ[r][half * DH + d], ak[d]);
                }
            }
        }
    }
    if (row_ok) {
        T* pk = dk + (head + row) * D + half * DH;
        T* pv = dv + (head + row) * D + half * DH;
#pragma unroll
        for (int d = 0; d < DH; ++d) {
            from_f(pk + d, ak[d] * scale);
            from_f(pv + d, av[d]);
        }
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// Launchers

template <typename T, int D>
static cudaError_t simt_fwd_d(const T* q, const T* k, const T* v, T* out, float* lse, int BH,
                              const ScaleTable& st, float scale, cudaStream_t stream) {
    const int L = st.start[st.n_scales];
    dim3 grid((L + ROWS - 1) / ROWS, BH);
    simt_fwd_kernel<T, D><<<grid, 128, 0, stream>>>(q, k, v, nullptr, nullptr, out, lse, st, L, L, 0, 0, scale);
    count_launch(1);
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t simt_scale_step_d(const T* q, const T* k_prev, const T* v_prev, const T* k_cur, const T* v_cur,
                                     T* out, float* lse, int BH, int n_prev, int n_cur, float scale,
                                     cudaStream_t stream) {
    ScaleTable st{};
    dim3 grid((n_cur + ROWS - 1) / ROWS, BH);
    if (n_prev > 0)
        simt_fwd_kernel<T, D><<<grid, 128, 0, stream>>>(q, k_prev, v_prev, k_cur, v_cur, out, lse, st,
                                                     n_cur, n_prev, n_cur, 1, scale);
    else
        simt_fwd_kernel<T, D><<<grid, 128, 0, stream>>>(q, k_cur, v_cur, nullptr, nullptr, out, lse, st,
                                                     n_cur, n_cur, 0, 1, scale);
    count_launch(1);
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t simt_bwd_d(const T* q, const T* k, const T* v, const T* out, const float* lse, const T* dout,
                              T* dq, T* dk, T* dv, float* delta, int BH, const ScaleTable& st, float scale,
                              cudaStream_t stream) {
    const int L = st.start[st.n_scales];
    const size_t n_rows = (size_t)BH * L;
    simt_delta_kernel<T, D><<<(unsigned)((n_rows + ROWS - 1) / ROWS), 128, 0, stream>>>(out, dout, delta, n_rows);
    dim3 grid((L + ROWS - 1) / ROWS, BH);
    simt_dq_kernel<T, D><<<grid, 128, 0, stream>>>(q, k, v, dout, lse, delta, dq, st, L, scale);
    simt_dkdv_kernel<T, D><<<grid, 128, 0, stream>>>(q, k, v, dout, lse, delta, dk, dv, st, L, scale);
    count_launch(3);
    return cudaGetLastError();
}

// The public launchers pick the instantiation for the head dimension (32, 64 or 128; checked by the caller).
#define HMAR_BY_D(call32, call64, call128) (D == 32 ? (call32) : (D == 128 ? (call128) : (call64)))

template <typename T>
cudaError_t simt_fwd(const T* q, const T* k, const T* v, T* out, float* lse, int BH, int D,
                     const ScaleTable& st, float scale, cudaStream_t stream) {
    return HMAR_BY_D((simt_fwd_d<T, 32>(q, k, v, out, lse, BH, st, scale, stream)), (simt_fwd_d<T, 64>(q, k, v, out, lse, BH, st, scale, stream)),
                     (simt_fwd_d<T, 128>(q, k, v, out, lse, BH, st, scale, stream)));
}

template <typename T>
cudaError_t simt_scale_step(const T* q, const T* k_prev, const T* v_prev, const T* k_cur, const T* v_cur,
                            T* out, float* lse, int BH, int D, int n_prev, int n_cur, float scale,
                            cudaStream_t stream) {
    return HMAR_BY_D((simt_scale_step_d<T, 32>(q, k_prev, v_prev, k_cur, v_cur, out, lse, BH, n_prev, n_cur, scale, stream)),
                     (simt_scale_step_d<T, 64>(q, k_prev, v_prev, k_cur, v_cur, out, lse, BH, n_prev, n_cur, scale, stream)),
                     (simt_scale_step_d<T, 128>(q, k_prev, v_prev, k_cur, v_cur, out, lse, BH, n_prev, n_cur, scale, stream)));
}

template <typename T>
cudaError_t simt_bwd(const T* q, const T* k, const T* v, const T* out, const float* lse, const T* dout,
                     T* dq, T* dk, T* dv, float* delta, int BH, int D, const ScaleTable& st, float scale,
                     cudaStream_t stream) {
    return HMAR_BY_D((simt_bwd_d<T, 32>(q, k, v, out, lse, dout, dq, dk, dv, delta, BH, st, scale, stream)),
                     (simt_bwd_d<T, 64>(q, k, v, out, lse, dout, dq, dk, dv, delta, BH, st, scale, stream)),
                     (simt_bwd_d<T, 128>(q, k, v, out, lse, dout, dq, dk, dv, delta, BH, st, scale, stream)));
}

#define INSTANTIATE(T)                                                                                        \
    template cudaError_t simt_fwd<T>(const T*, const T*, const T*, T*, float*, int, int, const ScaleTable&,   \
                                     float, cudaStream_t);                                                    \
    template cudaError_t simt_scale_step<T>(const T*, const T*, const T*, const T*, const T*, T*, float*,     \
                                            int, int, int, int, float, cudaStream_t);                         \
    template cudaError_t simt_bwd<T>(const T*, const T*, const T*, const T*, const float*, const T*, T*,      \
                                     T*, T*, float*, int, int, const ScaleTable&, float, cudaStream_t);
INSTANTIATE(float)
INSTANTIATE(__nv_bfloat16)

}  // namespace hmar
