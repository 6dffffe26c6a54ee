// Inference step for the small scales (paper Sec. 4.2: every scale is refined over several masked
// sub-steps, so the coarse scales run many times; Sec. 4.1: the step sees the previous scale and its own).
//
// A scale step with at most kSmallMaxKeys keys in its window (previous scale + current scale) is far too
// small for the 128 x 128 tcgen05 tiles of the main kernel: one query row at scale 1, 81 at scale 6 of
// the 512 x 512 schedule.  Here one block takes one head: the head's K and V rows (previous scale, then
// current scale) are copied once into shared memory with plain 16-byte loads, and every warp owns 32
// query rows: S = Q K^T and O = P V with warp-level m16n8k16 bf16 products (fp32 accumulation), the
// softmax on the accumulator fragments in registers (online over chunks of 64 keys), P rounded to bf16
// before the second product as in the large kernels.  No TMEM, no tensor maps, no barriers besides one
// __syncthreads, so a launch costs little more than its latency; the arithmetic per head is below a
// microsecond and the kernel is bound by reading K, V, Q and writing O once (HBM) or by launch latency.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "hmar_common.h"
#include "launchers.h"
#include "tc_launchers.h"

namespace hmar {
namespace {

constexpr int D = kHeadDim;
constexpr int ROW_BYTES = D * 2 + 16;     // 144: rows 36 words apart, so fragment loads and ldmatrix hit 32 distinct banks
constexpr int CHUNK = 64;                 // keys per softmax chunk

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t smem_addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr));
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

struct StepArgs {
    const __nv_bfloat16 *q, *k_prev, *v_prev, *k_cur, *v_cur;
    __nv_bfloat16* out;
    float* lse;                 // [BH, n_cur] or nullptr
    long long q_head_stride, kv_prev_head_stride, kv_cur_head_stride, out_head_stride;    // elements
    int n_prev, n_cur;
    float scale_log2;
    int n_heads;
    int* status;                // device status word (checking build), may be nullptr
};

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gptr) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}

// One block per head, 32 query rows (two m16 row groups) per warp: every K and V fragment read from shared
// memory feeds two products, which keeps the shared-memory traffic (64 KB per 32 rows at 256 keys) below the
// time the head's rows take to arrive from HBM.
__global__ void __launch_bounds__(kSmallMaxQueries, 4)
hmar_step_small_kernel(const StepArgs a) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int bh = blockIdx.x;
    if (!HMAR_IN_BOUNDS(bh < a.n_heads && a.n_cur <= kSmallMaxQueries && a.n_prev + a.n_cur <= kSmallMaxKeys, a.status, 0xB301)) return;
    const int n_keys = a.n_prev + a.n_cur;
    const int keys_pad = (n_keys + 15) & ~15;
    uint8_t* sk = smem;
    uint8_t* sv = smem + (size_t)keys_pad * ROW_BYTES;
    const uint32_t sk_addr = static_cast<uint32_t>(__cvta_generic_to_shared(sk));
    const uint32_t sv_addr = static_cast<uint32_t>(__cvta_generic_to_shared(sv));

    // ---- K and V rows of the head into shared memory: asynchronous 16-byte copies, all in flight at once;
    // the rows between the end of the window and the next multiple of 16 are zeros
    {
        const __nv_bfloat16* kp = a.k_prev + bh * a.kv_prev_head_stride;
        const __nv_bfloat16* vp = a.v_prev + bh * a.kv_prev_head_stride;
        const __nv_bfloat16* kc = a.k_cur + bh * a.kv_cur_head_stride;
        const __nv_bfloat16* vc = a.v_cur + bh * a.kv_cur_head_stride;
        for (int idx = threadIdx.x; idx < keys_pad * 8; idx += blockDim.x) {
            const int row = idx >> 3, part = idx & 7;
            const uint32_t off = row * ROW_BYTES + part * 16;
            if (row < a.n_prev) {
                cp_async16(sk_addr + off, kp + (size_t)row * D + part * 8);
                cp_async16(sv_addr + off, vp + (size_t)row * D + part * 8);
            } else if (row < n_keys) {
                cp_async16(sk_addr + off, kc + (size_t)(row - a.n_prev) * D + part * 8);
                cp_async16(sv_addr + off, vc + (size_t)(row - a.n_prev) * D + part * 8);
            } else {
                *reinterpret_cast<uint4*>(sk + off) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(sv + off) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    // ---- this warp's 32 query rows as A fragments (two row groups, 4 steps of 16 head dimensions each)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    uint32_t qa[2][4][4];
    {
        const __nv_bfloat16* qh = a.q + bh * a.q_head_stride;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row0 = warp * 32 + r * 16 + g, row1 = row0 + 8;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int c = ks * 16 + t * 2;
                qa[r][ks][0] = row0 < a.n_cur ? __ldg(reinterpret_cast<const uint32_t*>(qh + (size_t)row0 * D + c)) : 0u;
                qa[r][ks][1] = row1 < a.n_cur ? __ldg(reinterpret_cast<const uint32_t*>(qh + (size_t)row1 * D + c)) : 0u;
                qa[r][ks][2] = row0 < a.n_cur ? __ldg(reinterpret_cast<const uint32_t*>(qh + (size_t)row0 * D + c + 8)) : 0u;
                qa[r][ks][3] = row1 < a.n_cur ? __ldg(reinterpret_cast<const uint32_t*>(qh + (size_t)row1 * D + c + 8)) : 0u;
            }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const bool second = warp * 32 + 16 < a.n_cur;      // the warp's second row group holds rows of the head

    float o[2][8][4];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int d = 0; d < 8; ++d) o[r][d][0] = o[r][d][1] = o[r][d][2] = o[r][d][3] = 0.f;
    // running maximum (log2 units) and row sum of this thread's four rows: [row group][row g / row g + 8]
    float m[2][2] = {{-INFINITY, -INFINITY}, {-INFINITY, -INFINITY}}, l[2][2] = {{0.f, 0.f}, {0.f, 0.f}};

    for (int c0 = 0; c0 < keys_pad; c0 += CHUNK) {
        const int n_tiles = min(CHUNK, keys_pad - c0) >> 3;        // 8-key tiles in this chunk (even)
        float s[2][CHUNK / 8][4];
        // S = Q K^T: fragment (g, t) of tile j holds keys c0 + 8 j + 2 t + {0, 1} for rows g (s[..][0..1]) and g + 8 (s[..][2..3])
#pragma unroll
        for (int j = 0; j < CHUNK / 8; ++j) {
#pragma unroll
            for (int r = 0; r < 2; ++r) s[r][j][0] = s[r][j][1] = s[r][j][2] = s[r][j][3] = 0.f;
            if (j < n_tiles) {
                const uint8_t* krow = sk + (c0 + j * 8 + g) * ROW_BYTES + t * 4;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint32_t b0 = *reinterpret_cast<const uint32_t*>(krow + ks * 32);
                    const uint32_t b1 = *reinterpret_cast<const uint32_t*>(krow + ks * 32 + 16);
                    mma_bf16_16816(s[0][j], qa[0][ks], b0, b1);
                    if (second) mma_bf16_16816(s[1][j], qa[1][ks], b0, b1);
                }
            }
        }
        // scaled logits in log2 units (keys past the end of the window masked), chunk maxima, rescale of the running state
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int j = 0; j < CHUNK / 8; ++j) {
                if (j < n_tiles) {
                    const int key = c0 + j * 8 + t * 2;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float x = (key + (e & 1) < n_keys) ? s[r][j][e] * a.scale_log2 : -INFINITY;
                        s[r][j][e] = x;
                        if (e < 2) mx0 = fmaxf(mx0, x); else mx1 = fmaxf(mx1, x);
                    }
                }
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m[r][0], mx0), mn1 = fmaxf(m[r][1], mx1);   // finite: every chunk holds at least one real key
            const float f0 = ex2f(m[r][0] - mn0), f1 = ex2f(m[r][1] - mn1);     // 0 for the first chunk (m = -inf)
            m[r][0] = mn0; m[r][1] = mn1;
            l[r][0] *= f0; l[r][1] *= f1;
#pragma unroll
            for (int d = 0; d < 8; ++d) { o[r][d][0] *= f0; o[r][d][1] *= f0; o[r][d][2] *= f1; o[r][d][3] *= f1; }
        }
        // P = 2^(s - m), O += P V, sixteen keys at a time
#pragma unroll
        for (int kk = 0; kk < CHUNK / 16; ++kk) {
            if (2 * kk < n_tiles) {
                uint32_t pa[2][4];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    float p[8];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        p[e] = ex2f(s[r][2 * kk][e] - m[r][e >> 1]);
                        p[4 + e] = ex2f(s[r][2 * kk + 1][e] - m[r][e >> 1]);
                    }
                    l[r][0] += p[0] + p[1] + p[4] + p[5];
                    l[r][1] += p[2] + p[3] + p[6] + p[7];
                    pa[r][0] = pack2(p[0], p[1]); pa[r][1] = pack2(p[2], p[3]);
                    pa[r][2] = pack2(p[4], p[5]); pa[r][3] = pack2(p[6], p[7]);
                }
                // V fragments: ldmatrix.trans of a 16 keys x 16 dimensions block gives the (k, n) fragments of two dimension tiles
                const uint32_t vbase = sv_addr + (c0 + kk * 16 + (lane & 15)) * ROW_BYTES + (lane >> 4) * 16;
#pragma unroll
                for (int dp = 0; dp < 4; ++dp) {
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, vbase + dp * 32);
                    mma_bf16_16816(o[0][2 * dp], pa[0], vb[0], vb[1]);
                    mma_bf16_16816(o[0][2 * dp + 1], pa[0], vb[2], vb[3]);
                    if (second) {
                        mma_bf16_16816(o[1][2 * dp], pa[1], vb[0], vb[1]);
                        mma_bf16_16816(o[1][2 * dp + 1], pa[1], vb[2], vb[3]);
                    }
                }
            }
        }
    }
    __nv_bfloat16* oh = a.out + bh * a.out_head_stride;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row0 = warp * 32 + r * 16 + g, row1 = row0 + 8;
        // row sums over the four lanes that share a row
        float l0 = l[r][0], l1 = l[r][1];
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        const float inv0 = 1.f / l0, inv1 = 1.f / l1;
#pragma unroll
        for (int d = 0; d < 8; ++d) {
            const int c = d * 8 + t * 2;
            if (row0 < a.n_cur && HMAR_IN_BOUNDS(c + 2 <= D, a.status, 0xB302)) *reinterpret_cast<uint32_t*>(oh + (size_t)row0 * D + c) = pack2(o[r][d][0] * inv0, o[r][d][1] * inv0);
            if (row1 < a.n_cur) *reinterpret_cast<uint32_t*>(oh + (size_t)row1 * D + c) = pack2(o[r][d][2] * inv1, o[r][d][3] * inv1);
        }
        if (a.lse != nullptr && t == 0) {
            if (row0 < a.n_cur) a.lse[(size_t)bh * a.n_cur + row0] = (m[r][0] + log2f(l0)) * 0.6931471805599453f;
            if (row1 < a.n_cur) a.lse[(size_t)bh * a.n_cur + row1] = (m[r][1] + log2f(l1)) * 0.6931471805599453f;
        }
    }
}

}  // namespace

bool step_small_applies(int n_prev, int n_cur) { return n_prev + n_cur <= kSmallMaxKeys && n_cur <= kSmallMaxQueries; }

int step_small(const __nv_bfloat16* q, const __nv_bfloat16* k_prev, const __nv_bfloat16* v_prev,
               const __nv_bfloat16* k_cur, const __nv_bfloat16* v_cur, __nv_bfloat16* out, float* lse, int BH, int n_prev,
               int n_cur, long long q_head_stride, long long kv_prev_head_stride, long long kv_cur_head_stride,
               long long out_head_stride, float scale, int* status, cudaStream_t stream) {
    StepArgs a;
    a.q = q; a.k_prev = k_prev; a.v_prev = v_prev; a.k_cur = k_cur; a.v_cur = v_cur;
    a.out = out; a.lse = lse;
    a.q_head_stride = q_head_stride; a.kv_prev_head_stride = kv_prev_head_stride;
    a.kv_cur_head_stride = kv_cur_head_stride; a.out_head_stride = out_head_stride;
    a.n_prev = n_prev; a.n_cur = n_cur;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.n_heads = BH;
    a.status = status;
    const int warps = (n_cur + 31) / 32;
    const int keys_pad = (n_prev + n_cur + 15) & ~15;
    const size_t smem = (size_t)2 * keys_pad * ROW_BYTES;
    // the largest window needs more than the default 48 KB of dynamic shared memory (per function and device; cheap to repeat)
    if (cudaFuncSetAttribute(hmar_step_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             2 * kSmallMaxKeys * ROW_BYTES) != cudaSuccess)
        return HMAR_ERR_CUDA;
    {
        KernelTimer timer("hmar_step_small_kernel", stream);
        hmar_step_small_kernel<<<BH, warps * 32, smem, stream>>>(a);
    }
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

}  // namespace hmar
