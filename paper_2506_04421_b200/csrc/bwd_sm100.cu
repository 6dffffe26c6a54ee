// Backward kernels of HMAR's Markovian block-sparse attention for sm_100a.
//
// The gradient of exact softmax attention is recomputed from the forward's lse (the paper benchmarks
// this pass in App. B.4; Sec. 4.1 builds the kernel on FlashAttention, whose backward this follows):
//   P = exp(scale * Q K^T - lse),  dV = P^T dO,  dP = dO V^T,  dS = P o (dP - delta),
//   dQ = scale * dS K,  dK = scale * dS^T Q,  delta_i = sum_d dO_id O_id.
//
// Main kernel: one block owns one tile of up to 128 key rows of one head and walks over the
// contiguous range of query rows that may see them under the mask (queries of the keys' own scale and
// of the next scale; paper Sec. 4.1, Fig. attn-mask), 128 queries at a time:
//   warp 8      TMA producer: K, V once; then Q_i, dO_i through a 3-stage ring
//   warp 10     loads lse_i, delta_i with plain loads (their row offsets are not 16-byte aligned) into
//               an 8-deep ring
//   warp 9      issues tcgen05.mma: S^T = K Q_i^T and dP^T = V dO_i^T into TMEM; after the compute
//               warps are done: dV += P^T dO_i (P^T read from TMEM), dK += dS^T Q_i and
//               dQ_i = dS K (dS read from shared memory, once as a K-major and once as an
//               MN-major operand)
//   warps 0-7   one key row per thread, two threads per row splitting the 128 query columns:
//               P^T and dS^T in fp32, P^T (bf16) back to TMEM over S^T, dS^T (bf16) to shared memory;
//               then they drain dQ_i from TMEM into the fp32 accumulator with vector atomics
// TMEM columns: S^T [0,128) (P^T of queries 0-63 over columns [0,32), of queries 64-127 over
// [64,96)), dP^T [128,256), dK [256,320), dV [320,384), dQ_i [384,448).
// dK and dV stay in TMEM for the whole block and are written once at the end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "hmar_common.h"
#include "launchers.h"
#include "ptx_sm100.cuh"
#include "tc_common.h"

namespace hmar {
namespace {

using namespace ptx;

constexpr int BKV = 128;             // key rows per block
constexpr int BQ = 128;              // query rows per step
constexpr int D = kHeadDim;
constexpr int NSTAGE = 3;
constexpr int AUX_STAGES = 8;        // ring of lse / delta rows, loaded this many steps ahead
constexpr int TILE_BYTES = 128 * D * 2;          // 16 KB
constexpr int NUM_COMPUTE_WARPS = 8;
constexpr int PRODUCER_WARP = 8, MMA_WARP = 9, AUX_WARP = 10;
constexpr int NUM_THREADS = 352;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_ST = 0, COL_DPT = 128, COL_DK = 256, COL_DV = 320, COL_DQ = 384;

struct __align__(1024) SharedStorage {
    uint8_t k[TILE_BYTES];
    uint8_t v[TILE_BYTES];
    uint8_t q[NSTAGE][TILE_BYTES];
    uint8_t dout[NSTAGE][TILE_BYTES];
    uint8_t ds[2][2][TILE_BYTES];           // dS^T, double buffered: [step parity][64-query half][key row][64 queries], 128B swizzle
    float lse2[AUX_STAGES][BQ];             // lse * log2(e); +inf for query rows outside the range
    float delta[AUX_STAGES][BQ];
    uint64_t kv_full;
    uint64_t qdo_full[NSTAGE], q_empty[NSTAGE], aux_full[AUX_STAGES], aux_empty[AUX_STAGES];
    uint64_t s_full[2], p_full[2], dq_full;   // [half of the step]
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void report_timeout(int* status, int where) {
    if (status != nullptr) {
        atomicCAS(status, 0, HMAR_ERR_DEVICE_TIMEOUT);
        atomicCAS(status + 1, 0, where);
    }
}

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c),
                 "f"(d)
                 : "memory");
}

#ifdef HMAR_STAMPS
// Developer build only: per-phase clock totals of compute warp 0 and of the MMA thread, summed over blocks.
__device__ unsigned long long g_bwd_stamps[16];
#define STAMP_DECL unsigned long long st_acc[16] = {0}; long long st_t = clock64();
#define STAMP(idx) { long long st_n = clock64(); st_acc[idx] += (unsigned long long)(st_n - st_t); st_t = st_n; }
#define STAMP_FLUSH(lo, hi) { for (int st_i = lo; st_i < hi; ++st_i) atomicAdd(&g_bwd_stamps[st_i], st_acc[st_i]); }
#else
#define STAMP_DECL
#define STAMP(idx) {}
#define STAMP_FLUSH(lo, hi) {}
#endif

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
hmar_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                   const BwdArgs args) {
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& sm = *reinterpret_cast<SharedStorage*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (args.status != nullptr && *reinterpret_cast<volatile int*>(args.status) != 0) return;

    const int bh = blockIdx.x / args.n_work;
    const BwdWork w = args.work[blockIdx.x % args.n_work];
    const int n_steps = (w.q_end - w.q_begin + BQ - 1) / BQ;
    const int L = args.L;

    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.kv_full, 1);
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(&sm.qdo_full[s], 1);
            mbar_init(&sm.q_empty[s], 1);
        }
        for (int s = 0; s < AUX_STAGES; ++s) {
            mbar_init(&sm.aux_full[s], 32);
            mbar_init(&sm.aux_empty[s], NUM_COMPUTE_WARPS * 32);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(&sm.s_full[h], 1);
            mbar_init(&sm.p_full[h], NUM_COMPUTE_WARPS * 32);
        }
        mbar_init(&sm.dq_full, 1);
        fence_mbar_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(&sm.tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;

    if (warp == PRODUCER_WARP) {
        // ================================================================== producer
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            prefetch_tensormap(&map_do);
            mbar_arrive_expect_tx(&sm.kv_full, 2 * TILE_BYTES);
            tma_load_3d(sm.k, &map_k, &sm.kv_full, 0, w.row_begin, bh);
            tma_load_3d(sm.v, &map_v, &sm.kv_full, 0, w.row_begin, bh);
        }
        bool ok = true;
        if (lane == 0) {
            for (int i = 0; i < n_steps; ++i) {
                const int slot = i % NSTAGE;
                const int q0 = w.q_begin + i * BQ;
                if (i >= NSTAGE) {
                    ok = mbar_wait(&sm.q_empty[slot], ((i / NSTAGE) & 1) ^ 1, abort_flag);
                    if (!ok) { report_timeout(args.status, 0x1100 + i); break; }
                }
                mbar_arrive_expect_tx(&sm.qdo_full[slot], 2 * TILE_BYTES);
                tma_load_3d(sm.q[slot], &map_q, &sm.qdo_full[slot], 0, q0, bh);
                tma_load_3d(sm.dout[slot], &map_do, &sm.qdo_full[slot], 0, q0, bh);
            }
        }
        if (!ok && lane == 0) {
            const uint64_t t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) { }
        }
    } else if (warp == AUX_WARP) {
        // ================================================================== lse / delta loader
        // lse and delta rows of step i go to ring slot i % AUX_STAGES, several steps ahead of their use
        // (plain loads: their row offsets are not 16-byte aligned, so TMA cannot fetch them).
        STAMP_DECL
        for (int i = 0; i < n_steps; ++i) {
            const int aslot = i % AUX_STAGES;
            STAMP(13)
            if (i >= AUX_STAGES) {
                const bool ok = __all_sync(0xffffffffu,
                                           mbar_wait(&sm.aux_empty[aslot], ((i / AUX_STAGES) & 1) ^ 1, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x1700 + i); break; }
            }
            STAMP(12)
            const int q0 = w.q_begin + i * BQ;
            // all loads first, then the stores: stores to shared memory in between would serialise them
            float lv[BQ / 32], dv[BQ / 32];
#pragma unroll
            for (int t = 0; t < BQ / 32; ++t) {
                const int row = q0 + t * 32 + lane;
                const bool in = row < w.q_end;
                lv[t] = in ? __ldg(args.lse + (size_t)bh * L + row) : INFINITY;
                dv[t] = in ? __ldg(args.delta + (size_t)bh * L + row) : 0.f;
            }
#pragma unroll
            for (int t = 0; t < BQ / 32; ++t) {
                sm.lse2[aslot][t * 32 + lane] = lv[t] * 1.4426950408889634f;
                sm.delta[aslot][t * 32 + lane] = dv[t];
            }
            mbar_arrive(&sm.aux_full[aslot]);
        }
        STAMP(13)
        if (lane == 0) STAMP_FLUSH(12, 14)
    } else if (warp == MMA_WARP) {
        // ================================================================== MMA issuer
        // A step of 128 queries is split into two halves of 64 (a: queries 0-63, b: 64-127), each with
        // its own S^T / dP^T columns and barriers, so that the compute warps work on one half while
        // the tensor core produces the scores of the other half or consumes the finished one.
        // The whole warp runs the control flow; one elected lane issues.  Descriptors are built once and
        // advanced by adding (byte offset >> 4) to them, so issuing an MMA costs a few instructions.
        {
            const bool leader = elect_one();
            STAMP_DECL
            bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.kv_full, 0, abort_flag));
            if (!ok && lane == 0) report_timeout(args.status, 0x1200);
            STAMP(8)
            const uint64_t k_kd = smem_desc_sw128(smem_u32(sm.k), 16);          // K rows, K-major (A of S^T)
            const uint64_t v_kd = smem_desc_sw128(smem_u32(sm.v), 16);          // V rows, K-major (A of dP^T)
            const uint64_t k_mn = smem_desc_sw128(smem_u32(sm.k), 1024);        // K as MN-major B of dQ
            // the ring slots and the dS buffers are 16 KB apart: descriptor of slot s = base + s * 1024
            const uint64_t q_kd0 = smem_desc_sw128(smem_u32(sm.q[0]), 16), do_kd0 = smem_desc_sw128(smem_u32(sm.dout[0]), 16);
            const uint64_t q_mn0 = smem_desc_sw128(smem_u32(sm.q[0]), 1024), do_mn0 = smem_desc_sw128(smem_u32(sm.dout[0]), 1024);
            const uint64_t ds_kd0 = smem_desc_sw128(smem_u32(sm.ds[0][0]), 16);
            const uint64_t ds_mn0 = smem_desc_sw128(smem_u32(sm.ds[0][0]), TILE_BYTES);
            constexpr uint32_t idesc_acc = idesc_bf16_f32(BKV, D, false, true);    // A K-major / TMEM, B MN-major
            constexpr uint32_t idesc_dq = idesc_bf16_f32(BQ, D, true, true);

            auto n_eff_half = [&](int i, int h) {
                const int n_valid = min(BQ, w.q_end - (w.q_begin + i * BQ));
                const int n_eff = (n_valid + 15) & ~15;
                return h == 0 ? min(n_eff, 64) : max(n_eff - 64, 0);
            };
            // S^T_h = K Q_h^T,  dP^T_h = V dO_h^T  for half h of step i
            auto issue_scores = [&](int i, int h) -> bool {
                const int slot = i % NSTAGE;
                const int n = n_eff_half(i, h);
                if (n == 0) return true;
                STAMP(11)
                if (!__all_sync(0xffffffffu, mbar_wait(&sm.qdo_full[slot], (i / NSTAGE) & 1, abort_flag))) {
                    if (lane == 0) report_timeout(args.status, 0x1300 + i);
                    return false;
                }
                STAMP(9)
                tc_fence_after();
                if (leader) {
                    const uint32_t idesc = idesc_bf16_f32(BKV, n, false, false);
                    const uint64_t qd = q_kd0 + slot * 1024 + h * 512, dd = do_kd0 + slot * 1024 + h * 512;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_ss(tmem + COL_ST + h * 64, k_kd + ks * 2, qd + ks * 2, idesc, ks > 0);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_ss(tmem + COL_DPT + h * 64, v_kd + ks * 2, dd + ks * 2, idesc, ks > 0);
                    tc_commit(&sm.s_full[h]);
                }
                __syncwarp();
                return true;
            };
            // dV += P_h^T dO_h,  dK += dS_h^T Q_h  for half h of step i
            auto issue_grads = [&](int i, int h) -> bool {
                const int slot = i % NSTAGE;
                const int n = n_eff_half(i, h);
                if (n == 0) return true;
                STAMP(11)
                if (!__all_sync(0xffffffffu, mbar_wait(&sm.p_full[h], i & 1, abort_flag))) {
                    if (lane == 0) report_timeout(args.status, 0x1400 + i);
                    return false;
                }
                STAMP(10)
                tc_fence_after();
                if (leader) {
                    const int nk = n / 16;
                    const uint64_t dod = do_mn0 + slot * 1024 + h * 512, qd = q_mn0 + slot * 1024 + h * 512;
                    const uint64_t dsd = ds_kd0 + ((i & 1) * 2 + h) * 1024;
                    const uint32_t p_base = tmem + COL_ST + h * 64;
                    const bool first = (i == 0) && (h == 0);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        if (ks < nk)
                            mma_ts(tmem + COL_DV, p_base + (ks / 2) * 32 + (ks % 2) * 8, dod + ks * 128, idesc_acc,
                                   !first || (ks > 0));
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        if (ks < nk)
                            mma_ss(tmem + COL_DK, dsd + ks * 2, qd + ks * 128, idesc_acc, !first || (ks > 0));
                }
                __syncwarp();
                return true;
            };

            if (ok) ok = issue_scores(0, 0);
            if (ok) ok = issue_scores(0, 1);
            for (int i = 0; i < n_steps && ok; ++i) {
                ok = issue_grads(i, 0);
                if (ok && i + 1 < n_steps) ok = issue_scores(i + 1, 0);
                if (ok) ok = issue_grads(i, 1);
                if (!ok) break;
                // dQ_i = dS K over both halves: A = dS (queries x keys) read as an MN-major operand.  When
                // the step has no second half its rows are stale data and are never drained.
                if (leader) {
                    const uint64_t dsd = ds_mn0 + (i & 1) * 2048;
#pragma unroll
                    for (int ks = 0; ks < BKV / 16; ++ks)
                        mma_ss(tmem + COL_DQ, dsd + ks * 128, k_mn + ks * 128, idesc_dq, ks > 0);
                    tc_commit(&sm.q_empty[i % NSTAGE]);
                    tc_commit(&sm.dq_full);
                }
                __syncwarp();
                if (i + 1 < n_steps) ok = issue_scores(i + 1, 1);
            }
            STAMP(11)
            if (lane == 0) STAMP_FLUSH(8, 12)
        }
    } else {
        // ================================================================== compute warps
        const int quarter = warp & 3;
        const int grp = warp >> 2;                          // which 32 query columns of a half
        const int j = quarter * 32 + lane;                  // key row inside the tile
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const bool row_ok = j < w.row_count;
        int qlo = w.q_begin, qhi = w.q_end;                 // queries that may see this key row
        if (!w.uniform && row_ok) {
            const int s = scale_of_row(args.st, w.row_begin + j);
            qlo = args.st.start[s];
            qhi = args.st.start[min(s + 2, args.st.n_scales)];
        }
        const bool tile_masked = (!w.uniform) || (w.row_count < BKV);
        const float sl2 = args.scale_log2;
        const int ds_row_off = (j >> 3) * 1024 + (j & 7) * 128;
        bool ok = true;
        uint32_t s_buf[32], dp_buf[32];
        STAMP_DECL

        // drains dQ of step `i` from TMEM into the fp32 accumulator (this thread: one query row, 32 dims)
        auto drain_dq = [&](int i) -> bool {
            if (!__all_sync(0xffffffffu, mbar_wait(&sm.dq_full, i & 1, abort_flag))) {
                if (lane == 0) report_timeout(args.status, 0x1600 + i);
                return false;
            }
            STAMP(3)
            tc_fence_after();
            const int q0 = w.q_begin + i * BQ;
            const int n_valid = min(BQ, w.q_end - q0);
            tmem_ld32(lane_base + COL_DQ + grp * 32, s_buf);
            tmem_ld_wait();
            if (j < n_valid) {
                float* dst = args.dq_acc + ((size_t)bh * L + q0 + j) * D + grp * 32;
#pragma unroll
                for (int t = 0; t < 32; t += 4)
                    red_add_v4(dst + t, __uint_as_float(s_buf[t]), __uint_as_float(s_buf[t + 1]),
                               __uint_as_float(s_buf[t + 2]), __uint_as_float(s_buf[t + 3]));
            }
            tc_fence_before();
            STAMP(4)
            return true;
        };

        for (int i = 0; i < n_steps && ok; ++i) {
            const int slot = i % NSTAGE;
            const int q0 = w.q_begin + i * BQ;
            const int n_valid = min(BQ, w.q_end - q0);
            const int n_eff = (n_valid + 15) & ~15;
            // visible query columns of this key row in this step: [c_lo, c_hi)
            const int c_lo = row_ok ? max(qlo - q0, 0) : 0;
            const int c_hi = row_ok ? min(qhi - q0, n_valid) : 0;

            const int aslot = i % AUX_STAGES;
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.aux_full[aslot], (i / AUX_STAGES) & 1, abort_flag));
            if (!ok) { if (lane == 0) report_timeout(args.status, 0x1500 + i); break; }
#ifdef HMAR_STAMPS
            if (i == 0) STAMP(6) else STAMP(0)
#endif

            // dQ of the previous step must leave TMEM before this step's dQ is issued, i.e. before the
            // last arrival of this step.  With two halves it is drained between them (the tensor core
            // has finished it by then); a step with a single half drains it first.
            const bool has_b = n_eff > 64;
            if (i > 0 && !has_b) ok = drain_dq(i - 1);

            for (int h = 0; h < 2 && ok; ++h) {
                if (h == 1 && !has_b) break;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[h], i & 1, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x1580 + i); break; }
                STAMP(1)
                tc_fence_after();
                const int c0 = h * 64 + grp * 32;           // first query column of this thread's chunk
                if (c0 < n_eff) {
                    tmem_ld32(lane_base + COL_ST + c0, s_buf);
                    tmem_ld32(lane_base + COL_DPT + c0, dp_buf);
                    // lse / delta of the chunk's 32 queries while the TMEM loads are in flight
                    float4 ls[8], de[8];
                    const float4* lse4 = reinterpret_cast<const float4*>(&sm.lse2[aslot][c0]);
                    const float4* del4 = reinterpret_cast<const float4*>(&sm.delta[aslot][c0]);
#pragma unroll
                    for (int t = 0; t < 8; ++t) { ls[t] = lse4[t]; de[t] = del4[t]; }
                    tmem_ld_wait();
                    STAMP(14)
                    uint32_t p_pack[16], ds_pack[16];
#pragma unroll
                    for (int t = 0; t < 32; t += 4) {
                        float p0 = ex2(fmaf(__uint_as_float(s_buf[t]), sl2, -ls[t / 4].x));
                        float p1 = ex2(fmaf(__uint_as_float(s_buf[t + 1]), sl2, -ls[t / 4].y));
                        float p2 = ex2(fmaf(__uint_as_float(s_buf[t + 2]), sl2, -ls[t / 4].z));
                        float p3 = ex2(fmaf(__uint_as_float(s_buf[t + 3]), sl2, -ls[t / 4].w));
                        if (tile_masked) {
                            p0 = (c0 + t >= c_lo && c0 + t < c_hi) ? p0 : 0.f;
                            p1 = (c0 + t + 1 >= c_lo && c0 + t + 1 < c_hi) ? p1 : 0.f;
                            p2 = (c0 + t + 2 >= c_lo && c0 + t + 2 < c_hi) ? p2 : 0.f;
                            p3 = (c0 + t + 3 >= c_lo && c0 + t + 3 < c_hi) ? p3 : 0.f;
                        }
                        const float d0 = p0 * (__uint_as_float(dp_buf[t]) - de[t / 4].x);
                        const float d1 = p1 * (__uint_as_float(dp_buf[t + 1]) - de[t / 4].y);
                        const float d2 = p2 * (__uint_as_float(dp_buf[t + 2]) - de[t / 4].z);
                        const float d3 = p3 * (__uint_as_float(dp_buf[t + 3]) - de[t / 4].w);
                        p_pack[t / 2] = pack_bf16(p0, p1);
                        p_pack[t / 2 + 1] = pack_bf16(p2, p3);
                        ds_pack[t / 2] = pack_bf16(d0, d1);
                        ds_pack[t / 2 + 1] = pack_bf16(d2, d3);
                    }
                    STAMP(15)
                    // P^T over S^T: the 16 packed columns written here start at this thread's own first
                    // fp32 column, which it has already read
                    tmem_st16(lane_base + COL_ST + c0, p_pack);
                    // dS^T to shared memory: 4 chunks of 8 queries, 128-byte swizzle on the key row
                    uint8_t* ds_row = sm.ds[i & 1][h] + ds_row_off;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const int chunk = grp * 4 + ch;
                        uint4 val = make_uint4(ds_pack[4 * ch], ds_pack[4 * ch + 1], ds_pack[4 * ch + 2], ds_pack[4 * ch + 3]);
                        *reinterpret_cast<uint4*>(ds_row + ((chunk ^ (j & 7)) << 4)) = val;
                    }
                    tmem_st_wait();
                }
                tc_fence_before();
                fence_proxy_async_smem();
                mbar_arrive(&sm.p_full[h]);
                STAMP(2)
                if (h == 0 && i > 0 && has_b) ok = drain_dq(i - 1);
            }
            mbar_arrive(&sm.aux_empty[aslot]);      // this thread is done with the step's lse / delta
        }
        if (ok) ok = drain_dq(n_steps - 1);
        const int half = grp;

        // ---- epilogue: dK (warps 0-3) and dV (warps 4-7); the last dq_full also covers them
        if (ok) {
            const uint32_t col = half == 0 ? COL_DK : COL_DV;
            const float mul = half == 0 ? args.softmax_scale : 1.f;
            __nv_bfloat16* base = half == 0 ? args.dk : args.dv;
            __nv_bfloat16* orow = base + ((size_t)bh * L + w.row_begin + j) * D;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                tmem_ld32(lane_base + col + h * 32, s_buf);
                tmem_ld_wait();
                if (row_ok) {
                    uint4* dst = reinterpret_cast<uint4*>(orow + h * 32);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(s_buf[8 * t + 0]) * mul, __uint_as_float(s_buf[8 * t + 1]) * mul);
                        o.y = pack_bf16(__uint_as_float(s_buf[8 * t + 2]) * mul, __uint_as_float(s_buf[8 * t + 3]) * mul);
                        o.z = pack_bf16(__uint_as_float(s_buf[8 * t + 4]) * mul, __uint_as_float(s_buf[8 * t + 5]) * mul);
                        o.w = pack_bf16(__uint_as_float(s_buf[8 * t + 6]) * mul, __uint_as_float(s_buf[8 * t + 7]) * mul);
                        dst[t] = o;
                    }
                }
            }
        }
        STAMP(5)
        if (warp == 0 && lane == 0) { STAMP_FLUSH(0, 7) STAMP_FLUSH(14, 16) }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

#ifdef HMAR_STAMPS
}  // namespace
extern "C" int hmar_debug_bwd_stamps(unsigned long long* out16) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(out16, g_bwd_stamps, sizeof(g_bwd_stamps)) != cudaSuccess) return -1;
    unsigned long long zero[16] = {0};
    cudaMemcpyToSymbol(g_bwd_stamps, zero, sizeof(zero));
    return 0;
}
namespace {
#endif

// ------------------------------------------------------------------------------------------------
// delta_i = sum_d dO_id * O_id  (one warp per 4 rows: 8 lanes x 16 bytes cover a row)
__global__ void __launch_bounds__(256)
hmar_bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                      float* __restrict__ delta, size_t n_rows) {
    const size_t row = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
    const int part = threadIdx.x & 7;
    float acc = 0.f;
    if (row < n_rows) {
        const uint4 a = *reinterpret_cast<const uint4*>(out + row * D + part * 8);
        const uint4 b = *reinterpret_cast<const uint4*>(dout + row * D + part * 8);
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const float2 fa = __bfloat1622float2(pa[t]), fb = __bfloat1622float2(pb[t]);
            acc = fmaf(fa.x, fb.x, acc);
            acc = fmaf(fa.y, fb.y, acc);
        }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    if (row < n_rows && part == 0) delta[row] = acc;
}

// dq = bf16(scale * dq_acc)
__global__ void __launch_bounds__(256)
hmar_bwd_dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, float scale, size_t n8) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n8) return;
    const float4 a = reinterpret_cast<const float4*>(acc)[2 * idx];
    const float4 b = reinterpret_cast<const float4*>(acc)[2 * idx + 1];
    uint4 o;
    o.x = pack_bf16(a.x * scale, a.y * scale);
    o.y = pack_bf16(a.z * scale, a.w * scale);
    o.z = pack_bf16(b.x * scale, b.y * scale);
    o.w = pack_bf16(b.z * scale, b.w * scale);
    reinterpret_cast<uint4*>(dq)[idx] = o;
}

}  // namespace

cudaError_t launch_bwd_tc(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& dout_map,
                          const BwdArgs& args, const __nv_bfloat16* out, const __nv_bfloat16* dout,
                          __nv_bfloat16* dq, int BH, cudaStream_t stream) {
    const size_t smem = sizeof(SharedStorage) + 1024;
    cudaError_t e = cudaFuncSetAttribute(hmar_bwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const size_t n_rows = (size_t)BH * args.L;
    {
        KernelTimer timer("memset_dq_acc", stream);
        e = cudaMemsetAsync(args.dq_acc, 0, n_rows * D * sizeof(float), stream);
        if (e != cudaSuccess) return e;
    }
    {
        KernelTimer timer("hmar_bwd_delta_kernel", stream);
        hmar_bwd_delta_kernel<<<(unsigned)((n_rows * 8 + 255) / 256), 256, 0, stream>>>(out, dout, args.delta_w, n_rows);
    }
    {
        KernelTimer timer("hmar_bwd_tc_kernel", stream);
        hmar_bwd_tc_kernel<<<(unsigned)BH * (unsigned)args.n_work, NUM_THREADS, smem, stream>>>(q, k, v, dout_map, args);
    }
    const size_t n8 = n_rows * D / 8;
    {
        KernelTimer timer("hmar_bwd_dq_convert_kernel", stream);
        hmar_bwd_dq_convert_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, stream>>>(args.dq_acc, dq, args.softmax_scale, n8);
    }
    count_launch(3);
    return cudaGetLastError();
}

}  // namespace hmar
