// Forward kernel of HMAR's Markovian block-sparse attention for sm_100a, and the inference step.
//
// One block handles one work tile: up to 128 consecutive query rows of one head and the contiguous
// key range those rows may see under the mask (paper Sec. 4.1, Fig. attn-mask).  It is the usual
// IO-aware tiling with an online softmax (Sec. 4.1: the kernel extends FlashAttention), laid out for
// Blackwell:
//   warp 0      TMA producer: Q once, then K and V tiles of 128 keys through a shared-memory ring
//   warp 1      issues tcgen05.mma.  Q is copied to TMEM once and is the A operand of S = Q K^T; a key
//               tile is handled as two halves of 64 keys with their own S columns and barriers, so the
//               tensor core computes one half while the softmax warps work on the other.  P replaces S
//               in place (bf16) and is the TMEM A operand of O += P V.
//   warps 2-5   one query row per thread.  A half's 64 logits are read from TMEM once; the running
//               maximum is kept unless the half exceeds it by more than 2^8 (then O and the row sum are
//               rescaled first), P = 2^(s - m) goes back to TMEM as bf16.
// TMEM columns: S/P half a [0,64), half b [64,128), O [128,192), Q [192,224).  Two blocks fit on one SM.
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

constexpr int BM = 128;              // query rows per block
constexpr int BN = 128;              // keys per tile
constexpr int HN = 64;               // keys per half tile
constexpr int D = kHeadDim;
constexpr int NSTAGE = 2;
constexpr int TILE_BYTES = BN * D * 2;          // 16 KB
constexpr int NUM_THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;
constexpr uint32_t COL_S = 0, COL_O = 128, COL_Q = 192;
constexpr float kRescaleThreshold = 8.0f;       // in log2 units

struct __align__(1024) SharedStorage {
    uint8_t q[TILE_BYTES];
    uint8_t k[NSTAGE][TILE_BYTES];
    uint8_t v[NSTAGE][TILE_BYTES];
    uint64_t q_full, q_tmem;
    uint64_t k_full[NSTAGE], k_empty[NSTAGE], v_full[NSTAGE], v_empty[NSTAGE];
    uint64_t s_full[2], p_full[2], pv_done, o_done;
    uint32_t tmem_base;
    int abort_flag;
};

struct KvTile {
    int seg;        // 0 or 1
    int coord;      // first row of the tile inside its tensor
    int n_valid;    // valid keys in the tile (1..128)
};

__device__ __forceinline__ KvTile kv_tile(const FwdWork& w, int tiles0, int j) {
    KvTile t;
    if (j < tiles0) {
        t.seg = 0;
        t.coord = w.s0_begin + j * BN;
        t.n_valid = min(BN, w.s0_end - t.coord);
    } else {
        t.seg = 1;
        t.coord = w.s1_begin + (j - tiles0) * BN;
        t.n_valid = min(BN, w.s1_end - t.coord);
    }
    return t;
}

// columns issued for half h of a tile with n_valid keys (multiple of 16, 0 if the half is empty)
__device__ __forceinline__ int half_cols(int n_valid, int h) {
    const int n_eff = (n_valid + 15) & ~15;
    return h == 0 ? min(n_eff, HN) : max(n_eff - HN, 0);
}

__device__ __forceinline__ void report_timeout(int* status, int where) {
    if (status != nullptr) {
        atomicCAS(status, 0, HMAR_ERR_DEVICE_TIMEOUT);
        atomicCAS(status + 1, 0, where);
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 2)
hmar_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k0,
                   const __grid_constant__ CUtensorMap map_v0, const __grid_constant__ CUtensorMap map_k1,
                   const __grid_constant__ CUtensorMap map_v1, const FwdArgs args) {
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& sm = *reinterpret_cast<SharedStorage*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // A block of this launch (or an earlier one) already gave up on a wait: do no further work.
    if (args.status != nullptr && *reinterpret_cast<volatile int*>(args.status) != 0) return;

    // ---- which tile of which head
    const int bh = blockIdx.x / args.n_work;
    const int wi = blockIdx.x % args.n_work;
    FwdWork w;
    if (args.work != nullptr) {
        w = args.work[wi];
    } else {   // inference step: dense window, previous scale then current scale
        w.row_begin = wi * BM;
        w.row_count = min(BM, args.n_q_rows - w.row_begin);
        w.s0_begin = 0; w.s0_end = args.n0;
        w.s1_begin = 0; w.s1_end = args.n1;
        w.uniform = 1;
    }
    const int tiles0 = (w.s0_end - w.s0_begin + BN - 1) / BN;
    const int tiles1 = (w.s1_end - w.s1_begin + BN - 1) / BN;
    const int n_tiles = tiles0 + tiles1;

    // ---- set-up
    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_tmem, 128);
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(&sm.k_full[s], 1);
            mbar_init(&sm.k_empty[s], 1);
            mbar_init(&sm.v_full[s], 1);
            mbar_init(&sm.v_empty[s], 1);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(&sm.s_full[h], 1);
            mbar_init(&sm.p_full[h], 128);
        }
        mbar_init(&sm.pv_done, 1);
        mbar_init(&sm.o_done, 1);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(&sm.tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;

    if (warp == 0) {
        // ================================================================== TMA producer
        // The whole warp runs the control flow; one elected lane issues the copies (a warp that has split
        // into one running lane and 31 parked ones issues far more slowly).
        const bool leader = elect_one();
        if (leader) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k0);
            prefetch_tensormap(&map_v0);
            mbar_arrive_expect_tx(&sm.q_full, TILE_BYTES);
            tma_load_3d(sm.q, &map_q, &sm.q_full, 0, w.row_begin, bh);
        }
        __syncwarp();
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int slot = j % NSTAGE;
            const uint32_t par = ((j / NSTAGE) & 1) ^ 1;     // parity of the previous use of the slot
            const KvTile t = kv_tile(w, tiles0, j);
            if (j >= NSTAGE) ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_empty[slot], par, abort_flag));
            if (!ok) { if (lane == 0) report_timeout(args.status, 0x100 + j); break; }
            if (leader) {
                mbar_arrive_expect_tx(&sm.k_full[slot], TILE_BYTES);
                tma_load_3d(sm.k[slot], t.seg ? &map_k1 : &map_k0, &sm.k_full[slot], 0, t.coord, bh);
            }
            __syncwarp();
            if (j >= NSTAGE) ok = __all_sync(0xffffffffu, mbar_wait(&sm.v_empty[slot], par, abort_flag));
            if (!ok) { if (lane == 0) report_timeout(args.status, 0x200 + j); break; }
            if (leader) {
                mbar_arrive_expect_tx(&sm.v_full[slot], TILE_BYTES);
                tma_load_3d(sm.v[slot], t.seg ? &map_v1 : &map_v0, &sm.v_full[slot], 0, t.coord, bh);
            }
            __syncwarp();
        }
        if (!ok) {
            // give the copies already issued a bounded chance to land before the block exits
            const uint64_t t0 = globaltimer_ns();
            while (globaltimer_ns() - t0 < 2000000ull) { }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        // The whole warp runs the control flow; one elected lane issues.  Descriptors are built once and
        // advanced by adding (byte offset >> 4), so issuing an MMA costs a few instructions.
        const bool leader = elect_one();
        const uint64_t k_kd0 = smem_desc_sw128(smem_u32(sm.k[0]), 16);      // ring slots are 16 KB apart
        const uint64_t v_mn0 = smem_desc_sw128(smem_u32(sm.v[0]), 1024);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(BM, D, false, true);
        int p_seen[2] = {0, 0};                                 // completed phases of p_full[h] consumed so far
        bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_tmem, 0, abort_flag));
        if (!ok && lane == 0) report_timeout(args.status, 0x300);

        // S_h = Q K_h^T for half h of tile j (Q from TMEM, 64 keys of the tile from shared memory)
        auto issue_s = [&](int j, int h) -> bool {
            const int slot = j % NSTAGE;
            const int n = half_cols(kv_tile(w, tiles0, j).n_valid, h);
            if (n == 0) return true;
            if (h == 0 && !__all_sync(0xffffffffu, mbar_wait(&sm.k_full[slot], (j / NSTAGE) & 1, abort_flag))) {
                if (lane == 0) report_timeout(args.status, 0x400 + j);
                return false;
            }
            tc_fence_after();
            if (leader) {
                const uint32_t idesc = idesc_bf16_f32(BM, n, false, false);
                const uint64_t kd = k_kd0 + slot * 1024 + h * 512;              // + 64 rows
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_ts(tmem + COL_S + h * HN, tmem + COL_Q + ks * 8, kd + ks * 2, idesc, ks > 0);
                tc_commit(&sm.s_full[h]);
            }
            __syncwarp();
            return true;
        };
        // O += P_h V_h for half h of tile j; the tile's last half releases its K and V slots
        auto issue_pv = [&](int j, int h) -> bool {
            const int slot = j % NSTAGE;
            const int n_valid = kv_tile(w, tiles0, j).n_valid;
            const int n = half_cols(n_valid, h);
            if (n == 0) return true;
            const int par = h == 0 ? (p_seen[0]++ & 1) : (p_seen[1]++ & 1);
            if (!__all_sync(0xffffffffu, mbar_wait(&sm.p_full[h], par, abort_flag))) {
                if (lane == 0) report_timeout(args.status, 0x600 + j);
                return false;
            }
            if (h == 0 && !__all_sync(0xffffffffu, mbar_wait(&sm.v_full[slot], (j / NSTAGE) & 1, abort_flag))) {
                if (lane == 0) report_timeout(args.status, 0x500 + j);
                return false;
            }
            tc_fence_after();
            if (leader) {
                const int nk = n / 16;
                const uint64_t vd = v_mn0 + slot * 1024 + h * 512;
                const bool first = (j == 0) && (h == 0);
#pragma unroll
                for (int ks = 0; ks < HN / 16; ++ks)
                    if (ks < nk)
                        mma_ts(tmem + COL_O, tmem + COL_S + h * HN + ks * 8, vd + ks * 128, idesc_pv, !first || (ks > 0));
                // Nobody waits for the slots of the last NSTAGE tiles to become free, and the block may exit as
                // soon as the softmax warps have seen the last pv_done: an arrival that lands after that would
                // hit the barriers of the next block on this SM.  So those slots are not signalled at all, and
                // pv_done / o_done are signalled last.
                if ((h == 1 || half_cols(n_valid, 1) == 0) && j + NSTAGE < n_tiles) {      // last half of the tile
                    tc_commit(&sm.k_empty[slot]);
                    tc_commit(&sm.v_empty[slot]);
                }
                tc_commit(&sm.pv_done);
                // the last product of the block also completes o_done, which the epilogue waits for: a warp
                // may be two halves ahead of the tensor core there, too far for pv_done's parity to tell
                if (j + 1 == n_tiles && (h == 1 || half_cols(n_valid, 1) == 0)) tc_commit(&sm.o_done);
            }
            __syncwarp();
            return true;
        };

        if (ok) ok = issue_s(0, 0);
        if (ok) ok = issue_s(0, 1);
        for (int j = 0; j < n_tiles && ok; ++j) {
            ok = issue_pv(j, 0);
            if (ok && j + 1 < n_tiles) ok = issue_s(j + 1, 0);
            if (ok) ok = issue_pv(j, 1);
            if (ok && j + 1 < n_tiles) ok = issue_s(j + 1, 1);
        }
    } else {
        // ================================================================== softmax + epilogue
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;                     // row inside the tile
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const int row = w.row_begin + r;
        const bool row_ok = r < w.row_count;
        int lo = w.s0_begin, hi = w.s0_end;                    // per-row key bounds (training, packed tiles)
        if (!w.uniform && row_ok) {
            const int s = scale_of_row(args.st, row);
            lo = args.st.start[s > 0 ? s - 1 : 0];
            hi = args.st.start[s + 1];
        }
        const float sl2 = args.scale_log2;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        int pv_issued = 0;                                     // halves handed to the tensor core so far
        int s_seen[2] = {0, 0};                                // completed phases of s_full[h] consumed so far
        uint32_t b0[32], b1[32];

        // ---- Q row to TMEM (A operand of S = Q K^T): undo the 128-byte swizzle of the TMA tile
        ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full, 0, abort_flag));
        if (!ok && lane == 0) report_timeout(args.status, 0x700);
        if (ok) {
            const uint8_t* qrow = sm.q + r * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 val = *reinterpret_cast<const uint4*>(qrow + ((c ^ (r & 7)) << 4));
                b0[4 * c] = val.x; b0[4 * c + 1] = val.y; b0[4 * c + 2] = val.z; b0[4 * c + 3] = val.w;
            }
            tmem_st32(lane_base + COL_Q, b0);
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&sm.q_tmem);
        }

        for (int j = 0; j < n_tiles && ok; ++j) {
            const KvTile t = kv_tile(w, tiles0, j);
            // key c of the tile is visible to this row iff c in [c_lo, c_hi)
            const int c_lo = w.uniform ? 0 : max(lo - t.coord, 0);
            const int c_hi = w.uniform ? t.n_valid : min(hi - t.coord, t.n_valid);

            for (int h = 0; h < 2 && ok; ++h) {
                const int n = half_cols(t.n_valid, h);
                if (n == 0) break;
                const int col0 = h * HN;                           // first key of the half inside the tile
                const bool two = n > 32;                           // second 32-column chunk present
                const bool need_mask = (!w.uniform) || (t.n_valid < col0 + (two ? 64 : 32));
                const uint32_t s_addr = lane_base + COL_S + col0;

                const int par = h == 0 ? (s_seen[0]++ & 1) : (s_seen[1]++ & 1);
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[h], par, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x800 + j); break; }
                tc_fence_after();

                tmem_ld32(s_addr, b0);
                if (two) tmem_ld32(s_addr + 32, b1);
                tmem_ld_wait();

                // masked logits become -inf once, so the maximum and the exponentials treat them alike
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (!(col0 + i >= c_lo && col0 + i < c_hi)) b0[i] = 0xff800000u;
                        if (!(col0 + 32 + i >= c_lo && col0 + 32 + i < c_hi)) b1[i] = 0xff800000u;
                    }
                }
                float mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(b0[i]));
                if (two) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(b1[i]));
                }
                mx *= sl2;                                          // softmax_scale > 0

                // Keep the running maximum unless this half exceeds it by more than the threshold.
                const bool grow = mx > m_used + kRescaleThreshold;  // false for -inf > -inf
                if (__any_sync(0xffffffffu, grow)) {
                    // O must be quiet: wait for every P V product handed over so far
                    if (pv_issued > 0) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&sm.pv_done, (pv_issued - 1) & 1, abort_flag));
                        if (!ok) { if (lane == 0) report_timeout(args.status, 0x900 + j); break; }
                        tc_fence_after();
                    }
                    const float m_new = fmaxf(m_used, mx);
                    const float f = (m_used == -INFINITY) ? 0.f : ex2(m_used - m_new);
                    m_used = m_new;
                    l *= f;
                    if (pv_issued > 0) {
                        uint32_t o[32];
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            tmem_ld32(lane_base + COL_O + hh * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                            tmem_st32(lane_base + COL_O + hh * 32, o);
                        }
                    }
                }
                const float m_sub = (m_used == -INFINITY) ? 0.f : m_used;

                // P = 2^(s * scale - m): fp32 row sum, bf16 P written over the S columns already read
                uint32_t packed[16];
                float l_add = 0.f;
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = ex2(fmaf(__uint_as_float(b0[i]), sl2, -m_sub));
                    const float p1 = ex2(fmaf(__uint_as_float(b0[i + 1]), sl2, -m_sub));
                    l_add += p0 + p1;
                    packed[i / 2] = pack_bf16(p0, p1);
                }
                tmem_st16(s_addr, packed);
                if (two) {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float p0 = ex2(fmaf(__uint_as_float(b1[i]), sl2, -m_sub));
                        const float p1 = ex2(fmaf(__uint_as_float(b1[i + 1]), sl2, -m_sub));
                        l_add += p0 + p1;
                        packed[i / 2] = pack_bf16(p0, p1);
                    }
                    tmem_st16(s_addr + 16, packed);
                }
                l += l_add;
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&sm.p_full[h]);
                ++pv_issued;
            }
        }

        if (ok) {
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_done, 0, abort_flag));
            if (!ok && lane == 0) report_timeout(args.status, 0xA00);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            __nv_bfloat16* orow = args.out + ((size_t)bh * args.n_q_rows + row) * D;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                tmem_ld32(lane_base + COL_O + h * 32, b0);
                tmem_ld_wait();
                if (row_ok) {
                    uint4* dst = reinterpret_cast<uint4*>(orow + h * 32);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 v4;
                        v4.x = pack_bf16(__uint_as_float(b0[8 * i + 0]) * inv, __uint_as_float(b0[8 * i + 1]) * inv);
                        v4.y = pack_bf16(__uint_as_float(b0[8 * i + 2]) * inv, __uint_as_float(b0[8 * i + 3]) * inv);
                        v4.z = pack_bf16(__uint_as_float(b0[8 * i + 4]) * inv, __uint_as_float(b0[8 * i + 5]) * inv);
                        v4.w = pack_bf16(__uint_as_float(b0[8 * i + 6]) * inv, __uint_as_float(b0[8 * i + 7]) * inv);
                        dst[i] = v4;
                    }
                }
            }
            if (row_ok && args.lse != nullptr)
                args.lse[(size_t)bh * args.n_q_rows + row] = (m_used + log2f(l)) * 0.6931471805599453f;
        }
    }

    // ---- tear-down
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

}  // namespace

size_t fwd_tc_smem_bytes() { return sizeof(SharedStorage) + 1024; }

cudaError_t launch_fwd_tc(const CUtensorMap& q, const CUtensorMap& k0, const CUtensorMap& v0, const CUtensorMap& k1,
                          const CUtensorMap& v1, const FwdArgs& args, int BH, cudaStream_t stream) {
    const size_t smem = fwd_tc_smem_bytes();
    cudaError_t e = cudaFuncSetAttribute(hmar_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)BH * (unsigned)args.n_work;
    {
        KernelTimer timer(args.work != nullptr ? "hmar_fwd_tc_kernel" : "hmar_fwd_tc_kernel/scale_step", stream);
        hmar_fwd_tc_kernel<<<grid, NUM_THREADS, smem, stream>>>(q, k0, v0, k1, v1, args);
    }
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace hmar
