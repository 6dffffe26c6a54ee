// Forward kernel of HMAR's Markovian block-sparse attention for sm_100a, and the inference step.
//
// One block handles one work tile: up to 128 consecutive query rows of one head and the contiguous
// key range those rows may see under the mask (paper Sec. 4.1, Fig. attn-mask).  It is the usual
// IO-aware tiling with an online softmax (Sec. 4.1: the kernel extends FlashAttention), laid out for
// Blackwell.  The key range is walked 64 keys at a time, and a block is ONE softmax chain:
//   logits ready -> softmax warpgroup -> P ready -> tensor core (O += P V, next logits) -> ...
// A chain spends most of its time waiting for the other side (the round trip through the barriers and the
// tensor core's queue is longer than either side's work), so what keeps an SM busy is the number of
// independent chains on it: a block is kept small (256 threads, 128 TMEM columns, 50 KB of shared memory)
// and FOUR blocks share an SM.  Each block's set-up, first copies and epilogue, during which it computes
// nothing, are then overlapped by three running chains instead of being a quarter of its life.
//   warps 0-3   softmax: one query row per thread, 64 logits per tile read from TMEM once; the running
//               maximum is kept unless the tile exceeds it by more than 2^8 (then O and the row sum are
//               rescaled first), P = 2^(s - m) goes back to TMEM as bf16 over S; at the end O / l -> out
//   warp 4      TMA producer: K and V tiles of 64 keys through a shared-memory ring (Q and the first K, V
//               tiles are requested by thread 0 during the set-up).  The tensor maps are 4-D (64, rows,
//               heads, batches) with the tensor's own strides, so contiguous [B,H,L,64] tensors and the
//               packed [B,L,3,H,64] projection output go through the same code; the output address is
//               formed from three strides
//   warp 5      issues tcgen05.mma: S = Q K^T (both operands in shared memory), O += P V (P from TMEM, V an
//               MN-major shared-memory operand), one burst per tile: O += P V of tile j, then S of tile
//               j + 1 into the columns P has just left
//   warps 6-7   idle: setmaxnreg works on whole warpgroups (four warps), so the producer and the MMA warp
//               sit in a full second warpgroup (a block of 192 threads cannot redistribute its registers;
//               without the redistribution the softmax warps spill and the kernel is 4 % slower)
// TMEM columns: S/P [0,64), O [64,128).
// Registers: the block starts with 64 per thread (four blocks per SM); the softmax warpgroup raises its
// to 88 and the second warpgroup drops to 40 (setmaxnreg), the same total.
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
constexpr int BN = 64;               // keys per tile
constexpr int D = kHeadDim;
constexpr int NSTAGE = 2;
constexpr int Q_BYTES = BM * D * 2;             // 16 KB
constexpr int TILE_BYTES = BN * D * 2;          // 8 KB
constexpr int NUM_THREADS = 256;
constexpr int NUM_SOFTMAX_THREADS = 128;
constexpr int PRODUCER_WARP = 4, MMA_WARP = 5;
constexpr int REGS_START = 64, REGS_SOFTMAX = 88, REGS_MISC = 40;
static_assert(4 * REGS_SOFTMAX + 4 * REGS_MISC == 8 * REGS_START, "register budget of the block");
constexpr uint32_t TMEM_COLS = 128;
constexpr uint32_t COL_S = 0, COL_O = 64;
constexpr float kRescaleThreshold = 8.0f;       // in log2 units

struct __align__(1024) SharedStorage {
    uint8_t q[Q_BYTES];
    uint8_t k[NSTAGE][TILE_BYTES];
    uint8_t v[NSTAGE][TILE_BYTES];
    uint64_t q_full;
    uint64_t k_full[NSTAGE], k_empty[NSTAGE], v_full[NSTAGE], v_empty[NSTAGE];
    uint64_t s_full, p_full, o_done;
    uint32_t tmem_base;
    int abort_flag;
};

struct KvTile {
    int seg;        // 0 or 1
    int coord;      // first row of the tile inside its tensor
    int n_valid;    // valid keys in the tile (1..64)
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

// columns issued for a tile with n_valid keys (a multiple of 16)
__device__ __forceinline__ int tile_cols(int n_valid) { return (n_valid + 15) & ~15; }

__device__ __forceinline__ void report_timeout(int* status, int where) {
    if (status != nullptr) {
        atomicCAS(status, 0, HMAR_ERR_DEVICE_TIMEOUT);
        atomicCAS(status + 1, 0, where);
    }
}

template <int N> __device__ __forceinline__ void reg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void reg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

__global__ void __launch_bounds__(NUM_THREADS, 4)
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
    const int batch = bh / args.heads_per_batch, head = bh - batch * args.heads_per_batch;
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
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(&sm.k_full[s], 1);
            mbar_init(&sm.k_empty[s], 1);
            mbar_init(&sm.v_full[s], 1);
            mbar_init(&sm.v_empty[s], 1);
        }
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.p_full, NUM_SOFTMAX_THREADS);
        mbar_init(&sm.o_done, 1);
        fence_mbar_init();
        // The block's first copies (Q, first K and V tiles) start here, before the TMEM allocation and the
        // block-wide barrier, so that their latency overlaps the rest of the set-up.
        const KvTile t0 = kv_tile(w, tiles0, 0);
        mbar_arrive_expect_tx(&sm.q_full, Q_BYTES);
        tma_load_4d(sm.q, &map_q, &sm.q_full, 0, w.row_begin, head, batch);
        mbar_arrive_expect_tx(&sm.k_full[0], TILE_BYTES);
        tma_load_4d(sm.k[0], t0.seg ? &map_k1 : &map_k0, &sm.k_full[0], 0, t0.coord, head, batch);
        mbar_arrive_expect_tx(&sm.v_full[0], TILE_BYTES);
        tma_load_4d(sm.v[0], t0.seg ? &map_v1 : &map_v0, &sm.v_full[0], 0, t0.coord, head, batch);
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

    if (warp >= PRODUCER_WARP) {
        reg_dec<REGS_MISC>();
        if (warp == PRODUCER_WARP) {
            // ================================================================== TMA producer
            // The whole warp runs the control flow; one elected lane issues the copies (a warp that has split
            // into one running lane and 31 parked ones issues far more slowly).
            const bool leader = elect_one();
            if (leader) {
                prefetch_tensormap(&map_q);
                prefetch_tensormap(&map_k0);
                prefetch_tensormap(&map_v0);
            }
            __syncwarp();
            bool ok = true;
            for (int j = 1; j < n_tiles && ok; ++j) {           // tile 0 was requested during the set-up
                const int slot = j % NSTAGE;
                const uint32_t par = ((j / NSTAGE) & 1) ^ 1;     // parity of the previous use of the slot
                const KvTile t = kv_tile(w, tiles0, j);
                if (j >= NSTAGE) ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_empty[slot], par, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x100 + j); break; }
                if (leader) {
                    mbar_arrive_expect_tx(&sm.k_full[slot], TILE_BYTES);
                    tma_load_4d(sm.k[slot], t.seg ? &map_k1 : &map_k0, &sm.k_full[slot], 0, t.coord, head, batch);
                }
                __syncwarp();
                if (j >= NSTAGE) ok = __all_sync(0xffffffffu, mbar_wait(&sm.v_empty[slot], par, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x200 + j); break; }
                if (leader) {
                    mbar_arrive_expect_tx(&sm.v_full[slot], TILE_BYTES);
                    tma_load_4d(sm.v[slot], t.seg ? &map_v1 : &map_v0, &sm.v_full[slot], 0, t.coord, head, batch);
                }
                __syncwarp();
            }
            if (!ok) {
                // give the copies already issued a bounded chance to land before the block exits
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 2000000ull) { }
            }
        } else if (warp == MMA_WARP) {
            // ================================================================== MMA issuer
            // The whole warp runs the control flow; one elected lane issues.  Descriptors are built once and
            // advanced by adding (byte offset >> 4), so issuing an MMA costs a few instructions.
            const bool leader = elect_one();
            const uint64_t q_kd = smem_desc_sw128(smem_u32(sm.q), 16);
            const uint64_t k_kd0 = smem_desc_sw128(smem_u32(sm.k[0]), 16);      // ring slots are 8 KB apart
            const uint64_t v_mn0 = smem_desc_sw128(smem_u32(sm.v[0]), 1024);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(BM, D, false, true);
            constexpr uint32_t SLOT_UNITS = TILE_BYTES >> 4;
            auto wait = [&](uint64_t* bar, uint32_t parity, int code) -> bool {
                if (__all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag))) return true;
                if (lane == 0) report_timeout(args.status, code);
                return false;
            };
            // S = Q K^T for n keys of the tile in ring slot `slot`
            auto issue_s = [&](int n, int slot) {
                const uint32_t idesc = idesc_bf16_f32(BM, n, false, false);
                const uint64_t kd = k_kd0 + slot * SLOT_UNITS;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_ss(tmem + COL_S, q_kd + ks * 2, kd + ks * 2, idesc, ks > 0);
                tc_commit(&sm.s_full);
            };
            // O += P V for n keys
            auto issue_pv = [&](int n, int slot, bool first) {
                const int nk = n / 16;
                const uint64_t vd = v_mn0 + slot * SLOT_UNITS;
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks)
                    if (ks < nk)
                        mma_ts(tmem + COL_O, tmem + COL_S + ks * 8, vd + ks * 128, idesc_pv, !first || (ks > 0));
            };

            bool ok = true;
            {
                const bool rq = mbar_try_wait(&sm.q_full, 0), rk = mbar_try_wait(&sm.k_full[0], 0);
                if (!__all_sync(0xffffffffu, rq && rk))
                    ok = (rq || wait(&sm.q_full, 0, 0x300)) && (rk || wait(&sm.k_full[0], 0, 0x400));
            }
            if (ok) {
                tc_fence_after();
                if (leader) {
                    issue_s(tile_cols(kv_tile(w, tiles0, 0).n_valid), 0);
                    if (NSTAGE < n_tiles) tc_commit(&sm.k_empty[0]);
                }
                __syncwarp();
            }
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int slot = j % NSTAGE, slot_next = (j + 1) % NSTAGE;
                const bool more = j + 1 < n_tiles;
                const int n = tile_cols(kv_tile(w, tiles0, j).n_valid);
                const int n_next = more ? tile_cols(kv_tile(w, tiles0, j + 1).n_valid) : 0;
                // one burst: O += P V of tile j, then S of tile j + 1 over the columns P leaves.  The copies are
                // looked at first (normally long complete), both looks sent before either answer is used: a look
                // at a barrier is a shared-memory round trip, and after the softmax warps' arrival every such trip
                // delays the products they are waiting for.
                {
                    const bool rv = mbar_try_wait(&sm.v_full[slot], (j / NSTAGE) & 1);
                    const bool rk = !more || mbar_try_wait(&sm.k_full[slot_next], ((j + 1) / NSTAGE) & 1);
                    if (!__all_sync(0xffffffffu, rv && rk))
                        ok = (rv || wait(&sm.v_full[slot], (j / NSTAGE) & 1, 0x500 + j)) &&
                             (rk || wait(&sm.k_full[slot_next], ((j + 1) / NSTAGE) & 1, 0x400 + j));
                }
                // The last tile of a key segment may be ragged: the rows between its last key and the next multiple of
                // 16 (the granularity of the product over keys) belong to another scale, or to nobody.  Their P is
                // exactly 0, but 0 x (Inf or NaN) is NaN, so these V rows are cleared before O += P V reads them:
                // a non-finite value outside a row's window cannot reach its output.  (Whole rows: the 128-byte swizzle
                // permutes 16-byte pieces inside a row only.)
                if (ok) {
                    const int n_valid = kv_tile(w, tiles0, j).n_valid;
                    if (n_valid < n) {
                        for (int idx = n_valid * 8 + lane; idx < n * 8; idx += 32)
                            *reinterpret_cast<uint4*>(sm.v[slot] + idx * 16) = make_uint4(0u, 0u, 0u, 0u);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                if (ok) ok = wait(&sm.p_full, j & 1, 0x600 + j);
                if (!ok) break;
                tc_fence_after();
                if (leader) {
                    issue_pv(n, slot, j == 0);
                    if (n_next > 0) issue_s(n_next, slot_next);
                    // V of tile j and K of tile j + 1 have been handed to their last readers; a slot is signalled
                    // free only if a later tile will use it (the block may exit as soon as the softmax warps have
                    // seen o_done: an arrival that lands after that would hit the barriers of the next block on
                    // this SM)
                    if (j + NSTAGE < n_tiles) tc_commit(&sm.v_empty[slot]);
                    if (j + 1 + NSTAGE < n_tiles) tc_commit(&sm.k_empty[slot_next]);
                    if (!more) tc_commit(&sm.o_done);
                }
                __syncwarp();
            }
        }
    } else {
        // ================================================================== softmax warps + epilogue
        reg_inc<REGS_SOFTMAX>();
        const int r = warp * 32 + lane;                        // row inside the tile
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const int row = w.row_begin + r;
        const bool row_ok = r < w.row_count;
        int lo = w.s0_begin, hi = w.s0_end;                    // per-row key bounds (training, packed tiles)
        if (!w.uniform && row_ok) {
            const int s = scale_of_row(args.st, row);
            lo = args.st.start[first_key_scale(args.st.window, s)];
            hi = args.st.start[last_key_scale(args.st.window, s) + 1];
        }
        const float sl2 = args.scale_log2;
        const uint32_t s_addr = lane_base + COL_S;
        const uint32_t o_addr = lane_base + COL_O;
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        uint32_t b0[32], b1[32];

        for (int j = 0; j < n_tiles && ok; ++j) {
            const KvTile t = kv_tile(w, tiles0, j);
            const int n = tile_cols(t.n_valid);
            // key c of the tile is visible to this row iff c in [c_lo, c_hi)
            const int c_lo = w.uniform ? 0 : max(lo - t.coord, 0);
            const int c_hi = w.uniform ? t.n_valid : min(hi - t.coord, t.n_valid);
            const bool two = n > 32;                           // second 32-column chunk present
            const bool need_mask = (!w.uniform) || (t.n_valid < (two ? 64 : 32));

            ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, j & 1, abort_flag));
            if (!ok) { if (lane == 0) report_timeout(args.status, 0x800 + j); break; }
            tc_fence_after();

            tmem_ld32(s_addr, b0);
            if (two) tmem_ld32(s_addr + 32, b1);
            tmem_ld_wait();

            // masked logits become -inf once, so the maximum and the exponentials treat them alike (columns the
            // tensor core did not write hold stale values and lie outside [c_lo, c_hi) too)
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (!(i >= c_lo && i < c_hi)) b0[i] = 0xff800000u;
                    if (!(32 + i >= c_lo && 32 + i < c_hi)) b1[i] = 0xff800000u;
                }
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};     // four chains of maxima, not one of 64
#pragma unroll
            for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(b0[i]));
            if (two) {
#pragma unroll
                for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(b1[i]));
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;     // softmax_scale > 0

            // Keep the running maximum unless this tile exceeds it by more than the threshold.  O is quiet
            // here: the product that precedes S of this tile in the tensor core's queue is the last one that
            // wrote it, and the next one waits for these warps.
            const bool grow = mx > m_used + kRescaleThreshold;  // false for -inf > -inf
            if (__any_sync(0xffffffffu, grow)) {
                const float m_new = fmaxf(m_used, mx);
                const float f = (m_used == -INFINITY) ? 0.f : ex2(m_used - m_new);
                m_used = m_new;
                l *= f;
                if (j > 0) {
#pragma unroll 1
                    for (int piece = 0; piece < 4; ++piece) {
                        uint32_t o[16];
                        tmem_ld16(o_addr + piece * 16, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                        tmem_st16(o_addr + piece * 16, o);
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
            mbar_arrive(&sm.p_full);
        }

        // ---- epilogue: out = O / l, lse = ln(l) + m (natural log of the scaled logits' sum)
        if (ok) {
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_done, 0, abort_flag));
            if (!ok && lane == 0) report_timeout(args.status, 0xA00);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            tmem_ld32(o_addr, b0);
            tmem_ld32(o_addr + 32, b1);
            tmem_ld_wait();
            const long long out_off = batch * args.out_batch_stride + head * args.out_head_stride + row * args.out_row_stride;
            const long long lse_off = (long long)bh * args.n_q_rows + row;
            if (row_ok && HMAR_IN_BOUNDS(out_off >= 0 && out_off + D <= args.out_extent, args.status, 0xB101) &&
                HMAR_IN_BOUNDS(args.lse == nullptr || (lse_off >= 0 && lse_off < args.lse_extent), args.status, 0xB102)) {
                uint4* dst = reinterpret_cast<uint4*>(args.out + out_off);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 v4;
                    v4.x = pack_bf16(__uint_as_float(b0[8 * i + 0]) * inv, __uint_as_float(b0[8 * i + 1]) * inv);
                    v4.y = pack_bf16(__uint_as_float(b0[8 * i + 2]) * inv, __uint_as_float(b0[8 * i + 3]) * inv);
                    v4.z = pack_bf16(__uint_as_float(b0[8 * i + 4]) * inv, __uint_as_float(b0[8 * i + 5]) * inv);
                    v4.w = pack_bf16(__uint_as_float(b0[8 * i + 6]) * inv, __uint_as_float(b0[8 * i + 7]) * inv);
                    dst[i] = v4;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 v4;
                    v4.x = pack_bf16(__uint_as_float(b1[8 * i + 0]) * inv, __uint_as_float(b1[8 * i + 1]) * inv);
                    v4.y = pack_bf16(__uint_as_float(b1[8 * i + 2]) * inv, __uint_as_float(b1[8 * i + 3]) * inv);
                    v4.z = pack_bf16(__uint_as_float(b1[8 * i + 4]) * inv, __uint_as_float(b1[8 * i + 5]) * inv);
                    v4.w = pack_bf16(__uint_as_float(b1[8 * i + 6]) * inv, __uint_as_float(b1[8 * i + 7]) * inv);
                    dst[4 + i] = v4;
                }
                if (args.lse != nullptr)
                    args.lse[lse_off] = (m_used + log2f(l)) * 0.6931471805599453f;
            }
        }
    }

    // ---- tear-down
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// Self-test of the bounded waits: one block waits on a barrier that nothing ever arrives on, with a limit of
// one millisecond, through the very wait and report functions the kernels use.  The wait gives up, the block
// records HMAR_ERR_DEVICE_TIMEOUT with location 0xD1A6 in the status word and returns; nothing traps.
__global__ void hmar_selftest_wait_kernel(int* status) {
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&never, 1);
        fence_mbar_init();
    }
    __syncthreads();
    const bool ok = __all_sync(0xffffffffu, mbar_wait(&never, 0, &abort_flag, 1000000ull));
    if (!ok && threadIdx.x == 0) report_timeout(status, 0xD1A6);
}

}  // namespace

cudaError_t launch_selftest_wait(int* status, cudaStream_t stream) {
    hmar_selftest_wait_kernel<<<1, 32, 0, stream>>>(status);
    count_launch(1);
    return cudaGetLastError();
}

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
