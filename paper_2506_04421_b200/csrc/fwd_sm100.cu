// Forward kernel of HMAR's Markovian block-sparse attention for sm_100a, and the inference step.
//
// One block handles one work tile: up to 128 consecutive query rows of one head and the contiguous
// key range those rows may see under the mask (paper Sec. 4.1, Fig. attn-mask).  It is the usual
// IO-aware tiling with an online softmax (Sec. 4.1: the kernel extends FlashAttention), laid out for
// Blackwell:
//   warp 0      TMA producer: Q once, then K and V tiles of 128 keys through a shared-memory ring
//   warp 1      issues tcgen05.mma: S = Q K^T into TMEM, then O += P V with P read from TMEM
//   warps 2-5   one query row per thread: read S from TMEM, mask, running max / sum in fp32,
//               write P (bf16) back to TMEM, rescale O only when the running max grew by > 2^8,
//               and finally normalise O and write out / lse
// TMEM columns: S fp32 [0,128), P bf16 [128,192), O fp32 [192,256).  Two blocks fit on one SM
// (256 TMEM columns and ~82 KB of shared memory each), so one block's softmax overlaps the other
// block's matrix products.
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
constexpr int D = kHeadDim;
constexpr int NSTAGE = 2;
constexpr int TILE_BYTES = BN * D * 2;          // 16 KB
constexpr int NUM_THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;
constexpr uint32_t COL_S = 0, COL_P = 128, COL_O = 192;
constexpr float kRescaleThreshold = 8.0f;       // in log2 units

struct __align__(1024) SharedStorage {
    uint8_t q[TILE_BYTES];
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
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(&sm.k_full[s], 1);
            mbar_init(&sm.k_empty[s], 1);
            mbar_init(&sm.v_full[s], 1);
            mbar_init(&sm.v_empty[s], 1);
        }
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.p_full, 128);
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
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k0);
            prefetch_tensormap(&map_v0);
            mbar_arrive_expect_tx(&sm.q_full, TILE_BYTES);
            tma_load_3d(sm.q, &map_q, &sm.q_full, 0, w.row_begin, bh);
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int slot = j % NSTAGE;
                const uint32_t par = ((j / NSTAGE) & 1) ^ 1;     // parity of the previous use of the slot
                const KvTile t = kv_tile(w, tiles0, j);
                if (j >= NSTAGE) ok = mbar_wait(&sm.k_empty[slot], par, abort_flag);
                if (!ok) { report_timeout(args.status, 0x100 + j); break; }
                mbar_arrive_expect_tx(&sm.k_full[slot], TILE_BYTES);
                tma_load_3d(sm.k[slot], t.seg ? &map_k1 : &map_k0, &sm.k_full[slot], 0, t.coord, bh);
                if (j >= NSTAGE) ok = mbar_wait(&sm.v_empty[slot], par, abort_flag);
                if (!ok) { report_timeout(args.status, 0x200 + j); break; }
                mbar_arrive_expect_tx(&sm.v_full[slot], TILE_BYTES);
                tma_load_3d(sm.v[slot], t.seg ? &map_v1 : &map_v0, &sm.v_full[slot], 0, t.coord, bh);
            }
            if (!ok) {
                // give the copies already issued a bounded chance to land before the block exits
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 2000000ull) { }
            }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        // The whole warp runs the control flow; one elected lane issues.  Descriptors are built once and
        // advanced by adding (byte offset >> 4), so issuing an MMA costs a few instructions.
        {
            const bool leader = elect_one();
            const uint64_t q_kd = smem_desc_sw128(smem_u32(sm.q), 16);
            const uint64_t k_kd0 = smem_desc_sw128(smem_u32(sm.k[0]), 16);      // ring slots are 16 KB apart
            const uint64_t v_mn0 = smem_desc_sw128(smem_u32(sm.v[0]), 1024);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(BM, D, false, true);
            bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full, 0, abort_flag));
            if (!ok && lane == 0) report_timeout(args.status, 0x300);
            auto issue_pv = [&](int j) -> bool {      // O += P_j V_j
                const int slot = j % NSTAGE;
                const KvTile t = kv_tile(w, tiles0, j);
                const int nk = ((t.n_valid + 15) & ~15) / 16;
                if (!__all_sync(0xffffffffu, mbar_wait(&sm.v_full[slot], (j / NSTAGE) & 1, abort_flag))) {
                    if (lane == 0) report_timeout(args.status, 0x500 + j);
                    return false;
                }
                tc_fence_after();
                if (leader) {
                    const uint64_t vd = v_mn0 + slot * 1024;
#pragma unroll
                    for (int ks = 0; ks < BN / 16; ++ks)
                        if (ks < nk)
                            mma_ts(tmem + COL_O, tmem + COL_P + ks * 8, vd + ks * 128, idesc_pv, (j > 0) || (ks > 0));
                    tc_commit(&sm.v_empty[slot]);
                    tc_commit(&sm.o_done);
                }
                __syncwarp();
                return true;
            };
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int slot = j % NSTAGE;
                const KvTile t = kv_tile(w, tiles0, j);
                const int n_eff = (t.n_valid + 15) & ~15;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[slot], (j / NSTAGE) & 1, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x400 + j); break; }
                if (j > 0) {   // S buffer free and P_{j-1} written
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.p_full, (j - 1) & 1, abort_flag));
                    if (!ok) { if (lane == 0) report_timeout(args.status, 0x600 + j); break; }
                }
                tc_fence_after();
                if (leader) {
                    const uint32_t idesc = idesc_bf16_f32(BM, n_eff, false, false);
                    const uint64_t kd = k_kd0 + slot * 1024;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) mma_ss(tmem + COL_S, q_kd + ks * 2, kd + ks * 2, idesc, ks > 0);
                    tc_commit(&sm.k_empty[slot]);
                    tc_commit(&sm.s_full);
                }
                __syncwarp();
                if (j > 0) ok = issue_pv(j - 1);
            }
            if (ok) {
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.p_full, (n_tiles - 1) & 1, abort_flag));
                if (!ok && lane == 0) report_timeout(args.status, 0x700);
                if (ok) {
                    tc_fence_after();
                    issue_pv(n_tiles - 1);
                }
            }
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
        uint32_t buf[32];

        for (int j = 0; j < n_tiles; ++j) {
            const KvTile t = kv_tile(w, tiles0, j);
            const int n_eff = (t.n_valid + 15) & ~15;
            const int n_chunks = (n_eff + 31) / 32;
            const bool need_mask = (!w.uniform) || (t.n_valid < n_chunks * 32);
            // key c of the tile is visible iff c in [c_lo, c_hi)
            const int c_lo = w.uniform ? 0 : max(lo - t.coord, 0);
            const int c_hi = w.uniform ? t.n_valid : min(hi - t.coord, t.n_valid);

            ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full, j & 1, abort_flag));
            if (!ok) { if (lane == 0) report_timeout(args.status, 0x800 + j); break; }
            tc_fence_after();

            // ---- pass 1: row maximum of the scaled logits (log2 units)
            float mx = -INFINITY;
            for (int ch = 0; ch < n_chunks; ++ch) {
                tmem_ld32(lane_base + COL_S + ch * 32, buf);
                tmem_ld_wait();
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int c = ch * 32 + i;
                        const float s = __uint_as_float(buf[i]) * sl2;
                        mx = fmaxf(mx, (c >= c_lo && c < c_hi) ? s : -INFINITY);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(buf[i]) * sl2);
                }
            }
            const float m_new = fmaxf(m_used, mx);
            const float m_old = m_used;
            const bool want = (j == 0) || (m_new > m_used + kRescaleThreshold);
            const bool any = __any_sync(0xffffffffu, want);

            if (j > 0) {    // P buffer free again, O not being accumulated into
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_done, (j - 1) & 1, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x900 + j); break; }
                tc_fence_after();
            }
            if (any) {
                m_used = m_new;
                if (j > 0) {
                    const float f = (m_old == -INFINITY) ? 0.f : ex2(m_old - m_used);
                    l *= f;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        tmem_ld32(lane_base + COL_O + h * 32, buf);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) buf[i] = __float_as_uint(__uint_as_float(buf[i]) * f);
                        tmem_st32(lane_base + COL_O + h * 32, buf);
                    }
                }
            }
            const float m_sub = (m_used == -INFINITY) ? 0.f : m_used;

            // ---- pass 2: P = 2^(s - m), row sum, bf16 P back to TMEM
            for (int ch = 0; ch < n_chunks; ++ch) {
                tmem_ld32(lane_base + COL_S + ch * 32, buf);
                tmem_ld_wait();
                uint32_t packed[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = ex2(fmaf(__uint_as_float(buf[i]), sl2, -m_sub));
                    float p1 = ex2(fmaf(__uint_as_float(buf[i + 1]), sl2, -m_sub));
                    if (need_mask) {
                        const int c = ch * 32 + i;
                        p0 = (c >= c_lo && c < c_hi) ? p0 : 0.f;
                        p1 = (c + 1 >= c_lo && c + 1 < c_hi) ? p1 : 0.f;
                    }
                    l += p0 + p1;
                    packed[i / 2] = pack_bf16(p0, p1);
                }
                tmem_st16(lane_base + COL_P + ch * 16, packed);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&sm.p_full);
        }

        if (ok) {
            ok = __all_sync(0xffffffffu, mbar_wait(&sm.o_done, (n_tiles - 1) & 1, abort_flag));
            if (!ok && lane == 0) report_timeout(args.status, 0xA00);
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            __nv_bfloat16* orow = args.out + ((size_t)bh * args.n_q_rows + row) * D;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                tmem_ld32(lane_base + COL_O + h * 32, buf);
                tmem_ld_wait();
                if (row_ok) {
                    uint4* dst = reinterpret_cast<uint4*>(orow + h * 32);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(buf[8 * i + 0]) * inv, __uint_as_float(buf[8 * i + 1]) * inv);
                        o.y = pack_bf16(__uint_as_float(buf[8 * i + 2]) * inv, __uint_as_float(buf[8 * i + 3]) * inv);
                        o.z = pack_bf16(__uint_as_float(buf[8 * i + 4]) * inv, __uint_as_float(buf[8 * i + 5]) * inv);
                        o.w = pack_bf16(__uint_as_float(buf[8 * i + 6]) * inv, __uint_as_float(buf[8 * i + 7]) * inv);
                        dst[i] = o;
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
