// Backward kernels of HMAR's Markovian block-sparse attention for sm_100a.
//
// The gradient of exact softmax attention is recomputed from the forward's lse (the paper benchmarks
// this pass in App. B.4; Sec. 4.1 builds the kernel on FlashAttention, whose backward this follows):
//   P = exp(scale * Q K^T - lse),  dV = P^T dO,  dP = dO V^T,  dS = P o (dP - delta),
//   dQ = scale * dS K,  dK = scale * dS^T Q,  delta_i = sum_d dO_id O_id.
//
// Main kernel: persistent blocks, one per SM.  A work item is one tile of up to 128 key rows of one
// head; the block walks over the contiguous range of query rows that may see them under the mask
// (queries of the keys' own scale and of the next scale; paper Sec. 4.1, Fig. attn-mask), 128 queries
// (one step) at a time.  A step is split into two halves of 64 queries with their own TMEM columns and
// barriers; each half belongs to one compute warpgroup, so the two warpgroups and the tensor core work
// on different halves at the same time.  The steps of all items of a block form one pipeline: while the
// warpgroups work on an item's last step the tensor core already computes the next item's first scores.
//   warps 0-3   compute warpgroup of half 0: 32 key rows per warp, 64 query columns.  P^T and dS^T in
//               fp32 with packed two-float instructions; P^T (bf16) goes back to TMEM over S^T, dS^T
//               (bf16) goes to TMEM over dP^T (A operand of dK) and to shared memory (A operand of dQ)
//   warps 4-7   the same for half 1
//   warps 8-11  per step: drain dQ_i from TMEM through a staging buffer into the fp32 accumulator with
//               bulk tensor reductions (cp.reduce.async.bulk.tensor).  Per item: copy the next item's K
//               and V rows into TMEM as soon as the current item's last scores are done, and write the
//               finished dK, dV (scaled, bf16)
//   warp 12     TMA producer: K per item (two buffers); Q_i, dO_i through a 3-stage ring
//   warp 13     issues tcgen05.mma.  K and V in TMEM are the A operands of S^T = K Q_i^T and
//               dP^T = V dO_i^T; dV += P^T dO_i and dK += dS^T Q_i read their A operand from TMEM too;
//               dQ_i = dS K reads dS from shared memory as an MN-major operand
//   warp 14     loads -lse_i * log2(e) and -delta_i with plain loads (their row offsets are not 16-byte
//               aligned) into an 8-deep ring
// TMEM columns: S^T [0,128) (half h at h*64; P^T of half h over its first 32 columns), dP^T [128,256)
// (dS^T likewise), dK [256,320), dV [320,384), dQ_i [384,448), K [448,480), V [480,512).
// dK and dV stay in TMEM for a whole item and are written once at its end.
// Registers: the block starts with 128 per thread; the compute warpgroups raise theirs and the other
// two warpgroups lower theirs (setmaxnreg) within the same total.
// The SMs of a cluster share the instruction cache behind the small per-partition one, and this kernel's
// speed depends on how much code it streams through it: changes that only add instructions (more unrolled
// variants, code that never runs) have cost up to a tenth of the time, so variants are kept few.
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

constexpr int BKV = 128;             // key rows per item
constexpr int BQ = 128;              // query rows per step
constexpr int HQ = 64;               // query rows per half step
constexpr int D = kHeadDim;
constexpr int NSTAGE = 3;
constexpr int AUX_STAGES = 8;        // ring of lse / delta rows, loaded this many steps ahead
constexpr int TILE_BYTES = 128 * D * 2;          // 16 KB
constexpr int WORK_CACHE = 64;       // work tiles of a head kept in shared memory
constexpr int MAX_CHUNKS = 64;       // runs of consecutive items a block can be given
constexpr int NUM_COMPUTE_THREADS = 256;
constexpr int DRAIN_WARP0 = 8, PRODUCER_WARP = 12, MMA_WARP = 13, AUX_WARP = 14;
constexpr int NUM_THREADS = 512;
constexpr int REGS_COMPUTE = 160, REGS_DRAIN = 88, REGS_MISC = 104;
static_assert(2 * REGS_COMPUTE + REGS_DRAIN + REGS_MISC == 4 * 128, "register budget of the block");
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t COL_ST = 0, COL_DPT = 128, COL_DK = 256, COL_DV = 320, COL_DQ = 384, COL_K = 448, COL_V = 480;

struct __align__(1024) SharedStorage {
    uint8_t k[2][TILE_BYTES];               // K of the current item and of the next one (B operand of dQ)
    uint8_t q[NSTAGE][TILE_BYTES];
    uint8_t dout[NSTAGE][TILE_BYTES];
    uint8_t ds[2][2][TILE_BYTES];           // dS^T, double buffered: [step parity][64-query half][key row][64 queries], 128B swizzle
    uint8_t dq_stage[TILE_BYTES];           // per drain warp: 32 query rows x 32 fp32 columns of dQ_i on their way to the accumulator, 128B swizzle
    float lse2[AUX_STAGES][BQ];             // -lse * log2(e); -inf for query rows outside the range
    float delta[AUX_STAGES][BQ];            // -delta
    uint64_t k_full[2], k_free[2];          // [item parity]: K tile in shared memory / no longer read
    uint64_t kv_tmem, kv_free;              // K, V rows in TMEM / no longer read
    uint64_t qdo_full[NSTAGE], q_empty[NSTAGE], aux_full[AUX_STAGES], aux_empty[AUX_STAGES];
    uint64_t s_full[2], p_full[2];            // [half of the step]
    uint64_t dq_full, dq_empty, acc_full, acc_empty;
    BwdWork work[WORK_CACHE];               // the head's work list (its first WORK_CACHE tiles)
    uint32_t tmem_base;
    int abort_flag;
    // The block's items: n_chunks runs of consecutive items; run c starts at item chunk_item[c] and holds the
    // block's items number chunk_first[c] .. chunk_first[c + 1] - 1.
    int chunk_item[MAX_CHUNKS], chunk_first[MAX_CHUNKS + 1];
    int n_chunks;
};

__device__ __forceinline__ void report_timeout(int* status, int where) {
    if (status != nullptr) {
        atomicCAS(status, 0, HMAR_ERR_DEVICE_TIMEOUT);
        atomicCAS(status + 1, 0, where);
    }
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Adds a [32 rows x 32 fp32] tile in shared memory (128-byte swizzle) to global memory at (column c0, row c1).
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* m, const void* smem_src, int c0, int c1) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

template <int N> __device__ __forceinline__ void reg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void reg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// One row of a 128-byte-swizzled [128 rows x 64 bf16] tile, as 32 packed words in row order.
__device__ __forceinline__ void load_swizzled_row(const uint8_t* tile, int r, uint32_t (&dst)[32]) {
    const uint8_t* row = tile + r * 128;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint4 val = *reinterpret_cast<const uint4*>(row + ((c ^ (r & 7)) << 4));
        dst[4 * c] = val.x; dst[4 * c + 1] = val.y; dst[4 * c + 2] = val.z; dst[4 * c + 3] = val.w;
    }
}

// The 64 query columns of one half step for the 32 key rows of one warp:
// P^T = 2^(S^T * scale * log2e - lse * log2e) and dS^T = P^T o (dP^T - delta) in fp32.
// S^T and dP^T are read 16 key rows at a time in the layout in which a thread holds, of two rows, the
// column pairs 8k + 2(t % 4) + {0, 1}: a thread then needs lse and delta of 16 columns only (eight 8-byte
// loads each, one shared-memory wavefront per load; one key row per thread would need all 64 columns as
// broadcast loads, which were the largest share of the shared-memory traffic of the LSU).  A column pair
// packs into one bf16x2: P^T goes back to TMEM over S^T and dS^T over dP^T with the matching store layout
// (the 32 packed columns start at the half's first column, which this warp has already read for these
// rows), and dS^T also goes to shared memory, 4 bytes per pair (a warp's store covers 16 bytes of 8 rows,
// 128-byte swizzle on the key row: no bank conflicts).
// MODE 2: row i of this thread's four rows sees only columns [c_lo[i], c_hi[i]) of the step.
// MODE 1: every row either sees all columns or is past the end of the key tile (c_hi[i] <= 0).  Such a row
// holds another tile's keys; its P^T and dS^T only reach rows of dV and dK that are never written, but in
// dQ = dS K it would be summed over, so the copy of dS in shared memory gets zeros there.
// MODE 0: all rows see all columns.
template <int MODE>
__device__ __forceinline__ void softmax_grad_half(uint32_t lane_base, int cbase, const float* neg_lse2, const float* neg_delta,
                                                  float sl2, const int (&c_lo)[4], const int (&c_hi)[4], uint8_t* ds_tile,
                                                  int quarter, int lane) {
    const int tq = lane & 3, tr = lane >> 2;
    // -lse * log2(e) and -delta of this thread's column pairs; the arithmetic works on pairs of columns
    // with packed fp32 instructions (half as many instructions to issue and to fetch)
    uint64_t nls[8], nde[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        nls[k] = *reinterpret_cast<const uint64_t*>(neg_lse2 + cbase + 8 * k + 2 * tq);
        nde[k] = *reinterpret_cast<const uint64_t*>(neg_delta + cbase + 8 * k + 2 * tq);
    }
    const uint64_t sl2_2 = f32x2(sl2, sl2);
#pragma unroll
    for (int hl = 0; hl < 2; ++hl) {                    // lanes 0-15, then 16-31 of the warp's quarter
        const uint32_t taddr = lane_base + ((uint32_t)(hl * 16) << 16);
        uint32_t s_buf[32], dp_buf[32];
        tmem_ld_16x256b_x8(taddr + COL_ST + cbase, s_buf);
        tmem_ld_16x256b_x8(taddr + COL_DPT + cbase, dp_buf);
        tmem_ld_wait();
        uint32_t p_pack[16], ds_pack[16];
        // key rows of this thread: quarter * 32 + hl * 16 + tr (+ 8); both have (row & 7) == tr
        uint8_t* ds_row = ds_tile + (quarter * 4 + hl * 2) * 1024 + tr * 128 + tq * 4;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
#pragma unroll
            for (int rs = 0; rs < 2; ++rs) {
                float x0, x1;
                f32x2_split(ffma2(f32x2(__uint_as_float(s_buf[4 * k + 2 * rs]), __uint_as_float(s_buf[4 * k + 2 * rs + 1])),
                                  sl2_2, nls[k]), x0, x1);
                float p0 = ex2(x0), p1 = ex2(x1);
                if (MODE == 2) {
                    const int c = cbase + 8 * k + 2 * tq, i = hl * 2 + rs;
                    p0 = (c >= c_lo[i] && c < c_hi[i]) ? p0 : 0.f;
                    p1 = (c + 1 >= c_lo[i] && c + 1 < c_hi[i]) ? p1 : 0.f;
                }
                float d0, d1;
                f32x2_split(fmul2(f32x2(p0, p1),
                                  fadd2(f32x2(__uint_as_float(dp_buf[4 * k + 2 * rs]), __uint_as_float(dp_buf[4 * k + 2 * rs + 1])),
                                        nde[k])), d0, d1);
                p_pack[2 * k + rs] = pack_bf16(p0, p1);
                ds_pack[2 * k + rs] = pack_bf16(d0, d1);
                // 8-row groups are 1024 bytes apart; 16-byte piece k of a row sits at position k ^ (row & 7)
                *reinterpret_cast<uint32_t*>(ds_row + rs * 1024 + ((k ^ tr) << 4)) =
                    (MODE == 1 && c_hi[hl * 2 + rs] <= 0) ? 0u : ds_pack[2 * k + rs];
            }
        }
        tmem_st_16x128b_x8(taddr + COL_ST + cbase, p_pack);
        tmem_st_16x128b_x8(taddr + COL_DPT + cbase, ds_pack);
    }
}

// Work items of one block.  Item g is tile g % n_work of head g / n_work; items are ordered head by
// head (a head's Q and dO tiles stay in L2 while its key tiles are processed) and every block takes a
// contiguous run of items of about the same total cost (steps plus a constant per item).
__device__ __forceinline__ int first_item_at_cost(const BwdArgs& args, long long cost) {
    const long long head = cost / args.head_cost;
    const int rem = (int)(cost - head * args.head_cost);
    int lo = 0, hi = args.n_work;                       // first tile whose starting cost is >= rem
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(&args.work[mid].cost_begin) >= rem) hi = mid; else lo = mid + 1;
    }
    return (int)head * args.n_work + lo;
}

// CHUNKED: the block's items are several runs (long sequences, see the launcher); otherwise one contiguous run,
// and the item loops compile to plain counting.
// STRIDED: the bf16 tensors have the strides given in the arguments (packed projection layouts); otherwise they are
// dense [BH, L, 64] and every address is formed with compile-time strides (the dense instantiation is the one the
// benchmarks run: the extra address arithmetic and code of the strided one cost it a tenth of its speed).
// ONE_MASK: every tile goes through the variant of the softmax-gradient code with per-element bounds, so that the
// block's code holds one variant instead of three.  It is the instantiation for side lists whose tiles are mostly
// partial or packed (L = 680: 11 % faster, a third of the instruction-cache requests of the three-variant code
// miss there); where most steps belong to full tiles the plain variant's shorter arithmetic wins (L = 2240: the
// one-variant code is 4 % slower).
template <bool CHUNKED, bool STRIDED, bool ONE_MASK>
__global__ void __launch_bounds__(NUM_THREADS, 1)
hmar_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                   const __grid_constant__ CUtensorMap map_dq, const BwdArgs args) {
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& sm = *reinterpret_cast<SharedStorage*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (args.status != nullptr && *reinterpret_cast<volatile int*>(args.status) != 0) return;

    const int L = args.L;
    const int n_work = args.n_work;

    if (threadIdx.x == 0) {
        sm.abort_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.k_full[b], 1);
            mbar_init(&sm.k_free[b], 1);
        }
        mbar_init(&sm.kv_tmem, 128);
        mbar_init(&sm.kv_free, 1);
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(&sm.qdo_full[s], 1);
            mbar_init(&sm.q_empty[s], 1);
        }
        for (int s = 0; s < AUX_STAGES; ++s) {
            mbar_init(&sm.aux_full[s], 32);
            mbar_init(&sm.aux_empty[s], NUM_COMPUTE_THREADS);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(&sm.s_full[h], 1);
            mbar_init(&sm.p_full[h], NUM_COMPUTE_THREADS / 2);
        }
        mbar_init(&sm.dq_full, 1);
        mbar_init(&sm.dq_empty, 128);
        mbar_init(&sm.acc_full, 1);
        mbar_init(&sm.acc_empty, 128);
        fence_mbar_init();
        int nch = 0, cnt = 0;
        if (!CHUNKED) {
            // one run: a contiguous stretch of the item list of about 1 / gridDim.x of the total cost
            const long long total = (long long)args.n_heads * args.head_cost;
            const int ib = first_item_at_cost(args, total * blockIdx.x / gridDim.x);
            const int ie = blockIdx.x + 1 == gridDim.x ? args.n_heads * n_work
                                                       : first_item_at_cost(args, total * (blockIdx.x + 1) / gridDim.x);
            if (ie > ib) { sm.chunk_item[0] = ib; sm.chunk_first[0] = 0; cnt = ie - ib; nch = 1; }
        } else {
            // Long sequences: every head is cut into `split` runs of equal cost, and the runs are dealt to the blocks
            // in turn.  The blocks then work on gridDim.x / split heads at a time instead of one head each, so that
            // the fp32 dQ accumulator lines of the heads in flight (and their Q, dO tiles) stay in L2.
            const int n_runs = args.n_heads * args.split;
            for (int k = blockIdx.x; k < n_runs && nch < MAX_CHUNKS; k += gridDim.x) {
                const int head = k / args.split, c = k - head * args.split;
                const int lo_cost = (int)((long long)args.head_cost * c / args.split);
                const int hi_cost = (int)((long long)args.head_cost * (c + 1) / args.split);
                const int tb = first_item_at_cost(args, lo_cost);                       // tile index: the head is 0 here
                const int te = c + 1 == args.split ? n_work : first_item_at_cost(args, hi_cost);
                if (te > tb) { sm.chunk_item[nch] = head * n_work + tb; sm.chunk_first[nch] = cnt; cnt += te - tb; ++nch; }
            }
        }
        sm.chunk_first[nch] = cnt;
        sm.n_chunks = nch;
    }
    for (int t = threadIdx.x; t < min(n_work, WORK_CACHE); t += NUM_THREADS) sm.work[t] = args.work[t];
    if (warp == MMA_WARP) {
        tmem_alloc(&sm.tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const int n_chunks = sm.n_chunks, n_items = sm.chunk_first[n_chunks];
    // item number n of this block (n rises, or steps back by one or two, from call to call: `run` follows it)
    const int first_item = sm.chunk_item[0];
    auto item_at = [&](int n, int& run) -> int {
        if (!CHUNKED) return first_item + n;
        while (n >= sm.chunk_first[run + 1] && run + 1 < n_chunks) ++run;
        while (n < sm.chunk_first[run] && run > 0) --run;
        return sm.chunk_item[run] + (n - sm.chunk_first[run]);
    };
    volatile int* abort_flag = &sm.abort_flag;

    auto get_work = [&](int g) -> BwdWork {
        const int t = g % n_work;
        return t < WORK_CACHE ? sm.work[t] : args.work[t];
    };
    auto steps_of = [](const BwdWork& w) { return (w.q_end - w.q_begin + BQ - 1) / BQ; };
    // number of query columns of half h of step i handed to the tensor core (a multiple of 16)
    auto half_cols = [](const BwdWork& w, int i, int h) {
        const int n_valid = min(BQ, w.q_end - (w.q_begin + i * BQ));
        const int n_eff = (n_valid + 15) & ~15;
        return h == 0 ? min(n_eff, HQ) : max(n_eff - HQ, 0);
    };

    if (warp >= PRODUCER_WARP) {
        reg_dec<REGS_MISC>();
        if (warp == PRODUCER_WARP) {
            // ================================================================== producer
            // The whole warp runs the control flow; one elected lane issues the copies.
            const bool leader = elect_one();
            if (leader) {
                prefetch_tensormap(&map_q);
                prefetch_tensormap(&map_k);
                prefetch_tensormap(&map_v);
                prefetch_tensormap(&map_do);
            }
            bool ok = true;
            int gs = 0;                                     // steps issued so far, over all items
            int run = 0;
            for (int item = 0; item < n_items && ok; ++item) {
                const int g = item_at(item, run);
                const int bh = g / n_work;
                const int batch = STRIDED ? bh / args.heads_per_batch : 0, head = STRIDED ? bh - batch * args.heads_per_batch : bh;
                const BwdWork w = get_work(g);
                const int n_steps = steps_of(w);
                if (item >= 2) {
                    // the buffer held K of the item before the previous one, read by its dQ products
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_free[item & 1], ((item >> 1) & 1) ^ 1, abort_flag));
                    if (!ok) { if (lane == 0) report_timeout(args.status, 0x1000); break; }
                }
                if (leader) {
                    mbar_arrive_expect_tx(&sm.k_full[item & 1], TILE_BYTES);
                    tma_load_4d(sm.k[item & 1], &map_k, &sm.k_full[item & 1], 0, w.row_begin, head, batch);
                    // the V rows are read by the drain warps a few steps from now: bring them into L2
                    tma_prefetch_4d(&map_v, 0, w.row_begin, head, batch);
                }
                __syncwarp();
                for (int i = 0; i < n_steps; ++i, ++gs) {
                    const int slot = gs % NSTAGE;
                    const int q0 = w.q_begin + i * BQ;
                    if (gs >= NSTAGE) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_empty[slot], ((gs / NSTAGE) & 1) ^ 1, abort_flag));
                        if (!ok) { if (lane == 0) report_timeout(args.status, 0x1100 + i); break; }
                    }
                    if (leader) {
                        mbar_arrive_expect_tx(&sm.qdo_full[slot], 2 * TILE_BYTES);
                        tma_load_4d(sm.q[slot], &map_q, &sm.qdo_full[slot], 0, q0, head, batch);
                        tma_load_4d(sm.dout[slot], &map_do, &sm.qdo_full[slot], 0, q0, head, batch);
                    }
                    __syncwarp();
                }
            }
            if (!ok) {
                // give the copies already issued a bounded chance to land before the block exits
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 2000000ull) { }
            }
        } else if (warp == AUX_WARP) {
            // ================================================================== lse / delta loader
            // lse and delta rows of a step go to ring slot (step count) % AUX_STAGES, several steps ahead of
            // their use (plain loads: their row offsets are not 16-byte aligned, so TMA cannot fetch them).
            bool ok = true;
            int gs = 0;
            int run = 0;
            for (int item = 0; item < n_items && ok; ++item) {
                const int g = item_at(item, run);
                const int bh = g / n_work;
                const BwdWork w = get_work(g);
                const int n_steps = steps_of(w);
                for (int i = 0; i < n_steps; ++i, ++gs) {
                    const int aslot = gs % AUX_STAGES;
                    if (gs >= AUX_STAGES) {
                        ok = __all_sync(0xffffffffu,
                                        mbar_wait(&sm.aux_empty[aslot], ((gs / AUX_STAGES) & 1) ^ 1, abort_flag));
                        if (!ok) { if (lane == 0) report_timeout(args.status, 0x1700 + i); break; }
                    }
                    const int q0 = w.q_begin + i * BQ;
                    // all loads first, then the stores: stores to shared memory in between would serialise them
                    float lv[BQ / 32], dv[BQ / 32];
#pragma unroll
                    for (int t = 0; t < BQ / 32; ++t) {
                        const int row = q0 + t * 32 + lane;
                        const bool in = row < w.q_end &&
                                        HMAR_IN_BOUNDS(row >= 0 && row < L && bh >= 0 && bh < args.n_heads, args.status, 0xB201);
                        lv[t] = in ? __ldg(args.lse + (size_t)bh * L + row) : INFINITY;
                        dv[t] = in ? __ldg(args.delta + (size_t)bh * L + row) : 0.f;
                    }
#pragma unroll
                    for (int t = 0; t < BQ / 32; ++t) {
                        sm.lse2[aslot][t * 32 + lane] = lv[t] * -1.4426950408889634f;
                        sm.delta[aslot][t * 32 + lane] = -dv[t];
                    }
                    mbar_arrive(&sm.aux_full[aslot]);
                }
            }
        } else if (warp == MMA_WARP) {
            // ================================================================== MMA issuer
            // The whole warp runs the control flow and one elected lane issues (a warp that has split into
            // one running lane and 31 parked ones issues far more slowly).  Descriptors are built once and
            // advanced by adding (byte offset >> 4) to them.
            // The tensor core's queue holds only a few products, and a product issued to an idle tensor core
            // costs about a hundred clocks before it starts, so a step is issued as two uninterrupted bursts:
            //   X_i = dV,dK of half 0 of step i, then S^T,dP^T of half 0 of step i+1
            //   Y_i = dV,dK of half 1 of step i, then S^T,dP^T of half 1 of step i+1, then dQ_i
            // each preceded by one look at the barriers it depends on (two at a time, both usually complete).
            const bool leader = elect_one();
            const uint64_t k_mn0 = smem_desc_sw128(smem_u32(sm.k[0]), 1024);    // K as MN-major B of dQ
            // the ring slots and the dS buffers are 16 KB apart: descriptor of slot s = base + s * 1024
            const uint64_t q_kd0 = smem_desc_sw128(smem_u32(sm.q[0]), 16), do_kd0 = smem_desc_sw128(smem_u32(sm.dout[0]), 16);
            const uint64_t q_mn0 = smem_desc_sw128(smem_u32(sm.q[0]), 1024), do_mn0 = smem_desc_sw128(smem_u32(sm.dout[0]), 1024);
            const uint64_t ds_mn0 = smem_desc_sw128(smem_u32(sm.ds[0][0]), TILE_BYTES);
            constexpr uint32_t idesc_acc = idesc_bf16_f32(BKV, D, false, true);    // A from TMEM, B MN-major
            constexpr uint32_t idesc_dq = idesc_bf16_f32(BQ, D, true, true);
            bool ok = true;
            int gs = 0;                                         // steps issued so far (ring slot, dQ parity)
            int ng[2] = {0, 0};                                 // gradient halves issued so far, per half
            // waits for barrier a and, if have_b, barrier b; the two first looks overlap
            auto wait2 = [&](uint64_t* a, uint32_t pa, uint64_t* b, uint32_t pb, bool have_b, int code) -> bool {
                const bool ra = mbar_try_wait(a, pa);
                const bool rb = !have_b || mbar_try_wait(b, pb);
                if (__all_sync(0xffffffffu, ra && rb)) return true;
                // a barrier seen complete is not looked at again: a look is a shared-memory round trip behind the
                // compute warps' stores, on the critical path of the step
                const bool done = (ra || mbar_wait(a, pa, abort_flag)) && (rb || mbar_wait(b, pb, abort_flag));
                if (__all_sync(0xffffffffu, done)) return true;
                if (lane == 0) report_timeout(args.status, code);
                return false;
            };
            // S^T_h = K Q_h^T,  dP^T_h = V dO_h^T : n query columns of half h, Q / dO tile in ring slot `slot`
            auto scores = [&](int h, int n, int slot) {
                const uint32_t idesc = idesc_bf16_f32(BKV, n, false, false);
                const uint64_t qd = q_kd0 + slot * 1024 + h * 512, dd = do_kd0 + slot * 1024 + h * 512;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_ts(tmem + COL_ST + h * HQ, tmem + COL_K + ks * 8, qd + ks * 2, idesc, ks > 0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_ts(tmem + COL_DPT + h * HQ, tmem + COL_V + ks * 8, dd + ks * 2, idesc, ks > 0);
                tc_commit(&sm.s_full[h]);
            };
            // dV += P_h^T dO_h,  dK += dS_h^T Q_h : n query columns of half h
            auto grads = [&](int h, int n, int slot, bool first) {
                const int nk = n / 16;
                const uint64_t dod = do_mn0 + slot * 1024 + h * 512, qd = q_mn0 + slot * 1024 + h * 512;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    if (ks < nk)
                        mma_ts(tmem + COL_DV, tmem + COL_ST + h * HQ + ks * 8, dod + ks * 128, idesc_acc, !first || (ks > 0));
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    if (ks < nk)
                        mma_ts(tmem + COL_DK, tmem + COL_DPT + h * HQ + ks * 8, qd + ks * 128, idesc_acc, !first || (ks > 0));
            };

            auto wait1 = [&](uint64_t* a, uint32_t pa, int code) -> bool {
                if (__all_sync(0xffffffffu, mbar_wait(a, pa, abort_flag))) return true;
                if (lane == 0) report_timeout(args.status, code);
                return false;
            };
            // The steps of all items form one sequence: while the compute warpgroups work on a step, the
            // tensor core gets the next step's S^T, dP^T even when that step belongs to the next item (whose
            // K, V rows the drain warps have put into TMEM by then).
            int run = 0;
            if (n_items > 0) {
                const BwdWork w0 = get_work(item_at(0, run));
                ok = wait2(&sm.kv_tmem, 0, &sm.qdo_full[0], 0, true, 0x1200);
                if (ok) {
                    tc_fence_after();
                    if (leader) {
                        scores(0, half_cols(w0, 0, 0), 0);
                        const int n1 = half_cols(w0, 0, 1);
                        if (n1 > 0) scores(1, n1, 0);
                        if (steps_of(w0) == 1 && 1 < n_items) tc_commit(&sm.kv_free);
                    }
                    __syncwarp();
                }
            }
            for (int item = 0; item < n_items && ok; ++item) {
                const BwdWork w = get_work(item_at(item, run));
                const int n_steps = steps_of(w);
                const bool next_item = item + 1 < n_items;
                const BwdWork wn = next_item ? get_work(item_at(item + 1, run)) : w;
                const int n_steps_next = steps_of(wn);
                const uint64_t k_mn = k_mn0 + (item & 1) * 1024;
                for (int i = 0; i < n_steps && ok; ++i, ++gs) {
                    const int slot = gs % NSTAGE, slot_next = (gs + 1) % NSTAGE;
                    const bool more = i + 1 < n_steps;          // the item has another step
                    const bool cross = !more && next_item;      // the next step is the next item's first
                    const bool any_next = more || cross;
                    const int n0 = half_cols(w, i, 0), n1 = half_cols(w, i, 1);
                    const int m0 = more ? half_cols(w, i + 1, 0) : cross ? half_cols(wn, 0, 0) : 0;
                    const int m1 = more ? half_cols(w, i + 1, 1) : cross ? half_cols(wn, 0, 1) : 0;
                    // the next step is the last one that reads its item's K, V rows in TMEM, and another item follows
                    const bool frees_kv = more ? (i + 2 == n_steps && next_item) : (cross && n_steps_next == 1 && item + 2 < n_items);
                    // ---- burst X: needs P^T, dS^T of half 0 and the next step's Q / dO tile
                    ok = wait2(&sm.p_full[0], ng[0] & 1, &sm.qdo_full[slot_next], ((gs + 1) / NSTAGE) & 1, any_next, 0x1400 + i);
                    if (!ok) break;
                    ++ng[0];
                    if (cross) {                                // K, V of the next item in TMEM
                        ok = wait1(&sm.kv_tmem, (item + 1) & 1, 0x1200);
                        if (!ok) break;
                    }
                    if (i == 0 && item > 0) {                   // dK, dV of the previous item read out
                        ok = wait1(&sm.acc_empty, (item - 1) & 1, 0x1B00);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    if (leader) {
                        grads(0, n0, slot, i == 0);
                        if (m0 > 0) scores(0, m0, slot_next);
                    }
                    __syncwarp();
                    // ---- burst Y: needs P^T, dS^T of half 1 (if the step has one) and dQ of the previous
                    // step drained from TMEM
                    if (n1 > 0) {
                        ok = wait2(&sm.p_full[1], ng[1] & 1, &sm.dq_empty, (gs - 1) & 1, gs > 0, 0x1800 + i);
                        ++ng[1];
                    } else if (gs > 0) {
                        ok = wait2(&sm.dq_empty, (gs - 1) & 1, nullptr, 0, false, 0x1800 + i);
                    }
                    if (!ok) break;
                    if (i == 0) {                               // K of this item in shared memory (B operand of dQ)
                        ok = wait1(&sm.k_full[item & 1], (item >> 1) & 1, 0x1C00);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    if (leader) {
                        if (n1 > 0) grads(1, n1, slot, false);
                        tc_commit(&sm.q_empty[slot]);           // Q_i, dO_i are not read again
                        if (!more) tc_commit(&sm.acc_full);     // dK, dV of the item are complete
                        // the next scores of half 1 go first: the compute warpgroup is waiting for them, dQ_i
                        // is not needed before the drain warps get to it
                        if (m1 > 0) scores(1, m1, slot_next);
                        if (frees_kv) tc_commit(&sm.kv_free);
                        // dQ_i = dS K over both halves: A = dS (queries x keys) read as an MN-major operand.  When
                        // the step has no second half its rows are stale data and are never drained.
                        const uint64_t dsd = ds_mn0 + (gs & 1) * 2048;
#pragma unroll
                        for (int ks = 0; ks < BKV / 16; ++ks)
                            mma_ss(tmem + COL_DQ, dsd + ks * 128, k_mn + ks * 128, idesc_dq, ks > 0);
                        tc_commit(&sm.dq_full);
                        if (!more) tc_commit(&sm.k_free[item & 1]);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp >= DRAIN_WARP0) {
        // ================================================================== dQ drain
        // One query row per thread, and every warp on its own: dQ_i leaves TMEM 32 columns at a time, is
        // staged in the warp's 4 KB of shared memory and added to the fp32 accumulator by one bulk tensor
        // reduction per 32 x 32 piece (whole cache lines, issued by the copy engine; per-thread reductions
        // would be 16-byte pieces of 32 different lines).  Rows past the end of the query range are staged
        // as zeros.
        reg_dec<REGS_DRAIN>();
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        uint8_t* stage = sm.dq_stage + quarter * 4096;
        uint8_t* stage_row = stage + (lane >> 3) * 1024 + (lane & 7) * 128;
        if (lane == 0) prefetch_tensormap(&map_dq);
        uint32_t buf[32];
        bool ok = true;
        int gs = 0;
        auto wait1 = [&](uint64_t* a, uint32_t pa, int code) -> bool {
            if (__all_sync(0xffffffffu, mbar_wait(a, pa, abort_flag))) return true;
            if (lane == 0) report_timeout(args.status, code);
            return false;
        };
        // K and V rows of item gc (the block's item number `item`) to TMEM, one key row per thread: the A
        // operands of S^T = K Q^T and dP^T = V dO^T.  The V row comes straight from global memory and waits
        // in registers until the previous item's last scores have been computed; the K row is read from the
        // tile that the copy engine has put into shared memory for the dQ products.  Rows past the end of
        // the sequence are zeros.
        auto copy_kv = [&](int gc, int item, bool wait_free) -> bool {
            const BwdWork wc = get_work(gc);
            const int row = wc.row_begin + r;
            const uint4* vsrc;
            if (STRIDED) {
                const int cbh = gc / n_work, cb = cbh / args.heads_per_batch, ch = cbh - cb * args.heads_per_batch;
                vsrc = reinterpret_cast<const uint4*>(args.v + cb * args.in_batch + ch * args.in_head + (long long)row * args.in_row);
            } else {
                vsrc = reinterpret_cast<const uint4*>(args.v + ((size_t)(gc / n_work) * L + row) * D);
            }
            const long long v_off = reinterpret_cast<const __nv_bfloat16*>(vsrc) - args.v;
            const bool v_in = row < L && HMAR_IN_BOUNDS(v_off >= 0 && v_off + D <= args.in_extent, args.status, 0xB202);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 val = v_in ? __ldg(vsrc + c) : make_uint4(0u, 0u, 0u, 0u);
                buf[4 * c] = val.x; buf[4 * c + 1] = val.y; buf[4 * c + 2] = val.z; buf[4 * c + 3] = val.w;
            }
            if (wait_free) {
                if (!wait1(&sm.kv_free, (item - 1) & 1, 0x1900)) return false;
                tc_fence_after();
            }
            tmem_st32(lane_base + COL_V, buf);
            if (!wait1(&sm.k_full[item & 1], (item >> 1) & 1, 0x1980)) return false;
            load_swizzled_row(sm.k[item & 1], r, buf);
            tmem_st32(lane_base + COL_K, buf);
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&sm.kv_tmem);
            return true;
        };
        int run = 0;
        if (n_items > 0) {
            ok = copy_kv(item_at(0, run), 0, false);
            if (ok && steps_of(get_work(item_at(0, run))) == 1 && 1 < n_items) ok = copy_kv(item_at(1, run), 1, true);
        }
        for (int item = 0; item < n_items && ok; ++item) {
            const int g = item_at(item, run);
            const int bh = g / n_work;
            const BwdWork w = get_work(g);
            const int n_steps = steps_of(w);
            const bool next_item = item + 1 < n_items;
            const int n_steps_next = next_item ? steps_of(get_work(item_at(item + 1, run))) : 0;
            for (int i = 0; i < n_steps; ++i, ++gs) {
                const bool more = i + 1 < n_steps;
                // the next step is the last one of its item and another item follows: that item's K, V rows
                // go to TMEM as soon as the next step's scores are complete
                if (more ? (i + 2 == n_steps && next_item) : (next_item && n_steps_next == 1 && item + 2 < n_items)) {
                    const int nc = more ? item + 1 : item + 2;
                    ok = copy_kv(item_at(nc, run), nc, true);
                    if (!ok) break;
                }
                if (!more) {
                    // ---- end of the item: dK and dV, one key row per thread, scaled and rounded to bf16
                    ok = wait1(&sm.acc_full, item & 1, 0x1A00);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int part = 0; part < 4; ++part) {
                        tmem_ld32(lane_base + (part < 2 ? COL_DK : COL_DV) + (part & 1) * 32, buf);
                        tmem_ld_wait();
                        if (part == 3) {
                            tc_fence_before();
                            mbar_arrive(&sm.acc_empty);         // the next item's products may overwrite dK / dV
                        }
                        if (r < w.row_count) {
                            const float mul = part < 2 ? args.softmax_scale : 1.f;
                            __nv_bfloat16* base = part < 2 ? args.dk : args.dv;
                            uint4* dst;
                            if (STRIDED) {
                                const int ob = bh / args.heads_per_batch, oh = bh - ob * args.heads_per_batch;
                                dst = reinterpret_cast<uint4*>(base + ob * args.g_batch + oh * args.g_head +
                                                               (long long)(w.row_begin + r) * args.g_row + (part & 1) * 32);
                            } else {
                                dst = reinterpret_cast<uint4*>(base + ((size_t)bh * L + w.row_begin + r) * D + (part & 1) * 32);
                            }
                            const long long g_off = reinterpret_cast<__nv_bfloat16*>(dst) - base;
                            const bool g_in = HMAR_IN_BOUNDS(g_off >= 0 && g_off + 32 <= args.g_extent, args.status, 0xB203);
#pragma unroll
                            for (int t = 0; t < 4 && g_in; ++t) {
                                uint4 o;
                                o.x = pack_bf16(__uint_as_float(buf[8 * t + 0]) * mul, __uint_as_float(buf[8 * t + 1]) * mul);
                                o.y = pack_bf16(__uint_as_float(buf[8 * t + 2]) * mul, __uint_as_float(buf[8 * t + 3]) * mul);
                                o.z = pack_bf16(__uint_as_float(buf[8 * t + 4]) * mul, __uint_as_float(buf[8 * t + 5]) * mul);
                                o.w = pack_bf16(__uint_as_float(buf[8 * t + 6]) * mul, __uint_as_float(buf[8 * t + 7]) * mul);
                                dst[t] = o;
                            }
                        }
                    }
                }
                if (!__all_sync(0xffffffffu, mbar_wait(&sm.dq_full, gs & 1, abort_flag))) {
                    if (lane == 0) report_timeout(args.status, 0x1600 + i);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const int q0 = w.q_begin + i * BQ;
                const bool row_in = r < min(BQ, w.q_end - q0);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    tmem_ld32(lane_base + COL_DQ + c * 32, buf);
                    tmem_ld_wait();
                    if (c == 1) {
                        tc_fence_before();
                        mbar_arrive(&sm.dq_empty);
                    }
                    // the previous piece must have been read out of the staging buffer
                    if (lane == 0) bulk_wait_read_all();
                    __syncwarp();
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const uint4 val = row_in ? make_uint4(buf[4 * t], buf[4 * t + 1], buf[4 * t + 2], buf[4 * t + 3])
                                                 : make_uint4(0u, 0u, 0u, 0u);
                        *reinterpret_cast<uint4*>(stage_row + ((t ^ (lane & 7)) << 4)) = val;
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_reduce_add_2d(&map_dq, stage, c * 32, bh * L + q0 + quarter * 32);
                        bulk_commit_group();
                    }
                }
            }
        }
        if (lane == 0) bulk_wait_all();         // the staging buffer must outlive the last reduction's read
    } else {
        // ================================================================== compute warpgroups
        reg_inc<REGS_COMPUTE>();
        const int quarter = warp & 3;
        const int h = warp >> 2;                            // the half of every step this warpgroup owns
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const float sl2 = args.scale_log2;
        bool ok = true;
        int gs = 0;                                         // steps seen so far (aux ring, dS buffer parity)
        int nsh = 0;                                        // non-empty halves of this warpgroup seen so far

        int run = 0;
        for (int item = 0; item < n_items && ok; ++item) {
            const BwdWork w = get_work(item_at(item, run));
            const int n_steps = steps_of(w);
            // the four key rows this thread works on in the softmax-gradient layout, and the queries that may see them
            const bool tile_masked = ONE_MASK || (!w.uniform) || (w.row_count < BKV);
            const bool rows_only = !ONE_MASK && w.uniform != 0;   // only rows past the end of the tile are hidden
            int qlo[4], qhi[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int rr = quarter * 32 + (i >> 1) * 16 + (lane >> 2) + (i & 1) * 8;
                qlo[i] = w.q_begin; qhi[i] = w.q_end;
                if (tile_masked) {
                    if (rr >= w.row_count) { qlo[i] = 0; qhi[i] = 0; }
                    else if (!w.uniform) {
                        const int sc = scale_of_row(args.st, w.row_begin + rr);
                        qlo[i] = args.st.start[first_query_scale(args.st.window, sc)];
                        qhi[i] = args.st.start[last_query_scale(args.st.window, sc, args.st.n_scales) + 1];
                    }
                }
            }

            for (int i = 0; i < n_steps && ok; ++i, ++gs) {
                const int q0 = w.q_begin + i * BQ;
                const int n_valid = min(BQ, w.q_end - q0);
                const int n_cols = half_cols(w, i, h);
                const int cbase = h * HQ;                   // first query column of this half inside the step

                const int aslot = gs % AUX_STAGES;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.aux_full[aslot], (gs / AUX_STAGES) & 1, abort_flag));
                if (!ok) { if (lane == 0) report_timeout(args.status, 0x1500 + i); break; }

                if (n_cols > 0) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[h], nsh & 1, abort_flag));
                    if (!ok) { if (lane == 0) report_timeout(args.status, 0x1580 + i); break; }
                    ++nsh;
                    tc_fence_after();
                    // tiles whose rows all see every column skip the mask code
                    if (tile_masked) {
                        int c_lo[4], c_hi[4];               // visible query columns of the four rows in this step
#pragma unroll
                        for (int r4 = 0; r4 < 4; ++r4) {
                            c_lo[r4] = max(qlo[r4] - q0, 0);
                            c_hi[r4] = min(qhi[r4] - q0, n_valid);
                        }
                        if (rows_only)
                            softmax_grad_half<1>(lane_base, cbase, sm.lse2[aslot], sm.delta[aslot], sl2, c_lo, c_hi,
                                                 sm.ds[gs & 1][h], quarter, lane);
                        else
                            softmax_grad_half<2>(lane_base, cbase, sm.lse2[aslot], sm.delta[aslot], sl2, c_lo, c_hi,
                                                 sm.ds[gs & 1][h], quarter, lane);
                    } else {
                        const int none[4] = {0, 0, 0, 0};
                        softmax_grad_half<0>(lane_base, cbase, sm.lse2[aslot], sm.delta[aslot], sl2, none, none,
                                                 sm.ds[gs & 1][h], quarter, lane);
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    fence_proxy_async_smem();
                    mbar_arrive(&sm.p_full[h]);
                }
                mbar_arrive(&sm.aux_empty[aslot]);      // this thread is done with the step's lse / delta
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// Offset (elements) of row `row` (= bh * L + l) of a strided bf16 tensor.
struct RowLayout {
    int L, heads_per_batch;
    long long row, head, batch;
    template <bool STRIDED>
    __device__ __forceinline__ long long offset(size_t r) const {
        if (!STRIDED) return (long long)r * D;
        const int bh = (int)(r / (size_t)L), l = (int)(r - (size_t)bh * L);
        const int b = bh / heads_per_batch, h = bh - b * heads_per_batch;
        return b * batch + h * head + l * row;
    }
};

// delta_i = sum_d dO_id * O_id  (one warp per 4 rows: 8 lanes x 16 bytes cover a row).  The same pass
// clears the fp32 dQ accumulator (32 bytes per lane), which saves a separate pass over it.
template <bool STRIDED>
__global__ void __launch_bounds__(256)
hmar_bwd_delta_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                      float* __restrict__ delta, float* __restrict__ dq_acc, size_t n_rows, const RowLayout lay) {
    const size_t row = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3;
    const int part = threadIdx.x & 7;
    float acc = 0.f;
    if (row < n_rows) {
        float4* z = reinterpret_cast<float4*>(dq_acc + row * D + part * 8);
        z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        const long long off = lay.template offset<STRIDED>(row) + part * 8;
        const uint4 a = *reinterpret_cast<const uint4*>(out + off);
        const uint4 b = *reinterpret_cast<const uint4*>(dout + off);
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
template <bool STRIDED>
__global__ void __launch_bounds__(256)
hmar_bwd_dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, float scale, size_t n8,
                           const RowLayout lay) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n8) return;
    const float4 a = reinterpret_cast<const float4*>(acc)[2 * idx];
    const float4 b = reinterpret_cast<const float4*>(acc)[2 * idx + 1];
    uint4 o;
    o.x = pack_bf16(a.x * scale, a.y * scale);
    o.y = pack_bf16(a.z * scale, a.w * scale);
    o.z = pack_bf16(b.x * scale, b.y * scale);
    o.w = pack_bf16(b.z * scale, b.w * scale);
    *reinterpret_cast<uint4*>(dq + lay.template offset<STRIDED>(idx >> 3) + (idx & 7) * 8) = o;
}

}  // namespace

// Number of SMs of the current device (one persistent block each), looked up once per device.
static int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 1;
        cached[dev] = n;
    }
    return cached[dev];
}

// Side lists with fewer than this share (in thousandths) of their steps in full tiles run the one-variant
// instantiation (L = 680 has 42 %, L = 2240 has 82 %).
constexpr int kOneMaskBelowPermille = 600;

template <bool STRIDED>
static cudaError_t launch_bwd_tc_layout(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& dout_map,
                                        const CUtensorMap& dq_acc_map, const BwdArgs& args, const __nv_bfloat16* out,
                                        const __nv_bfloat16* dout, __nv_bfloat16* dq, int BH, cudaStream_t stream) {
    const size_t smem = sizeof(SharedStorage) + 1024;
    cudaError_t e = cudaFuncSetAttribute(hmar_bwd_tc_kernel<false, STRIDED, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hmar_bwd_tc_kernel<true, STRIDED, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(hmar_bwd_tc_kernel<false, STRIDED, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const size_t n_rows = (size_t)BH * args.L;
    {
        KernelTimer timer("hmar_bwd_delta_kernel", stream);
        const RowLayout lay{args.L, args.heads_per_batch, args.od_row, args.od_head, args.od_batch};
        hmar_bwd_delta_kernel<STRIDED><<<(unsigned)((n_rows * 8 + 255) / 256), 256, 0, stream>>>(out, dout, args.delta_w, args.dq_acc, n_rows, lay);
    }
    {
        KernelTimer timer("hmar_bwd_tc_kernel", stream);
        const long long items = (long long)BH * args.n_work;
        const unsigned grid = (unsigned)(items < sm_count() ? items : sm_count());
        BwdArgs a = args;
        // Long sequences only (measured: at L = 2240 the kernel does not care how many heads are in flight, at
        // L = 9451 it is a fifth slower with one head per block): 8 runs per head, fewer if a block would get
        // more runs than its table holds.
        a.split = 0;
        if (args.L >= 4096 && (unsigned)BH >= grid) {       // (with fewer heads than blocks the runs would not balance)
            a.split = 8;
            while (a.split > 0 && ((long long)BH * a.split + grid - 1) / grid > MAX_CHUNKS) a.split >>= 1;
        }
        if (a.split > 0)
            hmar_bwd_tc_kernel<true, STRIDED, false><<<grid, NUM_THREADS, smem, stream>>>(q, k, v, dout_map, dq_acc_map, a);
        else if (args.plain_permille < kOneMaskBelowPermille)
            hmar_bwd_tc_kernel<false, STRIDED, true><<<grid, NUM_THREADS, smem, stream>>>(q, k, v, dout_map, dq_acc_map, a);
        else
            hmar_bwd_tc_kernel<false, STRIDED, false><<<grid, NUM_THREADS, smem, stream>>>(q, k, v, dout_map, dq_acc_map, a);
    }
    const size_t n8 = n_rows * D / 8;
    {
        KernelTimer timer("hmar_bwd_dq_convert_kernel", stream);
        const RowLayout lay{args.L, args.heads_per_batch, args.g_row, args.g_head, args.g_batch};
        hmar_bwd_dq_convert_kernel<STRIDED><<<(unsigned)((n8 + 255) / 256), 256, 0, stream>>>(args.dq_acc, dq, args.softmax_scale, n8, lay);
    }
    count_launch(3);
    return cudaGetLastError();
}

cudaError_t launch_bwd_tc(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& dout_map,
                          const CUtensorMap& dq_acc_map, const BwdArgs& args, const __nv_bfloat16* out, const __nv_bfloat16* dout,
                          __nv_bfloat16* dq, int BH, cudaStream_t stream) {
    // dense [BH, L, 64] everywhere: the instantiation with compile-time strides
    const long long row = D, head = (long long)args.L * D;
    const bool dense = args.in_row == row && args.od_row == row && args.g_row == row && args.in_head == head &&
                       args.od_head == head && args.g_head == head &&
                       (args.heads_per_batch == BH || (args.in_batch == args.heads_per_batch * head &&
                                                       args.od_batch == args.in_batch && args.g_batch == args.in_batch));
    return dense ? launch_bwd_tc_layout<false>(q, k, v, dout_map, dq_acc_map, args, out, dout, dq, BH, stream)
                 : launch_bwd_tc_layout<true>(q, k, v, dout_map, dq_acc_map, args, out, dout, dq, BH, stream);
}

}  // namespace hmar
