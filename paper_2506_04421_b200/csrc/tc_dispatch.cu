// Host-side dispatch of the bf16 entry points to the tensor-core kernels: the per-schedule plan
// cache (device work lists) and the TMA tensor maps.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <vector>

#include "launchers.h"
#include "tc_common.h"
#include "tc_launchers.h"

namespace hmar {

typedef __nv_bfloat16 bf16;

// ------------------------------------------------------------------------------------------------
// cuTensorMapEncodeTiled is fetched through the runtime so the library has no link-time dependency
// on libcuda (it must load on machines without a driver, where only host-side calls are used).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    });
    return fn;
}

// 4-D map (64 elements, rows, heads, batches) with the strides of the tensor in elements; boxes of `box_rows`
// rows of one head.  Serves the contiguous [B, H, rows, 64] layout and a packed [B, rows, 3, H, 64] one alike.
constexpr int kFwdKeyRows = 64;      // key rows per tile of the forward kernel (its query tiles are kTileRows high)
static bool make_rows_map4(CUtensorMap* map, const void* base, int batches, int heads, int rows, long long row_stride,
                           long long head_stride, long long batch_stride, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batches};
    const cuuint64_t strides[3] = {(cuuint64_t)row_stride * 2, (cuuint64_t)head_stride * 2, (cuuint64_t)batch_stride * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kHeadDim, (cuuint32_t)box_rows, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the fp32 dQ accumulator seen as [rows, 64]: boxes of 32 rows x 32 columns (128 bytes,
// 128-byte swizzle), the unit in which a warp of the backward kernel adds dQ pieces to it.
static bool make_acc_map(CUtensorMap* map, const float* base, size_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ------------------------------------------------------------------------------------------------
// Plan cache: one entry per (device, side length list).
struct Plan {
    FwdWork* fwd_work = nullptr;     // one allocation: forward tiles, then backward tiles
    BwdWork* bwd_work = nullptr;
    int n_fwd = 0;
    int n_bwd = 0;
    int bwd_head_cost = 0;
    int bwd_plain_permille = 1000;
    int zero_begin = 0, zero_end = 0;   // key rows of a head that no query sees: their dK, dV are zeros
};

struct PlanKey {
    int device;
    std::vector<int> starts;
    bool operator<(const PlanKey& o) const {
        return device != o.device ? device < o.device : starts < o.starts;
    }
};

static std::mutex g_plan_mu;
static std::map<PlanKey, Plan> g_plans;

// The backward's work list of one head: a tile of 128 key rows each, with the query range that may see it.
// Key tiles that no query sees (the last scale under HMAR_WINDOW_PREV) are not work items: the backward
// kernel's pipeline wants at least one step per item.  Their rows are one stretch at the end of the head,
// returned in [zero_begin, zero_end) (their dK, dV are zeros).
static std::vector<BwdWork> make_bwd_work(const ScaleTable& st, int& zero_begin, int& zero_end) {
    std::vector<Tile> btiles = build_tiles(st, 1);
    std::vector<Tile> live;
    zero_begin = zero_end = 0;
    for (const Tile& t : btiles) {
        if (t.partner_end > t.partner_begin) { live.push_back(t); continue; }
        if (zero_end == zero_begin) { zero_begin = t.row_begin; zero_end = t.row_begin + t.row_count; }
        zero_begin = std::min(zero_begin, (int)t.row_begin);
        zero_end = std::max(zero_end, (int)(t.row_begin + t.row_count));
    }
    std::vector<BwdWork> bwork(live.size());
    for (size_t i = 0; i < live.size(); ++i) {
        bwork[i] = BwdWork{};
        bwork[i].row_begin = live[i].row_begin;
        bwork[i].row_count = live[i].row_count;
        bwork[i].q_begin = live[i].partner_begin;
        bwork[i].q_end = live[i].partner_end;
        bwork[i].uniform = live[i].uniform;
    }
    return bwork;
}

int tc_bwd_full_tile_permille(const ScaleTable& st) {
    int zb = 0, ze = 0;
    std::vector<BwdWork> bwork = make_bwd_work(st, zb, ze);
    return bwd_plain_permille(bwork.data(), (int)bwork.size());
}

static const Plan* get_plan(const ScaleTable& st) {
    PlanKey key;
    if (cudaGetDevice(&key.device) != cudaSuccess) return nullptr;
    key.starts.assign(st.start, st.start + st.n_scales + 1);
    key.starts.push_back(st.window);
    std::lock_guard<std::mutex> lock(g_plan_mu);
    auto it = g_plans.find(key);
    if (it != g_plans.end()) return &it->second;

    std::vector<Tile> tiles = build_tiles(st, 0);
    std::vector<FwdWork> work(tiles.size());
    for (size_t i = 0; i < tiles.size(); ++i) {
        work[i].row_begin = tiles[i].row_begin;
        work[i].row_count = tiles[i].row_count;
        work[i].s0_begin = tiles[i].partner_begin;
        work[i].s0_end = tiles[i].partner_end;
        work[i].s1_begin = work[i].s1_end = 0;
        work[i].uniform = tiles[i].uniform;
        work[i].pad = 0;
    }
    Plan plan;
    std::vector<BwdWork> bwork = make_bwd_work(st, plan.zero_begin, plan.zero_end);
    static_assert(sizeof(FwdWork) == sizeof(BwdWork), "work tiles share one allocation");
    plan.bwd_head_cost = bwd_fill_costs(bwork.data(), (int)bwork.size());
    plan.bwd_plain_permille = bwd_plain_permille(bwork.data(), (int)bwork.size());
    plan.n_fwd = (int)work.size();
    plan.n_bwd = (int)bwork.size();
    const size_t fwd_bytes = work.size() * sizeof(FwdWork), bwd_bytes = bwork.size() * sizeof(BwdWork);
    cudaStream_t s = nullptr;
    bool ok = cudaMalloc(&plan.fwd_work, fwd_bytes + bwd_bytes) == cudaSuccess &&
              cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) == cudaSuccess &&
              cudaMemcpyAsync(plan.fwd_work, work.data(), fwd_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess &&
              cudaMemcpyAsync(reinterpret_cast<char*>(plan.fwd_work) + fwd_bytes, bwork.data(), bwd_bytes,
                              cudaMemcpyHostToDevice, s) == cudaSuccess &&
              cudaStreamSynchronize(s) == cudaSuccess;
    plan.bwd_work = reinterpret_cast<BwdWork*>(reinterpret_cast<char*>(plan.fwd_work) + fwd_bytes);
    if (s != nullptr) cudaStreamDestroy(s);
    if (!ok) {
        cudaGetLastError();
        if (plan.fwd_work) cudaFree(plan.fwd_work);
        return nullptr;
    }
    return &(g_plans[key] = plan);
}

void tc_release_plans() {
    std::lock_guard<std::mutex> lock(g_plan_mu);
    int current = 0;
    const bool have_dev = cudaGetDevice(&current) == cudaSuccess;
    for (auto& kv : g_plans) {
        if (have_dev) cudaSetDevice(kv.first.device);
        if (kv.second.fwd_work) cudaFree(kv.second.fwd_work);
    }
    if (have_dev) cudaSetDevice(current);
    g_plans.clear();
    cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Forward on tensors whose layout is given by strides (elements): q, k, v share one layout, out has its own.
static int tc_fwd_strided(const bf16* q, const bf16* k, const bf16* v, bf16* out, float* lse, int B, int H,
                          const ScaleTable& st, float scale, long long in_row, long long in_head, long long in_batch,
                          long long out_row, long long out_head, long long out_batch, int* status, cudaStream_t stream) {
    const Plan* plan = get_plan(st);
    if (plan == nullptr) return HMAR_ERR_CUDA;
    const int L = st.start[st.n_scales];
    CUtensorMap mq, mk, mv;
    if (!make_rows_map4(&mq, q, B, H, L, in_row, in_head, in_batch, kTileRows) ||
        !make_rows_map4(&mk, k, B, H, L, in_row, in_head, in_batch, kFwdKeyRows) ||
        !make_rows_map4(&mv, v, B, H, L, in_row, in_head, in_batch, kFwdKeyRows))
        return HMAR_ERR_CUDA;
    FwdArgs a{};
    a.work = plan->fwd_work;
    a.n_work = plan->n_fwd;
    a.n_q_rows = L;
    a.heads_per_batch = H;
    a.out_row_stride = out_row;
    a.out_head_stride = out_head;
    a.out_batch_stride = out_batch;
    a.out_extent = (B - 1) * out_batch + (H - 1) * out_head + (long long)(L - 1) * out_row + kHeadDim;
    a.lse_extent = (long long)B * H * L;
    a.n0 = L;
    a.n1 = 0;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.out = out;
    a.lse = lse;
    a.status = status;
    a.st = st;
    return launch_fwd_tc(mq, mk, mv, mk, mv, a, B * H, stream) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

// Contiguous [B*H, L, 64] tensors: one "batch" of BH heads.
int tc_fwd(const bf16* q, const bf16* k, const bf16* v, bf16* out, float* lse, int BH, const ScaleTable& st,
           float scale, int* status, cudaStream_t stream) {
    const long long L = st.start[st.n_scales];
    return tc_fwd_strided(q, k, v, out, lse, 1, BH, st, scale, kHeadDim, L * kHeadDim, (long long)BH * L * kHeadDim,
                          kHeadDim, L * kHeadDim, (long long)BH * L * kHeadDim, status, stream);
}

// Packed projection output qkv [B, L, 3, H, 64] (q, k, v of a token side by side), out [B, L, H, 64].
int tc_fwd_packed(const bf16* qkv, bf16* out, float* lse, int B, int H, const ScaleTable& st, float scale, int* status,
                  cudaStream_t stream) {
    const long long L = st.start[st.n_scales], HD = (long long)H * kHeadDim;
    return tc_fwd_strided(qkv, qkv + HD, qkv + 2 * HD, out, lse, B, H, st, scale, 3 * HD, kHeadDim, L * 3 * HD,
                          HD, kHeadDim, L * HD, status, stream);
}

int tc_scale_step(const bf16* q, const bf16* k_prev, const bf16* v_prev, const bf16* k_cur, const bf16* v_cur,
                  bf16* out, float* lse, int BH, int n_prev, int n_cur, const StepStrides& st, float scale, int* status,
                  cudaStream_t stream) {
    if (step_small_applies(n_prev, n_cur))
        return step_small(q, k_prev, v_prev, k_cur, v_cur, out, lse, BH, n_prev, n_cur, st.q, st.kv_prev, st.kv_cur, st.out,
                          scale, status, stream);
    CUtensorMap mq, mk0, mv0, mk1, mv1;
    auto rows_map = [&](CUtensorMap* m, const bf16* base, int rows, long long head_stride, int box_rows) {
        return make_rows_map4(m, base, 1, BH, rows, kHeadDim, head_stride, (long long)BH * head_stride, box_rows);
    };
    if (!rows_map(&mq, q, n_cur, st.q, kTileRows) || !rows_map(&mk1, k_cur, n_cur, st.kv_cur, kFwdKeyRows) ||
        !rows_map(&mv1, v_cur, n_cur, st.kv_cur, kFwdKeyRows))
        return HMAR_ERR_CUDA;
    if (n_prev > 0) {
        if (!rows_map(&mk0, k_prev, n_prev, st.kv_prev, kFwdKeyRows) || !rows_map(&mv0, v_prev, n_prev, st.kv_prev, kFwdKeyRows))
            return HMAR_ERR_CUDA;
    } else {
        mk0 = mk1;
        mv0 = mv1;
    }
    FwdArgs a{};
    a.work = nullptr;
    a.n_work = (n_cur + kTileRows - 1) / kTileRows;
    a.n_q_rows = n_cur;
    a.heads_per_batch = BH;
    a.out_row_stride = kHeadDim;
    a.out_head_stride = st.out;
    a.out_batch_stride = (long long)BH * st.out;
    a.out_extent = (long long)(BH - 1) * st.out + (long long)n_cur * kHeadDim;
    a.lse_extent = (long long)BH * n_cur;
    a.n0 = n_prev;
    a.n1 = n_cur;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.out = out;
    a.lse = lse;
    a.status = status;
    a.st.n_scales = 0;
    a.st.window = HMAR_WINDOW_MARKOV;
    return launch_fwd_tc(mq, mk0, mv0, mk1, mv1, a, BH, stream) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

// Backward on tensors whose layout is given by strides (elements): q, k, v share one layout, out and dout another,
// dq, dk, dv a third.
struct Strides3 { long long row, head, batch; };
static int tc_bwd_strided(const bf16* q, const bf16* k, const bf16* v, const bf16* out, const float* lse, const bf16* dout,
                          bf16* dq, bf16* dk, bf16* dv, float* delta, float* dq_acc, int B, int H, const ScaleTable& st,
                          float scale, Strides3 in, Strides3 od, Strides3 g, int* status, cudaStream_t stream) {
    const Plan* plan = get_plan(st);
    if (plan == nullptr) return HMAR_ERR_CUDA;
    const int L = st.start[st.n_scales];
    const int BH = B * H;
    CUtensorMap mq, mk, mv, mdo, macc;
    if (!make_rows_map4(&mq, q, B, H, L, in.row, in.head, in.batch, kTileRows) ||
        !make_rows_map4(&mk, k, B, H, L, in.row, in.head, in.batch, kTileRows) ||
        !make_rows_map4(&mv, v, B, H, L, in.row, in.head, in.batch, kTileRows) ||
        !make_rows_map4(&mdo, dout, B, H, L, od.row, od.head, od.batch, kTileRows) || !make_acc_map(&macc, dq_acc, (size_t)BH * L))
        return HMAR_ERR_CUDA;
    BwdArgs a{};
    a.work = plan->bwd_work;
    a.n_work = plan->n_bwd;
    a.n_heads = BH;
    a.head_cost = plan->bwd_head_cost;
    a.plain_permille = plan->bwd_plain_permille;
    a.L = L;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.softmax_scale = scale;
    a.lse = lse;
    a.delta = delta;
    a.delta_w = delta;
    a.dq_acc = dq_acc;
    a.heads_per_batch = H;
    a.in_row = in.row; a.in_head = in.head; a.in_batch = in.batch;
    a.od_row = od.row; a.od_head = od.head; a.od_batch = od.batch;
    a.g_row = g.row; a.g_head = g.head; a.g_batch = g.batch;
    a.in_extent = (B - 1) * in.batch + (H - 1) * in.head + (long long)(L - 1) * in.row + kHeadDim;
    a.g_extent = (B - 1) * g.batch + (H - 1) * g.head + (long long)(L - 1) * g.row + kHeadDim;
    a.v = v;
    a.dk = dk;
    a.dv = dv;
    a.status = status;
    a.st = st;
    if (plan->zero_end > plan->zero_begin) {
        // rows of keys that no query sees: zeros in dK and dV.  Dense heads [BH, L, 64] take one strided fill per
        // tensor; other layouts one per head.
        const size_t rows = (size_t)(plan->zero_end - plan->zero_begin);
        if (g.row == kHeadDim && g.head == (long long)L * kHeadDim && (B == 1 || g.batch == (long long)H * g.head)) {
            const size_t pitch = (size_t)L * kHeadDim * sizeof(bf16), width = rows * kHeadDim * sizeof(bf16);
            if (cudaMemset2DAsync(dk + (size_t)plan->zero_begin * kHeadDim, pitch, 0, width, BH, stream) != cudaSuccess ||
                cudaMemset2DAsync(dv + (size_t)plan->zero_begin * kHeadDim, pitch, 0, width, BH, stream) != cudaSuccess)
                return HMAR_ERR_CUDA;
        } else {
            for (int b = 0; b < B; ++b)
                for (int h = 0; h < H; ++h) {
                    const long long off = b * g.batch + h * g.head + (long long)plan->zero_begin * g.row;
                    if (cudaMemset2DAsync(dk + off, (size_t)g.row * sizeof(bf16), 0, kHeadDim * sizeof(bf16), rows, stream) != cudaSuccess ||
                        cudaMemset2DAsync(dv + off, (size_t)g.row * sizeof(bf16), 0, kHeadDim * sizeof(bf16), rows, stream) != cudaSuccess)
                        return HMAR_ERR_CUDA;
                }
        }
    }
    return launch_bwd_tc(mq, mk, mv, mdo, macc, a, out, dout, dq, BH, stream) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

// Contiguous [B*H, L, 64] tensors: one "batch" of BH heads.
int tc_bwd(const bf16* q, const bf16* k, const bf16* v, const bf16* out, const float* lse, const bf16* dout,
           bf16* dq, bf16* dk, bf16* dv, float* delta, float* dq_acc, int BH, const ScaleTable& st, float scale,
           int* status, cudaStream_t stream) {
    const long long L = st.start[st.n_scales];
    const Strides3 dense{kHeadDim, L * kHeadDim, (long long)BH * L * kHeadDim};
    return tc_bwd_strided(q, k, v, out, lse, dout, dq, dk, dv, delta, dq_acc, 1, BH, st, scale, dense, dense, dense, status, stream);
}

// Packed projection layouts: qkv and dqkv [B, L, 3, H, 64], out and dout [B, L, H, 64].
int tc_bwd_packed(const bf16* qkv, const bf16* out, const float* lse, const bf16* dout, bf16* dqkv, float* delta,
                  float* dq_acc, int B, int H, const ScaleTable& st, float scale, int* status, cudaStream_t stream) {
    const long long L = st.start[st.n_scales], HD = (long long)H * kHeadDim;
    const Strides3 packed{3 * HD, kHeadDim, L * 3 * HD}, od{HD, kHeadDim, L * HD};
    return tc_bwd_strided(qkv, qkv + HD, qkv + 2 * HD, out, lse, dout, dqkv, dqkv + HD, dqkv + 2 * HD, delta, dq_acc, B, H, st,
                          scale, packed, od, packed, status, stream);
}

// The same tensor maps for code outside this file.
bool make_rows_map_bf16(CUtensorMap* map, const void* base, int heads, int rows) {
    return make_rows_map4(map, base, 1, heads, rows, kHeadDim, (long long)rows * kHeadDim, (long long)heads * rows * kHeadDim, kTileRows);
}
bool make_dq_acc_map(CUtensorMap* map, const float* base, size_t rows) { return make_acc_map(map, base, rows); }

}  // namespace hmar
