// Backward entry point that allocates nothing.
//
// Some callers cannot allocate device memory at the moment they need a backward pass: code running
// under a framework that has handed its whole memory budget to its own pool and forbids further
// cudaMalloc calls, plug-ins of inference servers that must not grow the process footprint after
// start-up, and code that is not allowed to call anything that may synchronise the device (cudaMalloc
// and cudaFree may).  hmar_attn_bwd needs a caller-provided workspace and, on first use of a side
// length list, creates a device work list with cudaMalloc; neither is possible for such callers.
//
// hmar_attn_bwd_noalloc therefore keeps all of its scratch - the work list, delta and the fp32 dQ
// accumulator - in one fixed device array that is part of the library image.  Every GPU that loads
// the library holds the array (about 8.6 MB) until the process exits.  The price is a size limit,
// kMaxRows rows in total, and that all calls share the array (see include/hmar.h).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "hmar_common.h"
#include "launchers.h"
#include "tc_common.h"
#include "tc_launchers.h"

namespace hmar {

constexpr size_t kMaxRows = HMAR_NOALLOC_MAX_ROWS;             // B * H * L
// Backward work tiles of one head: a scale of n rows gives at most n / 128 + 1 tiles and a packed tile ends at a
// scale boundary, so a head has at most L / 128 + 2 * n_scales tiles; the size check below can therefore not be
// passed by a list that does not fit here.
constexpr size_t kMaxWork = kMaxRows / 128 + 2 * HMAR_MAX_SCALES;
constexpr size_t kWorkBytes = kMaxWork * sizeof(BwdWork);      // 12 KB
constexpr size_t kDeltaBytes = kMaxRows * sizeof(float);
constexpr size_t kAccBytes = kMaxRows * kHeadDim * sizeof(float);
constexpr size_t kScratchBytes = kWorkBytes + kDeltaBytes + kAccBytes;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an
// address a kernel may be given.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Device address of the scratch on the current device, looked up once per device.
static unsigned char* scratch_address() {
    static std::mutex mu;
    static unsigned char* addr[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return nullptr; }
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        unsigned char* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        addr[dev] = p;
    }
    return addr[dev];
}

// The work list reaches the scratch as kernel parameters: parameters are copied when the launch is enqueued,
// so no host buffer has to outlive the call and no host-to-device copy (which, from pageable memory, may make
// the host wait for the stream) is involved.
constexpr int kFillChunk = 96;                                 // 96 x 32 bytes of parameters per launch
struct WorkChunk { BwdWork w[kFillChunk]; };
static __global__ void noalloc_fill_work_kernel(const WorkChunk chunk, int first, int count) {
    BwdWork* dst = reinterpret_cast<BwdWork*>(g_noalloc_scratch);
    for (int i = threadIdx.x; i < count; i += blockDim.x) dst[first + i] = chunk.w[i];
}

bool make_rows_map_bf16(CUtensorMap* map, const void* base, int heads, int rows);
bool make_dq_acc_map(CUtensorMap* map, const float* base, size_t rows);

}  // namespace hmar

using namespace hmar;

extern "C" int hmar_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* out,
                                     const float* lse, const void* dout, void* dq, void* dk, void* dv,
                                     int B, int H, int D, int n_scales, const int* side_lens,
                                     float softmax_scale, void* stream) {
    if (B <= 0 || H <= 0 || D <= 0 || (long long)B * H > 65535) return HMAR_ERR_BAD_ARG;
    if (D != kHeadDim) return HMAR_ERR_UNSUPPORTED;
    if (!(softmax_scale > 0.f && softmax_scale < 1e30f)) return HMAR_ERR_BAD_ARG;
    if (n_scales <= 0 || n_scales > HMAR_MAX_SCALES || side_lens == nullptr) return HMAR_ERR_BAD_ARG;
    long long L = 0;
    for (int s = 0; s < n_scales; ++s) {
        if (side_lens[s] <= 0 || side_lens[s] > 4096) return HMAR_ERR_BAD_ARG;
        L += (long long)side_lens[s] * side_lens[s];
    }
    const void* ptrs[] = {q, k, v, out, lse, dout, dq, dk, dv};
    for (const void* p : ptrs)
        if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15u) != 0) return HMAR_ERR_BAD_ARG;
    if ((unsigned long long)L * B * H > kMaxRows) return HMAR_ERR_WORKSPACE;     // beyond the fixed scratch

    ScaleTable st;
    build_scale_table(n_scales, side_lens, HMAR_WINDOW_MARKOV, &st);
    const std::vector<Tile> tiles = build_tiles(st, 1);
    if (tiles.size() > kMaxWork) return HMAR_ERR_WORKSPACE;     // cannot happen (see kMaxWork); kept as a guard

    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return HMAR_ERR_CUDA;
    }
    if (major != 10) return HMAR_ERR_UNSUPPORTED;
    unsigned char* scratch = scratch_address();
    if (scratch == nullptr) return HMAR_ERR_CUDA;

    static thread_local BwdWork host_work[kMaxWork];
    for (size_t i = 0; i < tiles.size(); ++i) {
        host_work[i] = BwdWork{};
        host_work[i].row_begin = tiles[i].row_begin;
        host_work[i].row_count = tiles[i].row_count;
        host_work[i].q_begin = tiles[i].partner_begin;
        host_work[i].q_end = tiles[i].partner_end;
        host_work[i].uniform = tiles[i].uniform;
    }
    const int head_cost = bwd_fill_costs(host_work, (int)tiles.size());
    const int plain_permille = bwd_plain_permille(host_work, (int)tiles.size());
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (size_t first = 0; first < tiles.size(); first += kFillChunk) {
        WorkChunk chunk;
        const int count = (int)std::min<size_t>(kFillChunk, tiles.size() - first);
        for (int i = 0; i < count; ++i) chunk.w[i] = host_work[first + i];
        for (int i = count; i < kFillChunk; ++i) chunk.w[i] = BwdWork{};
        noalloc_fill_work_kernel<<<1, 128, 0, s>>>(chunk, (int)first, count);
    }
    if (cudaGetLastError() != cudaSuccess) return HMAR_ERR_CUDA;
    count_launch((int)((tiles.size() + kFillChunk - 1) / kFillChunk));

    const int BH = B * H;
    CUtensorMap mq, mk, mv, mdo, macc;
    if (!make_rows_map_bf16(&mq, q, BH, (int)L) || !make_rows_map_bf16(&mk, k, BH, (int)L) ||
        !make_rows_map_bf16(&mv, v, BH, (int)L) || !make_rows_map_bf16(&mdo, dout, BH, (int)L) ||
        !make_dq_acc_map(&macc, reinterpret_cast<const float*>(scratch + kWorkBytes + kDeltaBytes), (size_t)BH * L))
        return HMAR_ERR_CUDA;
    BwdArgs a{};
    a.work = reinterpret_cast<const BwdWork*>(scratch);
    a.n_work = (int)tiles.size();
    a.n_heads = BH;
    a.head_cost = head_cost;
    a.plain_permille = plain_permille;
    a.L = (int)L;
    a.scale_log2 = softmax_scale * 1.4426950408889634f;
    a.softmax_scale = softmax_scale;
    a.lse = lse;
    a.delta = reinterpret_cast<float*>(scratch + kWorkBytes);
    a.delta_w = reinterpret_cast<float*>(scratch + kWorkBytes);
    a.dq_acc = reinterpret_cast<float*>(scratch + kWorkBytes + kDeltaBytes);    // cleared by the launcher
    a.heads_per_batch = BH;
    a.in_row = a.od_row = a.g_row = kHeadDim;
    a.in_head = a.od_head = a.g_head = L * kHeadDim;
    a.in_batch = a.od_batch = a.g_batch = (long long)BH * L * kHeadDim;
    a.in_extent = a.g_extent = (long long)BH * L * kHeadDim;
    a.v = static_cast<const __nv_bfloat16*>(v);
    a.dk = static_cast<__nv_bfloat16*>(dk);
    a.dv = static_cast<__nv_bfloat16*>(dv);
    a.status = nullptr;
    a.st = st;
    return launch_bwd_tc(mq, mk, mv, mdo, macc, a, static_cast<const __nv_bfloat16*>(out),
                         static_cast<const __nv_bfloat16*>(dout), static_cast<__nv_bfloat16*>(dq), BH, s) == cudaSuccess
               ? HMAR_OK : HMAR_ERR_CUDA;
}
