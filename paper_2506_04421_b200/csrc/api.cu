// C-ABI layer: argument validation, plan cache, dispatch to the kernel launchers.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <type_traits>
#include <vector>

#include "hmar_common.h"
#include "launchers.h"
#include "tc_common.h"
#include "tc_launchers.h"

namespace hmar {

static std::atomic<long long> g_launches{0};
static std::atomic<int> g_force_simt{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- per-kernel timing
struct TimedLaunch { const char* name; cudaEvent_t begin, end; };
static std::atomic<int> g_profile_on{0};
static std::mutex g_profile_mu;
static std::vector<TimedLaunch> g_profile_log;

bool profile_enabled() { return g_profile_on.load(std::memory_order_relaxed) != 0; }

KernelTimer::KernelTimer(const char* name, cudaStream_t stream)
    : name_(name), stream_(stream), begin_(nullptr), on_(profile_enabled()) {
    if (on_ && (cudaEventCreate(&begin_) != cudaSuccess || cudaEventRecord(begin_, stream_) != cudaSuccess)) {
        cudaGetLastError();
        on_ = false;
    }
}

KernelTimer::~KernelTimer() {
    if (!on_) return;
    cudaEvent_t end = nullptr;
    if (cudaEventCreate(&end) == cudaSuccess && cudaEventRecord(end, stream_) == cudaSuccess) {
        std::lock_guard<std::mutex> lock(g_profile_mu);
        g_profile_log.push_back(TimedLaunch{name_, begin_, end});
    } else {
        cudaGetLastError();
    }
}

// Device status word written by kernels whose bounded waits ran out: {code, detail}.
__device__ int g_device_status[2];

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_scale(float softmax_scale) {
    // the kernels take maxima before scaling, so the scale must be positive (and finite)
    return (softmax_scale > 0.f && softmax_scale < 1e30f) ? HMAR_OK : HMAR_ERR_BAD_ARG;
}

// any_d: the entry point also runs the plain kernels, which exist for head dimensions 32, 64 and 128; the
// tensor-core kernels (and every entry point that has nothing else) take 64 only
static int check_shape(int B, int H, int D, bool any_d = false) {
    if (B <= 0 || H <= 0 || D <= 0) return HMAR_ERR_BAD_ARG;
    if ((long long)B * H > 65535) return HMAR_ERR_BAD_ARG;   // heads map to gridDim.y
    if (D != kHeadDim && !(any_d && (D == 32 || D == 128))) return HMAR_ERR_UNSUPPORTED;
    return HMAR_OK;
}

static int check_sides(int n_scales, const int* side_lens, int window, ScaleTable* st) {
    if (n_scales <= 0 || n_scales > HMAR_MAX_SCALES || side_lens == nullptr) return HMAR_ERR_BAD_ARG;
    if (window < HMAR_WINDOW_MARKOV || window > HMAR_WINDOW_PREV) return HMAR_ERR_BAD_ARG;
    long long total = 0;
    for (int s = 0; s < n_scales; ++s) {
        if (side_lens[s] <= 0 || side_lens[s] > 4096) return HMAR_ERR_BAD_ARG;
        total += (long long)side_lens[s] * side_lens[s];
    }
    if (total > (1 << 24)) return HMAR_ERR_BAD_ARG;
    build_scale_table(n_scales, side_lens, window, st);
    return HMAR_OK;
}

static int check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return HMAR_ERR_CUDA;
    }
    return major == 10 ? HMAR_OK : HMAR_ERR_UNSUPPORTED;
}

static size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

static int* device_status_ptr() {
    // One address per device; looked up on first use with that device current.
    static std::mutex mu;
    static std::map<int, int*> ptrs;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    auto it = ptrs.find(dev);
    if (it != ptrs.end()) return it->second;
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_device_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    ptrs[dev] = p;
    return p;
}

// ------------------------------------------------------------------------------------------------
template <typename T>
static int fwd_impl(const T* q, const T* k, const T* v, T* out, float* lse, int B, int H, int D,
                    int n_scales, const int* side_lens, int window, float softmax_scale, void* stream, bool tensor_core) {
    int rc = check_shape(B, H, D, true);
    tensor_core = tensor_core && D == kHeadDim;
    if (rc != HMAR_OK) return rc;
    ScaleTable st;
    rc = check_sides(n_scales, side_lens, window, &st);
    if (rc != HMAR_OK) return rc;
    if (check_scale(softmax_scale) != HMAR_OK) return HMAR_ERR_BAD_ARG;
    if (!q || !k || !v || !out || !lse) return HMAR_ERR_BAD_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(lse))
        return HMAR_ERR_BAD_ARG;
    rc = check_device();
    if (rc != HMAR_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (tensor_core && !g_force_simt.load())
            return tc_fwd(q, k, v, out, lse, B * H, st, softmax_scale, device_status_ptr(), s);
    }
    return simt_fwd<T>(q, k, v, out, lse, B * H, D, st, softmax_scale, s) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

template <typename T>
static int bwd_impl(const T* q, const T* k, const T* v, const T* out, const float* lse, const T* dout,
                    T* dq, T* dk, T* dv, void* workspace, size_t workspace_bytes, int B, int H, int D,
                    int n_scales, const int* side_lens, int window, float softmax_scale, void* stream, bool tensor_core) {
    int rc = check_shape(B, H, D, true);
    tensor_core = tensor_core && D == kHeadDim;
    if (rc != HMAR_OK) return rc;
    ScaleTable st;
    rc = check_sides(n_scales, side_lens, window, &st);
    if (rc != HMAR_OK) return rc;
    if (check_scale(softmax_scale) != HMAR_OK) return HMAR_ERR_BAD_ARG;
    if (!q || !k || !v || !out || !lse || !dout || !dq || !dk || !dv) return HMAR_ERR_BAD_ARG;
    const void* ptrs[] = {q, k, v, out, lse, dout, dq, dk, dv};
    for (const void* p : ptrs)
        if (!aligned16(p)) return HMAR_ERR_BAD_ARG;
    const size_t need = hmar_attn_bwd_workspace_bytes(B, H, D, n_scales, side_lens);
    if (workspace == nullptr || workspace_bytes < need) return HMAR_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return HMAR_ERR_BAD_ARG;
    rc = check_device();
    if (rc != HMAR_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int L = st.start[st.n_scales];
    float* delta = static_cast<float*>(workspace);
    float* dq_acc = reinterpret_cast<float*>(static_cast<char*>(workspace) + round256((size_t)B * H * L * sizeof(float)));
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (tensor_core && !g_force_simt.load())
            return tc_bwd(q, k, v, out, lse, dout, dq, dk, dv, delta, dq_acc, B * H, st, softmax_scale,
                          device_status_ptr(), s);
    }
    (void)dq_acc;
    return simt_bwd<T>(q, k, v, out, lse, dout, dq, dk, dv, delta, B * H, D, st, softmax_scale, s) == cudaSuccess
               ? HMAR_OK : HMAR_ERR_CUDA;
}

// strides == nullptr: dense [B,H,n,D] tensors
template <typename T>
static int step_impl(const T* q, const T* k_prev, const T* v_prev, const T* k_cur, const T* v_cur, T* out,
                     float* lse, int B, int H, int D, int side_prev, int side_cur, const StepStrides* strides,
                     float softmax_scale, void* stream, bool tensor_core) {
    int rc = check_shape(B, H, D, strides == nullptr);
    tensor_core = tensor_core && D == kHeadDim;
    if (rc != HMAR_OK) return rc;
    if (side_cur <= 0 || side_cur > 4096 || side_prev < 0 || side_prev > 4096) return HMAR_ERR_BAD_ARG;
    if (check_scale(softmax_scale) != HMAR_OK) return HMAR_ERR_BAD_ARG;
    if (!q || !k_cur || !v_cur || !out) return HMAR_ERR_BAD_ARG;
    if ((side_prev == 0) != (k_prev == nullptr) || (k_prev == nullptr) != (v_prev == nullptr))
        return HMAR_ERR_BAD_ARG;
    const void* ptrs[] = {q, k_prev, v_prev, k_cur, v_cur, out, lse};
    for (const void* p : ptrs)
        if (!aligned16(p)) return HMAR_ERR_BAD_ARG;
    const int n_prev = side_prev * side_prev, n_cur = side_cur * side_cur;
    StepStrides st{(long long)n_cur * D, (long long)n_prev * D, (long long)n_cur * D, (long long)n_cur * D};
    bool dense = true;
    if (strides != nullptr) {
        // a head must hold its rows, and heads must start on 16-byte boundaries
        if (strides->q < st.q || strides->kv_cur < st.kv_cur || strides->out < st.out ||
            (n_prev > 0 && strides->kv_prev < st.kv_prev))
            return HMAR_ERR_BAD_ARG;
        if (((strides->q | strides->kv_prev | strides->kv_cur | strides->out) & 7) != 0) return HMAR_ERR_BAD_ARG;
        dense = strides->q == st.q && strides->kv_cur == st.kv_cur && strides->out == st.out &&
                (n_prev == 0 || strides->kv_prev == st.kv_prev);
        st = *strides;
    }
    rc = check_device();
    if (rc != HMAR_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (tensor_core && !g_force_simt.load())
            return tc_scale_step(q, k_prev, v_prev, k_cur, v_cur, out, lse, B * H, n_prev, n_cur, st, softmax_scale,
                                 device_status_ptr(), s);
    }
    if (!dense) return HMAR_ERR_UNSUPPORTED;      // the plain kernels take dense tensors only
    return simt_scale_step<T>(q, k_prev, v_prev, k_cur, v_cur, out, lse, B * H, D, n_prev, n_cur, softmax_scale, s)
                   == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

}  // namespace hmar

using namespace hmar;
typedef __nv_bfloat16 bf16;

extern "C" {

int hmar_attn_fwd_window(const void* q, const void* k, const void* v, void* out, float* lse, int B, int H, int D,
                         int n_scales, const int* side_lens, int window, float softmax_scale, void* stream) {
    return fwd_impl<bf16>((const bf16*)q, (const bf16*)k, (const bf16*)v, (bf16*)out, lse, B, H, D, n_scales,
                          side_lens, window, softmax_scale, stream, true);
}

int hmar_attn_fwd_window_f32(const float* q, const float* k, const float* v, float* out, float* lse, int B, int H,
                             int D, int n_scales, const int* side_lens, int window, float softmax_scale, void* stream) {
    return fwd_impl<float>(q, k, v, out, lse, B, H, D, n_scales, side_lens, window, softmax_scale, stream, false);
}

int hmar_attn_fwd_packed(const void* qkv, void* out, float* lse, int B, int H, int D, int n_scales,
                         const int* side_lens, float softmax_scale, void* stream) {
    int rc = check_shape(B, H, D);
    if (rc != HMAR_OK) return rc;
    ScaleTable st;
    rc = check_sides(n_scales, side_lens, HMAR_WINDOW_MARKOV, &st);
    if (rc != HMAR_OK) return rc;
    if (check_scale(softmax_scale) != HMAR_OK) return HMAR_ERR_BAD_ARG;
    if (!qkv || !out || !lse) return HMAR_ERR_BAD_ARG;
    if (!aligned16(qkv) || !aligned16(out) || !aligned16(lse)) return HMAR_ERR_BAD_ARG;
    rc = check_device();
    if (rc != HMAR_OK) return rc;
    if (g_force_simt.load()) return HMAR_ERR_UNSUPPORTED;      // the fall-back kernels read contiguous tensors only
    return tc_fwd_packed((const bf16*)qkv, (bf16*)out, lse, B, H, st, softmax_scale, device_status_ptr(),
                         static_cast<cudaStream_t>(stream));
}

int hmar_attn_bwd_packed(const void* qkv, const void* out, const float* lse, const void* dout, void* dqkv,
                         void* workspace, size_t workspace_bytes, int B, int H, int D, int n_scales,
                         const int* side_lens, float softmax_scale, void* stream) {
    int rc = check_shape(B, H, D);
    if (rc != HMAR_OK) return rc;
    ScaleTable st;
    rc = check_sides(n_scales, side_lens, HMAR_WINDOW_MARKOV, &st);
    if (rc != HMAR_OK) return rc;
    if (check_scale(softmax_scale) != HMAR_OK) return HMAR_ERR_BAD_ARG;
    const void* ptrs[] = {qkv, out, lse, dout, dqkv};
    for (const void* p : ptrs)
        if (p == nullptr || !aligned16(p)) return HMAR_ERR_BAD_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 ||
        workspace_bytes < hmar_attn_bwd_workspace_bytes(B, H, D, n_scales, side_lens))
        return HMAR_ERR_WORKSPACE;
    rc = check_device();
    if (rc != HMAR_OK) return rc;
    if (g_force_simt.load()) return HMAR_ERR_UNSUPPORTED;      // the fall-back kernels read contiguous tensors only
    const int L = st.start[st.n_scales];
    float* delta = static_cast<float*>(workspace);
    float* dq_acc = reinterpret_cast<float*>(static_cast<char*>(workspace) + round256((size_t)B * H * L * sizeof(float)));
    return tc_bwd_packed((const bf16*)qkv, (const bf16*)out, lse, (const bf16*)dout, (bf16*)dqkv, delta, dq_acc, B, H, st,
                         softmax_scale, device_status_ptr(), static_cast<cudaStream_t>(stream));
}

int hmar_attn_fwd(const void* q, const void* k, const void* v, void* out, float* lse, int B, int H, int D,
                  int n_scales, const int* side_lens, float softmax_scale, void* stream) {
    return hmar_attn_fwd_window(q, k, v, out, lse, B, H, D, n_scales, side_lens, HMAR_WINDOW_MARKOV, softmax_scale, stream);
}

int hmar_attn_fwd_f32(const float* q, const float* k, const float* v, float* out, float* lse, int B, int H,
                      int D, int n_scales, const int* side_lens, float softmax_scale, void* stream) {
    return hmar_attn_fwd_window_f32(q, k, v, out, lse, B, H, D, n_scales, side_lens, HMAR_WINDOW_MARKOV, softmax_scale, stream);
}

size_t hmar_attn_bwd_workspace_bytes(int B, int H, int D, int n_scales, const int* side_lens) {
    ScaleTable st;
    if (check_shape(B, H, D, true) != HMAR_OK || check_sides(n_scales, side_lens, HMAR_WINDOW_MARKOV, &st) != HMAR_OK) return 0;
    const size_t rows = (size_t)B * H * st.start[st.n_scales];
    return round256(rows * sizeof(float)) + round256(rows * D * sizeof(float));
}

int hmar_attn_bwd_window(const void* q, const void* k, const void* v, const void* out, const float* lse,
                         const void* dout, void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes,
                         int B, int H, int D, int n_scales, const int* side_lens, int window, float softmax_scale,
                         void* stream) {
    return bwd_impl<bf16>((const bf16*)q, (const bf16*)k, (const bf16*)v, (const bf16*)out, lse,
                          (const bf16*)dout, (bf16*)dq, (bf16*)dk, (bf16*)dv, workspace, workspace_bytes, B, H,
                          D, n_scales, side_lens, window, softmax_scale, stream, true);
}

int hmar_attn_bwd_window_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                             const float* dout, float* dq, float* dk, float* dv, void* workspace,
                             size_t workspace_bytes, int B, int H, int D, int n_scales, const int* side_lens,
                             int window, float softmax_scale, void* stream) {
    return bwd_impl<float>(q, k, v, out, lse, dout, dq, dk, dv, workspace, workspace_bytes, B, H, D, n_scales,
                           side_lens, window, softmax_scale, stream, false);
}

int hmar_attn_bwd(const void* q, const void* k, const void* v, const void* out, const float* lse,
                  const void* dout, void* dq, void* dk, void* dv, void* workspace, size_t workspace_bytes,
                  int B, int H, int D, int n_scales, const int* side_lens, float softmax_scale, void* stream) {
    return hmar_attn_bwd_window(q, k, v, out, lse, dout, dq, dk, dv, workspace, workspace_bytes, B, H, D, n_scales,
                                side_lens, HMAR_WINDOW_MARKOV, softmax_scale, stream);
}

int hmar_attn_bwd_f32(const float* q, const float* k, const float* v, const float* out, const float* lse,
                      const float* dout, float* dq, float* dk, float* dv, void* workspace,
                      size_t workspace_bytes, int B, int H, int D, int n_scales, const int* side_lens,
                      float softmax_scale, void* stream) {
    return hmar_attn_bwd_window_f32(q, k, v, out, lse, dout, dq, dk, dv, workspace, workspace_bytes, B, H, D,
                                    n_scales, side_lens, HMAR_WINDOW_MARKOV, softmax_scale, stream);
}

int hmar_attn_scale_step(const void* q, const void* k_prev, const void* v_prev, const void* k_cur,
                         const void* v_cur, void* out, float* lse, int B, int H, int D, int side_prev,
                         int side_cur, float softmax_scale, void* stream) {
    return step_impl<bf16>((const bf16*)q, (const bf16*)k_prev, (const bf16*)v_prev, (const bf16*)k_cur,
                           (const bf16*)v_cur, (bf16*)out, lse, B, H, D, side_prev, side_cur, nullptr, softmax_scale,
                           stream, true);
}

int hmar_attn_scale_step_strided(const void* q, const void* k_prev, const void* v_prev, const void* k_cur,
                                 const void* v_cur, void* out, float* lse, int B, int H, int D, int side_prev,
                                 int side_cur, long long q_head_stride, long long kv_prev_head_stride,
                                 long long kv_cur_head_stride, long long out_head_stride, float softmax_scale,
                                 void* stream) {
    const StepStrides st{q_head_stride, kv_prev_head_stride, kv_cur_head_stride, out_head_stride};
    return step_impl<bf16>((const bf16*)q, (const bf16*)k_prev, (const bf16*)v_prev, (const bf16*)k_cur,
                           (const bf16*)v_cur, (bf16*)out, lse, B, H, D, side_prev, side_cur, &st, softmax_scale,
                           stream, true);
}

int hmar_attn_scale_step_f32(const float* q, const float* k_prev, const float* v_prev, const float* k_cur,
                             const float* v_cur, float* out, float* lse, int B, int H, int D, int side_prev,
                             int side_cur, float softmax_scale, void* stream) {
    return step_impl<float>(q, k_prev, v_prev, k_cur, v_cur, out, lse, B, H, D, side_prev, side_cur, nullptr,
                            softmax_scale, stream, false);
}

int hmar_schedule_tiles(int n_scales, const int* side_lens, int direction, int32_t* tiles, int max_tiles) {
    return hmar_schedule_tiles_window(n_scales, side_lens, HMAR_WINDOW_MARKOV, direction, tiles, max_tiles);
}

int hmar_schedule_tiles_window(int n_scales, const int* side_lens, int window, int direction, int32_t* tiles,
                               int max_tiles) {
    ScaleTable st;
    int rc = check_sides(n_scales, side_lens, window, &st);
    if (rc != HMAR_OK) return rc;
    if (direction != 0 && direction != 1) return HMAR_ERR_BAD_ARG;
    std::vector<Tile> t = build_tiles(st, direction);
    if (tiles != nullptr) {
        const int n = (int)t.size() < max_tiles ? (int)t.size() : max_tiles;
        for (int i = 0; i < n; ++i) std::memcpy(tiles + 6 * i, &t[i], sizeof(Tile));
    }
    return (int)t.size();
}

int hmar_schedule_bwd_full_tile_share(int n_scales, const int* side_lens, int window) {
    ScaleTable st;
    int rc = check_sides(n_scales, side_lens, window, &st);
    if (rc != HMAR_OK) return rc;
    return tc_bwd_full_tile_permille(st);
}

int hmar_device_status(int* detail) {
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    int host[2] = {0, 0};
    if (cudaMemcpyFromSymbol(host, g_device_status, sizeof(host)) != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    const int zero[2] = {0, 0};
    if (cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero)) != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    if (detail) *detail = host[1];
    return host[0];
}

void hmar_profile_begin(void) {
    std::lock_guard<std::mutex> lock(g_profile_mu);
    for (auto& t : g_profile_log) { cudaEventDestroy(t.begin); cudaEventDestroy(t.end); }
    g_profile_log.clear();
    g_profile_on.store(1);
}

int hmar_profile_end(char* report, size_t capacity) {
    g_profile_on.store(0);
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_profile_mu);
    std::map<std::string, std::pair<int, double>> acc;
    for (auto& t : g_profile_log) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.begin, t.end) == cudaSuccess) {
            auto& a = acc[t.name];
            a.first += 1;
            a.second += ms;
        } else {
            cudaGetLastError();
        }
        cudaEventDestroy(t.begin);
        cudaEventDestroy(t.end);
    }
    g_profile_log.clear();
    std::string text;
    for (auto& kv : acc) {
        char line[160];
        snprintf(line, sizeof(line), "%s %d %.6f\n", kv.first.c_str(), kv.second.first, kv.second.second);
        text += line;
    }
    if (report != nullptr && capacity > 0) {
        const size_t n = text.size() < capacity - 1 ? text.size() : capacity - 1;
        std::memcpy(report, text.data(), n);
        report[n] = 0;
    }
    return HMAR_OK;
}

int hmar_recon_accumulate(float* xhat, const float* codebook, const int* tokens_old, const int* tokens_new,
                          const unsigned char* mask, int* tokens_out, int B, int C, int V, int side, int out_side,
                          void* stream) {
    if (B <= 0 || C <= 0 || V <= 0 || side <= 0 || out_side <= 0 || side > 4096 || out_side > 4096 || C > 4096) return HMAR_ERR_BAD_ARG;
    if (side > out_side) return HMAR_ERR_BAD_ARG;                       // the step only ever enlarges a token map
    if (xhat == nullptr || codebook == nullptr || tokens_new == nullptr) return HMAR_ERR_BAD_ARG;
    if (mask != nullptr && tokens_old == nullptr) return HMAR_ERR_BAD_ARG;
    if (tokens_out != nullptr && (tokens_out == tokens_new || tokens_out == tokens_old)) return HMAR_ERR_BAD_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    return launch_recon_accumulate(xhat, codebook, tokens_old, tokens_new, mask, tokens_out, B, C, V, side, out_side,
                                   static_cast<cudaStream_t>(stream)) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

int hmar_recon_downsample(const float* xhat, float* out, int B, int C, int in_side, int out_side, void* stream) {
    if (B <= 0 || C <= 0 || in_side <= 0 || out_side <= 0 || in_side > 4096 || C > 4096) return HMAR_ERR_BAD_ARG;
    if (out_side > in_side) return HMAR_ERR_BAD_ARG;                    // the step only ever shrinks the image
    if (xhat == nullptr || out == nullptr || xhat == out) return HMAR_ERR_BAD_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return HMAR_ERR_CUDA; }
    return launch_recon_downsample(xhat, out, B, C, in_side, out_side, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? HMAR_OK : HMAR_ERR_CUDA;
}

int hmar_selftest_bounded_wait(void* stream) {
    int rc = check_device();
    if (rc != HMAR_OK) return rc;
    int* status = device_status_ptr();
    if (status == nullptr) return HMAR_ERR_CUDA;
    return launch_selftest_wait(status, static_cast<cudaStream_t>(stream)) == cudaSuccess ? HMAR_OK : HMAR_ERR_CUDA;
}

int hmar_debug_force_simt(int enable) { return g_force_simt.exchange(enable ? 1 : 0); }

long long hmar_launch_count(void) { return g_launches.load(); }

void hmar_shutdown(void) { tc_release_plans(); }

const char* hmar_status_string(int status) {
    switch (status) {
        case HMAR_OK: return "ok";
        case HMAR_ERR_BAD_ARG: return "bad argument";
        case HMAR_ERR_UNSUPPORTED: return "unsupported head dimension or device";
        case HMAR_ERR_CUDA: return "CUDA call failed";
        case HMAR_ERR_WORKSPACE: return "workspace missing or too small";
        case HMAR_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case HMAR_ERR_BOUNDS: return "checking build: a kernel formed an address outside its tensor";
        default: return "unknown status";
    }
}

}  // extern "C"
