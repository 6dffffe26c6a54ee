// Shared host/device declarations of the HMAR attention library (internal).
#pragma once
#include <cstdint>
#include <vector>
#include "../../include/hmar.h"

namespace hmar {

constexpr int kHeadDim = 64;
constexpr int kTileRows = 128;   // rows of one work tile (query rows forward, key rows backward)

// Offsets of the scales in the flattened sequence; passed to kernels by value.
struct ScaleTable {
    int n_scales;
    int window;                       // hmar_window: which scales a query of scale s sees
    int start[HMAR_MAX_SCALES + 1];   // start[n_scales] == L
};

#if defined(__CUDACC__)
#define HMAR_HD __host__ __device__ __forceinline__
#else
#define HMAR_HD inline
#endif
// The keys a query of scale s sees are the scales first_key_scale(s) .. last_key_scale(s), a contiguous range of
// the flattened sequence; the queries that see a key of scale s are the scales first_query_scale(s) ..
// last_query_scale(s), also contiguous - and empty (first > last) for the keys of the last scale under
// HMAR_WINDOW_PREV, which no query looks at.
HMAR_HD int first_key_scale(int window, int s) {
    return window == HMAR_WINDOW_CAUSAL ? 0 : (window == HMAR_WINDOW_SELF ? s : (s > 0 ? s - 1 : 0));
}
HMAR_HD int last_key_scale(int window, int s) {
    return (window == HMAR_WINDOW_PREV && s > 0) ? s - 1 : s;
}
HMAR_HD int first_query_scale(int window, int s) {
    return (window == HMAR_WINDOW_PREV && s > 0) ? s + 1 : s;       // may be n_scales: no query sees the key
}
HMAR_HD int last_query_scale(int window, int s, int n_scales) {
    return window == HMAR_WINDOW_CAUSAL ? n_scales - 1 : (window == HMAR_WINDOW_SELF ? s : (s + 1 < n_scales ? s + 1 : s));
}

// One unit of work: `row_count` consecutive rows starting at `row_begin`, and the contiguous range
// [partner_begin, partner_end) of the other operand those rows touch.
// Forward: rows are queries, partners are keys.  Backward: rows are keys, partners are queries.
struct Tile {
    int32_t row_begin;
    int32_t row_count;
    int32_t partner_begin;
    int32_t partner_end;
    int32_t uniform;   // 1: every row sees the whole partner range; 0: rows have their own bounds
    int32_t cost;      // number of kTileRows-wide partner tiles (for ordering)
};

// Forward bounds of query row `i` of scale s: keys [start[first_key_scale(s)], start[last_key_scale(s)+1]).
// Backward bounds of key row `j` of scale s: queries [start[first_query_scale(s)], start[last_query_scale(s)+1]).
void build_scale_table(int n_scales, const int* side_lens, int window, ScaleTable* out);
std::vector<Tile> build_tiles(const ScaleTable& st, int direction);

#if defined(__CUDACC__)
// Checking build (-DHMAR_BOUNDS_CHECK, a separate library used by the tests): every address the kernels form by
// their own arithmetic for a plain load or store (TMA copies are clipped by the hardware against the tensor map)
// is compared with the extent of its tensor first.  An offset outside records HMAR_ERR_BOUNDS with the site's
// code in the status word and the access is skipped; nothing traps.  In the normal build the check folds away.
#if defined(HMAR_BOUNDS_CHECK)
__device__ __forceinline__ bool hmar_bounds_fail(int* status, int site) {
    if (status != nullptr) {
        atomicCAS(status, 0, HMAR_ERR_BOUNDS);
        atomicCAS(status + 1, 0, site);
    }
    return false;
}
#define HMAR_IN_BOUNDS(cond, status, site) ((cond) ? true : hmar_bounds_fail((status), (site)))
#else
#define HMAR_IN_BOUNDS(cond, status, site) true
#endif

__device__ __forceinline__ int scale_of_row(const ScaleTable& st, int row) {
    int s = 0;
    while (s + 1 < st.n_scales && row >= st.start[s + 1]) ++s;
    return s;
}
#endif

}  // namespace hmar
