// Host-side scale-block scheduler: side lengths -> work tiles that cover only the live blocks of
// HMAR's Markovian mask (paper Sec. 4.1, Fig. attn-mask).
//
// Scales k-1 and k are neighbours in the flattened sequence, so the keys a query of scale k may see
// form ONE contiguous range [start[k-1], start[k+1]); likewise the queries that see a key of scale k
// are [start[k], start[k+2]).  A tile whose rows all belong to one scale therefore needs no
// element-wise mask beyond its ragged ends.  Scales smaller than a tile are packed together, several
// per tile, and those tiles carry per-row bounds instead.
#include <algorithm>
#include "hmar_common.h"

namespace hmar {

void build_scale_table(int n_scales, const int* side_lens, int window, ScaleTable* out) {
    out->n_scales = n_scales;
    out->window = window;
    out->start[0] = 0;
    for (int s = 0; s < n_scales; ++s)
        out->start[s + 1] = out->start[s] + side_lens[s] * side_lens[s];
}

static void partner_range(const ScaleTable& st, int direction, int s_first, int s_last,
                          int* begin, int* end) {
    const int K = st.n_scales;
    if (direction == 0) {           // queries of scales s_first..s_last -> keys
        *begin = st.start[first_key_scale(st.window, s_first)];
        *end = st.start[last_key_scale(st.window, s_last) + 1];
    } else {                        // keys of scales s_first..s_last -> queries (possibly none)
        *begin = st.start[first_query_scale(st.window, s_first)];
        *end = st.start[last_query_scale(st.window, s_last, K) + 1];
        if (*end < *begin) *end = *begin;
    }
}

std::vector<Tile> build_tiles(const ScaleTable& st, int direction) {
    std::vector<Tile> tiles;
    const int K = st.n_scales;
    auto emit = [&](int row_begin, int row_count, int s_first, int s_last) {
        Tile t;
        t.row_begin = row_begin;
        t.row_count = row_count;
        partner_range(st, direction, s_first, s_last, &t.partner_begin, &t.partner_end);
        // uniform: every scale of the tile has the whole partner range as its own
        t.uniform = 1;
        for (int s = s_first; s <= s_last; ++s) {
            int b, e;
            partner_range(st, direction, s, s, &b, &e);
            if (b != t.partner_begin || e != t.partner_end) t.uniform = 0;
        }
        t.cost = (t.partner_end - t.partner_begin + kTileRows - 1) / kTileRows;
        tiles.push_back(t);
    };
    int pack_first = -1;            // first scale of the packed tile being grown, -1 if none
    for (int s = 0; s < K; ++s) {
        const int n = st.start[s + 1] - st.start[s];
        if (pack_first >= 0 && st.start[s + 1] - st.start[pack_first] > kTileRows) {
            emit(st.start[pack_first], st.start[s] - st.start[pack_first], pack_first, s - 1);
            pack_first = -1;
        }
        if (n >= kTileRows) {
            for (int r = 0; r < n; r += kTileRows)
                emit(st.start[s] + r, std::min(kTileRows, n - r), s, s);
        } else if (pack_first < 0) {
            pack_first = s;
        }
    }
    if (pack_first >= 0)
        emit(st.start[pack_first], st.start[K] - st.start[pack_first], pack_first, K - 1);
    // Longest first, so the heaviest tiles of a head are dispatched before its light ones.
    std::stable_sort(tiles.begin(), tiles.end(),
                     [](const Tile& a, const Tile& b) { return a.cost > b.cost; });
    return tiles;
}

}  // namespace hmar
