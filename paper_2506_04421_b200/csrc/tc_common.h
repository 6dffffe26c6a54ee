// Argument structures shared by the tensor-core kernels and their host-side dispatch (internal).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "hmar_common.h"

namespace hmar {

// Device form of a forward work tile: query rows [row_begin, row_begin + row_count) and up to two key
// segments (second one used by the inference step only: previous scale, then current scale).
struct FwdWork {
    int32_t row_begin, row_count;
    int32_t s0_begin, s0_end;
    int32_t s1_begin, s1_end;
    int32_t uniform;
    int32_t pad;
};

struct FwdArgs {
    const FwdWork* work;     // n_work tiles per head; nullptr = inference step (tiles derived in-kernel)
    int n_work;
    int n_q_rows;            // rows per head of q / out / lse
    int heads_per_batch;     // H: head bh is head bh % H of batch bh / H (the tensor maps are 4-D: D, rows, H, B)
    long long out_row_stride, out_head_stride, out_batch_stride;   // of `out`, in elements (lse is always [B*H, rows])
    long long out_extent, lse_extent;   // elements reachable through out / lse (read by the checking build only)
    int n0, n1;              // inference step: rows of the previous / current scale's keys
    float scale_log2;        // softmax_scale * log2(e)
    __nv_bfloat16* out;
    float* lse;              // may be nullptr
    int* status;             // device status word {code, detail}, may be nullptr
    ScaleTable st;
};

// Backward work tile: key rows [row_begin, row_begin + row_count) and the query range that may see them.
struct BwdWork {
    int32_t row_begin, row_count;
    int32_t q_begin, q_end;
    int32_t uniform;
    int32_t cost_begin;      // cost of the head's tiles before this one (see bwd_fill_costs)
    int32_t pad[2];
};

// Cost model of the backward's persistent blocks: a tile costs its number of 128-query steps plus a
// constant for the work at its start and end.  Fills cost_begin and returns the cost of a whole head.
inline int bwd_fill_costs(BwdWork* work, int n) {
    int acc = 0;
    for (int i = 0; i < n; ++i) {
        work[i].cost_begin = acc;
        acc += (work[i].q_end - work[i].q_begin + 127) / 128 + 2;
    }
    return acc;
}

// Share, in thousandths, of a head's steps that belong to full tiles (128 key rows that all see the whole query
// range): those run without any mask code.
inline int bwd_plain_permille(const BwdWork* work, int n) {
    long long plain = 0, total = 0;
    for (int i = 0; i < n; ++i) {
        const int steps = (work[i].q_end - work[i].q_begin + 127) / 128;
        total += steps;
        if (work[i].uniform && work[i].row_count == 128) plain += steps;
    }
    return total > 0 ? (int)(plain * 1000 / total) : 1000;
}

struct BwdArgs {
    const BwdWork* work;
    int n_work;
    int n_heads;             // B * H
    int head_cost;           // from bwd_fill_costs
    int plain_permille;      // from bwd_plain_permille: picks the instantiation of the main kernel
    int split;               // set by the launcher: runs per head dealt to the blocks in turn (0: one contiguous run per block)
    int L;
    float scale_log2;        // softmax_scale * log2(e)
    float softmax_scale;
    const float* lse;        // [BH, L] from the forward
    const float* delta;      // [BH, L] rowsum(dO o O) (read by the main kernel)
    float* delta_w;          // same buffer, written by the preprocess kernel
    float* dq_acc;           // [BH, L, 64] fp32 accumulator
    // Layout of the bf16 tensors: head bh is head bh % heads_per_batch of batch bh / heads_per_batch, and element
    // (batch, head, row, d) sits at batch * *_batch + head * *_head + row * *_row + d (strides in elements).  q, k, v
    // share the `in` strides, out and dout the `od` strides, dq, dk, dv the `g` strides; lse, delta and the fp32 dQ
    // accumulator are always dense [BH, L(, 64)].
    int heads_per_batch;
    long long in_row, in_head, in_batch;
    long long od_row, od_head, od_batch;
    long long g_row, g_head, g_batch;
    long long in_extent, g_extent;      // elements reachable through v and through dk / dv (checking build only)
    const __nv_bfloat16* v;  // read directly for the rows that go to TMEM
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    ScaleTable st;
};

size_t fwd_tc_smem_bytes();
cudaError_t launch_selftest_wait(int* status, cudaStream_t stream);
cudaError_t launch_bwd_tc(const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& dout_map,
                          const CUtensorMap& dq_acc_map, const BwdArgs& args, const __nv_bfloat16* out, const __nv_bfloat16* dout,
                          __nv_bfloat16* dq, int BH, cudaStream_t stream);
cudaError_t launch_fwd_tc(const CUtensorMap& q, const CUtensorMap& k0, const CUtensorMap& v0, const CUtensorMap& k1,
                          const CUtensorMap& v1, const FwdArgs& args, int BH, cudaStream_t stream);

}  // namespace hmar
