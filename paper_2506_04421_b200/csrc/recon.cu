// The sampler's step next to the attention at inference: the running multi-scale reconstruction
// (paper Alg. 2, "Multi-scale VQ-VAE Reconstruction": x~_k = interpolate(lookup(V, r_k), H_K, W_K),
// x~_{1:k} = x~_{1:k-1} + x~_k) fused with the token selection of a masked refinement sub-step (Sec. 4.2:
// only the positions in the sub-step's mask take the newly generated token).
//
// One pass does, per output pixel of the final resolution: select the 4 x 4 neighbourhood's token ids
// (new where the mask is set, old elsewhere), look their code vectors up, interpolate bicubically
// (a = -0.75, half-pixel sample positions, border indices clamped) and add the result to the running
// reconstruction in place.  The reconstruction is read and written exactly once (the algorithmic HBM bytes
// of the step); the codebook (V x C fp32, 512 KB for V = 4096, C = 32) and the token maps stay in L2 / L1.
// Two kernels: for token maps of at most 32 x 32 (every scale of the paper's schedules) a block takes one image
// and stages the looked-up coarse map in shared memory; larger maps go through the plain kernel, in which a
// thread owns one output pixel and walks the channels.  In both a warp's accesses to the [B, C, H, W] tensor
// are 128-byte rows.
#include <cuda_runtime.h>

#include "hmar_common.h"
#include "launchers.h"

namespace hmar {
namespace {

__device__ __forceinline__ void cubic_weights(float t, float (&w)[4]) {
    const float a = -0.75f;
    const float x0 = t + 1.f, x1 = t, x2 = 1.f - t, x3 = 2.f - t;
    w[0] = ((a * x0 - 5.f * a) * x0 + 8.f * a) * x0 - 4.f * a;
    w[1] = ((a + 2.f) * x1 - (a + 3.f)) * x1 * x1 + 1.f;
    w[2] = ((a + 2.f) * x2 - (a + 3.f)) * x2 * x2 + 1.f;
    w[3] = ((a * x3 - 5.f * a) * x3 + 8.f * a) * x3 - 4.f * a;
}

__global__ void __launch_bounds__(256)
hmar_recon_accumulate_kernel(float* __restrict__ xhat, const float* __restrict__ codebook,
                             const int* __restrict__ tokens_old, const int* __restrict__ tokens_new,
                             const unsigned char* __restrict__ mask, int* __restrict__ tokens_out,
                             int B, int C, int V, int side, int out_side) {
    const long long pix = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n_pix = (long long)B * out_side * out_side;
    // the selected token map is also written back (one thread per coarse position), for the next sub-step
    if (tokens_out != nullptr && pix < (long long)B * side * side) {
        const int keep = (mask == nullptr || mask[pix] != 0) ? tokens_new[pix] : tokens_old[pix];
        tokens_out[pix] = keep;
    }
    if (pix >= n_pix) return;
    const int ox = (int)(pix % out_side), oy = (int)((pix / out_side) % out_side), b = (int)(pix / ((long long)out_side * out_side));
    const float ratio = (float)side / (float)out_side;
    const float sy = (oy + 0.5f) * ratio - 0.5f, sx = (ox + 0.5f) * ratio - 0.5f;
    const int iy = (int)floorf(sy), ix = (int)floorf(sx);
    float wy[4], wx[4];
    cubic_weights(sy - (float)iy, wy);
    cubic_weights(sx - (float)ix, wx);
    // ids of the 16 neighbours, selected, clamped into the codebook (an id outside [0, V) reads code 0 or V - 1)
    int id[16];
    float wgt[16];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int yy = min(max(iy - 1 + a, 0), side - 1);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int xx = min(max(ix - 1 + c, 0), side - 1);
            const long long pos = ((long long)b * side + yy) * side + xx;
            int t = (mask == nullptr || mask[pos] != 0) ? tokens_new[pos] : tokens_old[pos];
            id[a * 4 + c] = min(max(t, 0), V - 1);
            wgt[a * 4 + c] = wy[a] * wx[c];
        }
    }
    float* dst = xhat + ((long long)b * C) * out_side * out_side + (long long)oy * out_side + ox;
    const long long plane = (long long)out_side * out_side;
    for (int ch = 0; ch < C; ++ch) {
        float acc = 0.f;
#pragma unroll
        for (int n = 0; n < 16; ++n) acc = fmaf(wgt[n], __ldg(codebook + (long long)id[n] * C + ch), acc);
        dst[ch * plane] += acc;
    }
}

// Staged variant for token maps of at most 32 x 32 and reconstructions of at most 64 x 64: one block per image
// and group of 8 channels.  The selected tokens' code values are gathered once into shared memory as a
// channel-major coarse map (channel rows padded to 4 words past a multiple of 32, so the transposing stores spread
// over the banks), then every warp takes a channel and walks down the output rows, interpolating separably from
// shared memory and adding one 128-byte row segment into the reconstruction at a time.  Each code vector is
// fetched once per image instead of once per output pixel and tap, and a launch at the sampler's batch still has
// a few hundred blocks.
constexpr int kStageMaxSide = 32;
constexpr int kStageChannels = 8;
constexpr int kStageMaxOut = 64;

__global__ void __launch_bounds__(256)
hmar_recon_accumulate_staged_kernel(float* __restrict__ xhat, const float* __restrict__ codebook,
                                    const int* __restrict__ tokens_old, const int* __restrict__ tokens_new,
                                    const unsigned char* __restrict__ mask, int* __restrict__ tokens_out,
                                    int C, int V, int side, int out_side, int n_groups) {
    __shared__ float coarse[kStageChannels * (kStageMaxSide * kStageMaxSide + 4)];
    __shared__ int ids[kStageMaxSide * kStageMaxSide];
    __shared__ float4 row_w[kStageMaxOut];                  // per output row: the four vertical weights ...
    __shared__ int row_src[kStageMaxOut];                   // ... and the source row of the second one
    const int b = blockIdx.x / n_groups, grp = blockIdx.x - b * n_groups;
    const int c0 = grp * kStageChannels, nc = min(kStageChannels, C - c0);
    const int n_tok = side * side;
    const int stride = n_tok + ((4 - n_tok) & 31);          // = 4 mod 32: the gather's transposing stores miss each other's banks
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    const float ratio = (float)side / (float)out_side;
    if (threadIdx.x < out_side) {
        const float sy = (threadIdx.x + 0.5f) * ratio - 0.5f;
        const int iy = (int)floorf(sy);
        float wy[4];
        cubic_weights(sy - (float)iy, wy);
        row_w[threadIdx.x] = make_float4(wy[0], wy[1], wy[2], wy[3]);
        row_src[threadIdx.x] = iy;
    }
    // ---- token selection (written out by the image's first channel group)
    for (int pos = threadIdx.x; pos < n_tok; pos += blockDim.x) {
        const long long gp = (long long)b * n_tok + pos;
        const int t = (mask == nullptr || mask[gp] != 0) ? tokens_new[gp] : tokens_old[gp];
        if (tokens_out != nullptr && grp == 0) tokens_out[gp] = t;
        ids[pos] = min(max(t, 0), V - 1);
    }
    __syncthreads();
    // ---- gather: a pair of lanes per token reads the group's 8 channels (32 bytes, one sector) as two 16-byte
    // loads, so that one instruction of a warp covers 16 whole sectors; a group cut short by C, or a codebook
    // whose rows do not start on 16-byte boundaries, goes one value at a time
    if (nc == kStageChannels && (C & 3) == 0 && (reinterpret_cast<unsigned long long>(codebook) & 15ull) == 0) {
#pragma unroll 4
        for (int idx = threadIdx.x; idx < 2 * n_tok; idx += blockDim.x) {
            const int pos = idx >> 1, half = idx & 1;
            const float4 v = __ldg(reinterpret_cast<const float4*>(codebook + (long long)ids[pos] * C + c0) + half);
            float* dst = coarse + (half * 4) * stride + pos;
            dst[0 * stride] = v.x; dst[1 * stride] = v.y; dst[2 * stride] = v.z; dst[3 * stride] = v.w;
        }
    } else {
        for (int idx = threadIdx.x; idx < n_tok * kStageChannels; idx += blockDim.x) {
            const int pos = idx / kStageChannels, ch = idx - pos * kStageChannels;
            if (ch < nc) coarse[ch * stride + pos] = __ldg(codebook + (long long)ids[pos] * C + c0 + ch);
        }
    }
    __syncthreads();
    // ---- interpolate and accumulate: lane per output column, warp per channel, walking down the output rows.
    // The interpolation is separable: a source row's four horizontal taps are combined once (h) and reused by
    // every output row whose vertical window holds that source row; going down, the window of four h values
    // moves by at most one source row per output row (the step only ever enlarges a map), so an output value costs
    // one to four shared-memory loads instead of sixteen.  Each element of the reconstruction gets exactly one
    // addition, issued as a reduction to memory: nothing waits for the old value, and with a single addend per
    // element the result does not depend on the order in which the reductions land.
    const long long plane = (long long)out_side * out_side;
    for (int ox = lane; ox < out_side; ox += 32) {
        const float sx = (ox + 0.5f) * ratio - 0.5f;
        const int ix = (int)floorf(sx);
        float wx[4];
        cubic_weights(sx - (float)ix, wx);
        int xx[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) xx[c] = min(max(ix - 1 + c, 0), side - 1);
        for (int ch = warp; ch < nc; ch += n_warps) {
            const float* src = coarse + ch * stride;
            auto hrow = [&](int r) -> float {
                const float* row = src + min(max(r, 0), side - 1) * side;
                float h = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) h = fmaf(wx[c], row[xx[c]], h);
                return h;
            };
            float* dst = xhat + ((long long)b * C + c0 + ch) * plane + ox;
            int cur = -1000000;                             // source row of the window's second entry
            float h0 = 0.f, h1 = 0.f, h2 = 0.f, h3 = 0.f;
#pragma unroll 4
            for (int oy = 0; oy < out_side; ++oy, dst += out_side) {
                const int iy = row_src[oy];
                const float4 wy = row_w[oy];
                if (iy == cur + 1) {
                    h0 = h1; h1 = h2; h2 = h3; h3 = hrow(iy + 2);
                } else if (iy != cur) {
                    h0 = hrow(iy - 1); h1 = hrow(iy); h2 = hrow(iy + 1); h3 = hrow(iy + 2);
                }
                cur = iy;
                atomicAdd(dst, fmaf(wy.w, h3, fmaf(wy.z, h2, fmaf(wy.y, h1, wy.x * h0))));
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// The running reconstruction brought down to a scale's resolution (Sec. 4.1: the scale is conditioned on the
// interpolated x~_{1:k-1}): area interpolation, out(i, j) = mean of the input over rows
// [floor(i * S / s), ceil((i + 1) * S / s)) and the like columns.
//
// Staged kernel: a warp per image plane.  The plane is read once, coalesced, into shared memory (rows padded by
// one word); lane = input row sums the row's column bins (partial sums, row stride odd so the lanes hit
// different banks); lane = output column sums those over the row bins, divides by the bin's size and writes
// a coalesced output row.  One read of the reconstruction, which is all the traffic that counts.  Equal sizes are
// a plain copy (the launcher does it).
constexpr int kDownStageMaxSide = 64;
constexpr size_t kDownStageSmem = 96 * 1024;

__device__ __forceinline__ int bin_begin(int i, int in, int out) { return (i * in) / out; }
__device__ __forceinline__ int bin_end(int i, int in, int out) { return ((i + 1) * in + out - 1) / out; }

// SF: the input side as a compile-time constant (16, 32, 64: the latents of the paper's resolutions), so that a
// lane's loads of the plane are all issued before the first is used -- a warp's 1 to 16 KB in flight is what brings
// the read near the HBM rate; 0 = any side up to 64, eight loads at a time.
template <int SF>
__global__ void __launch_bounds__(256)
hmar_recon_downsample_staged_kernel(const float* __restrict__ xhat, float* __restrict__ out, long long n_planes,
                                    int S_any, int s, int warps_per_block) {
    const int S = SF ? SF : S_any;
    extern __shared__ float down_smem[];
    __shared__ int2 bins[kDownStageMaxSide];               // [begin, end) of every output index (rows and columns alike)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < s; i += blockDim.x) bins[i] = make_int2(bin_begin(i, S, s), bin_end(i, S, s));
    __syncthreads();
    const int ts = s | 1;                                   // row stride of the partial sums
    const int per_warp = S * (S + 1) + (S + 1) * ts;
    float* tile = down_smem + warp * per_warp;
    float* part = tile + S * (S + 1);
    const long long plane = (long long)blockIdx.x * warps_per_block + warp;
    if (warp >= warps_per_block || plane >= n_planes) return;
    const float* src = xhat + plane * S * S;
    if (SF) {
        constexpr int N = SF ? SF * SF / 32 : 1;           // values per lane
        constexpr int CH = N < 32 ? N : 32;                // ... fetched CH at a time
#pragma unroll 1
        for (int i0 = 0; i0 < N; i0 += CH) {
            float v[CH];
#pragma unroll
            for (int k = 0; k < CH; ++k) v[k] = src[(i0 + k) * 32 + lane];
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                const int i = (i0 + k) * 32 + lane, r = i / S, c = i - r * S;
                tile[r * (S + 1) + c] = v[k];
            }
        }
    } else {
        const float inv = 1.f / (float)S;
#pragma unroll 8
        for (int i = lane; i < S * S; i += 32) {
            const int r = (int)(((float)i + 0.5f) * inv), c = i - r * S;      // i / S: exact for i < 4096, S <= 64
            tile[r * (S + 1) + c] = src[i];
        }
    }
    __syncwarp();
    float* dst0 = out + plane * s * s;
    if (SF) {
        // Compile-time side: running sums.  Lane = input row turns its row into exclusive running sums in place (the
        // padded row has exactly S + 1 slots), so a column bin's sum is one difference; lane = output column does the
        // same down the partial sums' columns.  Everything is straight-line code over registers, and the loops over
        // the bins have independent iterations.
        constexpr int SS = SF ? SF : 1;
        for (int r = lane; r < SS; r += 32) {
            float* row = tile + r * (SS + 1);
            float v[SS];
#pragma unroll
            for (int c = 0; c < SS; ++c) v[c] = row[c];
            float run = 0.f;
#pragma unroll
            for (int c = 0; c < SS; ++c) {
                row[c] = run;
                run += v[c];
            }
            row[SS] = run;
#pragma unroll 4
            for (int ox = 0; ox < s; ++ox) {
                const int2 cb = bins[ox];
                part[r * ts + ox] = row[cb.y] - row[cb.x];
            }
        }
        __syncwarp();
        for (int ox = lane; ox < s; ox += 32) {
            const int2 cbx = bins[ox];
            const int nc = cbx.y - cbx.x;
            float* col = part + ox;
            float v[SS];
#pragma unroll
            for (int r = 0; r < SS; ++r) v[r] = col[r * ts];
            float run = 0.f;
#pragma unroll
            for (int r = 0; r < SS; ++r) {
                col[r * ts] = run;
                run += v[r];
            }
            col[SS * ts] = run;
#pragma unroll 4
            for (int oy = 0; oy < s; ++oy) {
                const int2 rb = bins[oy];
                dst0[oy * s + ox] = (col[rb.y * ts] - col[rb.x * ts]) / (float)((rb.y - rb.x) * nc);
            }
        }
        return;
    }
    // Any other side: the bins one after the other.
    for (int r = lane; r < S; r += 32) {
        const float* row = tile + r * (S + 1);
        for (int ox = 0; ox < s; ++ox) {
            const int2 cb = bins[ox];
            float acc = 0.f;
            for (int c = cb.x; c < cb.y; ++c) acc += row[c];
            part[r * ts + ox] = acc;
        }
    }
    __syncwarp();
    for (int ox = lane; ox < s; ox += 32) {
        const int2 cb = bins[ox];
        const int nc = cb.y - cb.x;
        for (int oy = 0; oy < s; ++oy) {
            const int2 rb = bins[oy];
            float acc = 0.f;
            for (int r = rb.x; r < rb.y; ++r) acc += part[r * ts + ox];
            dst0[oy * s + ox] = acc / (float)((rb.y - rb.x) * nc);
        }
    }
}

// Plain kernel for planes too large to stage: a thread per output pixel sums its bin from global memory.
__global__ void __launch_bounds__(256)
hmar_recon_downsample_kernel(const float* __restrict__ xhat, float* __restrict__ out, long long n_out, int S, int s) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_out) return;
    const int ox = (int)(idx % s), oy = (int)((idx / s) % s);
    const long long plane = idx / ((long long)s * s);
    const int r0 = bin_begin(oy, S, s), r1 = bin_end(oy, S, s), c0 = bin_begin(ox, S, s), c1 = bin_end(ox, S, s);
    const float* src = xhat + plane * S * S;
    float acc = 0.f;
    for (int r = r0; r < r1; ++r) {
        float row = 0.f;
        for (int c = c0; c < c1; ++c) row += __ldg(src + (long long)r * S + c);
        acc += row;
    }
    out[idx] = acc / (float)((r1 - r0) * (c1 - c0));
}

}  // namespace

cudaError_t launch_recon_accumulate(float* xhat, const float* codebook, const int* tokens_old, const int* tokens_new,
                                    const unsigned char* mask, int* tokens_out, int B, int C, int V, int side, int out_side,
                                    cudaStream_t stream) {
    if (side <= kStageMaxSide && out_side <= kStageMaxOut) {
        const int n_groups = (C + kStageChannels - 1) / kStageChannels;
        {
            KernelTimer timer("hmar_recon_accumulate_kernel", stream);
            hmar_recon_accumulate_staged_kernel<<<(unsigned)B * n_groups, 256, 0, stream>>>(xhat, codebook, tokens_old, tokens_new, mask,
                                                                                            tokens_out, C, V, side, out_side, n_groups);
        }
        count_launch(1);
        return cudaGetLastError();
    }
    const long long n_pix = (long long)B * out_side * out_side;
    const unsigned grid = (unsigned)((n_pix + 255) / 256);
    {
        KernelTimer timer("hmar_recon_accumulate_kernel", stream);
        hmar_recon_accumulate_kernel<<<grid, 256, 0, stream>>>(xhat, codebook, tokens_old, tokens_new, mask, tokens_out, B, C, V,
                                                              side, out_side);
    }
    count_launch(1);
    return cudaGetLastError();
}


cudaError_t launch_recon_downsample(const float* xhat, float* out, int B, int C, int in_side, int out_side,
                                    cudaStream_t stream) {
    const long long n_planes = (long long)B * C;
    if (in_side == out_side) {                              // every bin is one pixel: a copy, bit for bit
        return cudaMemcpyAsync(out, xhat, (size_t)n_planes * in_side * in_side * sizeof(float), cudaMemcpyDeviceToDevice, stream);
    }
    if (in_side <= kDownStageMaxSide) {
        const size_t per_warp = ((size_t)in_side * (in_side + 1) + (size_t)(in_side + 1) * (out_side | 1)) * sizeof(float);
        int warps = (int)(kDownStageSmem / per_warp);
        warps = warps > 8 ? 8 : warps;                      // >= 2 at the largest staged plane
        const size_t smem = per_warp * warps;
        const unsigned grid = (unsigned)((n_planes + warps - 1) / warps);
        cudaError_t e = cudaSuccess;
        KernelTimer timer("hmar_recon_downsample_kernel", stream);
        auto go = [&](auto kernel) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDownStageSmem);
            if (e == cudaSuccess) kernel<<<grid, warps * 32, smem, stream>>>(xhat, out, n_planes, in_side, out_side, warps);
        };
        if (in_side == 16) go(hmar_recon_downsample_staged_kernel<16>);
        else if (in_side == 32) go(hmar_recon_downsample_staged_kernel<32>);
        else if (in_side == 64) go(hmar_recon_downsample_staged_kernel<64>);
        else go(hmar_recon_downsample_staged_kernel<0>);
        if (e != cudaSuccess) return e;
        count_launch(1);
        return cudaGetLastError();
    }
    const long long n_out = n_planes * out_side * out_side;
    {
        KernelTimer timer("hmar_recon_downsample_kernel", stream);
        hmar_recon_downsample_kernel<<<(unsigned)((n_out + 255) / 256), 256, 0, stream>>>(xhat, out, n_out, in_side, out_side);
    }
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace hmar
