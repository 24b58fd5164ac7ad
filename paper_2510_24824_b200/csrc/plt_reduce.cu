// Merge kernel of the CLP decode attention: combines the split partials of the shared-cache
// attention (y_global of Algorithm 3) and of the window attention (y_local of Algorithm 3) by their
// running maxima, normalises each, and applies the sigmoid gate mix of Eq. 2:
//   O = g * y_local + (1 - g) * y_global for loops 2..L,  O = y_global for loop 1.
// One block per (sequence, KV-head group, chunk of 8 packed rows); one warp per output row. Which
// blocks of the main kernel hold pieces of an item is read from the table those blocks left.
#include <cuda_bf16.h>

#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"

namespace plt {

namespace {

constexpr int kReduceWarps = 8;

template <int D>
struct Vec {
    static constexpr int N = D / 32;  // elements per lane
    float v[N];
};

template <int D>
__device__ __forceinline__ void load_vec(const float* src, Vec<D>& x) {
    if constexpr (Vec<D>::N == 4) {
        const float4 t = *(const float4*)src;
        x.v[0] = t.x; x.v[1] = t.y; x.v[2] = t.z; x.v[3] = t.w;
    } else {
        const float2 t = *(const float2*)src;
        x.v[0] = t.x; x.v[1] = t.y;
    }
}

// Sum over the pieces held by blocks [c0, c1] of one item, rescaled to a common maximum. Returns the denominator.
// An item of a small batch is spread over many blocks (one sequence of a batch of four over dozens), so the loads
// must not wait for one another: the lanes of the warp read the (maximum, denominator) pairs of 32 pieces at a time,
// the common maximum and the denominator come from warp reductions, and the partial vectors are read four pieces at a
// time with the scale factors handed round by shuffles. The order of every sum is fixed by the piece index alone.
template <int D>
__device__ __forceinline__ float merge_item(const Params& p, int item, int hl, int r, int c0, int c1, int lane,
                                            Vec<D>& y) {
#pragma unroll
    for (int i = 0; i < Vec<D>::N; ++i) y.v[i] = 0.f;
    if (c0 > c1) return 0.f;
    const int64_t row0 = (slot_of(item, c0) * p.hpc + hl) * p.R + r;
    const int64_t step = (int64_t)p.hpc * p.R;  // rows between the slots of consecutive blocks
    if (c0 == c1) {
        // The usual case: the whole item was done by one block, nothing to rescale.
        const float2 ml = *(const float2*)(p.part_ml + row0 * 2);
        if (ml.x == -INFINITY) return 0.f;
        load_vec<D>(p.part_acc + row0 * D + lane * Vec<D>::N, y);
        return ml.y;
    }
    const int np = c1 - c0 + 1;
    // common maximum: every lane takes the pieces lane, lane + 32, ...
    float mstar = -INFINITY;
    for (int j = lane; j < np; j += 32) mstar = fmaxf(mstar, p.part_ml[(row0 + j * step) * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, o));
    if (mstar == -INFINITY) return 0.f;  // no visible key anywhere
    float denom = 0.f;
    for (int j0 = 0; j0 < np; j0 += 32) {
        // scale factor and weighted denominator of piece j0 + lane
        float sc = 0.f, dl = 0.f;
        if (j0 + lane < np) {
            const float2 ml = *(const float2*)(p.part_ml + (row0 + (j0 + lane) * step) * 2);
            sc = exp2f(ml.x - mstar);  // exp2f(-inf) = 0 for pieces that saw nothing
            dl = ml.y * sc;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dl += __shfl_xor_sync(0xffffffffu, dl, o);
        denom += dl;
        const int cnt = min(32, np - j0);
        for (int j = 0; j < cnt; j += 4) {
            Vec<D> a[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int jj = j + u < cnt ? j + u : cnt - 1;   // past the end: a load that is multiplied by 0
                load_vec<D>(p.part_acc + (row0 + (j0 + jj) * step) * D + lane * Vec<D>::N, a[u]);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float su = __shfl_sync(0xffffffffu, sc, (j + u) & 31);
                if (j + u >= cnt) su = 0.f;
#pragma unroll
                for (int i = 0; i < Vec<D>::N; ++i) y.v[i] = fmaf(a[u].v[i], su, y.v[i]);
            }
        }
    }
    return denom;
}

template <int D, bool BF16>
__global__ void __launch_bounds__(kReduceWarps * 32) plt_decode_reduce(const __grid_constant__ Params p, const int chunks) {
    // The next kernel in the stream (the main kernel of the following step, or whatever the caller enqueued with
    // programmatic serialisation) may be set up once every block of this grid has started.
    grid_launch_dependents();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int HG = p.Hkv / p.hpc;
    const int chunk = (int)(blockIdx.x % chunks);
    const int hg = (int)((blockIdx.x / chunks) % HG);
    const int b = (int)(blockIdx.x / (chunks * HG));
    const int row = chunk * kReduceWarps + wid;   // packed row of this head group: hl * R + r
    if (row >= p.hpc * p.R) return;
    const int hl = row / p.R, r = row - hl * p.R;
    const int lq = r / p.G, g = r - lq * p.G;        // lq = loop * Qn + token of the step
    const int l = lq / p.Qn, newer = p.Qn - 1 - lq % p.Qn;   // tokens of this loop in the step that are newer than the row's
    const int h = (hg * p.hpc + hl) * p.G + g;

    // What the caller passed (length, window length, gate logit) is read while the main kernel still drains; this
    // row's loop alone decides what is merged: cut = keys of the shared cache it may see, wl = its window's valid slots.
    uint32_t flags = 0;
    const int32_t n = seq_len_clamped(p, b, flags);
    int cut_loop = n - p.delta[l];                    // keys the loop's newest token sees
    cut_loop = cut_loop > 0 ? cut_loop : 0;
    int cut = cut_loop - newer;                       // keys this row sees
    cut = cut > 0 ? cut : 0;
    int wl = 0;
    float x = 0.f;
    if (l > 0) {
        wl = cut_loop < p.w ? cut_loop : p.w;
        if (p.win_lens != nullptr && cut_loop > 0) {
            wl = p.win_lens[b * (p.L - 1) + (l - 1)];
            wl = wl < 0 ? 0 : (wl > p.w ? p.w : wl);
        }
        // wl > 0 says that the loop's window item exists; a row that sees none of its slots finds an empty partial
        x = p.gate_logits[(((int64_t)b * (p.L - 1) + (l - 1)) * p.Qn + (lq - l * p.Qn)) * p.Hq + h];
    }
    const int item_g = item_index(p, b, hg, 0), item_l = item_index(p, b, hg, 1);

    // From here on the main kernel's results are read: first which of its blocks hold the pieces of the two items
    // (the table those blocks left), then the pieces. Both items' loads are issued together.
    grid_dependency_wait();
    int2 rg = make_int2(0, -1), rl = make_int2(0, -1);
    if (cut > 0) rg = *(const int2*)(p.item_blocks + 2 * item_g);
    if (wl > 0) rl = *(const int2*)(p.item_blocks + 2 * item_l);

    Vec<D> yg, yl;
    float out[Vec<D>::N];
    if (cut == 0) {
#pragma unroll
        for (int i = 0; i < Vec<D>::N; ++i) out[i] = 0.f;
    } else if (rg.x == rg.y && rl.x >= rl.y) {
        // The usual case: each item was done by one block (or the window is empty); nothing to rescale.
        const int64_t row_g = (slot_of(item_g, rg.x) * p.hpc + hl) * p.R + r;
        const int64_t row_l = (slot_of(item_l, rl.x) * p.hpc + hl) * p.R + r;
        const bool has_l = rl.x == rl.y;
        float2 mg = *(const float2*)(p.part_ml + row_g * 2), ml = make_float2(-INFINITY, 0.f);
        load_vec<D>(p.part_acc + row_g * D + lane * Vec<D>::N, yg);
        if (has_l) {
            ml = *(const float2*)(p.part_ml + row_l * 2);
            load_vec<D>(p.part_acc + row_l * D + lane * Vec<D>::N, yl);
        }
        const float ig = (mg.x != -INFINITY && mg.y > 0.f) ? 1.f / mg.y : 0.f;
        if (l == 0) {
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i) out[i] = yg.v[i] * ig;
        } else {
            const float il = (has_l && ml.x != -INFINITY && ml.y > 0.f) ? 1.f / ml.y : 0.f;  // empty window: y_local = 0
            const float gate = 1.f / (1.f + expf(-x));
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i)
                out[i] = gate * (has_l ? yl.v[i] * il : 0.f) + (1.f - gate) * (yg.v[i] * ig);
        }
    } else {
        const float dg = merge_item<D>(p, item_g, hl, r, rg.x, rg.y, lane, yg);
        const float ig = dg > 0.f ? 1.f / dg : 0.f;
        if (l == 0) {
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i) out[i] = yg.v[i] * ig;
        } else {
            const float dl = merge_item<D>(p, item_l, hl, r, rl.x, rl.y, lane, yl);
            const float il = dl > 0.f ? 1.f / dl : 0.f;  // empty window: y_local = 0
            const float gate = 1.f / (1.f + expf(-x));
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i) out[i] = gate * (yl.v[i] * il) + (1.f - gate) * (yg.v[i] * ig);
        }
    }
    const int64_t o = (((int64_t)b * p.L * p.Qn + lq) * p.Hq + h) * D + lane * Vec<D>::N;
    if (BF16) {
        __nv_bfloat16* dst = (__nv_bfloat16*)p.out + o;
        if constexpr (Vec<D>::N == 4) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(out[0], out[1]), hi = __floats2bfloat162_rn(out[2], out[3]);
            uint2 u;
            u.x = *(const uint32_t*)&lo;
            u.y = *(const uint32_t*)&hi;
            *(uint2*)dst = u;
        } else {
            *(__nv_bfloat162*)dst = __floats2bfloat162_rn(out[0], out[1]);
        }
    } else {
        float* dst = (float*)p.out + o;
        if constexpr (Vec<D>::N == 4) *(float4*)dst = make_float4(out[0], out[1], out[2], out[3]);
        else *(float2*)dst = make_float2(out[0], out[1]);
    }
}

template <int D, bool BF16>
cudaError_t launch_one(const Params& p, unsigned grid, int chunks, bool overlap, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kReduceWarps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, plt_decode_reduce<D, BF16>, p, chunks);
}

}  // namespace

// `overlap`: launch with programmatic stream serialisation, so that the blocks of this kernel are
// set up while the main kernel (the launch before it in the stream) drains; they wait for its
// completion in grid_dependency_wait() before reading anything it wrote.
cudaError_t launch_reduce(const Params& p, bool bf16, bool overlap, cudaStream_t stream) {
    const int rows = p.hpc * p.R;
    const int chunks = (rows + kReduceWarps - 1) / kReduceWarps;
    const int64_t blocks = (int64_t)p.B * (p.Hkv / p.hpc) * chunks;
    if (blocks == 0) return cudaSuccess;
    const unsigned grid = (unsigned)blocks;
    if (p.d == 128) return bf16 ? launch_one<128, true>(p, grid, chunks, overlap, stream)
                                : launch_one<128, false>(p, grid, chunks, overlap, stream);
    return bf16 ? launch_one<64, true>(p, grid, chunks, overlap, stream)
                : launch_one<64, false>(p, grid, chunks, overlap, stream);
}

}  // namespace plt
