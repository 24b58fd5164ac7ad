// Merge kernel of the CLP decode attention: combines the split partials of the shared-cache
// attention (y_global, Algorithm 3 line 2) and of the window attention (y_local, line 3) by their
// running maxima, normalises each, and applies the sigmoid gate mix of Eq. 2 (lines 4-5):
//   O = g * y_local + (1 - g) * y_global for loops 2..L,  O = y_global for loop 1.
// One warp per output row (b, l, h).
#include <cuda_bf16.h>

#include "plt_common.cuh"
#include "plt_host.h"

namespace plt {

template <int D>
struct Vec {
    static constexpr int N = D / 32;  // elements per lane
    float v[N];
};

// Sum over the pieces [s, e) of one item, rescaled to a common maximum. Returns the denominator.
template <int D>
__device__ __forceinline__ float merge_item(const Params& p, int item, int hl, int r, int64_t T, int64_t s, int64_t e,
                                            int lane, Vec<D>& y) {
#pragma unroll
    for (int i = 0; i < Vec<D>::N; ++i) y.v[i] = 0.f;
    if (s >= e) return 0.f;
    const int c0 = cta_of(T, s, p.num_ctas), c1 = cta_of(T, e - 1, p.num_ctas);
    float mstar = -INFINITY;
    for (int c = c0; c <= c1; ++c) {
        // With fewer tiles than blocks some blocks in between own nothing and wrote no partial.
        if (cta_begin(T, c, p.num_ctas) == cta_begin(T, c + 1, p.num_ctas)) continue;
        const int64_t row = (slot_of(item, c) * p.hpc + hl) * p.R + r;
        mstar = fmaxf(mstar, p.part_ml[row * 2]);
    }
    if (mstar == -INFINITY) return 0.f;  // no visible key anywhere
    float denom = 0.f;
    for (int c = c0; c <= c1; ++c) {
        if (cta_begin(T, c, p.num_ctas) == cta_begin(T, c + 1, p.num_ctas)) continue;
        const int64_t row = (slot_of(item, c) * p.hpc + hl) * p.R + r;
        const float2 ml = *(const float2*)(p.part_ml + row * 2);
        const float sc = exp2f(ml.x - mstar);  // exp2f(-inf) = 0 for pieces that saw nothing
        denom = fmaf(ml.y, sc, denom);
        const float* a = p.part_acc + row * D + lane * Vec<D>::N;
#pragma unroll
        for (int i = 0; i < Vec<D>::N; ++i) y.v[i] = fmaf(a[i], sc, y.v[i]);
    }
    return denom;
}

template <int D, bool BF16>
__global__ void __launch_bounds__(128) plt_decode_reduce(const __grid_constant__ Params p) {
    const int lane = threadIdx.x & 31;
    const int64_t row_id = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (row_id >= (int64_t)p.B * p.L * p.Hq) return;
    const int h = (int)(row_id % p.Hq);
    const int l = (int)((row_id / p.Hq) % p.L);
    const int b = (int)(row_id / ((int64_t)p.Hq * p.L));
    const int kvh = h / p.G, g = h - kvh * p.G;
    const int hg = kvh / p.hpc, hl = kvh - hg * p.hpc;
    const int r = l * p.G + g;

    uint32_t flags = 0;
    SeqPlan sp;
    seq_plan(p, b, sp, flags);
    const int64_t T = p.prefix[p.B];
    const int per = sp.gt + sp.lt;
    const int64_t base = (int64_t)p.prefix[b] + (int64_t)hg * per;

    Vec<D> yg, yl;
    float out[Vec<D>::N];
    int cut = 0;
#pragma unroll
    for (int k = 0; k < kMaxLoops; ++k)
        if (k == l) cut = sp.cut[k];
    if (cut == 0) {
#pragma unroll
        for (int i = 0; i < Vec<D>::N; ++i) out[i] = 0.f;
    } else {
        const float dg = merge_item<D>(p, item_index(p, b, hg, 0), hl, r, T, base, base + sp.gt, lane, yg);
        const float ig = dg > 0.f ? 1.f / dg : 0.f;
        if (l == 0) {
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i) out[i] = yg.v[i] * ig;
        } else {
            const float dl = merge_item<D>(p, item_index(p, b, hg, 1), hl, r, T, base + sp.gt, base + per, lane, yl);
            const float il = dl > 0.f ? 1.f / dl : 0.f;  // empty window: y_local = 0
            const float x = p.gate_logits[((int64_t)b * (p.L - 1) + (l - 1)) * p.Hq + h];
            const float gate = 1.f / (1.f + expf(-x));
#pragma unroll
            for (int i = 0; i < Vec<D>::N; ++i) out[i] = gate * (yl.v[i] * il) + (1.f - gate) * (yg.v[i] * ig);
        }
    }
    const int64_t o = row_id * D + lane * Vec<D>::N;
    if (BF16) {
        __nv_bfloat16* dst = (__nv_bfloat16*)p.out + o;
#pragma unroll
        for (int i = 0; i < Vec<D>::N; i += 2) *(__nv_bfloat162*)(dst + i) = __floats2bfloat162_rn(out[i], out[i + 1]);
    } else {
        float* dst = (float*)p.out + o;
#pragma unroll
        for (int i = 0; i < Vec<D>::N; ++i) dst[i] = out[i];
    }
}

cudaError_t launch_reduce(const Params& p, bool bf16, cudaStream_t stream) {
    const int64_t rows = (int64_t)p.B * p.L * p.Hq;
    if (rows == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((rows + 3) / 4);
    if (p.d == 128) {
        if (bf16) plt_decode_reduce<128, true><<<grid, 128, 0, stream>>>(p);
        else plt_decode_reduce<128, false><<<grid, 128, 0, stream>>>(p);
    } else {
        if (bf16) plt_decode_reduce<64, true><<<grid, 128, 0, stream>>>(p);
        else plt_decode_reduce<64, false><<<grid, 128, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace plt
