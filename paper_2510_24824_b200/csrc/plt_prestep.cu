// Pre-step kernel of a CLP decode step: puts what f_qkv of Algorithm 3 produced for this step where the
// attention reads it, and evaluates the head-wise gate linear f_gate of the same algorithm.
//   * the first loop's K, V row is appended to the shared cache at position cut_1 - 1 (Algorithm 1: the decode step returns the updated cache);
//   * each later loop's row replaces the oldest entry of its window, slot (cut_l - 1) mod w (a non-first loop keeps
//     only its w newest entries, Sec. 2.2.2);
//   * gate_logits[b, l, h] = <w_gate[h], Q[b, l, h]> + b_gate[h] for loops 2..L (one scalar per head).
// One block per (sequence, loop): the dot products of the gate (a warp takes four heads at a time), then 16-byte
// copies of the two rows.
// One launch instead of three; the attention kernels follow in the same stream.
#include <cuda_bf16.h>

#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"

namespace plt {

namespace {

constexpr int kPreThreads = 256;

// FP8: the caches hold E4M3 codes; the new rows (bf16) are quantised on the way in: code = round to nearest even of
// x / scale[head] in fp32, clamped to the largest finite magnitude.
// Eight bf16 values -> eight E4M3 codes for one scale.
__device__ __forceinline__ uint32_t e4m3x2_from(float lo, float hi) {
    unsigned short r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint2 quantise8(uint4 v, float scale) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __fdiv_rn(__uint_as_float(w[i] << 16), scale);
        const float hi = __fdiv_rn(__uint_as_float(w[i] & 0xffff0000u), scale);
        c[i] = e4m3x2_from(lo, hi);
    }
    return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

template <bool BF16, bool FP8>
__global__ void __launch_bounds__(kPreThreads) plt_decode_prestep(const __grid_constant__ Params p, const void* k_new,
                                                                  const void* v_new, const float* w_gate,
                                                                  const float* b_gate, float* gate_out) {
    using T = typename std::conditional<BF16, __nv_bfloat16, float>::type;
    grid_launch_dependents();   // the attention kernel's blocks may be set up meanwhile; they wait for this grid
    const int b = blockIdx.x / p.L, l = blockIdx.x % p.L;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;
    const int32_t n = seq_len_clamped(p, b, flags);
    int cut = n - p.delta[l];
    cut = cut > 0 ? cut : 0;

    if (l > 0) {
        // head-wise gate linear; written for every sequence and loop (the attention ignores it where cut = 0).
        // A warp takes kGateHeads heads at a time with all their loads in flight together.
        constexpr int kGateHeads = 4;
        for (int h0 = wid * kGateHeads; h0 < p.Hq; h0 += (kPreThreads / 32) * kGateHeads) {
            float acc[kGateHeads];
#pragma unroll
            for (int i = 0; i < kGateHeads; ++i) {
                const int h = h0 + i;
                acc[i] = 0.f;
                if (h < p.Hq) {
                    const T* q = (const T*)p.q + (((int64_t)b * p.L + l) * p.Hq + h) * p.d;
                    for (int j = lane; j < p.d; j += 32) {
                        float x;
                        if constexpr (BF16) x = __bfloat162float(q[j]);
                        else x = q[j];
                        acc[i] = fmaf(w_gate[(int64_t)h * p.d + j], x, acc[i]);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < kGateHeads; ++i) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
                const int h = h0 + i;
                if (lane == 0 && h < p.Hq) gate_out[((int64_t)b * (p.L - 1) + (l - 1)) * p.Hq + h] = acc[i] + b_gate[h];
            }
        }
    }

    if (cut > 0) {
        // destination rows of this loop's K and V: [Hkv] rows of d elements, kd elements apart
        using TD = typename std::conditional<FP8, uint8_t, T>::type;   // element of the caches and windows
        TD *kd, *vd;
        int64_t head_stride;
        if (l == 0) {
            const int pos = cut - 1;
            int64_t base;
            if (p.page_size > 0) {
                int page = p.page_table[(int64_t)b * p.max_pages + pos / p.page_size];
                if (page < 0 || page >= p.num_pool_pages) {
                    flags |= kDevPageIdClamped;
                    page = page < 0 ? 0 : p.num_pool_pages - 1;
                }
                base = (int64_t)page * p.kv_stride_b + (int64_t)(pos % p.page_size) * p.kv_stride_n;
            } else {
                base = (int64_t)b * p.kv_stride_b + (int64_t)pos * p.kv_stride_n;
            }
            kd = (TD*)p.k_cache + base;
            vd = (TD*)p.v_cache + base;
            head_stride = p.kv_stride_h;
        } else {
            const int slot = (cut - 1) % p.w;
            const int64_t base = ((((int64_t)b * (p.L - 1) + (l - 1)) * p.w + slot) * p.Hkv) * p.d;
            kd = (TD*)p.k_win + base;
            vd = (TD*)p.v_win + base;
            head_stride = p.d;
        }
        const int64_t src = (((int64_t)b * p.L + l) * p.Hkv) * p.d;
        const int per_row = p.d * (int)sizeof(T) / 16;   // 16-byte chunks per head row
        for (int i = tid; i < p.Hkv * per_row; i += kPreThreads) {
            const int h = i / per_row, c = i - h * per_row;
            const uint4 kk = *((const uint4*)((const T*)k_new + src + (int64_t)h * p.d) + c);
            const uint4 vv = *((const uint4*)((const T*)v_new + src + (int64_t)h * p.d) + c);
            if constexpr (FP8) {
                *((uint2*)(kd + h * head_stride) + c) = quantise8(kk, p.k_scale[h]);
                *((uint2*)(vd + h * head_stride) + c) = quantise8(vv, p.v_scale[h]);
            } else {
                *((uint4*)(kd + h * head_stride) + c) = kk;
                *((uint4*)(vd + h * head_stride) + c) = vv;
            }
        }
    }
    if (flags && tid == 0) atomicOr(p.status, flags);
}

}  // namespace

cudaError_t launch_prestep(const Params& p, bool bf16, const void* k_new, const void* v_new, const float* w_gate,
                           const float* b_gate, float* gate_out, cudaStream_t stream) {
    const unsigned grid = (unsigned)(p.B * p.L);
    if (grid == 0) return cudaSuccess;
    if (p.k_scale != nullptr) plt_decode_prestep<true, true><<<grid, kPreThreads, 0, stream>>>(p, k_new, v_new, w_gate, b_gate, gate_out);
    else if (bf16) plt_decode_prestep<true, false><<<grid, kPreThreads, 0, stream>>>(p, k_new, v_new, w_gate, b_gate, gate_out);
    else plt_decode_prestep<false, false><<<grid, kPreThreads, 0, stream>>>(p, k_new, v_new, w_gate, b_gate, gate_out);
    return cudaGetLastError();
}

}  // namespace plt
