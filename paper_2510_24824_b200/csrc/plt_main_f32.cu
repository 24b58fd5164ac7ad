// fp32 split-KV main kernel of the CLP decode attention (y_global and y_local of Algorithm 3 for all L loops).
// Plain SIMT fp32 FMA only (no tensor cores: a 1e-5 relative bound rules out tf32/bf16 products).
// Same tile plan and partial layout as the bf16 kernel: one persistent block walks its share of
// the line of 32-key tiles; the R = L * Hq/Hkv packed query rows of a KV head are kept in shared
// memory so that every K/V tile is read from global memory once for all loops.
#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"

namespace plt {

namespace {

constexpr int TK = kF32TileKeys;
constexpr int NT = kF32Threads;

template <int D>
struct F32Cfg {
    static constexpr int KROW = D + 4;              // padded K row (floats): conflict-free float4 reads
    static constexpr int RG = NT / D;               // row groups in the PV phase
    static constexpr int MAXK = kMaxRows / RG;      // accumulator rows per thread
    __host__ __device__ static size_t smem_bytes(int R, int max_batch) {
        return (size_t)(TK * KROW + TK * D + R * D + R * TK + 3 * R) * 4 + (size_t)(max_batch + 4) * 4;
    }
};

template <int D>
__global__ void __launch_bounds__(NT) plt_decode_main_f32(const __grid_constant__ Params p) {
    using C = F32Cfg<D>;
    extern __shared__ float4 smem_f4[];
    float* sK = (float*)smem_f4;                 // [TK][KROW]
    float* sV = sK + TK * C::KROW;               // [TK][D]
    float* sQ = sV + TK * D;                     // [R][D]
    float* sS = sQ + p.R * D;                    // [R][TK] scores, then probabilities
    float* sM = sS + p.R * TK;                   // [R] running max (log2 units)
    float* sL = sM + p.R;                        // [R] running sum
    float* sA = sL + p.R;                        // [R] rescale factor of the current tile
    int32_t* s_prefix = (int32_t*)(sA + p.R);

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int R = p.R;
    uint32_t flags = 0;
    grid_launch_dependents();  // the merge kernel may be set up meanwhile; it waits for this grid to complete
    build_prefix(p, s_prefix, flags);
    const int64_t T = s_prefix[p.B];
    const int cta = blockIdx.x;
    if (cta == 0)
        for (int b = tid; b <= p.B; b += NT) p.prefix[b] = s_prefix[b];
    const int nctas = plan_ctas(T, (int)gridDim.x);
    const bool in_plan = cta < nctas;
    const int64_t lo = in_plan ? cta_begin(T, cta, nctas) : 0, hi = in_plan ? cta_begin(T, cta + 1, nctas) : 0;

    const float* kc = (const float*)p.k_cache;
    const float* vc = (const float*)p.v_cache;
    const float* kwn = (const float*)p.k_win;
    const float* vwn = (const float*)p.v_win;
    const int pc_c = tid % D, pc_rg = tid / D;   // PV phase: column and row group of this thread

    PieceWalk walk(p, s_prefix, lo, hi);
    Piece pc;
    while (walk.next(pc, flags)) {
        const int kvh = pc.hg;  // one KV head per item on this path
        __syncthreads();
        for (int i = tid; i < R * D; i += NT) {
            const int r = i / D, c = i - r * D;
            const int l = r / p.G, g = r - l * p.G;
            sQ[i] = ((const float*)p.q)[(((int64_t)pc.b * p.L + l) * p.Hq + kvh * p.G + g) * D + c];
        }
        for (int r = tid; r < R; r += NT) {
            sM[r] = -INFINITY;
            sL[r] = 0.f;
        }
        float acc[C::MAXK];
#pragma unroll
        for (int k = 0; k < C::MAXK; ++k) acc[k] = 0.f;

        WinCursor cur;
        if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
        for (int t = pc.t0; t < pc.t1; ++t) {
            int key0, nvalid, wloop = 0;
            if (pc.kind == 0) {
                key0 = t * TK;
                nvalid = pc.sp.cmax - key0;
            } else {
                key0 = cur.key0;
                wloop = cur.l;
                nvalid = pc.sp.wl[wloop] - key0;
            }
            nvalid = nvalid < TK ? nvalid : TK;
            __syncthreads();  // previous tile fully consumed
            // ---- stage the K and V tile (rows at or beyond nvalid are zero) --------------------------
            for (int i = tid; i < TK * (D / 4); i += NT) {
                const int j = i / (D / 4), c4 = (i - j * (D / 4)) * 4;
                float4 kv4 = make_float4(0.f, 0.f, 0.f, 0.f), vv4 = kv4;
                if (j < nvalid) {
                    int64_t off;
                    const float *ks, *vs;
                    if (pc.kind == 0) {
                        const int key = key0 + j;
                        ks = kc;
                        vs = vc;
                        if (p.page_size > 0) {
                            int page = p.page_table[(int64_t)pc.b * p.max_pages + key / p.page_size];
                            if (page < 0 || page >= p.num_pool_pages) {
                                flags |= kDevPageIdClamped;
                                page = page < 0 ? 0 : p.num_pool_pages - 1;
                            }
                            off = (int64_t)page * p.kv_stride_b + (int64_t)(key % p.page_size) * p.kv_stride_n;
                        } else {
                            off = (int64_t)pc.b * p.kv_stride_b + (int64_t)key * p.kv_stride_n;
                        }
                        off += (int64_t)kvh * p.kv_stride_h + c4;
                    } else {
                        ks = kwn;
                        vs = vwn;
                        off = ((((int64_t)pc.b * (p.L - 1) + (wloop - 1)) * p.w + key0 + j) * p.Hkv + kvh) * D + c4;
                    }
                    kv4 = *(const float4*)(ks + off);
                    vv4 = *(const float4*)(vs + off);
                }
                *(float4*)(sK + j * C::KROW + c4) = kv4;
                *(float4*)(sV + j * D + c4) = vv4;
            }
            __syncthreads();
            // ---- scores: thread (row group wid, key lane) ---------------------------------------------
            for (int r = wid; r < R; r += NT / 32) {
                const int l = r / p.G;
                int lim;
                if (pc.kind == 0) lim = pc.sp.cut[l] - key0;
                else lim = (l == wloop) ? nvalid : 0;
                float s = 0.f;
                const float4* kr = (const float4*)(sK + lane * C::KROW);
                const float4* qr = (const float4*)(sQ + r * D);
#pragma unroll 8
                for (int c = 0; c < D / 4; ++c) {
                    const float4 a = qr[c], k4 = kr[c];
                    s = fmaf(a.x, k4.x, s);
                    s = fmaf(a.y, k4.y, s);
                    s = fmaf(a.z, k4.z, s);
                    s = fmaf(a.w, k4.w, s);
                }
                s = lane < lim ? s * p.scale_log2 : -INFINITY;
                // ---- online softmax for this row (the warp holds the whole tile row) ------------------
                float mx = s;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_old = sM[r];
                const float m_new = fmaxf(m_old, mx);
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float pj = exp2f(s - m_use);
                float sum = pj;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                sS[r * TK + lane] = pj;
                if (lane == 0) {
                    const float alpha = exp2f(m_old - m_use);
                    sA[r] = alpha;
                    sM[r] = m_new;
                    sL[r] = fmaf(sL[r], alpha, sum);
                }
            }
            __syncthreads();
            // ---- acc = acc * alpha + P V: thread (row group, column) ---------------------------------
#pragma unroll
            for (int k = 0; k < C::MAXK; ++k) {
                const int r = pc_rg + k * C::RG;
                if (r < R) {
                    float a = acc[k] * sA[r];
                    const float* pr = sS + r * TK;
#pragma unroll 8
                    for (int j = 0; j < TK; ++j) a = fmaf(pr[j], sV[j * D + pc_c], a);
                    acc[k] = a;
                }
            }
            if (pc.kind == 1) cur.advance(p, pc.sp);
        }
        __syncthreads();
        // ---- store the split partial ------------------------------------------------------------------
        const int64_t slot = slot_of(item_index(p, pc.b, pc.hg, pc.kind), cta);
        const int64_t prow = slot * R;
        if (tid == 0) note_piece(p, pc, cta);
#pragma unroll
        for (int k = 0; k < C::MAXK; ++k) {
            const int r = pc_rg + k * C::RG;
            if (r < R) p.part_acc[(prow + r) * D + pc_c] = acc[k];
        }
        for (int r = tid; r < R; r += NT) *(float2*)(p.part_ml + (prow + r) * 2) = make_float2(sM[r], sL[r]);
    }
    if (flags) atomicOr(p.status, flags);
}

}  // namespace

size_t main_f32_smem(int D, int R, int max_batch) {
    return D == 128 ? F32Cfg<128>::smem_bytes(R, max_batch) : F32Cfg<64>::smem_bytes(R, max_batch);
}

cudaError_t main_f32_prepare(int D, int R, int max_batch, int* blocks_per_sm) {
    const size_t smem = main_f32_smem(D, R, max_batch);
    const void* fn = D == 128 ? (const void*)plt_decode_main_f32<128> : (const void*)plt_decode_main_f32<64>;
    cudaError_t e = allow_max_dynamic_smem(fn);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, NT, smem);
}

cudaError_t launch_main_f32(const Params& p, int grid, size_t smem, cudaStream_t stream) {
    if (p.d == 128) plt_decode_main_f32<128><<<grid, NT, smem, stream>>>(p);
    else plt_decode_main_f32<64><<<grid, NT, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace plt
