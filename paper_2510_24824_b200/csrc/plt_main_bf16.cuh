// bf16 split-KV main kernel of the CLP decode attention (y_global and y_local of Algorithm 3 for all L loops),
// warp-level tensor-core products with the KEYS as the M dimension.
//
// One persistent thread block owns an equal share of the line of key tiles of all sequences. A
// producer warp streams K/V tiles of the shared first-loop cache (and of the windows of loops 2..L)
// into a shared-memory ring with tiled TMA loads (128-byte swizzle). Each consumer warp owns KS
// 16-key slices of a tile for one KV head and ALL packed query rows of that head (all L loop-queries
// times all GQA heads, 8 NT rows; RW warps split the rows when there are more than 32):
//
//   S^T [16 keys x 8 NT]   = K_slice [16 x d] . Q^T          A = K via ldmatrix, B = query rows in registers
//   O^T [d x 8 NT]        += V_slice^T [d x 16] . P^T         A = V via ldmatrix.trans, B = P^T via movmatrix
//   l   [. x 8 NT]        += ones [16 x 16] . P^T             softmax denominators, every row alike
//
// With the rows in the N dimension (granularity 8) nothing is padded to 16-row tiles, the K and V
// fragments are loaded once for all rows, and the softmax needs no shuffles on the per-tile path:
// the reference maximum of a row is updated lazily (a warp vote triggers the true row maxima and the
// rescale of the accumulators only when a score exceeds the reference by more than kSlack powers
// of two). Every K/V byte is read from HBM once and used by every loop.
#pragma once
#include <cuda_bf16.h>
#include "plt_common.cuh"
#include "plt_ptx.cuh"

namespace plt {

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every barrier wait gives up after ~2 s
constexpr float kSlack = 8.f;
constexpr float kNoMax = -1e30f;   // reference maximum of a row that has seen no key yet (finite, so that no select is needed)
constexpr uint32_t kOnesBf16x2 = 0x3f803f80u;
constexpr float kHeavyShareInv = 4.f;   // a probability above 1/4 of its row's denominator so far gets a second bf16 term

template <int D, int NT, int RW, int HPC, int KW, int KS, bool FP8 = false>
struct TCfg {
    static constexpr int ES = FP8 ? 1 : 2;          // bytes per cache element: E4M3 codes or bf16
    static constexpr int NH = D * ES / 128;         // 128-byte pieces of a head row (one TMA box each)
    static constexpr int TK = 16 * KW * KS;         // keys per tile: KW warps along the keys, KS 16-key slices each
    static constexpr int NCW = HPC * KW * RW;       // consumer warps
    static constexpr int NTHREADS = (NCW + 1) * 32;
    static constexpr int ROWS_W = 8 * NT;           // packed rows per warp
    // register budget: up to 16 rows per warp two to four blocks share an SM, above that one block has it all
    static constexpr int MIN_BLOCKS = NT <= 2 ? (NCW <= 2 ? 4 : (NCW <= 4 ? 2 : 1)) : 1;
    static constexpr int BOX_BYTES = 128 * TK * HPC;        // one TMA box: [HPC][TK][64 elements]
    static constexpr int TENSOR_BYTES = NH * BOX_BYTES;     // K (or V) part of a stage
    static constexpr int STAGE_BYTES = 2 * TENSOR_BYTES;
    static constexpr int MROW = D + 4;                      // padded row of the merge buffer (floats): no bank conflicts
    static constexpr int MERGE_ACC_FLOATS = KW > 1 ? HPC * RW * ROWS_W * MROW : 0;
    static constexpr int MERGE_ML_FLOATS = KW > 1 ? HPC * RW * KW * ROWS_W * 2 : 0;
    static constexpr int kMaxStages = 12;
    __host__ __device__ static constexpr size_t smem_bytes(int stages, int max_batch) {
        return 1024 /* alignment slack */ + (size_t)stages * STAGE_BYTES + 2 * kMaxStages * 8 +
               (size_t)(MERGE_ACC_FLOATS + MERGE_ML_FLOATS) * 4 + (size_t)(2 * max_batch + 4) * 4;
    }
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// The softmax part of a consumer-warp step, shared by the bf16 and the E4M3 kernels: masks (boundary tiles only) and the
// lazily updated reference maxima with the rescale of the accumulators when a score outruns its reference by more than
// kSlack powers of two.
template <int D, int NT, int KS, bool MASKED>
__device__ __forceinline__ void softmax_reference(float (&s)[KS][NT][4], float (&acc)[D / 16][NT][4], float (&mref)[NT][2],
                                                  float (&lacc)[NT][4], const int (&lim)[NT][2], float scale_log2,
                                                  int kbase, int grp) {
    // ---- per-loop causal cutoff / window length (only on boundary tiles) ------------------------------
    if (MASKED) {
#pragma unroll
        for (int ki = 0; ki < KS; ++ki)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int kk = kbase + ki * 16 + grp + (e >= 2 ? 8 : 0);
                    if (kk >= lim[nt][e & 1]) s[ki][nt][e] = -INFINITY;
                }
    }
    // ---- lazily updated reference maxima ----------------------------------------------------------------
    bool grow = false;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float mx = fmaxf(s[0][nt][j], s[0][nt][2 + j]);
#pragma unroll
            for (int ki = 1; ki < KS; ++ki) mx = fmaxf(mx, fmaxf(s[ki][nt][j], s[ki][nt][2 + j]));
            grow = grow || (fmaf(mx, scale_log2, -mref[nt][j]) > kSlack);  // true for a row's first visible key
        }
    if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float mx = fmaxf(s[0][nt][j], s[0][nt][2 + j]);
#pragma unroll
                for (int ki = 1; ki < KS; ++ki) mx = fmaxf(mx, fmaxf(s[ki][nt][j], s[ki][nt][2 + j]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                const float m_new = fmaxf(mref[nt][j], mx * scale_log2);
                const float alpha = fast_exp2(mref[nt][j] - m_new);   // 1 while the row is empty, 0 at its first key
                mref[nt][j] = m_new;
                lacc[nt][j] *= alpha;
                lacc[nt][2 + j] *= alpha;
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt) {
                    acc[mt][nt][j] *= alpha;
                    acc[mt][nt][2 + j] *= alpha;
                }
            }
    }
}

// Turns the scores of a step into probabilities in place (fp32, relative to the reference maxima) and, for bf16
// weights, says whether the tile is "heavy". bf16 probabilities carry 8 significant bits; where a single key holds a
// large share of a row's weight that rounding shows in the output (rows with a few dominant keys and large V: up to
// 1e-2 at |O| ~ 5), so heavy tiles are multiplied with V in two terms, p = hi + lo with hi = bf16(p), lo = bf16(p - hi),
// both also summed into the denominators. A tile is heavy when some probability of it exceeds 1/4 of the denominator
// its row has accumulated so far; the final denominator is at least that, so every key that ends up with more than
// 1/4 of a row's weight is covered, and so are the first tiles of every piece (about the first 64 keys on rows with
// N(0,1) scores). Measured: with the second term the worst error on rows with tripled K/V is the output rounding
// (0.83 of the 2e-2 bound for every launch variant and seed tried; 0.8-1.2 without it, where the lazily placed
// reference leaves the dominant key's weight inexact) at 0.5-3.6 % of the step time on the four bf16 workloads.
template <int NT, int KS, bool F16>
__device__ __forceinline__ bool softmax_probabilities(float (&s)[KS][NT][4], const float (&mref)[NT][2],
                                                      const float (&lacc)[NT][4], float scale_log2) {
    bool heavy = false;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float pm0 = 0.f, pm1 = 0.f;
#pragma unroll
        for (int ki = 0; ki < KS; ++ki) {
            s[ki][nt][0] = fast_exp2(fmaf(s[ki][nt][0], scale_log2, -mref[nt][0]));
            s[ki][nt][1] = fast_exp2(fmaf(s[ki][nt][1], scale_log2, -mref[nt][1]));
            s[ki][nt][2] = fast_exp2(fmaf(s[ki][nt][2], scale_log2, -mref[nt][0]));
            s[ki][nt][3] = fast_exp2(fmaf(s[ki][nt][3], scale_log2, -mref[nt][1]));
            pm0 = fmaxf(pm0, fmaxf(s[ki][nt][0], s[ki][nt][2]));
            pm1 = fmaxf(pm1, fmaxf(s[ki][nt][1], s[ki][nt][3]));
        }
        if (!F16) heavy = heavy || pm0 * kHeavyShareInv > lacc[nt][0] || pm1 * kHeavyShareInv > lacc[nt][1];
    }
    if (F16) return false;   // f16 weights carry 11 bits
    return __any_sync(0xffffffffu, heavy);
}

// The probabilities of a step, packed (bf16 or, F16, f16) and transposed into the B operand of the second product.
// LO: what the bf16 rounding of the probabilities dropped, p - bf16(p), instead of the probabilities themselves.
template <int NT, int KS, bool F16, bool LO>
__device__ __forceinline__ void softmax_weights(const float (&p)[KS][NT][4], uint32_t (&pb)[KS][NT][2]) {
#pragma unroll
    for (int ki = 0; ki < KS; ++ki)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float p0 = p[ki][nt][0], p1 = p[ki][nt][1], p2 = p[ki][nt][2], p3 = p[ki][nt][3];
            if (LO) {
                const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
                p0 -= __uint_as_float(h01 << 16);
                p1 -= __uint_as_float(h01 & 0xffff0000u);
                p2 -= __uint_as_float(h23 << 16);
                p3 -= __uint_as_float(h23 & 0xffff0000u);
            }
            pb[ki][nt][0] = movmatrix_trans((F16 ? pack_f16x2(p0, p1) : pack_bf16x2(p0, p1)));   // keys 0-7 of the slice
            pb[ki][nt][1] = movmatrix_trans((F16 ? pack_f16x2(p2, p3) : pack_bf16x2(p2, p3)));   // keys 8-15
        }
}

// One consumer-warp step: this warp's 16 KS keys of a tile against its 8 NT packed rows.
// Thread (grp = lane / 4, tq = lane % 4) holds of S^T, per 16-key slice ki, the keys grp and grp + 8 and, per 8-row
// group nt, the rows 2 tq and 2 tq + 1: s[ki][nt][0..1] = key grp, s[ki][nt][2..3] = key grp + 8. lim[nt][j] (keys
// visible to row 8 nt + 2 tq + j) and nvalid (keys that hold data) count from the first key of the tile and are used
// only when MASKED. mref[nt][j] is the reference maximum (log2 units; kNoMax while the row has seen no key) the
// accumulators of that row are scaled to; lacc[nt][j] the row's softmax denominator, accumulated on the tensor cores
// from exactly the bf16-rounded weights that multiply V.
template <int D, int NT, int KS, int HPC, int KW, int TKEYS, int BOXB, bool MASKED>
__device__ __forceinline__ void process_keys(uint32_t sK, uint32_t sV, const uint32_t (&qb)[D / 16][NT][2],
                                             float (&acc)[D / 16][NT][4], float (&mref)[NT][2], float (&lacc)[NT][4],
                                             const int (&lim)[NT][2], int nvalid, float scale_log2, int lane, int kw,
                                             int h_local) {
    const int grp = lane >> 2, tq = lane & 3;
    const int kbase = kw * 16 * KS;   // first key of this warp in the tile
    // ---- S^T = K Q^T ---------------------------------------------------------------------------------
    // Shared-memory rows are 128 bytes (64 elements) with the 16-byte chunks XOR-swizzled by (row & 7); the two
    // 64-element halves of a 128-wide head are BOXB bytes apart. Chunk (2 k + dhalf) ^ x of a row = base ^ (k << 5).
    float s[KS][NT][4];
#pragma unroll
    for (int ki = 0; ki < KS; ++ki)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) s[ki][nt][0] = s[ki][nt][1] = s[ki][nt][2] = s[ki][nt][3] = 0.f;
    {
        const int key = kbase + (lane & 7) + ((lane >> 3) & 1) * 8;
        const uint32_t base = sK + (uint32_t)((h_local * TKEYS + key) * 128 + (((lane >> 4) ^ (key & 7)) << 4));
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t addr = (base ^ (uint32_t)((ks & 3) << 5)) + (uint32_t)((ks >> 2) * BOXB);
#pragma unroll
            for (int ki = 0; ki < KS; ++ki) {
                uint32_t a[4];
                ldmatrix_x4(addr + (uint32_t)(ki * 16 * 128), a[0], a[1], a[2], a[3]);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(s[ki][nt], a, qb[ks][nt][0], qb[ks][nt][1]);
            }
        }
    }
    softmax_reference<D, NT, KS, MASKED>(s, acc, mref, lacc, lim, scale_log2, kbase, grp);
    const bool heavy = softmax_probabilities<NT, KS, false>(s, mref, lacc, scale_log2);   // s holds probabilities now
    // ---- O^T += V^T P^T, denominators += 1 P^T --------------------------------------------------------
    const int vkey = kbase + (lane & 7) + (lane >> 4) * 8;
    const uint32_t vbase = sV + (uint32_t)((h_local * TKEYS + vkey) * 128 + ((((lane >> 3) & 1) ^ (vkey & 7)) << 4));
    uint32_t mask_lo[KS], mask_hi[KS];
    if (MASKED) {
        // Rows at or beyond nvalid may hold anything (uninitialised cache slots): force them to 0 so that
        // 0 * garbage cannot produce NaN.
#pragma unroll
        for (int ki = 0; ki < KS; ++ki) {
            const int k0 = kbase + ki * 16 + 2 * tq;
            mask_lo[ki] = (k0 < nvalid ? 0x0000ffffu : 0u) | (k0 + 1 < nvalid ? 0xffff0000u : 0u);
            mask_hi[ki] = (k0 + 8 < nvalid ? 0x0000ffffu : 0u) | (k0 + 9 < nvalid ? 0xffff0000u : 0u);
        }
    }
    auto multiply_v = [&](const uint32_t (&pb)[KS][NT][2]) {
#pragma unroll
        for (int mt = 0; mt < D / 16; ++mt) {
            const uint32_t addr = (vbase ^ (uint32_t)((mt & 3) << 5)) + (uint32_t)((mt >> 2) * BOXB);
#pragma unroll
            for (int ki = 0; ki < KS; ++ki) {
                uint32_t a[4];
                ldmatrix_x4_trans(addr + (uint32_t)(ki * 16 * 128), a[0], a[1], a[2], a[3]);
                if (MASKED) {
                    a[0] &= mask_lo[ki];
                    a[1] &= mask_lo[ki];
                    a[2] &= mask_hi[ki];
                    a[3] &= mask_hi[ki];
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(acc[mt][nt], a, pb[ki][nt][0], pb[ki][nt][1]);
            }
        }
        const uint32_t ones[4] = {kOnesBf16x2, kOnesBf16x2, kOnesBf16x2, kOnesBf16x2};
#pragma unroll
        for (int ki = 0; ki < KS; ++ki)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(lacc[nt], ones, pb[ki][nt][0], pb[ki][nt][1]);
    };
    if (heavy) {   // rare: the second term of the probabilities first, in a pass of its own
        uint32_t pl[KS][NT][2];
        softmax_weights<NT, KS, false, true>(s, pl);
        multiply_v(pl);
    }
    uint32_t pb[KS][NT][2];
    softmax_weights<NT, KS, false, false>(s, pb);
    multiply_v(pb);
}

// The same step for caches of E4M3 codes (d = 128: one 128-byte row per key). The codes convert exactly to f16, so the
// products run as f16 mma with the query rows and the probabilities in f16. ldmatrix moves 16-bit units, i.e. PAIRS of
// codes, so the fragments come out permuted; both permutations are absorbed without data movement:
//   S^T: a thread gets d = 16 c + 4 tq .. + 3 of key grp (chunk c of 16 codes). The contraction index may be permuted
//        freely as long as B uses the same order: the query fragments qb are loaded in that order (see the caller).
//   O^T: ldmatrix.trans hands a thread the 2 x 2 block keys (2 tq, 2 tq + 1) x d (2 grp, 2 grp + 1); one byte
//        permute splits it into the rows d = 2 grp and d = 2 grp + 1, so accumulator row grp is d = 16 mt + 2 grp and
//        row grp + 8 is d = 16 mt + 2 grp + 1 (the caller stores accordingly).
// scale_log2 already contains the K scale of the head; the V scale is applied when the piece is stored.
template <int D, int NT, int KS, int HPC, int KW, int TKEYS, bool MASKED>
__device__ __forceinline__ void process_keys_fp8(uint32_t sK, uint32_t sV, const uint32_t (&qb)[D / 16][NT][2],
                                                 float (&acc)[D / 16][NT][4], float (&mref)[NT][2], float (&lacc)[NT][4],
                                                 const int (&lim)[NT][2], int nvalid, float scale_log2, int lane, int kw,
                                                 int h_local) {
    static_assert(D == 128, "E4M3 caches: head dimension 128 only");
    const int grp = lane >> 2, tq = lane & 3;
    const int kbase = kw * 16 * KS;
    float s[KS][NT][4];
#pragma unroll
    for (int ki = 0; ki < KS; ++ki)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) s[ki][nt][0] = s[ki][nt][1] = s[ki][nt][2] = s[ki][nt][3] = 0.f;
    {
        const int key = kbase + (lane & 7) + ((lane >> 3) & 1) * 8;
        const uint32_t base = sK + (uint32_t)((h_local * TKEYS + key) * 128 + (((lane >> 4) ^ (key & 7)) << 4));
#pragma unroll
        for (int j = 0; j < D / 32; ++j) {          // chunks 2 j and 2 j + 1 (16 codes each) of every key
            const uint32_t addr = base ^ (uint32_t)(j << 5);
#pragma unroll
            for (int ki = 0; ki < KS; ++ki) {
                uint32_t r[4];   // keys 0-7 / 8-15 of chunk 2 j, keys 0-7 / 8-15 of chunk 2 j + 1
                ldmatrix_x4(addr + (uint32_t)(ki * 16 * 128), r[0], r[1], r[2], r[3]);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const uint32_t a[4] = {e4m3x2_to_f16x2(r[2 * c]), e4m3x2_to_f16x2(r[2 * c + 1]),
                                           e4m3x2_to_f16x2(r[2 * c] >> 16), e4m3x2_to_f16x2(r[2 * c + 1] >> 16)};
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_f16_16816(s[ki][nt], a, qb[2 * j + c][nt][0], qb[2 * j + c][nt][1]);
                }
            }
        }
    }
    softmax_reference<D, NT, KS, MASKED>(s, acc, mref, lacc, lim, scale_log2, kbase, grp);
    softmax_probabilities<NT, KS, true>(s, mref, lacc, scale_log2);   // f16 weights carry 11 bits: no second term
    uint32_t pb[KS][NT][2];
    softmax_weights<NT, KS, true, false>(s, pb);
    {
        const int key = kbase + (lane & 7) + (lane >> 4) * 8;
        const uint32_t base = sV + (uint32_t)((h_local * TKEYS + key) * 128 + ((((lane >> 3) & 1) ^ (key & 7)) << 4));
        uint32_t mask_lo[KS], mask_hi[KS];
        if (MASKED) {
#pragma unroll
            for (int ki = 0; ki < KS; ++ki) {
                const int k0 = kbase + ki * 16 + 2 * tq;
                mask_lo[ki] = (k0 < nvalid ? 0x0000ffffu : 0u) | (k0 + 1 < nvalid ? 0xffff0000u : 0u);
                mask_hi[ki] = (k0 + 8 < nvalid ? 0x0000ffffu : 0u) | (k0 + 9 < nvalid ? 0xffff0000u : 0u);
            }
        }
#pragma unroll
        for (int j = 0; j < D / 32; ++j) {
            const uint32_t addr = base ^ (uint32_t)(j << 5);
#pragma unroll
            for (int ki = 0; ki < KS; ++ki) {
                uint32_t r[4];   // keys 0-7 of chunks 2 j, 2 j + 1, then keys 8-15 of chunks 2 j, 2 j + 1
                ldmatrix_x4_trans(addr + (uint32_t)(ki * 16 * 128), r[0], r[1], r[2], r[3]);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    // bytes (k0 d0, k0 d1, k1 d0, k1 d1) -> (k0 d0, k1 d0 | k0 d1, k1 d1)
                    const uint32_t lo = byte_perm(r[c], 0u, 0x3120u), hi = byte_perm(r[2 + c], 0u, 0x3120u);
                    uint32_t a[4] = {e4m3x2_to_f16x2(lo), e4m3x2_to_f16x2(lo >> 16), e4m3x2_to_f16x2(hi),
                                     e4m3x2_to_f16x2(hi >> 16)};
                    if (MASKED) {
                        a[0] &= mask_lo[ki];
                        a[1] &= mask_lo[ki];
                        a[2] &= mask_hi[ki];
                        a[3] &= mask_hi[ki];
                    }
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_f16_16816(acc[2 * j + c][nt], a, pb[ki][nt][0], pb[ki][nt][1]);
                }
            }
        }
        const uint32_t ones[4] = {0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u};   // f16 1.0
#pragma unroll
        for (int ki = 0; ki < KS; ++ki)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) mma_f16_16816(lacc[nt], ones, pb[ki][nt][0], pb[ki][nt][1]);
    }
}

template <int D, int NT, int RW, int HPC, int KW, int KS, bool FP8>
__global__ void __launch_bounds__(TCfg<D, NT, RW, HPC, KW, KS, FP8>::NTHREADS, TCfg<D, NT, RW, HPC, KW, KS, FP8>::MIN_BLOCKS)
plt_decode_main_bf16(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmKw, const __grid_constant__ CUtensorMap tmVw,
                     const __grid_constant__ Params p, const int stages) {
    using C = TCfg<D, NT, RW, HPC, KW, KS, FP8>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = (uint64_t*)(smem + (size_t)stages * C::STAGE_BYTES);
    uint64_t* empty_bar = full_bar + C::kMaxStages;
    float* merge_acc = (float*)(empty_bar + C::kMaxStages);
    float* merge_ml = merge_acc + C::MERGE_ACC_FLOATS;
    int32_t* s_ctl = (int32_t*)(merge_ml + C::MERGE_ML_FLOATS);  // [0] abort flag, [1] tiles issued
    int32_t* s_prefix = s_ctl + 2;                      // [B + 1] tile prefix
    int32_t* s_lens = s_prefix + p.B + 2;               // [B] clamped lengths, so that walking the pieces reads no global memory

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;
    bool ok = true;

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[1] = 0;
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], C::NCW);
        }
        mbar_fence_init();
    }
    build_prefix(p, s_prefix, flags, s_lens);  // contains __syncthreads
    // Everything above reads only what the caller passed (lengths) and writes only shared memory. This grid is launched
    // to overlap the end of the kernel before it in the stream (the pre-step kernel, or the merge kernel of the step
    // before, which still reads the partials): caches, windows and query rows are read, and the workspace is written,
    // only from here on.
    grid_dependency_wait();
    // The merge kernel may be set up from now on (it reads the gate logits, which the pre-step may have written, before
    // its own wait, hence not earlier); it waits for this grid to complete before it reads the partials.
    grid_launch_dependents();
    const int64_t T = s_prefix[p.B];
    const int cta = blockIdx.x, nctas = plan_ctas(T, (int)gridDim.x);
    if (cta == 0)
        for (int b = tid; b <= p.B; b += C::NTHREADS) p.prefix[b] = s_prefix[b];
    const bool in_plan = cta < nctas;
    const int64_t lo = in_plan ? cta_begin(T, cta, nctas) : 0, hi = in_plan ? cta_begin(T, cta + 1, nctas) : 0;

    if (wid == C::NCW) {
        // =========================== producer warp (one lane issues) ==============================
        if (lane == 0 && lo < hi) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            if (p.L > 1) {
                tma_prefetch_desc(&tmKw);
                tma_prefetch_desc(&tmVw);
            }
            const uint64_t stream_once = l2_evict_first_policy();
            uint32_t it = 0;
            int stage = 0;
            uint32_t use = 0;  // how many times `stage` has been filled before
            PieceWalk walk(p, s_prefix, lo, hi, s_lens);
            Piece pc;
            while (walk.next(pc, flags)) {
                const int head0 = pc.hg * HPC;
                WinCursor cur;
                if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
                // Paged cache: the id of the page in use and, loaded one page early so that its latency is off the
                // issue path, the id of the page after it.
                const int32_t* ptab = p.page_table + (int64_t)pc.b * p.max_pages;
                int pg = 0, in_page = 0, page_id = 0, page_next = 0;
                if (pc.kind == 0 && p.page_size > 0) {
                    pg = (pc.t0 * C::TK) / p.page_size;
                    in_page = pc.t0 * C::TK - pg * p.page_size;   // advanced by a tile per step: no division per tile
                    page_id = ptab[pg];
                    page_next = ptab[min(pg + 1, p.max_pages - 1)];
                }
                for (int t = pc.t0; t < pc.t1; ++t, ++it) {
                    const CUtensorMap *mk, *mv;
                    int c1, c3;
                    if (pc.kind == 0) {
                        const int key0 = t * C::TK;
                        mk = &tmK;
                        mv = &tmV;
                        if (p.page_size > 0) {
                            if (in_page == p.page_size) {
                                in_page = 0;
                                ++pg;
                                page_id = page_next;
                                page_next = ptab[min(pg + 1, p.max_pages - 1)];
                            }
                            int page = page_id;
                            if (page < 0 || page >= p.num_pool_pages) {
                                flags |= kDevPageIdClamped;
                                page = page < 0 ? 0 : p.num_pool_pages - 1;
                            }
                            c1 = in_page;
                            c3 = page;
                            in_page += C::TK;
                        } else {
                            c1 = key0;
                            c3 = pc.b;
                        }
                    } else {
                        mk = &tmKw;
                        mv = &tmVw;
                        c1 = cur.key0;
                        c3 = pc.b * (p.L - 1) + (cur.l - 1);
                        cur.advance(p, pc.sp);
                    }
                    if (use > 0 && ok) {
                        ok = mbar_wait_bounded(&empty_bar[stage], (use - 1) & 1, kWaitLimitNs);
                        if (!ok) flags |= kDevWaitTimeout;
                    }
                    if (ok) {
                        uint8_t* dst = smem + (size_t)stage * C::STAGE_BYTES;
                        mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
#pragma unroll
                        for (int hf = 0; hf < C::NH; ++hf) {
                            tma_load_4d(dst + hf * C::BOX_BYTES, mk, &full_bar[stage], hf * 64, c1, head0, c3, stream_once);
                            tma_load_4d(dst + C::TENSOR_BYTES + hf * C::BOX_BYTES, mv, &full_bar[stage], hf * 64, c1,
                                        head0, c3, stream_once);
                        }
                    }
                    if (!ok) break;
                    if (++stage == stages) {
                        stage = 0;
                        ++use;
                    }
                }
                if (!ok) break;
            }
            s_ctl[1] = (int32_t)it;
        }
    } else {
        // ================================= consumer warps =========================================
        const int h_local = wid / (KW * RW);
        const int rw = (wid % (KW * RW)) / KW;
        const int kw = wid % KW;
        const int grp = lane >> 2, tq = lane & 3;
        const int rb = rw * C::ROWS_W;              // first packed row of this warp
        const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q;
        // Rows as the accumulator fragments see them: column 2 tq + j of 8-row group nt.
        // loop (0-based) of the row in the low byte, kMaxLoops for rows beyond R; above it how many of the step's
        // tokens of that loop are NEWER than the row's (0 with one query token per loop): the row sees that many fewer
        // keys of the shared cache and that many fewer slots of its (age-ordered) window
        int lc[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int r = rb + nt * 8 + 2 * tq + j;
                const int lq = r / p.G;               // loop * Qn + token
                lc[nt][j] = r < p.R ? (lq / p.Qn) | ((p.Qn - 1 - lq % p.Qn) << 8) : kMaxLoops;
            }

        int stage = 0;
        uint32_t use = 0;
        int q_b = -1, q_hg = -1;   // (sequence, head group) whose query rows are in qb
        uint32_t qb[D / 16][NT][2];
        PieceWalk walk(p, s_prefix, lo, hi, s_lens);
        Piece pc;
        while (walk.next(pc, flags)) {
            const int kvh = pc.hg * HPC + h_local;
            // ---- packed query rows of this KV head: row r = loop * G + head-in-group, as B fragments (row = lane / 4)
            // (the windows item of a head group follows its shared-cache item: same rows, kept)
            if (pc.b != q_b || pc.hg != q_hg) {
                q_b = pc.b;
                q_hg = pc.hg;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int r = rb + nt * 8 + grp;
                    const bool v = r < p.R;
                    const int lq = v ? r / p.G : 0;       // loop * Qn + token: q is [B, L, Qn, Hq, d]
                    const int64_t qrow = (((int64_t)pc.b * p.L * p.Qn + lq) * p.Hq + kvh * p.G + (r - lq * p.G)) * D;
                    if constexpr (FP8) {
                        // contraction order of process_keys_fp8: k-step ks takes d = 16 ks + 4 tq .. + 3; bf16 -> f16
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            uint2 u = make_uint2(0u, 0u);
                            if (v) u = *(const uint2*)(qg + qrow + ks * 16 + 4 * tq);
                            qb[ks][nt][0] = pack_f16x2(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
                            qb[ks][nt][1] = pack_f16x2(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
                        }
                    } else {
                        const int64_t q0 = qrow + 2 * tq;
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            qb[ks][nt][0] = v ? *(const uint32_t*)(qg + q0 + ks * 16) : 0u;
                            qb[ks][nt][1] = v ? *(const uint32_t*)(qg + q0 + ks * 16 + 8) : 0u;
                        }
                    }
                }
            }
            int cutr[NT][2], cmin = 0x7fffffff;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) cutr[nt][0] = cutr[nt][1] = 0;
#pragma unroll
            for (int l = 0; l < kMaxLoops; ++l)
                if (l < p.L) {
                    const int c = pc.sp.cut[l];
                    cmin = min(cmin, max(c - (p.Qn - 1), 0));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        if ((lc[nt][0] & 0xff) == l) cutr[nt][0] = max(c - (lc[nt][0] >> 8), 0);
                        if ((lc[nt][1] & 0xff) == l) cutr[nt][1] = max(c - (lc[nt][1] >> 8), 0);
                    }
                }
            float acc[D / 16][NT][4], mref[NT][2], lacc[NT][4];
            // E4M3 caches: the K scale of the head is a score scale, the V scale is applied to the finished partial
            const float sc2 = FP8 ? p.scale_log2 * p.k_scale[kvh] : p.scale_log2;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                mref[nt][0] = mref[nt][1] = kNoMax;
                lacc[nt][0] = lacc[nt][1] = lacc[nt][2] = lacc[nt][3] = 0.f;
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;
            }

            WinCursor cur;
            if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
            for (int t = pc.t0; t < pc.t1; ++t) {
                if (ok) {
                    ok = mbar_wait_bounded(&full_bar[stage], use & 1, kWaitLimitNs);
                    if (!ok) flags |= kDevWaitTimeout;
                }
                const uint32_t sK = smem_u32(smem + (size_t)stage * C::STAGE_BYTES);
                const uint32_t sV = sK + C::TENSOR_BYTES;
                int lim[NT][2];
                if (pc.kind == 0) {
                    const int key0 = t * C::TK;
                    if (ok) {
                        if (key0 + C::TK <= cmin) {
                            if constexpr (FP8)
                                process_keys_fp8<D, NT, KS, HPC, KW, C::TK, false>(sK, sV, qb, acc, mref, lacc, cutr, 0, sc2,
                                                                                   lane, kw, h_local);
                            else
                                process_keys<D, NT, KS, HPC, KW, C::TK, C::BOX_BYTES, false>(sK, sV, qb, acc, mref, lacc,
                                                                                             cutr, 0, sc2, lane, kw, h_local);
                        } else {
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                lim[nt][0] = cutr[nt][0] - key0;
                                lim[nt][1] = cutr[nt][1] - key0;
                            }
                            if constexpr (FP8)
                                process_keys_fp8<D, NT, KS, HPC, KW, C::TK, true>(sK, sV, qb, acc, mref, lacc, lim,
                                                                                  pc.sp.cmax - key0, sc2, lane, kw, h_local);
                            else
                                process_keys<D, NT, KS, HPC, KW, C::TK, C::BOX_BYTES, true>(sK, sV, qb, acc, mref, lacc, lim,
                                                                                            pc.sp.cmax - key0, sc2, lane, kw,
                                                                                            h_local);
                        }
                    }
                } else {
                    // Window of loop cur.l: only the rows of that loop take part.
                    const int l = cur.l;
                    int wl = 0;
#pragma unroll
                    for (int k = 1; k < kMaxLoops; ++k)
                        if (k == l) wl = pc.sp.wl[k];
                    const int row_lo = l * p.Qn * p.G, row_hi = row_lo + p.Qn * p.G;
                    const bool any = row_lo < rb + C::ROWS_W && row_hi > rb;
                    if (ok && any) {
                        const int n = wl - cur.key0;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            lim[nt][0] = (lc[nt][0] & 0xff) == l ? n - (lc[nt][0] >> 8) : 0;
                            lim[nt][1] = (lc[nt][1] & 0xff) == l ? n - (lc[nt][1] >> 8) : 0;
                        }
                        if constexpr (FP8)
                            process_keys_fp8<D, NT, KS, HPC, KW, C::TK, true>(sK, sV, qb, acc, mref, lacc, lim, n, sc2, lane, kw,
                                                                              h_local);
                        else
                            process_keys<D, NT, KS, HPC, KW, C::TK, C::BOX_BYTES, true>(sK, sV, qb, acc, mref, lacc, lim, n, sc2,
                                                                                        lane, kw, h_local);
                    }
                    cur.advance(p, pc.sp);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[stage]);
                if (++stage == stages) {
                    stage = 0;
                    ++use;
                }
            }

            // ---- end of piece: merge the key slices and store the split partial ------------------
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    if (mref[nt][j] == kNoMax) mref[nt][j] = -INFINITY;   // the partial's "saw no key" mark
            // Accumulator fragment rows (lane / 4, lane / 4 + 8) of 16-row group mt are the head dimensions
            // 16 mt + dA and 16 mt + dB (E4M3 caches: see process_keys_fp8).
            const int dA = FP8 ? 2 * grp : grp, dB = FP8 ? 2 * grp + 1 : grp + 8;
            if constexpr (FP8) {
                const float vs = p.v_scale[kvh];
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[mt][nt][e] *= vs;
            }
            const int64_t slot = slot_of(item_index(p, pc.b, pc.hg, pc.kind), cta);
            const int64_t prow = (slot * HPC + h_local) * p.R + rb;
            if (tid == 0) note_piece(p, pc, cta);
            if (KW == 1) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        if (lc[nt][j] == kMaxLoops) continue;
                        const int64_t row = prow + nt * 8 + 2 * tq + j;
                        float* dst = p.part_acc + row * D;
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) {
                            dst[mt * 16 + dA] = acc[mt][nt][j];
                            dst[mt * 16 + dB] = acc[mt][nt][2 + j];
                        }
                        if (grp == 0) *(float2*)(p.part_ml + row * 2) = make_float2(mref[nt][j], lacc[nt][j]);
                    }
            } else {
                const int gidx = h_local * RW + rw;
                float* macc = merge_acc + gidx * C::ROWS_W * C::MROW;
                float* mml = merge_ml + gidx * KW * C::ROWS_W * 2;
                if (grp == 0) {
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int j = 0; j < 2; ++j)
                            *(float2*)(mml + (kw * C::ROWS_W + nt * 8 + 2 * tq + j) * 2) = make_float2(mref[nt][j], lacc[nt][j]);
                }
                named_barrier_sync(1, C::NCW * 32);
                float sc[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int lr = nt * 8 + 2 * tq + j;
                        float mm = -INFINITY;
#pragma unroll
                        for (int k = 0; k < KW; ++k) mm = fmaxf(mm, mml[(k * C::ROWS_W + lr) * 2]);
                        const float ms = (mm == -INFINITY) ? 0.f : mm;
                        sc[nt][j] = fast_exp2(mref[nt][j] - ms);
                        if (kw == 0 && grp == 0 && lc[nt][j] != kMaxLoops) {
                            float ll = 0.f;
#pragma unroll
                            for (int k = 0; k < KW; ++k) {
                                const float2 v = *(const float2*)(mml + (k * C::ROWS_W + lr) * 2);
                                ll = fmaf(v.y, fast_exp2(v.x - ms), ll);
                            }
                            *(float2*)(p.part_ml + (prow + lr) * 2) = make_float2(mm, ll);
                        }
                    }
#pragma unroll
                for (int k = 0; k < KW; ++k) {
                    if (kw == k) {
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                float* a = macc + (nt * 8 + 2 * tq + j) * C::MROW;
#pragma unroll
                                for (int mt = 0; mt < D / 16; ++mt) {
                                    float x0 = acc[mt][nt][j] * sc[nt][j], x1 = acc[mt][nt][2 + j] * sc[nt][j];
                                    if (k > 0) {
                                        x0 += a[mt * 16 + dA];
                                        x1 += a[mt * 16 + dB];
                                    }
                                    a[mt * 16 + dA] = x0;
                                    a[mt * 16 + dB] = x1;
                                }
                            }
                    }
                    named_barrier_sync(1, C::NCW * 32);
                }
                // The KW warps of the group copy the merged rows out, 16 bytes per thread per step.
                for (int i4 = kw * 32 + lane; i4 < C::ROWS_W * (D / 4); i4 += KW * 32) {
                    const int row = i4 / (D / 4), c = (i4 % (D / 4)) * 4;
                    if (rb + row < p.R)
                        *(float4*)(p.part_acc + (prow + row) * D + c) = *(const float4*)(macc + row * C::MROW + c);
                }
                named_barrier_sync(1, C::NCW * 32);
            }
        }
    }
    if (flags) atomicOr(p.status, flags);
    if (flags & kDevWaitTimeout) s_ctl[0] = 1;
    __syncthreads();
    // A wait ran out somewhere: before the block retires, give every copy that was issued a bounded
    // chance to land (in the normal path the consumers have waited for all of them already).
    if (s_ctl[0] != 0 && tid == 0) {
        const uint32_t it = (uint32_t)s_ctl[1];
        const uint32_t filled = it < (uint32_t)stages ? it : (uint32_t)stages;
        for (uint32_t s = 0; s < filled; ++s) {
            const uint32_t last_use = (it - 1 - s) / (uint32_t)stages;  // index of the last fill of stage s
            mbar_wait_bounded(&full_bar[s], last_use & 1, kWaitLimitNs);
        }
    }
    __syncthreads();
}

}  // namespace plt
