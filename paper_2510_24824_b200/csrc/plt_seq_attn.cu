// Sequence-shaped PLT attention (prefill / training-forward; Algorithm 2 with the attention of Algorithm 3) on the
// 5th-generation tensor cores: tcgen05.mma with the QUERIES as the M dimension and accumulators in tensor memory.
//
// One thread block owns two 128-row query tiles A and B of one (sequence, loop): the same 128 rows t of two query heads
// that share a KV head (any even GQA group), else 256 consecutive rows of one head. Each tile has its own score tile S
// (128 lanes x 128 fp32 columns of tensor memory) and output tile O (128 x 128).
//
//   S_X [128 rows x 128 keys] = Q_X [128 x d] . K_tile^T [d x 128]     A = Q tile, B = K tile, both as TMA wrote them
//                                                                      (K-major, 128-byte swizzle)
//   O_X [128 rows x d]       += P_X [128 x 128] . V_tile [128 x d]     A = probabilities in TENSOR MEMORY (bf16, two
//                                                                      per column, written over S by the softmax
//                                                                      threads), B = V tile as TMA wrote it (MN-major)
//
// Warp roles: warp 0 streams K and V tiles (and the two Q tiles) by TMA into a ring of 32 KB slots; warp 1 issues the
// products (one lane) and owns the tensor-memory allocation; warps 4-7 are the softmax of tile A, warps 8-11 of
// tile B (thread = query row = tensor-memory lane). The issue order PV_A(j), S_A(j+1), PV_B(j), S_B(j+1) keeps the
// tensor core busy with one tile's products while the other tile's softmax runs.
//
// A block walks a list of steps: first the key tiles of the shared first-loop K/V up to the causal cutoff of its rows
// (online softmax with a lazily updated reference maximum: the accumulator in tensor memory is rescaled only when a
// score outruns the reference by more than kSlack powers of two), then, for loops 2..L, the one to three key tiles of
// the loop's own K/V that its rows' windows touch, twice: a scores-only pass that yields the window softmax's maximum
// and denominator, and a pass whose probabilities are already normalised and gated, g * p / l_local, and accumulate into
// the same O, which the softmax threads have scaled to (1 - g) * y_global in between. Eq. 2 thus costs no second
// accumulator. Every wait on an mbarrier is bounded and reports through the status word.
#include "../../include/plt_seq_attn.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "plt_host.h"
#include "plt_ptx.cuh"

namespace plt {
namespace {

constexpr int SQ = 128;                    // query rows per tile
constexpr int SK = 128;                    // keys per tile
constexpr int SD = 128;                    // head dimension
constexpr int kTileBytes = SK * SD * 2;    // one Q, K or V tile
constexpr int kHalf = SK * 128;            // one 64-element half of a tile: [128 rows][128 bytes]
constexpr int kRing = 5;                   // K/V ring slots
constexpr int kSeqThreads = 384;
constexpr float kSeqBig = 256.f;           // probabilities stay below 2^8 of their row's reference, else the slow path
constexpr float kSeqNoMax = -1e30f;
constexpr uint64_t kSeqWaitNs = 1000000000ull;
constexpr int kSeqMaxLoops = 8;

// mbarriers
constexpr int SB_QFULL = 0;                // Q tiles landed
constexpr int SB_FULL = 1;                 // + slot: tile landed
constexpr int SB_EMPTY = SB_FULL + kRing;  // + slot: products reading the slot completed
constexpr int SB_SFULL = SB_EMPTY + kRing; // + X: S_X complete (and every product issued before it)
constexpr int SB_PFULL = SB_SFULL + 2;     // + X: softmax of X consumed S_X (and wrote P_X)
constexpr int SB_ODONE = SB_PFULL + 2;     // + X: every product into O_X completed
constexpr int SB_COUNT = SB_ODONE + 2;

constexpr size_t kSeqSmem = 1024 + 2 * kTileBytes + (size_t)kRing * kTileBytes + SB_COUNT * 8 + 64;

struct SeqParams {
    const float* gate;          // [B, L-1, T, Hq]
    const int32_t* seq_lens;    // [B]
    __nv_bfloat16* out;         // [B, L, T, Hq, d]
    uint32_t* status;
    int32_t B, L, T, Hq, Hkv, G, w, nqb;   // nqb: row blocks per sequence (128 rows with paired heads, else 256)
    int32_t pair_heads, heads_per_grid;      // tiles of a block = two heads of one KV group; grid entries per (row block, loop)
    float scale_log2;
    int32_t delta[kSeqMaxLoops];
};

// The steps of one block: nG tiles of the shared K/V (tile A takes part in the first ntA of them), then for loops
// 2..L the tiles [l0, l0 + nL) of the loop's own K/V that the windows of the block's rows touch, scores only (kind 1),
// then the same tiles again with the second product (kind 2). Tile A takes part in the own-K/V tiles [lA0, lA0 + nLA),
// tile B in [lB0, lB0 + nLB); where both do, the step is shared like a step of the first phase.
struct SeqPlan {
    int ntA, ntB, nG;
    int lA0, nLA, lB0, nLB;
    int l0, nL;
    int total;
};
struct SeqStep {
    int kind;    // 0 shared K/V, 1 own K/V scores only, 2 own K/V with the second product
    int jk;      // key tile
    int qmask;   // bit 0: tile A takes part, bit 1: tile B
};

__device__ __forceinline__ SeqStep seq_step_at(const SeqPlan& pl, int i) {
    SeqStep s;
    if (i < pl.nG) {
        s.kind = 0; s.jk = i; s.qmask = (i < pl.ntA ? 1 : 0) | (i < pl.ntB ? 2 : 0);
        return s;
    }
    i -= pl.nG;
    s.kind = 1;
    if (i >= pl.nL) { i -= pl.nL; s.kind = 2; }
    s.jk = pl.l0 + i;
    s.qmask = ((s.jk >= pl.lA0 && s.jk < pl.lA0 + pl.nLA) ? 1 : 0) | ((s.jk >= pl.lB0 && s.jk < pl.lB0 + pl.nLB) ? 2 : 0);
    return s;
}

// Shared-memory matrix descriptor of tcgen05.mma (start address, leading / stride byte offsets in 16-byte units,
// descriptor version 1, 128-byte swizzle).
__device__ __forceinline__ uint64_t seq_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, B majorness (0 = K-major, 1 = MN-major), N / 8, M / 16.
__host__ __device__ constexpr uint32_t seq_instr_desc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// Bounded wait that also gives up as soon as another thread of the block has given up.
__device__ __noinline__ bool seq_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3fu) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kSeqWaitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool seq_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_test_wait(bar, parity)) return true;
    return seq_wait_slow(bar, parity, abort_flag);
}

struct SeqRing {
    int slot;
    uint32_t parity;
    __device__ SeqRing() : slot(0), parity(0) {}
    __device__ __forceinline__ void advance() {
        if (++slot == kRing) {
            slot = 0;
            parity ^= 1u;
        }
    }
};

// What a softmax thread knows about its row.
struct RowCtx {
    int t;            // row (decode step) index
    int cut;          // shared keys the row may see: max(0, t + 1 - delta)
    int lo;           // first own key of the window: max(delta, t + 1 - w)
    bool live;        // t < n_b and cut > 0
};

// 32 scores of a row -> probabilities against the reference: packed bf16 into pk[16], summed (fp32, two lanes) and
// their packed maximum tracked (bf16 bit patterns of non-negative numbers order like integers).
template <bool FULL>
__device__ __forceinline__ void global_chunk(const uint32_t (&r)[32], int c, int lim, float2 sc2, float2 nm2, uint32_t* pk,
                                             float2& sum2, uint32_t& pmax) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        float2 t = __ffma2_rn(make_float2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2);
        if (!FULL) {
            if (c * 32 + i >= lim) t.x = -INFINITY;
            if (c * 32 + i + 1 >= lim) t.y = -INFINITY;
        }
        const float2 pr = make_float2(fast_exp2(t.x), fast_exp2(t.y));
        sum2 = __fadd2_rn(sum2, pr);
        const uint32_t h = pack_bf16x2(pr.x, pr.y);
        pk[i / 2] = h;
        asm("max.u16x2 %0, %0, %1;" : "+r"(pmax) : "r"(h));
    }
}

// One pass over the 128 scores of this thread's row (tensor-memory lane) of a shared-K/V step: probabilities against
// the reference mref, packed bf16 into pk[64], their sum and the largest probability. kbase: index of the tile's first
// key. full: no key of the tile is masked for any row of the block's tile. The loads of a chunk are in flight while
// the chunk before it is worked on.
__device__ __forceinline__ void global_pass(uint32_t tS, const RowCtx& rc, int kbase, bool full, float scale, float mref,
                                            uint32_t (&pk)[64], float& lsum, float& pbig) {
    const int lim = rc.cut - kbase;   // keys [0, lim) of the tile are visible to this row
    const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(-mref, -mref);
    float2 sum2 = make_float2(0.f, 0.f);
    uint32_t pmax = 0;
    uint32_t ra[32], rb[32];
    tmem_ld32(tS, ra);
    tmem_wait_ld();
    tmem_ld32(tS + 32, rb);
    if (full) global_chunk<true>(ra, 0, lim, sc2, nm2, &pk[0], sum2, pmax); else global_chunk<false>(ra, 0, lim, sc2, nm2, &pk[0], sum2, pmax);
    tmem_wait_ld();
    tmem_ld32(tS + 64, ra);
    if (full) global_chunk<true>(rb, 1, lim, sc2, nm2, &pk[16], sum2, pmax); else global_chunk<false>(rb, 1, lim, sc2, nm2, &pk[16], sum2, pmax);
    tmem_wait_ld();
    tmem_ld32(tS + 96, rb);
    if (full) global_chunk<true>(ra, 2, lim, sc2, nm2, &pk[32], sum2, pmax); else global_chunk<false>(ra, 2, lim, sc2, nm2, &pk[32], sum2, pmax);
    tmem_wait_ld();
    if (full) global_chunk<true>(rb, 3, lim, sc2, nm2, &pk[48], sum2, pmax); else global_chunk<false>(rb, 3, lim, sc2, nm2, &pk[48], sum2, pmax);
    lsum = sum2.x + sum2.y;
    pbig = fmaxf(__uint_as_float(pmax << 16), __uint_as_float(pmax & 0xffff0000u));
}

// Largest visible score of the row in the tile (slow path of the shared-K/V pass).
__device__ __forceinline__ float global_row_max(uint32_t tS, const RowCtx& rc, int kbase) {
    float mx = -INFINITY;
    const int lim = rc.cut - kbase;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(tS + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (c * 32 + i < lim) mx = fmaxf(mx, __uint_as_float(r[i]));
    }
    return mx;
}

// Scores-only pass over a tile of the loop's own keys: folds the visible columns [c_lo, c_hi] of this thread's row into
// the window softmax's exact running maximum ml (log2 units) and denominator ll. Rows without a visible key keep
// ml = -inf, ll = 0. Every lane runs every load (they are collective over the warp).
__device__ __forceinline__ void window_stats_chunk(const uint32_t (&r)[32], int c, int c_lo, int c_hi, float scale, float& ml,
                                                   float& ll) {
    float t[32], cmax = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int col = c * 32 + i;
        t[i] = (col >= c_lo && col <= c_hi) ? __uint_as_float(r[i]) * scale : -INFINITY;
        cmax = fmaxf(cmax, t[i]);
    }
    const float m_new = fmaxf(ml, cmax);
    const float m_use = m_new > -INFINITY ? m_new : 0.f;
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) sum += fast_exp2(t[i] - m_use);
    ll = ll * fast_exp2(ml - m_use) + sum;   // ml = -inf: the old denominator is 0 and stays 0
    ml = m_new;
}
__device__ __forceinline__ void window_stats(uint32_t tS, int c_lo, int c_hi, float scale, float& ml, float& ll) {
    uint32_t ra[32], rb[32];
    tmem_ld32(tS, ra);
    tmem_wait_ld();
    tmem_ld32(tS + 32, rb);
    window_stats_chunk(ra, 0, c_lo, c_hi, scale, ml, ll);
    tmem_wait_ld();
    tmem_ld32(tS + 64, ra);
    window_stats_chunk(rb, 1, c_lo, c_hi, scale, ml, ll);
    tmem_wait_ld();
    tmem_ld32(tS + 96, rb);
    window_stats_chunk(ra, 2, c_lo, c_hi, scale, ml, ll);
    tmem_wait_ld();
    window_stats_chunk(rb, 3, c_lo, c_hi, scale, ml, ll);
}

// Second pass over the same tile: the weights 2^(s * scale + negm) of the visible columns (0 elsewhere), packed bf16.
__device__ __forceinline__ void window_weights_chunk(const uint32_t (&r)[32], int c, int c_lo, int c_hi, float2 sc2, float2 nm2,
                                                     uint32_t* pk) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const int col = c * 32 + i;
        float2 t = __ffma2_rn(make_float2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2);
        if (!(col >= c_lo && col <= c_hi)) t.x = -INFINITY;
        if (!(col + 1 >= c_lo && col + 1 <= c_hi)) t.y = -INFINITY;
        pk[i / 2] = pack_bf16x2(fast_exp2(t.x), fast_exp2(t.y));
    }
}
__device__ __forceinline__ void window_weights(uint32_t tS, int c_lo, int c_hi, float scale, float negm, uint32_t (&pk)[64]) {
    const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(negm, negm);
    uint32_t ra[32], rb[32];
    tmem_ld32(tS, ra);
    tmem_wait_ld();
    tmem_ld32(tS + 32, rb);
    window_weights_chunk(ra, 0, c_lo, c_hi, sc2, nm2, &pk[0]);
    tmem_wait_ld();
    tmem_ld32(tS + 64, ra);
    window_weights_chunk(rb, 1, c_lo, c_hi, sc2, nm2, &pk[16]);
    tmem_wait_ld();
    tmem_ld32(tS + 96, rb);
    window_weights_chunk(ra, 2, c_lo, c_hi, sc2, nm2, &pk[32]);
    tmem_wait_ld();
    window_weights_chunk(rb, 3, c_lo, c_hi, sc2, nm2, &pk[48]);
}

// Multiplies this thread's row of O (128 fp32 columns) by f.
__device__ __forceinline__ void scale_o_row(uint32_t tO, float f) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(tO + c * 32, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
        tmem_st32(tO + c * 32, r);
    }
    tmem_wait_st();
}

__global__ void __launch_bounds__(kSeqThreads, 1)
plt_seq_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKl,
                    const __grid_constant__ CUtensorMap tmVl, const __grid_constant__ SeqParams p) {
    extern __shared__ uint8_t seq_smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)seq_smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* q_smem = smem;                              // [2][tile]
    uint8_t* ring = smem + 2 * kTileBytes;               // [kRing][tile]
    uint64_t* bars = (uint64_t*)(ring + (size_t)kRing * kTileBytes);
    int32_t* s_ctl = (int32_t*)(bars + SB_COUNT);        // [0] abort flag, [1] tensor-memory base, [2] loads issued
    volatile int* abort_flag = (volatile int*)s_ctl;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

    // ---- which rows ------------------------------------------------------------------------------------
    // Blocks with the most key tiles (the last rows of a sequence) come first in the grid.
    // The block's two tiles are, where two query heads share a KV head (an even GQA group), the SAME 128 rows of two
    // neighbouring heads: both then walk exactly the same key tiles with the same masks, every K/V tile in shared memory
    // serves two products and neither tile idles on a step. Otherwise they are two consecutive 128-row tiles of one head
    // (the second then has one more key tile than the first).
    int item = blockIdx.x;
    const int hh = item % p.heads_per_grid; item /= p.heads_per_grid;
    const int l = item % p.L; item /= p.L;
    const int b = item % p.B; item /= p.B;
    const int qb = p.nqb - 1 - item;
    const int hA = p.pair_heads ? 2 * hh : hh, hB = p.pair_heads ? 2 * hh + 1 : hh;
    uint32_t flags = 0;
    int n = p.seq_lens[b];
    if (n < 0 || n > p.T) {
        flags |= 1u;   // PLT_DEV_SEQ_LEN_CLAMPED
        n = n < 0 ? 0 : p.T;
    }
    const int delta = p.delta[l];
    const int r0A = p.pair_heads ? qb * SQ : qb * 2 * SQ, r0B = p.pair_heads ? r0A : r0A + SQ;
    const int kvh = hA / p.G;

    SeqPlan pl;
    {
        // shared K/V tiles of a query tile with first row r0: keys [0, min(n, r0 + 128 - delta))
        auto tiles_of = [&](int r0) {
            if (r0 >= n) return 0;
            int keys = min(n, r0 + SQ) - delta;
            return keys > 0 ? (keys + SK - 1) / SK : 0;
        };
        pl.ntA = tiles_of(r0A);
        pl.ntB = tiles_of(r0B);
        pl.nG = max(pl.ntA, pl.ntB);
        pl.lA0 = pl.nLA = pl.lB0 = pl.nLB = 0;
        if (l > 0) {
            // own keys of a query tile: from the window start of its first live row to its last live row
            auto own = [&](int r0, int nt, int& j0, int& cnt) {
                j0 = cnt = 0;
                if (nt == 0) return;
                const int first_row = max(r0, delta);            // first row with a token
                const int last_row = min(n, r0 + SQ) - 1;
                const int lo = max(delta, first_row + 1 - p.w);
                j0 = lo / SK;
                cnt = last_row / SK - j0 + 1;
            };
            own(r0A, pl.ntA, pl.lA0, pl.nLA);
            own(r0B, pl.ntB, pl.lB0, pl.nLB);
        }
        pl.l0 = pl.nL = 0;
        if (pl.nLA > 0 || pl.nLB > 0) {
            const int a0 = pl.nLA > 0 ? pl.lA0 : pl.lB0, b0 = pl.nLB > 0 ? pl.lB0 : pl.lA0;
            const int a1 = pl.nLA > 0 ? pl.lA0 + pl.nLA : 0, b1 = pl.nLB > 0 ? pl.lB0 + pl.nLB : 0;
            pl.l0 = min(a0, b0);
            pl.nL = max(a1, b1) - pl.l0;   // the two ranges overlap or touch: every tile in between belongs to one
        }
        pl.total = pl.nG + 2 * pl.nL;
    }
    const bool activeA = pl.ntA > 0, activeB = pl.ntB > 0;

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[2] = 0;
        mbar_init(&bars[SB_QFULL], 1);
        for (int s = 0; s < kRing; ++s) {
            mbar_init(&bars[SB_FULL + s], 1);
            mbar_init(&bars[SB_EMPTY + s], 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&bars[SB_SFULL + x], 1);
            mbar_init(&bars[SB_PFULL + x], 4);
            mbar_init(&bars[SB_ODONE + x], 1);
        }
        mbar_fence_init();
    }
    if (wid == 1) tmem_alloc((uint32_t*)&s_ctl[1], 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = (uint32_t)s_ctl[1];
    // columns: S_A 0..127 (P_A over 0..63), S_B 128..255, O_A 256..383, O_B 384..511

    if (wid == 0) {
        // =========================== TMA producer (one lane) ==============================================
        if (lane == 0 && pl.total > 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            const uint64_t keep = l2_evict_first_policy();   // K/V tiles are re-read by the other heads and loops from L2;
            // the policy only orders evictions among streamed data
            mbar_expect_tx(&bars[SB_QFULL], (activeA ? kTileBytes : 0) + (activeB ? kTileBytes : 0));
            for (int x = 0; x < 2; ++x) {
                if (!(x == 0 ? activeA : activeB)) continue;
                const int r0 = x == 0 ? r0A : r0B;
                for (int hf = 0; hf < 2; ++hf)
                    tma_load_4d(q_smem + x * kTileBytes + hf * kHalf, &tmQ, &bars[SB_QFULL], hf * 64, x == 0 ? hA : hB, r0, b * p.L + l, keep);
            }
            SeqRing rg;
            uint32_t issued = 0;
            bool ok = true;
            for (int i = 0; i < pl.total && ok; ++i) {
                const SeqStep st = seq_step_at(pl, i);
                const int ntens = st.kind == 1 ? 1 : 2;   // K, then V unless the step is scores only
                for (int which = 0; which < ntens && ok; ++which) {
                    if (issued >= (uint32_t)kRing) ok = seq_wait(&bars[SB_EMPTY + rg.slot], rg.parity ^ 1u, abort_flag);
                    if (!ok) break;
                    const CUtensorMap* m = st.kind == 0 ? (which == 0 ? &tmK : &tmV) : (which == 0 ? &tmKl : &tmVl);
                    const int c3 = st.kind == 0 ? b : b * (p.L - 1) + (l - 1);
                    uint8_t* dst = ring + (size_t)rg.slot * kTileBytes;
                    mbar_expect_tx(&bars[SB_FULL + rg.slot], kTileBytes);
                    for (int hf = 0; hf < 2; ++hf)
                        tma_load_4d(dst + hf * kHalf, m, &bars[SB_FULL + rg.slot], hf * 64, kvh, st.jk * SK, c3, keep);
                    ++issued;
                    rg.advance();
                }
            }
            s_ctl[2] = (int32_t)issued;
        }
    } else if (wid == 1) {
        // =========================== product issue (whole warp walks, lane 0 issues) =====================
        if (pl.total > 0) {
            constexpr uint32_t idesc_qk = seq_instr_desc(SQ, SK, 0);
            constexpr uint32_t idesc_pv = seq_instr_desc(SQ, SD, 1);
            const uint32_t q_a = smem_u32(q_smem), ring_a = smem_u32(ring);
            bool ok = seq_wait(&bars[SB_QFULL], 0, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            // Ring position of every step's tiles: K of step i, then its V. Walked twice (S products run one step
            // ahead of PV products), so positions are recomputed from a running count.
            // slot_of(count) = count % kRing, parity = (count / kRing) & 1
            uint32_t s_issued[2] = {0, 0};    // per tile: S products issued (= steps of that tile started)
            int s_mask_step[2] = {-1, -1}, s_mask[2] = {0, 0};   // tiles whose S of a step has been issued (two steps in flight at most)
            uint32_t p_parity[2] = {0, 0};    // parity of the next P_FULL wait per tile
            bool o_started[2] = {false, false};
            // tile count before step i: prefix over steps (1 or 2 tiles each)
            auto tiles_before = [&](int i) {
                // steps [0, nG) and kind-2 steps have two tiles, kind-1 steps one
                const int nl = pl.nL;
                if (i <= pl.nG) return 2 * i;
                if (i <= pl.nG + nl) return 2 * pl.nG + (i - pl.nG);
                return 2 * pl.nG + nl + 2 * (i - pl.nG - nl);
            };
            auto issue_s = [&](int i, int x) {   // S_x = Q_x . K(step i)^T
                const uint32_t cnt = (uint32_t)tiles_before(i);
                const int slot = cnt % kRing;
                const uint32_t par = (cnt / kRing) & 1u;
                const SeqStep st = seq_step_at(pl, i);
                if (ok) ok = seq_wait(&bars[SB_FULL + slot], par, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return;
                tc_fence_after_sync();
                if (lane == 0) {
                    const uint32_t ka = ring_a + (uint32_t)slot * kTileBytes, qa = q_a + (uint32_t)x * kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < SD / 16; ++kk)
                        umma_bf16(tmem_base + x * 128, seq_smem_desc(qa + (kk >> 2) * kHalf + (kk & 3) * 32, 16, 1024),
                                  seq_smem_desc(ka + (kk >> 2) * kHalf + (kk & 3) * 32, 16, 1024), idesc_qk, kk == 0 ? 0u : 1u);
                    umma_commit(&bars[SB_SFULL + x]);
                }
                // The K slot is free once every tile that takes part in the step has issued its S product; which of the
                // two comes last depends on which of them ran ahead.
                if (s_mask_step[i & 1] != i) {
                    s_mask_step[i & 1] = i;
                    s_mask[i & 1] = 0;
                }
                s_mask[i & 1] |= 1 << x;
                if (s_mask[i & 1] == st.qmask && lane == 0) umma_commit(&bars[SB_EMPTY + slot]);
                __syncwarp();
                ++s_issued[x];
            };
            // next step after i in which tile x takes part, or -1
            auto next_step_of = [&](int i, int x) {
                for (int k = i + 1; k < pl.total; ++k)
                    if (seq_step_at(pl, k).qmask & (1 << x)) return k;
                return -1;
            };
            // prologue: the first S of each active tile
            int first[2] = {activeA ? 0 : -1, activeB ? 0 : -1};
            for (int x = 0; x < 2; ++x)
                if (first[x] >= 0) issue_s(first[x], x);
            bool s_ahead[2] = {true, true};   // S of the tile's current step has been issued already
            for (int i = 0; i < pl.total && ok; ++i) {
                const SeqStep st = seq_step_at(pl, i);
                for (int x = 0; x < 2 && ok; ++x) {
                    if (!(st.qmask & (1 << x))) continue;
                    if (!s_ahead[x]) issue_s(i, x);
                    if (!ok) break;
                    // the softmax of tile x has read S_x (and, unless the step is scores only, written P_x)
                    ok = seq_wait(&bars[SB_PFULL + x], p_parity[x], abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    p_parity[x] ^= 1u;
                    if (!ok) break;
                    if (st.kind != 1) {
                        const uint32_t cnt = (uint32_t)tiles_before(i) + 1;
                        const int slot = cnt % kRing;
                        const uint32_t par = (cnt / kRing) & 1u;
                        ok = seq_wait(&bars[SB_FULL + slot], par, abort_flag);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        // Rows of the V tile at or beyond the sequence's length may hold anything: zero them, so that
                        // a probability of 0 times garbage cannot produce NaN. Done once per tile (first tile to use it).
                        const int vrow0 = n - st.jk * SK;
                        if (vrow0 < SK && x == ((st.qmask & 1) ? 0 : 1)) {
                            uint8_t* v = ring + (size_t)slot * kTileBytes;
                            for (int idx = lane; idx < (SK - max(vrow0, 0)) * 16; idx += 32) {
                                const int row = max(vrow0, 0) + idx / 16, ch = idx % 16;
                                *(uint4*)(v + (ch >> 3) * kHalf + row * 128 + (ch & 7) * 16) = make_uint4(0, 0, 0, 0);
                            }
                            fence_proxy_async_smem();
                            __syncwarp();
                        }
                        tc_fence_after_sync();
                        if (lane == 0) {
                            const uint32_t va = ring_a + (uint32_t)slot * kTileBytes;
#pragma unroll
                            for (int kk = 0; kk < SK / 16; ++kk)
                                umma_bf16_ts(tmem_base + 256 + x * 128, tmem_base + x * 128 + kk * 8,
                                             seq_smem_desc(va + kk * 2048, kHalf, 1024), idesc_pv,
                                             (o_started[x] || kk > 0) ? 1u : 0u);
                            if (x == ((st.qmask & 2) ? 1 : 0)) umma_commit(&bars[SB_EMPTY + slot]);   // last reader of this V
                        }
                        __syncwarp();
                        o_started[x] = true;
                    }
                    // run ahead: S of this tile's next step, if that is the very next step of the list (keeps the
                    // ring first-in first-out)
                    const int nx = next_step_of(i, x);
                    s_ahead[x] = false;
                    if (nx == i + 1) {
                        issue_s(nx, x);
                        s_ahead[x] = true;
                    } else if (nx < 0 && lane == 0) {
                        umma_commit(&bars[SB_ODONE + x]);   // everything into O_x has been issued
                    }
                    __syncwarp();
                }
            }
        }
    } else if (wid >= 4) {
        // =========================== softmax and epilogue ================================================
        const int x = (wid - 4) >> 2;                      // 0: tile A, 1: tile B
        const int wq = wid & 3;                            // lane quarter of tensor memory this warp may touch
        const bool active = x == 0 ? activeA : activeB;
        const int r0 = x == 0 ? r0A : r0B;
        const int h = x == 0 ? hA : hB;
        RowCtx rc;
        rc.t = r0 + wq * 32 + lane;
        rc.cut = max(0, min(rc.t, n - 1) + 1 - delta);
        rc.lo = max(delta, rc.t + 1 - p.w);
        rc.live = rc.t < n && rc.t + 1 - delta > 0;
        const uint32_t lane_off = (uint32_t)(wq * 32) << 16;
        const uint32_t tS = tmem_base + lane_off + x * 128, tO = tmem_base + lane_off + 256 + x * 128;
        const float scale = p.scale_log2;
        float mref = kSeqNoMax, lg = 0.f;       // shared-K/V softmax: reference maximum (log2 units) and denominator
        float ml = -INFINITY, ll = 0.f;          // window softmax: exact maximum (log2 units) and denominator
        float gate = 0.f;
        bool ok = true, o_scaled = false;
        uint32_t s_parity = 0;
        int gsteps = 0;
        if (active && l > 0 && rc.t < p.T) {
            const float z = p.gate[(((int64_t)b * (p.L - 1) + (l - 1)) * p.T + rc.t) * p.Hq + h];
            gate = 1.f / (1.f + __expf(-z));
        }
        if (active) {
            for (int i = 0; i < pl.total; ++i) {
                const SeqStep st = seq_step_at(pl, i);
                if (!(st.qmask & (1 << x))) continue;
                if (ok) ok = seq_wait(&bars[SB_SFULL + x], s_parity, abort_flag);
                ok = __all_sync(0xffffffffu, ok);      // the tensor-memory accesses below are collective over the warp
                s_parity ^= 1u;
                if (!ok) break;
                tc_fence_after_sync();
                const int kbase = st.jk * SK;
                if (st.kind == 0) {
                    // ---- shared K/V: online softmax against the lazily updated reference ----------------
                    const bool full = kbase + SK <= r0 + 1 - delta && kbase + SK <= n;
                    uint32_t pk[64];
                    float lsum, pbig;
                    global_pass(tS, rc, kbase, full, scale, mref, pk, lsum, pbig);
                    if (__any_sync(0xffffffffu, rc.live && !(pbig <= kSeqBig))) {   // a probability of a live row beyond 2^8 of its reference
                        // slow path: true maximum, rescale of this row of O (every product into it has completed: the
                        // commit behind S_FULL covers them), probabilities again
                        const float mx = global_row_max(tS, rc, kbase);
                        const float m_new = fmaxf(mref, mx * scale);
                        const float alpha = fast_exp2(mref - m_new);
                        mref = m_new;
                        lg *= alpha;
                        if (gsteps > 0) scale_o_row(tO, alpha);
                        global_pass(tS, rc, kbase, full, scale, mref, pk, lsum, pbig);
                    }
                    lg += lsum;
                    ++gsteps;
#pragma unroll
                    for (int c = 0; c < 2; ++c) tmem_st32(tS + c * 32, &pk[c * 32]);
                    tmem_wait_st();
                } else {
                    if (!o_scaled) {
                        // O_x holds the unnormalised shared-K/V sum: make it (1 - g) * y_global (Eq. 2)
                        o_scaled = true;
                        scale_o_row(tO, (rc.live && lg > 0.f) ? (1.f - gate) / lg : 0.f);
                    }
                    // own keys lo .. t of the row: columns [c_lo, c_hi] of the tile
                    const int c_lo = rc.lo - kbase, c_hi = rc.t - kbase;
                    if (st.kind == 1) {
                        window_stats(tS, c_lo, c_hi, scale, ml, ll);
                    } else {
                        // probabilities already normalised and gated: g * 2^(s - m) / l = 2^(s - m + log2(g / l))
                        const float beta = (rc.live && ll > 0.f) ? gate / ll : 0.f;
                        const float negm = beta > 0.f ? fast_log2(beta) - ml : -INFINITY;
                        uint32_t pk[64];
                        window_weights(tS, c_lo, c_hi, scale, negm, pk);
#pragma unroll
                        for (int c = 0; c < 2; ++c) tmem_st32(tS + c * 32, &pk[c * 32]);
                        tmem_wait_st();
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[SB_PFULL + x]);
            }
            // ---- epilogue: O_x out of tensor memory ---------------------------------------------------------
            if (ok) ok = seq_wait(&bars[SB_ODONE + x], 0, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
        }
        {
            // Every lane of the warp runs the loads (they are collective); only rows inside the tensor are stored.
            const bool in_tensor = rc.t < p.T;
            __nv_bfloat16* dst = p.out + ((((int64_t)b * p.L + l) * p.T + (in_tensor ? rc.t : 0)) * p.Hq + h) * SD;
            const bool have_o = active && ok;                  // warp-uniform
            const bool write = have_o && rc.live;
            // loop 1: O holds the unnormalised sum; loops 2..L: O is final (scaled before the window pass)
            const float f = l == 0 ? (lg > 0.f ? 1.f / lg : 0.f) : 1.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                if (have_o) {
                    tmem_ld32(tO + c * 32, r);
                    tmem_wait_ld();
                }
                if (in_tensor) {
#pragma unroll
                    for (int i2 = 0; i2 < 32; i2 += 8) {
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (write) {
                            v.x = pack_bf16x2(__uint_as_float(r[i2]) * f, __uint_as_float(r[i2 + 1]) * f);
                            v.y = pack_bf16x2(__uint_as_float(r[i2 + 2]) * f, __uint_as_float(r[i2 + 3]) * f);
                            v.z = pack_bf16x2(__uint_as_float(r[i2 + 4]) * f, __uint_as_float(r[i2 + 5]) * f);
                            v.w = pack_bf16x2(__uint_as_float(r[i2 + 6]) * f, __uint_as_float(r[i2 + 7]) * f);
                        }
                        *(uint4*)(dst + c * 32 + i2) = v;
                    }
                }
            }
        }
    }
    if (flags && tid == 0) atomicOr(p.status, flags);
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && s_ctl[0] != 0) {
        atomicOr(p.status, 4u);   // PLT_DEV_WAIT_TIMEOUT
        // give every copy that was issued a bounded chance to land before the block retires
        const uint32_t issued = (uint32_t)s_ctl[2];
        const uint32_t outstanding = issued < (uint32_t)kRing ? issued : (uint32_t)kRing;
        for (uint32_t k = 0; k < outstanding; ++k) {
            const uint32_t cnt = issued - 1 - k;
            mbar_wait_bounded(&bars[SB_FULL + cnt % kRing], (cnt / kRing) & 1u, kSeqWaitNs);
        }
        if (pl.total > 0) mbar_wait_bounded(&bars[SB_QFULL], 0, kSeqWaitNs);
    }
    __syncthreads();
    if (wid == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace
}  // namespace plt

// ===================================================================================================
// C ABI
// ===================================================================================================
using namespace plt;

namespace {

thread_local char g_seq_create_error[512] = "";

typedef CUresult (*SeqEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct plt_seq_attn {
    plt_seq_attn_config cfg;
    int32_t delta[kSeqMaxLoops];
    float scale_log2;
    uint32_t* status = nullptr;
    SeqEncodeFn encode = nullptr;
    CUtensorMap maps[5];
    const void* map_base[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    int map_batch[5] = {0, 0, 0, 0, 0};
    char err[512];
};

namespace {

plt_status seq_fail(plt_seq_attn_t h, plt_status code, const char* fmt, ...) {
    char* dst = h ? h->err : g_seq_create_error;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(dst, 512, fmt, ap);
    va_end(ap);
    return code;
}

// [outer][rows][heads][128] bf16, box = [1][128 rows][1 head][64 elements]
plt_status seq_encode(plt_seq_attn_t h, int idx, const void* base, int heads, int rows, int64_t outer) {
    if (h->map_base[idx] == base && h->map_batch[idx] == (int)outer) return PLT_OK;
    cuuint64_t dims[4] = {(cuuint64_t)SD, (cuuint64_t)heads, (cuuint64_t)rows, (cuuint64_t)outer};
    cuuint64_t strides[3] = {(cuuint64_t)SD * 2, (cuuint64_t)heads * SD * 2, (cuuint64_t)rows * heads * SD * 2};
    cuuint32_t box[4] = {64u, 1u, (cuuint32_t)SQ, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = h->encode(&h->maps[idx], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        h->map_base[idx] = nullptr;
        return seq_fail(h, PLT_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d for tensor %d", (int)r, idx);
    }
    h->map_base[idx] = base;
    h->map_batch[idx] = (int)outer;
    return PLT_OK;
}

bool seq_aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

#define PLT_API __attribute__((visibility("default")))
extern "C" {

PLT_API plt_status plt_seq_attn_create(const plt_seq_attn_config* c, plt_seq_attn_t* out_handle) {
    if (!out_handle) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "out_handle is NULL");
    *out_handle = nullptr;
    if (!c) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "config is NULL");
    if (c->struct_size != sizeof(plt_seq_attn_config))
        return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "config.struct_size %u != %zu", c->struct_size, sizeof(plt_seq_attn_config));
    if (c->max_batch < 1 || c->L < 1 || c->Hq < 1 || c->Hkv < 1 || c->max_seq_len < 1 || c->w < 0)
        return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "non-positive size in config");
    if (c->L > kSeqMaxLoops) return seq_fail(nullptr, PLT_ERR_UNSUPPORTED, "L %d > %d", c->L, kSeqMaxLoops);
    if (c->Hq % c->Hkv != 0) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "Hq %d is not a multiple of Hkv %d", c->Hq, c->Hkv);
    if (c->d != SD) return seq_fail(nullptr, PLT_ERR_UNSUPPORTED, "head dim %d (supported: 128)", c->d);
    if (c->L > 1 && c->w < 1) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "w must be >= 1 when L > 1");
    if (c->loop_offset)
        for (int l = 0; l < c->L; ++l)
            if (c->loop_offset[l] < 0) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "loop_offset[%d] < 0", l);
    const int64_t nqb = (c->max_seq_len + 2 * SQ - 1) / (2 * SQ);
    if ((double)nqb * c->max_batch * c->L * c->Hq >= 2147483647.0)
        return seq_fail(nullptr, PLT_ERR_UNSUPPORTED, "max_batch * L * Hq * max_seq_len too large for one grid");
    cudaError_t e = cudaSetDevice(c->device);
    if (e != cudaSuccess) return seq_fail(nullptr, PLT_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(e));
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, c->device);
    if (e != cudaSuccess) return seq_fail(nullptr, PLT_ERR_CUDA, "cudaGetDeviceProperties: %s", cudaGetErrorString(e));
    if (prop.major != 10)
        return seq_fail(nullptr, PLT_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", c->device,
                        prop.major, prop.minor);
    plt_seq_attn* h = new (std::nothrow) plt_seq_attn();
    if (!h) return seq_fail(nullptr, PLT_ERR_OUT_OF_MEMORY, "host allocation failed");
    h->cfg = *c;
    h->cfg.loop_offset = nullptr;
    for (int l = 0; l < kSeqMaxLoops; ++l) h->delta[l] = c->loop_offset && l < c->L ? c->loop_offset[l] : l;
    const float scale = c->sm_scale > 0.f ? c->sm_scale : 1.0f / sqrtf((float)c->d);
    h->scale_log2 = scale * 1.4426950408889634f;
    h->err[0] = 0;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) {
        delete h;
        return seq_fail(nullptr, PLT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    }
    h->encode = (SeqEncodeFn)fn;
    e = allow_max_dynamic_smem((const void*)plt_seq_attn_kernel);
    if (e != cudaSuccess) {
        delete h;
        return seq_fail(nullptr, PLT_ERR_CUDA, "preparing the kernel: %s", cudaGetErrorString(e));
    }
    e = cudaMalloc((void**)&h->status, 256);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete h;
        return seq_fail(nullptr, PLT_ERR_OUT_OF_MEMORY, "cudaMalloc of the status word failed");
    }
    e = cudaMemset(h->status, 0, 256);
    if (e != cudaSuccess) {
        cudaFree(h->status);
        delete h;
        return seq_fail(nullptr, PLT_ERR_CUDA, "cudaMemset: %s", cudaGetErrorString(e));
    }
    *out_handle = h;
    return PLT_OK;
}

PLT_API plt_status plt_seq_attn_run(plt_seq_attn_t h, const plt_seq_attn_args* a, void* cuda_stream) {
    if (!h) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if (!a) return seq_fail(h, PLT_ERR_INVALID_ARG, "args is NULL");
    if (a->struct_size != sizeof(plt_seq_attn_args))
        return seq_fail(h, PLT_ERR_INVALID_ARG, "args.struct_size %u != %zu", a->struct_size, sizeof(plt_seq_attn_args));
    const plt_seq_attn_config& c = h->cfg;
    if (a->batch < 0) return seq_fail(h, PLT_ERR_INVALID_ARG, "batch %d < 0", a->batch);
    if (a->batch > c.max_batch) return seq_fail(h, PLT_ERR_CAPACITY, "batch %d > max_batch %d", a->batch, c.max_batch);
    if (a->batch == 0) return PLT_OK;
    if (!a->q || !a->k_share || !a->v_share || !a->seq_lens || !a->out)
        return seq_fail(h, PLT_ERR_INVALID_ARG, "q, k_share, v_share, seq_lens and out must not be NULL");
    if (c.L > 1 && (!a->k_loc || !a->v_loc || !a->gate_logits))
        return seq_fail(h, PLT_ERR_INVALID_ARG, "k_loc, v_loc and gate_logits must not be NULL when L > 1");
    if (!seq_aligned16(a->q) || !seq_aligned16(a->k_share) || !seq_aligned16(a->v_share) || !seq_aligned16(a->out) ||
        (c.L > 1 && (!seq_aligned16(a->k_loc) || !seq_aligned16(a->v_loc))))
        return seq_fail(h, PLT_ERR_INVALID_ARG, "tensor base pointers must be 16-byte aligned");
    const int T = c.max_seq_len;
    plt_status s = seq_encode(h, 0, a->q, c.Hq, T, (int64_t)a->batch * c.L);
    if (s == PLT_OK) s = seq_encode(h, 1, a->k_share, c.Hkv, T, a->batch);
    if (s == PLT_OK) s = seq_encode(h, 2, a->v_share, c.Hkv, T, a->batch);
    if (s == PLT_OK && c.L > 1) s = seq_encode(h, 3, a->k_loc, c.Hkv, T, (int64_t)a->batch * (c.L - 1));
    if (s == PLT_OK && c.L > 1) s = seq_encode(h, 4, a->v_loc, c.Hkv, T, (int64_t)a->batch * (c.L - 1));
    if (s != PLT_OK) return s;
    if (c.L == 1) {
        h->maps[3] = h->maps[1];
        h->maps[4] = h->maps[2];
    }
    SeqParams p;
    memset(&p, 0, sizeof p);
    p.gate = a->gate_logits;
    p.seq_lens = a->seq_lens;
    p.out = (__nv_bfloat16*)a->out;
    p.status = h->status;
    p.B = a->batch; p.L = c.L; p.T = T; p.Hq = c.Hq; p.Hkv = c.Hkv; p.G = c.Hq / c.Hkv; p.w = c.w;
    p.pair_heads = (p.G % 2 == 0) ? 1 : 0;
    p.heads_per_grid = p.pair_heads ? p.Hq / 2 : p.Hq;
    p.nqb = p.pair_heads ? (T + SQ - 1) / SQ : (T + 2 * SQ - 1) / (2 * SQ);
    p.scale_log2 = h->scale_log2;
    for (int l = 0; l < kSeqMaxLoops; ++l) p.delta[l] = h->delta[l];
    const unsigned grid = (unsigned)((int64_t)p.nqb * p.B * p.L * p.heads_per_grid);
    plt_seq_attn_kernel<<<grid, kSeqThreads, kSeqSmem, (cudaStream_t)cuda_stream>>>(h->maps[0], h->maps[1], h->maps[2],
                                                                                    h->maps[3], h->maps[4], p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return seq_fail(h, PLT_ERR_CUDA, "launching the kernel: %s", cudaGetErrorString(e));
    return PLT_OK;
}

PLT_API plt_status plt_seq_attn_check(plt_seq_attn_t h, void* cuda_stream, uint32_t* out_bits) {
    if (!h) return seq_fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    uint32_t bits = 0;
    cudaError_t e = cudaMemcpyAsync(&bits, h->status, 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->status, 0, 4, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return seq_fail(h, PLT_ERR_CUDA, "reading the device status word: %s", cudaGetErrorString(e));
    if (out_bits) *out_bits = bits;
    if (bits == 0) return PLT_OK;
    return seq_fail(h, PLT_ERR_DEVICE_CHECK, "device status 0x%x:%s%s", bits,
                    (bits & PLT_DEV_SEQ_LEN_CLAMPED) ? " seq_lens entry out of range (clamped)" : "",
                    (bits & PLT_DEV_WAIT_TIMEOUT) ? " a bounded wait ran out (output invalid)" : "");
}

PLT_API plt_status plt_seq_attn_destroy(plt_seq_attn_t h) {
    if (!h) return PLT_OK;
    if (h->status) cudaFree(h->status);
    delete h;
    return PLT_OK;
}

PLT_API const char* plt_seq_attn_last_error(plt_seq_attn_t h) { return h ? h->err : g_seq_create_error; }

}  // extern "C"
