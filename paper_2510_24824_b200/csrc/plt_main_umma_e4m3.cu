// Split-KV main kernel of the CLP decode attention for E4M3 caches on the 5th-generation tensor cores
// (tcgen05.mma kind::f8f6f4 reading the codes from shared memory as TMA wrote them, accumulators in tensor
// memory), head dimension 128, up to 32 packed query rows.
//
// y_global and y_local of Algorithm 3 for all L loops, same tile plan and split-partial format as the other main
// kernels: one persistent block per SM walks its share of the line of 128-key tiles.
// No code is converted on the way: both products take 8-bit operands, so the bf16 queries and the fp32
// probabilities are each written as a SUM of E4M3 numbers and the terms are laid side by side along N:
//
//   S^T [128 keys x 2 RP]  = K_tile [128 x 128] . [Q_hi ; Q_lo]^T      A = K codes (K-major, 128-byte swizzle)
//   O^T [128 dims x 3 RP] += V_tile^T [128 x 128] . [P_hi ; 2^10 P_mid ; 2^14 P_lo]^T   A = V codes (MN-major)
//
// A bf16 number times a power of two IS the sum of two E4M3 numbers (8 significant bits = 4 + 4) as long as its low
// part stays above the E4M3 subnormal step, so the scores are those of the bf16 queries; a probability keeps 12
// significant bits in three terms, the second and third scaled up by 2^10 and 2^14 so that probabilities far below
// the E4M3 subnormal step (2^-9) still count: many keys of tiny weight next to one peak must not be dropped. The
// softmax threads add the two score columns of a row, and the epilogue adds the three accumulator columns. One
// tcgen05.mma costs the same issue slot whatever N is, so the extra terms are free on the tensor side: 8
// instructions per 32 KB step.
//
// A work item is one or two KV heads of a sequence, and its steps alternate between them tile by tile: the codes of
// a key of all heads lie side by side in memory, and neighbouring heads fetched within a short time of each other
// stream at 6.4 TB/s where one head's 128 bytes per key alone stream at 4.5 (measured on B200).
// Warp roles: one team of four softmax-and-epilogue warps per head of the item (thread = key = tensor-memory lane,
// all RP scores of it); then four warps with one working lane each: the TMA producer of the K tiles and that of the
// V tiles (a ring of 16 KB slots each), the issuer of the S^T products (which also copies the packed query images of
// the next piece with cp.async.bulk and owns the tensor-memory allocation) and the issuer of the O^T products.
// The query image (codes in the core-matrix order the instruction reads, and the power of two they were scaled
// by) is written per (sequence, KV head) by plt_decode_pack_q_e4m3, launched before this kernel.
// Online softmax with a lazily updated reference maximum, as in the bf16 tcgen05 kernel. Every wait is bounded.
// Paged caches: a tile is one TMA box when a page holds whole tiles and two boxes with pages of 64 tokens (template
// parameter HALVES), the page ids fetched one tile ahead by the producers' per-step loop; smaller pages go through
// an out-of-line path with a page-table read per box.
// Whatever the softmax teams call is inlined and takes no array or structure by reference: arguments in local
// memory cost an L2 round trip each beside 213 KB of shared memory (measured: 240 -> 218 us on B = 16, N = 32768).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"
#include "plt_umma_util.cuh"

namespace plt {

namespace {

constexpr int kTile8 = UK * UD;        // one K (or V) tile of one KV head: 128 keys x 128 codes = a ring slot
// K tiles and V tiles have a ring each: a K tile is done with as soon as its scores are formed (two steps ahead of
// the probabilities), a V tile only after the product that ends its step, so that one ring of K + V slots would
// keep most of its slots waiting for that product and leave two loads in flight (measured: 4.7 TB/s at best).
constexpr int kKRing8 = 4;             // K slots
constexpr int kMaxVRing8 = 4;          // V slots at most
// Threads of a block: one team of 128 softmax threads per KV head of the item, two producer warps, two issuer warps.
__host__ __device__ constexpr int threads8(int hpc) { return hpc * 128 + 128; }
// A probability may exceed the lazily updated reference by 3 powers of two at most (p <= 8), which fixes the powers of
// two the second and third term are scaled by: |p - hi| <= 2^-2 and |p - hi - mid| <= 2^-7 times 2^10 and 2^14 stay
// below 448. The third term then resolves 2^-23, the step of the f16 the probability is rounded to first.
constexpr float kSlack8 = 3.f;
constexpr uint32_t kMidScaleH2 = 0x64006400u;   // 2^10 as f16x2
constexpr uint32_t kLoScaleH2 = 0x4c004c00u;    // 2^4 as f16x2 (on top of the 2^10)
constexpr float kMidInv = 1.f / 1024.f, kLoInv = 1.f / 16384.f;

// mbarrier indices
constexpr int E_KFULL = 0, E_KEMPTY = 4, E_VFULL = 8, E_VEMPTY = 14, E_SFULL = 20 /* two */, E_SFREE = 22 /* two */,
              E_PFULL = 24 /* four */, E_PFREE = 28 /* four */, E_OFULL = 32 /* two */, E_OFREE = 34 /* two */,
              E_QFULL = 36 /* two */, E_DRAIN = 38 /* two */, E_COUNT = 40;
// Probability buffers: four, used in turn by the steps, so that a team (every other step with two heads) writes the
// probabilities of a step without waiting for the O^T product of its step before, which is still queued behind the
// S^T products of later steps on the tensor pipe (measured: 480 of a team's 3400 cycles per step).
constexpr int kPBufs = 4;

template <int RP>
struct ECfg {
    static constexpr int QLBO = 2 * RP * 16;   // bytes between the 16-code column chunks of the query image
    static constexpr int QBUF = 8 * QLBO;      // [8 chunks][2 RP rows: hi then lo][16 codes]
    static constexpr int PBUF = 3 * RP * UK;   // [3 RP / 16 row groups: hi, mid, lo][128 keys][16 codes]
    // Tensor memory: two S^T buffers of 2 RP columns (step parity), then O^T buffers of 3 RP columns, one per piece
    // parity and head of the item (two heads: 4 RP + 12 RP = 16 RP columns, all 512 at 32 rows).
    static constexpr int TMEM_COLS = RP == 16 ? 256 : 512;
    // hpc: KV heads per work item (their tiles take turns; each has its own query image, reference maxima and O^T)
    __host__ __device__ static constexpr size_t smem_bytes(int nslot, int hpc, int max_batch) {
        return 1024 + (size_t)nslot * kTile8 + kPBufs * PBUF + (size_t)2 * hpc * QBUF + E_COUNT * 8 +
               (size_t)RP * 4 * (12 * hpc + 1) + 64 + (size_t)(2 * max_batch + 4) * 4;
    }
};

// ---- the query image ---------------------------------------------------------------------------------------
// One block per (sequence, KV head), one thread per (packed row, 16-element chunk). q * 2^k = hi + lo with hi and lo
// E4M3 numbers; 2^k puts the largest |q| of the block's rows into [128, 256).
template <int RP>
__global__ void __launch_bounds__(RP * 8) plt_decode_pack_q_e4m3(const Params p, uint8_t* qimg, float* qinv) {
    using C = ECfg<RP>;
    __shared__ float wmax[RP * 8 / 32];
    grid_launch_dependents();   // the main kernel sets up and starts its cache loads meanwhile; it waits for this grid
                                // to complete before it touches a query image
    const int b = blockIdx.x / p.Hkv, hg = blockIdx.x - b * p.Hkv;
    const int r = threadIdx.x >> 3, c = threadIdx.x & 7;
    float x[16];
    float mx = 0.f;
    if (r < p.R) {
        const int l = r / p.G, g = r - l * p.G;
        const __nv_bfloat16* src = (const __nv_bfloat16*)p.q + (((int64_t)b * p.L + l) * p.Hq + hg * p.G + g) * UD + c * 16;
        uint4 raw[2] = {*(const uint4*)src, *(const uint4*)(src + 8)};
        const __nv_bfloat162* h2 = (const __nv_bfloat162*)raw;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float2 f = __bfloat1622float2(h2[i]);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
            mx = fmaxf(mx, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = 0.f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = wmax[0];
#pragma unroll
    for (int i = 1; i < RP * 8 / 32; ++i) mx = fmaxf(mx, wmax[i]);
    // k = 7 - floor(log2 max), kept inside the normal range; 0 for an all-zero or non-finite block
    int k = 0;
    if (mx > 0.f && mx < INFINITY) {
        k = 7 - ((int)((__float_as_uint(mx) >> 23) & 0xffu) - 127);
        k = k > 120 ? 120 : k;
    }
    const float qs = __uint_as_float((uint32_t)(127 + k) << 23);
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float a0 = x[2 * i] * qs, a1 = x[2 * i + 1] * qs;
        const uint32_t ch = f16x2_to_e4m3x2(pack_f16x2(a0, a1));   // a0, a1 are bf16 values below 2^8: exact in f16 above 2^-14
        const uint32_t bh = e4m3x2_to_f16x2(ch);
        const float2 back = __half22float2(*(const __half2*)&bh);
        const uint32_t cl = f16x2_to_e4m3x2(pack_f16x2(a0 - back.x, a1 - back.y));
        if (i & 1) {
            hi[i >> 1] |= ch << 16;
            lo[i >> 1] |= cl << 16;
        } else {
            hi[i >> 1] = ch;
            lo[i >> 1] = cl;
        }
    }
    uint8_t* img = qimg + ((size_t)b * p.Hkv + hg) * C::QBUF + c * C::QLBO;
    *(uint4*)(img + r * 16) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *(uint4*)(img + (RP + r) * 16) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    if (threadIdx.x == 0) qinv[b * p.Hkv + hg] = __uint_as_float((uint32_t)(127 - k) << 23);
}

// ---- the tile plan, walked with scalars only --------------------------------------------------------------
// The same plan as PieceWalk / SeqPlan (plt_common.cuh) yields, recomputed from the clamped sequence length with no
// per-loop arrays, so that every role keeps its position in registers: with 200+ KB of shared memory the L1 that
// would back a stack frame is a few KB, and a role that spills its plan there runs at a fraction of its speed.
__device__ __forceinline__ int e_cut(const Params& p, int n, int l) {
    const int c = n - p.delta[l];
    return c > 0 ? c : 0;
}
// Valid window slots of loop l (1 .. L-1) of sequence b.
__device__ __forceinline__ int e_wl(const Params& p, int b, int n, int l, uint32_t& flags) {
    const int c = e_cut(p, n, l);
    int wl = c < p.w ? c : p.w;
    if (p.win_lens != nullptr && c > 0) {
        wl = p.win_lens[b * (p.L - 1) + (l - 1)];
        if (wl < 0 || wl > p.w) {
            flags |= kDevWinLenClamped;
            wl = wl < 0 ? 0 : p.w;
        }
    }
    return wl;
}
// Largest cutoff over the loops, tiles of the shared cache and of all windows of sequence b.
__device__ __forceinline__ void e_counts(const Params& p, int b, int n, uint32_t& flags, int& cmax, int& gt, int& lt) {
    cmax = 0;
    lt = 0;
#pragma unroll 1
    for (int l = 0; l < p.L; ++l) {
        const int c = e_cut(p, n, l);
        cmax = c > cmax ? c : cmax;
        if (l >= 1) lt += ceil_div(e_wl(p, b, n, l, flags), UK);
    }
    gt = ceil_div(cmax, UK);
}

// One piece: tiles [t0, t1) of item (b, hg, kind); n = clamped length of b, cmax / total = what e_counts gave
// (total = tiles of the whole item).
struct EPiece {
    int b, hg, kind, t0, t1, n, cmax, total;
};

// The step to the next piece is out of line and shared by the three roles (it runs once per piece); the per-tile
// loops copy what they need of the piece into registers and stay small enough for the instruction cache.
struct EWalk {
    int pos, hi, b;
    __device__ __forceinline__ EWalk(const Params& p, const int32_t* sp, int lo_, int hi_) : pos(lo_), hi(hi_), b(0) {
        if (pos < hi) b = find_seq(sp, p.B, pos);
    }
    __device__ __forceinline__ bool next(const Params& p, const int32_t* sp, const int32_t* lens, EPiece& pc, uint32_t& flags) {
        for (;;) {
            if (pos >= hi) return false;
            while (sp[b + 1] <= pos) ++b;
            const int n = lens[b];
            int cmax, gt, lt;
            e_counts(p, b, n, flags, cmax, gt, lt);
            const int vg = line_len(p, gt), per = vg + line_len(p, lt);
            const int o = pos - sp[b];
            pc.b = b;
            pc.n = n;
            pc.cmax = cmax;
            pc.hg = o / per;
            const int o2 = o - pc.hg * per;
            int v0, item_end;
            if (o2 < vg) {
                pc.kind = 0;
                pc.total = gt;
                v0 = o2;
                item_end = pos + (vg - o2);
            } else {
                pc.kind = 1;
                pc.total = lt;
                v0 = o2 - vg;
                item_end = pos + (per - o2);
            }
            const int end = item_end < hi ? item_end : hi;
            const int v1 = v0 + (end - pos);
            pos = end;
            pc.t0 = v0 > p.piece_cost ? v0 - p.piece_cost : 0;
            pc.t1 = v1 > p.piece_cost ? v1 - p.piece_cost : 0;
            if (pc.t1 > pc.t0) return true;   // else: only the item's lead-in positions fell to this block
        }
    }
};

// Window tile cursor of a windows item: loop (1 .. L-1), first key of the tile inside that loop's window, and the
// window's length.
struct EWin {
    int l, key0, wl;
    __device__ __forceinline__ void seek(const Params& p, int b, int n, int t, uint32_t& flags) {
        l = 1;
        wl = e_wl(p, b, n, 1, flags);
        while (l < p.L - 1) {
            const int nt = ceil_div(wl, UK);
            if (t < nt) break;
            t -= nt;
            ++l;
            wl = e_wl(p, b, n, l, flags);
        }
        key0 = t * UK;
    }
    __device__ __forceinline__ void advance(const Params& p, int b, int n, uint32_t& flags) {
        key0 += UK;
        while (key0 >= wl && l < p.L - 1) {
            ++l;
            key0 = 0;
            wl = e_wl(p, b, n, l, flags);
        }
    }
};

// ---- softmax side: per-team context and the work that is off the per-step path -------------------------------
// One team of four softmax warps per KV head of the item (thread = key, all RP scores of it). The steps of an item
// alternate between its heads, so with two heads a team takes every other step and has two step times for each:
// heads share nothing (own reference maxima, denominators, accumulator, score and probability buffer), so the two
// teams never wait for one another.
struct ECtx {
    float* negm;       // [RP] of this team's head: minus the reference maximum of each row (1e30 while the row has none)
    float* mref;       // [RP] reference maximum, log2 units
    float* alpha;      // [RP] rescale factors of the slow path
    float* red;        // [4][RP] cross-warp reduction scratch
    float* mfin;       // [2][RP] reference maxima of a finished piece, by piece parity
    float* lfin;       // [2][RP] its denominators
    int32_t* lim;      // [RP] keys visible to each row in the current segment
    int32_t* rowloop;  // [RP] loop (0-based) of each packed row (shared by the teams, read-only)
    uint64_t* bars;
    volatile int* abort_flag;
    uint32_t lane_off;  // this warp's lane quarter in a tensor-memory address
    int R;              // packed rows
    int HPC;            // KV heads per work item = teams
    int hh;             // this team's head within the item
    int bar_id;         // named barrier of the team's 128 threads
    int ltid, lane, wq; // thread in the team (= key = output dimension), lane, warp in the team
};

// Slow path of the online softmax: true maxima of the tile over its 128 keys, new reference maxima, and (unless this
// is the head's first tile of the piece) the rescale of the three O^T column groups and of the denominators. The 128
// threads of a team call it together. `s`: the scores in log2 units; `done_bar` / `done_parity`: completion of the
// last product into this O^T.
template <int RP>
__device__ __forceinline__ bool e_slow_path(const float (&s)[RP], float (&lsum)[RP], const ECtx& cx, bool rescale,
                                         uint32_t tOb, uint64_t* done_bar, uint32_t done_parity, bool failed) {
    {
        float v[RP];
#pragma unroll
        for (int r = 0; r < RP; ++r) v[r] = s[r];
        warp_reduce_rows<RP, true>(v, cx.lane, cx.red + cx.wq * RP);
    }
    named_barrier_sync(cx.bar_id, kSmThreads);
    if (cx.ltid < RP) {
        const int t = cx.ltid;
        const float mo = cx.mref[t];
        const float mn = fmaxf(fmaxf(mo, fmaxf(cx.red[t], cx.red[RP + t])), fmaxf(cx.red[2 * RP + t], cx.red[3 * RP + t]));
        cx.alpha[t] = (mo == -INFINITY) ? 1.f : exp2f(mo - mn);
        cx.mref[t] = mn;
        // rows beyond R (padding of the instruction's N) keep a reference that makes every probability 0
        cx.negm[t] = t >= cx.R ? -1e30f : ((mn == -INFINITY) ? 1e30f : -mn);
    }
    named_barrier_sync(cx.bar_id, kSmThreads);
    if (rescale) {
        failed = sm_wait(done_bar, done_parity, cx.abort_flag, failed);
        if (!failed) {
            tc_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < 3 * RP / 16; ++c) {
                uint32_t o[16];
                tmem_ld16(tOb + cx.lane_off + c * 16, o);
                tmem_wait_ld();
                const int r0 = (c * 16) % RP;
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * cx.alpha[r0 + j]);
                tmem_st16(tOb + cx.lane_off + c * 16, o);
            }
            tmem_wait_st();
            tc_fence_before_sync();
        }
#pragma unroll
        for (int r = 0; r < RP; ++r) lsum[r] *= cx.alpha[r];
    }
    return failed;
}

// Epilogue of a finished piece for this team's head: the three column groups of O^T summed (the second and third
// scaled back), times the V scale of the head, and the denominators, out of tensor memory into the split partial.
// tOb: O^T of the head in the piece; ob: piece parity; prow: first row of the head's partial.
template <int RP>
__device__ __forceinline__ bool e_epilogue(const Params& p, const ECtx& cx, uint32_t tOb, int ob, uint32_t parity, int64_t prow,
                                        float vscale, bool failed) {
    failed = sm_wait(&cx.bars[E_OFULL + ob], parity, cx.abort_flag, failed);
    float* dst = p.part_acc + prow * UD + cx.ltid;
    // Eight rows at a time in a loop that is not unrolled: this code is cold every time it runs (the per-step loops of
    // six roles evict it) and a cold instruction line costs hundreds of cycles to fetch, so it is kept to a few lines.
#pragma unroll 1
    for (int c = 0; c < RP / 8; ++c) {
        if (!failed) {
            uint32_t o0[8], o1[8], o2[8];
            tc_fence_after_sync();
            tmem_ld8(tOb + cx.lane_off + c * 8, o0);
            tmem_ld8(tOb + cx.lane_off + RP + c * 8, o1);
            tmem_ld8(tOb + cx.lane_off + 2 * RP + c * 8, o2);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (c * 8 + j < p.R)
                    dst[(c * 8 + j) * UD] =
                        (__uint_as_float(o0[j]) + (__uint_as_float(o1[j]) * kMidInv + __uint_as_float(o2[j]) * kLoInv)) * vscale;
        }
    }
    tc_fence_before_sync();
    __syncwarp();
    if (cx.lane == 0) mbar_arrive(&cx.bars[E_OFREE + ob]);
    if (!failed && cx.ltid < p.R)
        *(float2*)(p.part_ml + (prow + cx.ltid) * 2) = make_float2(cx.mfin[ob * RP + cx.ltid], cx.lfin[ob * RP + cx.ltid]);
    return failed;
}

// V rows of a boundary tile that hold no data may contain anything (NaN codes too): zero them so that 0 * garbage
// stays 0. `vtile`: the V half of the slot. Called by the team that owns the step.
__device__ __forceinline__ bool e_zero_v_rows(uint8_t* vtile, int nvalid, uint64_t* full_bar, uint32_t parity, const ECtx& cx,
                                           bool failed) {
    failed = sm_wait(full_bar, parity, cx.abort_flag, failed);
    if (!failed && cx.ltid >= nvalid) {
        uint8_t* row = vtile + cx.ltid * 128;
#pragma unroll
        for (int i = 0; i < 8; ++i) *(uint4*)(row + i * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    return failed;
}

// Start of a piece (shared cache) or of a window inside a windows piece: the visibility limit of each row; at the
// start of a piece also the reference maxima. n: clamped length of the sequence.
__device__ __forceinline__ void e_set_limits(const Params& p, const ECtx& cx, int RP, int kind, int n, int win_loop, int wl,
                                          bool new_piece) {
    // Threads still forming the probabilities of the tile before read lim: nobody rewrites it earlier.
    named_barrier_sync(cx.bar_id, kSmThreads);
    if (cx.ltid < RP) {
        const int t = cx.ltid;
        if (new_piece) {
            cx.mref[t] = -INFINITY;
            cx.negm[t] = t >= cx.R ? -1e30f : 1e30f;
        }
        int lim = 0;
        if (t < cx.R) {
            if (kind == 0) lim = e_cut(p, n, cx.rowloop[t]);
            else if (cx.rowloop[t] == win_loop) lim = wl;
        }
        cx.lim[t] = lim;
    }
    named_barrier_sync(cx.bar_id, kSmThreads);
}

// ---- the four single-lane roles: what happens once per piece, or on tiles that are not plain shared-cache tiles, is
// out of line, so that the per-step loops of the producers and issuers are a few dozen instructions each. (Instruction
// fetch decides the speed of this kernel: six loops run side by side on one SM.) ----
struct ProdState {
    EWalk walk;
    EPiece pc;
    EWin win;
    int t;   // tile of the piece the next step belongs to
    __device__ ProdState(const Params& p, const int32_t* sp, int lo, int hi) : walk(p, sp, lo, hi), t(0) { pc.t0 = pc.t1 = 0; }
};

// Next piece of a producer. Returns the steps it has (tiles x heads); `plain`: shared-cache tiles that the per-step
// loop loads itself (a contiguous cache or pages that hold whole 128-key tiles: one TMA box each; pages of 64 keys:
// two boxes).
__device__ __noinline__ int prod_next_piece(const Params& p, const int32_t* sp, const int32_t* lens, ProdState& st, int hpc, bool& plain,
                                            uint32_t& flags) {
    st.walk.next(p, sp, lens, st.pc, flags);
    st.t = st.pc.t0;
    if (st.pc.kind == 1) st.win.seek(p, st.pc.b, st.pc.n, st.t, flags);
    plain = st.pc.kind == 0 && (p.page_size == 0 || p.page_size % UK == 0 || 2 * p.page_size == UK);
    return (st.pc.t1 - st.pc.t0) * hpc;
}

// Loads of a tile of a paged cache or of a window (head `hh` of the item; after the item's last head the window
// cursor moves on). `map`: the K or the V map of the tensor the tile belongs to.
__device__ __noinline__ void prod_issue_special(const Params& p, const UmmaGeom& geo, ProdState& st, int hh, int hpc, uint8_t* dst,
                                                uint64_t* full, const CUtensorMap* map, const CUtensorMap* wmap, uint64_t pol,
                                                uint32_t& flags) {
    const EPiece& pc = st.pc;
    const int head = pc.hg * hpc + hh;
    if (pc.kind == 0) {
        const int key0 = st.t * UK;
        const int rem = pc.cmax - key0;   // keys that hold data from key0 on (>= 1)
        const int nbox = (min(rem, UK) + geo.kbox - 1) / geo.kbox;
        mbar_expect_tx(full, (uint32_t)(nbox * geo.kbox * 128));
        for (int i = 0; i < nbox; ++i) {
            const int key = key0 + i * geo.kbox;
            int page = p.page_table[(int64_t)pc.b * p.max_pages + key / p.page_size];
            if (page < 0 || page >= p.num_pool_pages) {
                flags |= kDevPageIdClamped;
                page = page < 0 ? 0 : p.num_pool_pages - 1;
            }
            tma_load_4d(dst + i * geo.kbox * 128, map, full, 0, key % p.page_size, head, page, pol);
        }
    } else {
        mbar_expect_tx(full, (uint32_t)(geo.wbox * 128));
        tma_load_4d(dst, wmap, full, 0, st.win.key0, head, pc.b * (p.L - 1) + (st.win.l - 1), pol);
        if (hh == hpc - 1) st.win.advance(p, pc.b, pc.n, flags);
    }
}

// Steps a block takes: one per tile and head of every piece in its range of the line (the positions of the range that
// are lead-ins of items are not tiles).
__device__ __noinline__ int count_steps(const Params& p, const int32_t* sp, const int32_t* lens, int lo, int hi, int hpc, uint32_t& flags) {
    EWalk walk(p, sp, lo, hi);
    EPiece pc;
    int steps = 0;
    while (walk.next(p, sp, lens, pc, flags)) steps += (pc.t1 - pc.t0) * hpc;
    return steps;
}

// Next piece of an issuer: its steps (0: none left) and the index of its first query image.
__device__ __noinline__ int issuer_next_piece(const Params& p, const int32_t* sp, const int32_t* lens, EWalk& walk, int hpc, int& image,
                                              uint32_t& flags) {
    EPiece pc;
    if (!walk.next(p, sp, lens, pc, flags)) return 0;
    image = pc.b * p.Hkv + pc.hg * hpc;
    return (pc.t1 - pc.t0) * hpc;
}

template <int RP, int HPC, bool HALVES>
__global__ void __launch_bounds__(threads8(HPC), 1)
plt_decode_main_umma_e4m3(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                          const __grid_constant__ CUtensorMap tmKw, const __grid_constant__ CUtensorMap tmVw,
                          const __grid_constant__ Params p, const UmmaGeom geo, const uint8_t* __restrict__ qimg,
                          const float* __restrict__ qinv) {
    using C = ECfg<RP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int vring = geo.ring - kKRing8;                   // V slots (geo.ring counts all slots)
    uint8_t* kslots = smem;                                 // ring of K tiles, then ring of V tiles
    uint8_t* vslots = smem + (size_t)kKRing8 * kTile8;
    uint8_t* pbuf = smem + (size_t)geo.ring * kTile8;       // kPBufs buffers of PBUF (step modulo kPBufs)
    uint8_t* qbuf = pbuf + kPBufs * C::PBUF;                // two buffers (piece parity) of HPC query images
    uint64_t* bars = (uint64_t*)(qbuf + 2 * HPC * C::QBUF);
    // per team (= head of the item), kTeamFloats each: negm, mref, alpha [RP]; red [4][RP]; lim [RP]; mfin, lfin [2][RP]
    constexpr int kTeamFloats = 12 * RP;
    float* s_team = (float*)(bars + E_COUNT);
    int32_t* s_rowloop = (int32_t*)(s_team + HPC * kTeamFloats);
    int32_t* s_ctl = s_rowloop + RP;                        // [0] abort flag, [1] tensor-memory base, [2] K / [3] V tiles issued, [4] steps
    int32_t* s_prefix = s_ctl + 16;                         // [B + 1] tile prefix
    int32_t* s_len = s_prefix + p.B + 1;                    // [B] clamped sequence lengths
    volatile int* abort_flag = (volatile int*)&s_ctl[0];

    // One lane of each softmax warp arrives on the barriers they feed (a thread-wide count would put hundreds of
    // arrivals on one shared-memory word per step). With two heads a score / probability buffer belongs to one team.
    constexpr int kKProducerWarp = 4 * HPC, kVProducerWarp = 4 * HPC + 1, kSIssuerWarp = 4 * HPC + 2, kOIssuerWarp = 4 * HPC + 3;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[2] = 0;
        s_ctl[3] = 0;
        for (int s = 0; s < kKRing8; ++s) {
            mbar_init(&bars[E_KFULL + s], 1);
            mbar_init(&bars[E_KEMPTY + s], 1);
        }
        for (int s = 0; s < kMaxVRing8; ++s) {
            mbar_init(&bars[E_VFULL + s], 1);
            mbar_init(&bars[E_VEMPTY + s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars[E_SFULL + i], 1);
            mbar_init(&bars[E_SFREE + i], 4);
            mbar_init(&bars[E_OFULL + i], 1);
            mbar_init(&bars[E_OFREE + i], 4 * HPC);
            mbar_init(&bars[E_QFULL + i], 1);
        }
        for (int i = 0; i < kPBufs; ++i) {
            mbar_init(&bars[E_PFULL + i], 4);
            mbar_init(&bars[E_PFREE + i], 1);
        }
        mbar_init(&bars[E_DRAIN], 1);
        mbar_init(&bars[E_DRAIN + 1], 1);
        mbar_fence_init();
    }
    if (tid < RP) s_rowloop[tid] = tid / p.G;
    if (wid == kSIssuerWarp) tmem_alloc((uint32_t*)&s_ctl[1], C::TMEM_COLS);
    grid_launch_dependents();  // the merge kernel may be set up meanwhile; it waits for this grid to complete
    build_prefix(p, s_prefix, flags, s_len, /*small=*/true);  // contains __syncthreads
    if (tid == 0) {
        const int64_t t64 = s_prefix[p.B];
        const int c = blockIdx.x, nc = plan_ctas(t64, (int)gridDim.x);
        s_ctl[4] = c < nc ? count_steps(p, s_prefix, s_len, (int)cta_begin(t64, c, nc), (int)cta_begin(t64, c + 1, nc), HPC, flags) : 0;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = (uint32_t)s_ctl[1];
    // S^T of step parity g at tS + 2 RP g; O^T of piece parity b, head hh at tO + 3 RP (HPC b + hh)
    const uint32_t tS = tmem_base, tO = tmem_base + 4 * RP;

    const int64_t T64 = s_prefix[p.B];
    const int cta = blockIdx.x, nctas = plan_ctas(T64, (int)gridDim.x);
    if (cta == 0)
        for (int b = tid; b <= p.B; b += threads8(HPC)) p.prefix[b] = s_prefix[b];
    const bool in_plan = cta < nctas;
    const int lo = in_plan ? (int)cta_begin(T64, cta, nctas) : 0, hi = in_plan ? (int)cta_begin(T64, cta + 1, nctas) : 0;
    // Steps this block takes: one per (tile, head of the item) of the pieces in its range of the line. The heads of a
    // tile follow one another: a key's codes of all heads lie side by side in memory, and fetched within a short time
    // of each other they come at 6.4 TB/s where one head's 128 bytes per key alone come at 4.5 (measured on B200, 8
    // heads of 128 codes per key).
    const uint32_t U = (uint32_t)s_ctl[4];
    bool q_pending[2] = {false, false};       // issuer only: query images were asked for and not yet waited for
    uint32_t q_parity[2] = {0u, 0u};          // and the phase of their barrier that ends when they have landed

    if (wid == kKProducerWarp || wid == kVProducerWarp) {
        // ===================== TMA producers: one warp streams the K tiles, one the V tiles =====================
        // Each keeps at most `cap` of its tiles in flight (issued, not landed): more outstanding requests make the
        // memory system slower, not faster. cap <= ring, so the slot of the tile issued `cap` tiles ago has not been
        // refilled and its phase parity is unambiguous.
        if (lane == 0 && U > 0) {
            const bool is_v = wid == kVProducerWarp;
            const int ring = is_v ? vring : kKRing8, cap = geo.cap < ring ? geo.cap : ring;
            uint8_t* slots = is_v ? vslots : kslots;
            uint64_t* fullb = &bars[is_v ? E_VFULL : E_KFULL];
            uint64_t* emptyb = &bars[is_v ? E_VEMPTY : E_KEMPTY];
            const CUtensorMap* map = is_v ? &tmV : &tmK;
            const CUtensorMap* wmap = is_v ? &tmVw : &tmKw;
            tma_prefetch_desc(map);
            if (p.L > 1) tma_prefetch_desc(wmap);
            const uint64_t pol = l2_evict_first_policy();
            bool ok = true, plain = false;
            Ring cur, old;   // slot of tile n, slot of tile n - cap
            ProdState st(p, s_prefix, lo, hi);
            int left = 0, hh = 0, key0 = 0, head0 = 0, outer = 0;   // of a plain piece: next tile's first key, first head, sequence
            // ... and with pages: the tile's offset in its page, the page's index in the sequence's table, its id, and
            // the id of the next tile's page, fetched one tile ahead so that the load is never waited for
            // With pages of half a tile a tile is two boxes, the second only if it holds data; pidx then counts pages
            // of the tile's first half and page_cur2 / page_next2 are the ids of the second half.
            // (HALVES: a kernel of its own, so that the other page sizes' loop stays as short as it was.)
            const bool paged = p.page_size > 0;
            int poff = 0, pidx = 0, page_cur = 0, page_next = 0, page_cur2 = 0, page_next2 = 0, cmax = 0;
            const int32_t* table = p.page_table;
            uint32_t n = 0;
            for (; n < U && ok; ++n) {
                if (left == 0) {
                    left = prod_next_piece(p, s_prefix, s_len, st, HPC, plain, flags);
                    key0 = st.t * UK;
                    head0 = st.pc.hg * HPC;
                    outer = st.pc.b;
                    if (plain && paged) {
                        pidx = key0 / p.page_size;
                        poff = key0 - pidx * p.page_size;
                        table = p.page_table + (int64_t)outer * p.max_pages;
                        page_cur = table[pidx];
                        cmax = st.pc.cmax;
                        if (HALVES && key0 + UK / 2 < cmax) page_cur2 = table[pidx + 1];
                    }
                }
                if (n >= (uint32_t)cap) {
                    ok = wait_or_abort(&fullb[old.slot], old.parity, abort_flag);
                    old.advance(ring);
                }
                if (ok && n >= (uint32_t)ring) ok = wait_or_abort(&emptyb[cur.slot], cur.parity ^ 1u, abort_flag);
                if (!ok) break;
                uint8_t* dst = slots + (size_t)cur.slot * kTile8;
                uint64_t* full = &fullb[cur.slot];
                if (plain) {
                    if constexpr (HALVES) {
                        if (hh == 0 && left > HPC) {   // the piece has a next tile: the ids of its one or two pages
                            page_next = table[pidx + 2];
                            if (key0 + UK + UK / 2 < cmax) page_next2 = table[pidx + 3];
                        }
                        const bool two = key0 + UK / 2 < cmax;
                        int page = page_cur, page2 = page_cur2;
                        if (page < 0 || page >= p.num_pool_pages || (two && (page2 < 0 || page2 >= p.num_pool_pages))) {
                            flags |= kDevPageIdClamped;
                            page = page < 0 ? 0 : (page >= p.num_pool_pages ? p.num_pool_pages - 1 : page);
                            page2 = page2 < 0 ? 0 : (page2 >= p.num_pool_pages ? p.num_pool_pages - 1 : page2);
                        }
                        mbar_expect_tx(full, two ? (uint32_t)kTile8 : (uint32_t)(kTile8 / 2));
                        tma_load_4d(dst, map, full, 0, 0, head0 + hh, page, pol);
                        if (two) tma_load_4d(dst + kTile8 / 2, map, full, 0, 0, head0 + hh, page2, pol);
                    } else {
                        int c1 = key0, c3 = outer;
                        if (paged) {
                            if (hh == 0 && left > HPC)   // the piece has a next tile: its page id, if it starts a new page
                                page_next = poff + UK == p.page_size ? table[pidx + 1] : page_cur;
                            int page = page_cur;
                            if (page < 0 || page >= p.num_pool_pages) {
                                flags |= kDevPageIdClamped;
                                page = page < 0 ? 0 : p.num_pool_pages - 1;
                            }
                            c1 = poff;
                            c3 = page;
                        }
                        mbar_expect_tx(full, (uint32_t)(geo.kbox * 128));
                        tma_load_4d(dst, map, full, 0, c1, head0 + hh, c3, pol);
                    }
                } else {
                    prod_issue_special(p, geo, st, hh, HPC, dst, full, map, wmap, pol, flags);
                }
                cur.advance(ring);
                --left;
                if (++hh == HPC) {
                    hh = 0;
                    key0 += UK;
                    ++st.t;
                    if constexpr (HALVES) {
                        pidx += 2;
                        page_cur = page_next;
                        page_cur2 = page_next2;
                    } else if (paged) {
                        poff += UK;
                        if (poff == p.page_size) {
                            poff = 0;
                            ++pidx;
                        }
                        page_cur = page_next;
                    }
                }
            }
            s_ctl[is_v ? 3 : 2] = (int32_t)n;
        }
    } else if (wid == kSIssuerWarp) {
        // ============ S^T = K [Q_hi ; Q_lo]^T issuer (one lane); owner of tensor memory and of the query images ============
        // A score buffer is refilled as soon as the team that owns it has read the scores of its step before, so the
        // scores of a team's next step are ready long before it has formed the probabilities of this one. The O^T
        // products have an issuer of their own: each waits for its own conditions only.
        if (lane == 0 && U > 0) {
            constexpr uint32_t idesc_qk = instr_desc_e4m3(UK, 2 * RP, 0, 0);
            // descriptors of slot 0 / buffer 0; the others differ in the start-address field (16-byte units) only
            const uint64_t kdesc0 = smem_desc(smem_u32(kslots), 16, 1024, 2);
            const uint64_t qdesc0 = smem_desc(smem_u32(qbuf), C::QLBO, 128, 0);
            bool ok = true;
            grid_dependency_wait();   // the query images are complete (the pack kernel ran just before this one)
            EWalk walk(p, s_prefix, lo, hi);
            // steps left in the piece, and the piece after it (0 steps: none) with the index of its first image
            int next_image = 0, next_left = 0;
            int s_left = issuer_next_piece(p, s_prefix, s_len, walk, HPC, next_image, flags);
            bool s_first = true, want_q = true;   // want_q: the images of piece q_piece are to be copied
            uint32_t pis = 0, q_piece = 0, s_head = 0;
            Ring krs;
            for (uint32_t gs = 0; gs < U && ok; ++gs) {
                if (want_q) {
                    const uint32_t buf = q_piece & 1;
                    mbar_expect_tx(&bars[E_QFULL + buf], (uint32_t)(HPC * C::QBUF));
                    bulk_load(qbuf + buf * HPC * C::QBUF, qimg + (size_t)next_image * C::QBUF, (uint32_t)(HPC * C::QBUF),
                              &bars[E_QFULL + buf]);   // the images of an item's heads are consecutive
                    q_pending[buf] = true;
                    q_parity[buf] = (q_piece >> 1) & 1;
                    want_q = false;
                }
                const uint32_t sb = gs & 1;
                if (s_first) {
                    ok = wait_or_abort(&bars[E_QFULL + (pis & 1)], (pis >> 1) & 1, abort_flag);
                    if (ok) q_pending[pis & 1] = false;
                }
                if (ok && gs >= 2)   // the scores that were in this buffer (two steps ago) have been read out
                    ok = wait_or_abort(&bars[E_SFREE + sb], ((gs >> 1) & 1) ^ 1u, abort_flag);
                if (ok) ok = wait_or_abort(&bars[E_KFULL + krs.slot], krs.parity, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t kd = kdesc0 + (uint64_t)((uint32_t)krs.slot * (kTile8 >> 4));
                const uint64_t qd = qdesc0 + (uint64_t)(((pis & 1) * HPC + s_head) * (C::QBUF >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_f8(tS + sb * 2 * RP, kd + (uint64_t)(k * 2), qd + (uint64_t)(k * 2 * (C::QLBO >> 4)), idesc_qk, k == 0 ? 0u : 1u);
                umma_commit(&bars[E_SFULL + sb]);
                umma_commit(&bars[E_KEMPTY + krs.slot]);
                krs.advance(kKRing8);
                if (s_first) {
                    // The other image buffer was last read by the products of the piece before; the last of them
                    // (step gs - 1) must have completed before the next piece's images are copied into it.
                    if (gs > 0) ok = wait_or_abort(&bars[E_SFULL + (sb ^ 1)], ((gs - 1) >> 1) & 1, abort_flag);
                    next_left = ok ? issuer_next_piece(p, s_prefix, s_len, walk, HPC, next_image, flags) : 0;
                    if (next_left > 0) {
                        q_piece = pis + 1;
                        want_q = true;   // copied at the top of the next step
                    }
                    s_first = false;
                }
                if (++s_head == HPC) s_head = 0;
                if (--s_left == 0) {
                    s_left = next_left;
                    s_first = true;
                    ++pis;
                }
            }
        }
    } else if (wid == kOIssuerWarp) {
        // ===================== O^T += V^T [P_hi ; P_mid ; P_lo]^T issuer (one lane) =====================
        if (lane == 0 && U > 0) {
            constexpr uint32_t idesc_pv = instr_desc_e4m3(UD, 3 * RP, 1, 1);
            const uint64_t vdesc0 = smem_desc(smem_u32(vslots), kTile8, 1024, 2);
            const uint64_t pdesc0 = smem_desc(smem_u32(pbuf), 128, 2048, 0);
            bool ok = true;
            EWalk walk(p, s_prefix, lo, hi);
            int image_unused = 0;
            int o_left = issuer_next_piece(p, s_prefix, s_len, walk, HPC, image_unused, flags);
            uint32_t pio = 0, o_done = 0;   // o_done: steps of the piece done (the first HPC start an accumulator each)
            Ring vro;
            for (uint32_t g = 0; g < U && ok; ++g) {
                const uint32_t pb = g % kPBufs, ob = pio & 1, o_head = o_done % HPC;
                if (o_done == 0 && pio >= 2)   // the epilogue of the piece that used these O^T buffers before has read them
                    ok = wait_or_abort(&bars[E_OFREE + ob], ((pio >> 1) & 1) ^ 1u, abort_flag);
                if (ok) ok = wait_or_abort(&bars[E_VFULL + vro.slot], vro.parity, abort_flag);
                if (ok) ok = wait_or_abort(&bars[E_PFULL + pb], (g / kPBufs) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t vd = vdesc0 + (uint64_t)((uint32_t)vro.slot * (kTile8 >> 4));
                const uint64_t pd = pdesc0 + (uint64_t)(pb * (C::PBUF >> 4));
                const uint32_t tOb = tO + (ob * HPC + o_head) * 3 * RP;
                const bool o_start = o_done < (uint32_t)HPC;   // this head's first product of the piece
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_f8(tOb, vd + (uint64_t)(k * (4096 >> 4)), pd + (uint64_t)(k * (512 >> 4)), idesc_pv, (o_start && k == 0) ? 0u : 1u);
                umma_commit(&bars[E_PFREE + pb]);
                umma_commit(&bars[E_VEMPTY + vro.slot]);
                vro.advance(vring);
                ++o_done;
                if (--o_left == 0) {
                    umma_commit(&bars[E_OFULL + ob]);
                    if (g + 1 < U) {
                        o_left = issuer_next_piece(p, s_prefix, s_len, walk, HPC, image_unused, flags);
                        o_done = 0;
                        ++pio;
                    }
                }
            }
        }
    } else {
        // ============================ softmax and epilogue (warps 0 .. 4 HPC - 1) ============================
        // Team hh = warps 4 hh .. 4 hh + 3 takes the steps of head hh of every item. Thread ltid owns key ltid of
        // its tiles (tensor-memory lane ltid of S^T) and, in the epilogue, output dimension ltid (lane of O^T).
        const int hh = wid >> 2, ltid = tid & (kSmThreads - 1);
        float* tf = s_team + hh * kTeamFloats;
        float* s_negm = tf;
        int32_t* s_lim = (int32_t*)(tf + 7 * RP);
        float* s_red = tf + 3 * RP;
        float* s_mfin = tf + 8 * RP;
        float* s_lfin = tf + 10 * RP;
        ECtx cx;
        cx.negm = s_negm; cx.mref = tf + RP; cx.alpha = tf + 2 * RP; cx.red = s_red; cx.mfin = s_mfin; cx.lfin = s_lfin; cx.lim = s_lim;
        cx.rowloop = s_rowloop; cx.bars = bars; cx.abort_flag = abort_flag;
        cx.lane_off = (uint32_t)((wid & 3) * 32) << 16;
        cx.R = p.R;
        cx.HPC = HPC;
        cx.hh = hh; cx.bar_id = 1 + hh; cx.ltid = ltid; cx.lane = lane; cx.wq = wid & 3;
        const uint32_t lane_off = cx.lane_off;
        bool failed = false;    // a wait of this warp ran out; it stops touching data but keeps the common control flow
        bool aborted = false;   // agreed by the 128 threads of the team

        // The epilogue of a piece runs one piece late, while the next piece is already streaming.
        bool ep_pending = false;
        uint32_t ep_pi = 0;
        int64_t ep_prow = 0;
        float ep_vscale = 1.f;

        uint32_t g = (uint32_t)hh, pi = 0;   // this team's next step (all heads counted), pieces done
        Ring vr;                             // V slot of step g (only boundary tiles look at it)
        for (int i = 0; i < hh; ++i) vr.advance(vring);
        EWalk walk(p, s_prefix, lo, hi);
        EPiece pc;
        EWin win;
        bool have = walk.next(p, s_prefix, s_len, pc, flags);
        grid_dependency_wait();   // the scale factors of the query images are complete
        while (have && !aborted) {
            const uint32_t tOb = tO + ((pi & 1) * HPC + hh) * 3 * RP;   // O^T of this head in this piece
            const int kind = pc.kind, t0 = pc.t0, t1 = pc.t1, cmax = pc.cmax, pn = pc.n, pb_ = pc.b, head = pc.hg * HPC + hh;
            // raw score -> log2 units: softmax scale, K scale of the head, scaling of its query image
            const float scale = p.scale_log2 * p.k_scale[head] * qinv[pb_ * p.Hkv + head];
            int cmin = 0x7fffffff;
#pragma unroll 1
            for (int l = 0; l < p.L; ++l) cmin = min(cmin, e_cut(p, pn, l));
            int seg_l = -1;
            if (kind == 1) {
                win.seek(p, pb_, pn, t0, flags);
                seg_l = win.l;
            }
            e_set_limits(p, cx, RP, kind, pn, seg_l, kind == 1 ? win.wl : 0, true);
            float lsum[RP];    // this key's share of the denominators
#pragma unroll
            for (int r = 0; r < RP; ++r) lsum[r] = 0.f;

            for (int t = t0; t < t1; ++t, g += HPC) {
                int kbase, nvalid;
                bool masked;
                // fresh: a row may see its first key in this tile (first tile of the piece, first tile of a window)
                bool fresh = t == t0;
                if (kind == 0) {
                    kbase = t * UK;
                    nvalid = cmax - kbase;
                    masked = kbase + UK > cmin;
                } else {
                    if (win.l != seg_l) {   // a new window: only the rows of its loop see it
                        seg_l = win.l;
                        e_set_limits(p, cx, RP, kind, pn, seg_l, win.wl, false);
                        fresh = true;
                    }
                    kbase = win.key0;
                    nvalid = win.wl - kbase;
                    masked = true;
                }
                // ---- scores of this thread's key: the two terms of the queries added ----
                const uint32_t sb = g & 1;
                failed = sm_wait(&bars[E_SFULL + sb], (g >> 1) & 1, abort_flag, failed);
                float s[RP];
                if (!failed) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < RP / 16; ++c) {
                        uint32_t a[16], b[16];
                        tmem_ld16(tS + sb * 2 * RP + lane_off + c * 16, a);
                        tmem_ld16(tS + sb * 2 * RP + lane_off + RP + c * 16, b);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) s[c * 16 + j] = __uint_as_float(a[j]) + __uint_as_float(b[j]);
                    }
                    tc_fence_before_sync();
                } else {
#pragma unroll
                    for (int r = 0; r < RP; ++r) s[r] = -INFINITY;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[E_SFREE + sb]);
                if (masked) {
                    const int key = kbase + ltid;
#pragma unroll
                    for (int r = 0; r < RP; ++r)
                        if (key >= s_lim[r]) s[r] = -INFINITY;   // also replaces whatever a stale K row gave
                }
                // Exponents against the reference maxima (rows beyond R: -1e30, never the largest), in place. A fresh
                // tile takes the slow path in any case (its rows have no reference yet), on the scaled scores.
                float over = -INFINITY;
                if (fresh) {
#pragma unroll
                    for (int r = 0; r < RP; ++r) s[r] *= scale;
                } else {
#pragma unroll
                    for (int r = 0; r < RP; ++r) {
                        s[r] = fmaf(s[r], scale, s_negm[r]);
                        over = fmaxf(over, s[r]);
                    }
                }
                const bool trouble = failed || (*abort_flag != 0);
                if (named_barrier_or(cx.bar_id, kSmThreads, fresh || over > kSlack8 || trouble)) {
                    if (named_barrier_or(cx.bar_id, kSmThreads, trouble)) {
                        aborted = true;
                        break;
                    }
                    // Inlined: an out-of-line call would take the addresses of the score and denominator arrays and put
                    // them in local memory. The product before into this head's O^T was that of step g - HPC.
                    // Back to scaled scores first: outside a fresh tile a row either has a finite reference or has seen
                    // no key at all (its scores are -inf and stay so).
                    if (!fresh) {
#pragma unroll
                        for (int r = 0; r < RP; ++r) s[r] -= s_negm[r];
                    }
                    failed = e_slow_path<RP>(s, lsum, cx, t != t0, tOb, &bars[E_PFREE + ((g - HPC) % kPBufs)], ((g - HPC) / kPBufs) & 1, failed);
#pragma unroll
                    for (int r = 0; r < RP; ++r) s[r] += s_negm[r];   // against the new references
                }
                // ---- probabilities as three E4M3 terms into shared memory ----
                const uint32_t pb = g % kPBufs;   // last used by step g - kPBufs
                if (g >= (uint32_t)kPBufs) failed = sm_wait(&bars[E_PFREE + pb], ((g / kPBufs) & 1) ^ 1u, abort_flag, failed);
                uint8_t* pdst = pbuf + pb * C::PBUF + ltid * 16;   // [3 RP / 16 chunks][key][16 codes]
#pragma unroll
                for (int j = 0; j < RP / 16; ++j) {
                    uint32_t c_hi[4], c_mid[4], c_lo[4];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int r0 = j * 16 + 2 * q;
                        const float p0 = fast_exp2(s[r0]);
                        const float p1 = fast_exp2(s[r0 + 1]);
                        lsum[r0] += p0;
                        lsum[r0 + 1] += p1;
                        const uint32_t h2 = pack_f16x2(p0, p1);
                        const uint32_t c0 = f16x2_to_e4m3x2(h2);
                        const uint32_t r1 = mul_f16x2(sub_f16x2(h2, e4m3x2_to_f16x2(c0)), kMidScaleH2);   // exact
                        const uint32_t c1 = f16x2_to_e4m3x2(r1);
                        const uint32_t r2 = mul_f16x2(sub_f16x2(r1, e4m3x2_to_f16x2(c1)), kLoScaleH2);    // exact
                        const uint32_t c2 = f16x2_to_e4m3x2(r2);
                        if (q & 1) {
                            c_hi[q >> 1] = byte_perm(c_hi[q >> 1], c0, 0x5410);
                            c_mid[q >> 1] = byte_perm(c_mid[q >> 1], c1, 0x5410);
                            c_lo[q >> 1] = byte_perm(c_lo[q >> 1], c2, 0x5410);
                        } else {
                            c_hi[q >> 1] = c0;
                            c_mid[q >> 1] = c1;
                            c_lo[q >> 1] = c2;
                        }
                    }
                    if (!failed) {
                        *(uint4*)(pdst + j * 2048) = make_uint4(c_hi[0], c_hi[1], c_hi[2], c_hi[3]);
                        *(uint4*)(pdst + (RP / 16 + j) * 2048) = make_uint4(c_mid[0], c_mid[1], c_mid[2], c_mid[3]);
                        *(uint4*)(pdst + (2 * RP / 16 + j) * 2048) = make_uint4(c_lo[0], c_lo[1], c_lo[2], c_lo[3]);
                    }
                }
                if (masked && nvalid < UK)
                    failed = e_zero_v_rows(vslots + (size_t)vr.slot * kTile8, nvalid, &bars[E_VFULL + vr.slot], vr.parity, cx, failed);
                fence_proxy_async_smem();   // by every thread that wrote, then one arrival per warp
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[E_PFULL + pb]);
#pragma unroll
                for (int i = 0; i < HPC; ++i) vr.advance(vring);
                if (kind == 1) win.advance(p, pb_, pn, flags);
                if (t == t0 && ep_pending) {
                    // put off so that the pipeline restarts first: the partial of the piece before
                    failed = e_epilogue<RP>(p, cx, tO + ((ep_pi & 1) * HPC + hh) * 3 * RP, (int)(ep_pi & 1), (ep_pi >> 1) & 1, ep_prow,
                                            ep_vscale, failed);
                    ep_pending = false;
                }
            }
            if (aborted) break;

            // ---- end of piece: denominators across the 128 keys, parked with the reference maxima; the epilogue
            //      proper runs one piece late ----
            warp_reduce_rows<RP, false>(lsum, lane, s_red + cx.wq * RP);
            named_barrier_sync(cx.bar_id, kSmThreads);
            if (ltid < RP) {
                s_lfin[(pi & 1) * RP + ltid] = (s_red[ltid] + s_red[RP + ltid]) + (s_red[2 * RP + ltid] + s_red[3 * RP + ltid]);
                s_mfin[(pi & 1) * RP + ltid] = cx.mref[ltid];
            }
            const int item = item_index(p, pb_, pc.hg, kind);
            ep_pending = true;
            ep_pi = pi;
            ep_prow = (slot_of(item, cta) * HPC + hh) * p.R;
            ep_vscale = p.v_scale[head];
            if (tid == 0) {   // first and last block of the item, for the merge kernel
                if (t0 == 0) p.item_blocks[2 * item] = cta;
                if (t1 == pc.total) p.item_blocks[2 * item + 1] = cta;
            }
            have = walk.next(p, s_prefix, s_len, pc, flags);
            ++pi;
        }
        if (ep_pending && !aborted) {
            named_barrier_sync(cx.bar_id, kSmThreads);   // s_mfin of the last piece visible to the team
            failed = e_epilogue<RP>(p, cx, tO + ((ep_pi & 1) * HPC + hh) * 3 * RP, (int)(ep_pi & 1), (ep_pi >> 1) & 1, ep_prow, ep_vscale,
                                    failed);
        }
    }

    // ---- common exit: nothing of this block may still be in flight when tensor memory is freed ----
    __syncthreads();
    const bool gave_up = *abort_flag != 0;
    if ((wid == kSIssuerWarp || wid == kOIssuerWarp) && lane == 0) {
        uint64_t* drain = &bars[wid == kSIssuerWarp ? E_DRAIN : E_DRAIN + 1];
        umma_commit(drain);   // arrives once every product issued by this thread has completed
        mbar_wait_bounded(drain, 0, kUmmaWaitNs);
    }
    if (wid == kSIssuerWarp && lane == 0) {
        // query images that were asked for and never waited for get a bounded chance to land
        for (int i = 0; i < 2; ++i)
            if (q_pending[i]) mbar_wait_bounded(&bars[E_QFULL + i], q_parity[i], kUmmaWaitNs);
    }
    if ((wid == kKProducerWarp || wid == kVProducerWarp) && lane == 0 && gave_up) {
        // give every copy that was issued a bounded chance to land
        const bool is_v = wid == kVProducerWarp;
        const uint32_t ring = (uint32_t)(is_v ? vring : kKRing8), issued = (uint32_t)s_ctl[is_v ? 3 : 2];
        for (uint32_t m = issued > ring ? issued - ring : 0; m < issued; ++m)
            mbar_wait_bounded(&bars[(is_v ? E_VFULL : E_KFULL) + (int)(m % ring)], (m / ring) & 1, kUmmaWaitNs);
    }
    if (gave_up) flags |= kDevWaitTimeout;
    if (flags) atomicOr(p.status, flags);
    tc_fence_before_sync();
    __syncthreads();
    if (wid == kSIssuerWarp) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int RP, int HPC, bool HALVES>
cudaError_t e4m3_prepare(size_t smem, int* blocks_per_sm) {
    auto fn = plt_decode_main_umma_e4m3<RP, HPC, HALVES>;
    cudaError_t e = allow_max_dynamic_smem((const void*)fn);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, threads8(HPC), smem);
}

template <int RP, int HPC, bool HALVES>
cudaError_t e4m3_launch(const CUtensorMap maps[4], const Params& p, int grid, size_t smem, const UmmaGeom& geo,
                        const uint8_t* qimg, const float* qinv, cudaStream_t stream) {
    // Programmatic stream serialisation: the blocks set up and the producers start streaming the caches (which the
    // kernel before, the query pack kernel, does not touch) while that kernel still runs; whoever reads what it wrote
    // waits for it first. The partials this kernel writes were last read by the merge kernel of the step before,
    // which had completed before the pack kernel started.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads8(HPC));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, plt_decode_main_umma_e4m3<RP, HPC, HALVES>, maps[0], maps[1], maps[2], maps[3], p, geo, qimg, qinv);
}

}  // namespace

int main_umma_e4m3_rows(int R) { return R <= 16 ? 16 : 32; }

int main_umma_e4m3_max_slots() { return kKRing8 + kMaxVRing8; }

int main_umma_e4m3_min_slots() { return kKRing8 + 3; }

size_t main_umma_e4m3_smem(int R, int hpc, int nslot, int max_batch) {
    return main_umma_e4m3_rows(R) == 16 ? ECfg<16>::smem_bytes(nslot, hpc, max_batch) : ECfg<32>::smem_bytes(nslot, hpc, max_batch);
}

// Bytes of the query image of one (sequence, KV head).
size_t main_umma_e4m3_image_bytes(int R) { return main_umma_e4m3_rows(R) == 16 ? ECfg<16>::QBUF : ECfg<32>::QBUF; }

// `half_pages`: the cache is in pages of 64 tokens (half a tile), which have a kernel of their own.
cudaError_t main_umma_e4m3_prepare(int R, int hpc, bool half_pages, size_t smem, int* blocks_per_sm) {
    const int which = (main_umma_e4m3_rows(R) == 16 ? 0 : 4) + (hpc == 2 ? 2 : 0) + (half_pages ? 1 : 0);
    switch (which) {
        case 0: return e4m3_prepare<16, 1, false>(smem, blocks_per_sm);
        case 1: return e4m3_prepare<16, 1, true>(smem, blocks_per_sm);
        case 2: return e4m3_prepare<16, 2, false>(smem, blocks_per_sm);
        case 3: return e4m3_prepare<16, 2, true>(smem, blocks_per_sm);
        case 4: return e4m3_prepare<32, 1, false>(smem, blocks_per_sm);
        case 5: return e4m3_prepare<32, 1, true>(smem, blocks_per_sm);
        case 6: return e4m3_prepare<32, 2, false>(smem, blocks_per_sm);
        default: return e4m3_prepare<32, 2, true>(smem, blocks_per_sm);
    }
}

cudaError_t launch_pack_q_e4m3(const Params& p, uint8_t* qimg, float* qinv, cudaStream_t stream) {
    if (main_umma_e4m3_rows(p.R) == 16) plt_decode_pack_q_e4m3<16><<<p.B * p.Hkv, 128, 0, stream>>>(p, qimg, qinv);
    else plt_decode_pack_q_e4m3<32><<<p.B * p.Hkv, 256, 0, stream>>>(p, qimg, qinv);
    return cudaGetLastError();
}

cudaError_t launch_main_umma_e4m3(const CUtensorMap maps[4], const Params& p, int grid, size_t smem, int nslot, int kbox,
                                  int wbox, int cap, const uint8_t* qimg, const float* qinv, cudaStream_t stream) {
    const UmmaGeom geo{nslot, kbox, wbox, cap < 1 ? 1 : (cap > nslot ? nslot : cap)};
    const int which = (main_umma_e4m3_rows(p.R) == 16 ? 0 : 4) + (p.hpc == 2 ? 2 : 0) + (2 * p.page_size == UK ? 1 : 0);
    switch (which) {
        case 0: return e4m3_launch<16, 1, false>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 1: return e4m3_launch<16, 1, true>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 2: return e4m3_launch<16, 2, false>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 3: return e4m3_launch<16, 2, true>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 4: return e4m3_launch<32, 1, false>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 5: return e4m3_launch<32, 1, true>(maps, p, grid, smem, geo, qimg, qinv, stream);
        case 6: return e4m3_launch<32, 2, false>(maps, p, grid, smem, geo, qimg, qinv, stream);
        default: return e4m3_launch<32, 2, true>(maps, p, grid, smem, geo, qimg, qinv, stream);
    }
}

}  // namespace plt
