// Shared device-side definitions of the CLP decode-attention kernels: the kernel parameter block,
// the tile plan (how the key tiles of all sequences are laid on one line and cut into equal
// ranges, one per persistent thread block) and the layout of split partials.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace plt {

constexpr int kMaxLoops = 8;
constexpr int kMaxRows = 64;     // packed query rows per KV head: L * q_len * (Hq / Hkv)
constexpr int kMaxBatch = 4096;

// Device status bits (mirrors the PLT_DEV_* values of the public header).
constexpr uint32_t kDevSeqLenClamped = 1u;
constexpr uint32_t kDevPageIdClamped = 2u;
constexpr uint32_t kDevWaitTimeout = 4u;
constexpr uint32_t kDevWinLenClamped = 8u;

// Everything a kernel needs besides its TMA descriptors. Passed by value.
struct Params {
    const void* q;             // [B, L, Hq, d]
    const void* k_cache;       // only the fp32 path dereferences these directly
    const void* v_cache;
    const void* k_win;
    const void* v_win;
    const int32_t* seq_lens;   // [B]
    const int32_t* win_lens;   // [B, L-1] or null
    const int32_t* page_table; // [B, max_pages] or null
    const float* gate_logits;  // [B, L-1, Hq]
    const float* k_scale;      // [Hkv] dequantisation scales of E4M3 caches and windows, else null
    const float* v_scale;
    void* out;                 // [B, L, Hq, d]
    float* part_acc;           // [slots][hpc][R][d]  unnormalised sum of p * V
    float* part_ml;            // [slots][hpc][R][2]  running max (log2 units) and sum of p
    int32_t* prefix;           // [B + 1] tile prefix written by block 0 of the main kernel
    int32_t* item_blocks;      // [items][2] first and last main-kernel block holding a piece of the item (written by
                               // the blocks that own the item's first / last tile; items without tiles are not written)
    uint32_t* status;          // device status word
    int64_t kv_stride_b, kv_stride_n, kv_stride_h;  // elements
    int32_t B, L, Hq, Hkv, G, R, d, w;
    int32_t Qn;                // query tokens per loop in this step (multi-token decode); packed row = (loop * Qn + token) * G + head in group
    int32_t max_seq_len, page_size, max_pages, num_pool_pages;
    int32_t hpc;               // KV heads per work item
    int32_t tile_keys;         // keys per plan tile
    int32_t num_ctas;          // persistent grid size of the main kernel
    int32_t piece_cost;        // what starting and finishing an item costs a block, in tiles (balances the plan)
    float scale_log2;          // sm_scale * log2(e)
    int32_t delta[kMaxLoops];  // per-loop causal offset
};

// ---- per-sequence plan -------------------------------------------------------------------------
// Sequence b contributes, per group of `hpc` KV heads, gt tiles of the shared cache followed by the
// tiles of the windows of loops 2..L. All head groups of a sequence are laid one after the other.
struct SeqPlan {
    int32_t n;                 // clamped N_b
    int32_t cmax;              // largest cutoff over loops = keys of the shared cache that are read
    int32_t gt;                // tiles of the shared cache
    int32_t lt;                // tiles of all windows
    int32_t cut[kMaxLoops];    // keys loop l may see
    int32_t wl[kMaxLoops];     // wl[l] valid window slots of loop l (index 1..L-1; wl[0] unused)
};

__device__ __forceinline__ int32_t ceil_div(int32_t a, int32_t b) { return (a + b - 1) / b; }

// Length of sequence b, clamped to [0, capacity].
__device__ __forceinline__ int32_t seq_len_clamped(const Params& p, int b, uint32_t& flags) {
    int32_t n = p.seq_lens[b];
    if (n < 0 || n > p.max_seq_len) {
        flags |= kDevSeqLenClamped;
        n = n < 0 ? 0 : p.max_seq_len;
    }
    return n;
}

// One loop's share of the plan of sequence b (length n).
__device__ __forceinline__ void seq_plan_step(const Params& p, int b, int32_t n, int l, SeqPlan& s, uint32_t& flags) {
    s.cut[l] = 0;
    s.wl[l] = 0;
    if (l < p.L) {
        int32_t c = n - p.delta[l];
        c = c > 0 ? c : 0;
        s.cut[l] = c;
        s.cmax = c > s.cmax ? c : s.cmax;
        if (l >= 1) {
            int32_t wl = c < p.w ? c : p.w;
            if (p.win_lens != nullptr && c > 0) {
                wl = p.win_lens[b * (p.L - 1) + (l - 1)];
                if (wl < 0 || wl > p.w) {
                    flags |= kDevWinLenClamped;
                    wl = wl < 0 ? 0 : p.w;
                }
            }
            s.wl[l] = wl;
            s.lt += ceil_div(wl, p.tile_keys);
        }
    }
}

__device__ __forceinline__ void seq_plan_n(const Params& p, int b, int32_t n, SeqPlan& s, uint32_t& flags) {
    s.n = n;
    s.cmax = 0;
    s.lt = 0;
#pragma unroll
    for (int l = 0; l < kMaxLoops; ++l) seq_plan_step(p, b, n, l, s, flags);
    s.gt = ceil_div(s.cmax, p.tile_keys);
}

// The same plan, compiled small (a rolled loop, out of line) for kernels whose instruction footprint matters
// more than the few cycles this costs per piece.
static __device__ __noinline__ void seq_plan_small(const Params& p, int b, int32_t n, SeqPlan& s, uint32_t& flags) {
    s.n = n;
    s.cmax = 0;
    s.lt = 0;
#pragma unroll 1
    for (int l = 0; l < kMaxLoops; ++l) seq_plan_step(p, b, n, l, s, flags);
    s.gt = ceil_div(s.cmax, p.tile_keys);
}

__device__ __forceinline__ void seq_plan(const Params& p, int b, SeqPlan& s, uint32_t& flags) {
    seq_plan_n(p, b, seq_len_clamped(p, b, flags), s, flags);
}

// Positions an item of `tiles` tiles takes on the line: its tiles preceded by piece_cost positions that stand for the
// work of starting and finishing it (query rows, plan step, partial store). A block whose share of an item holds
// none of its tiles skips it. Blocks with many short items thus get fewer tiles than blocks inside a long one.
__device__ __forceinline__ int32_t line_len(const Params& p, int32_t tiles) { return tiles > 0 ? tiles + p.piece_cost : 0; }

// Positions sequence b puts on the line.
__device__ __forceinline__ int32_t seq_tiles(const Params& p, int b, uint32_t& flags) {
    SeqPlan s;
    seq_plan(p, b, s, flags);
    return (p.Hkv / p.hpc) * (line_len(p, s.gt) + line_len(p, s.lt));
}

// Blocks that take part in the plan: at least kMinLinePerBlock positions of the line each (so never more blocks than
// tiles, every taking-part block owns work, and the blocks of one item are consecutive). On small batches fewer,
// longer pieces are merged faster than many short ones: B=4, N=1024 measured 18.7 -> 13.7 us per step with 8.
constexpr int kMinLinePerBlock = 8;
__device__ __forceinline__ int plan_ctas(int64_t T, int launched) {
    int64_t c = T / kMinLinePerBlock;
    if (c < 1) c = 1;
    return c < launched ? (int)c : launched;
}

// Range of the tile line owned by block c of C: [c*T/C, (c+1)*T/C).
__device__ __forceinline__ int64_t cta_begin(int64_t T, int c, int C) { return (T * c) / C; }

// Work item index: (sequence, head group, kind) with kind 0 = shared cache, 1 = windows.
__device__ __forceinline__ int item_index(const Params& p, int b, int hg, int kind) {
    return (b * (p.Hkv / p.hpc) + hg) * 2 + kind;
}

// A piece (the part of an item done by one block) stores its partial in slot item + block.
__device__ __forceinline__ int64_t slot_of(int item, int cta) { return (int64_t)item + cta; }


// Block-wide exclusive prefix of seq_tiles into sp[0..B] (shared memory). All threads of the block call it.
// With `lens` (shared memory, B entries) the clamped lengths are kept for PieceWalk, so that walking the pieces
// reads no global memory.
__device__ __forceinline__ void build_prefix(const Params& p, int32_t* sp, uint32_t& flags, int32_t* lens = nullptr,
                                             bool small = false) {
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int b = tid; b < p.B; b += nt) {
        const int32_t n = seq_len_clamped(p, b, flags);
        if (lens != nullptr) lens[b] = n;
        SeqPlan s;
        if (small) seq_plan_small(p, b, n, s, flags);
        else seq_plan_n(p, b, n, s, flags);
        sp[b + 1] = (p.Hkv / p.hpc) * (line_len(p, s.gt) + line_len(p, s.lt));
    }
    if (tid == 0) sp[0] = 0;
    __syncthreads();
    if (tid < 32) {
        // warp 0: each lane owns a contiguous chunk, then a warp scan of the chunk sums
        const int per = (p.B + 31) / 32;
        const int lo = tid * per, hi = min(lo + per, p.B);
        int32_t sum = 0;
        for (int b = lo; b < hi; ++b) sum += sp[b + 1];
        int32_t incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int32_t v = __shfl_up_sync(0xffffffffu, incl, o);
            if (tid >= o) incl += v;
        }
        int32_t run = incl - sum;
        for (int b = lo; b < hi; ++b) {
            run += sp[b + 1];
            sp[b + 1] = run;
        }
    }
    __syncthreads();
}

// Largest b with sp[b] <= pos (pos < sp[B]).
__device__ __forceinline__ int find_seq(const int32_t* sp, int B, int64_t pos) {
    int lo = 0, hi = B;  // invariant: sp[lo] <= pos < sp[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((int64_t)sp[mid] <= pos) lo = mid; else hi = mid;
    }
    return lo;
}

// One piece of work: the tiles [t0, t1) of item (b, hg, kind).
struct Piece {
    int b, hg, kind;
    int t0, t1;
    SeqPlan sp;
};

// Walks the pieces of the range [pos, hi). Usage: PieceWalk w(p, sp, lo, hi); while (w.next(piece)) {...}
struct PieceWalk {
    const Params& p;
    const int32_t* sp;
    const int32_t* lens;   // clamped lengths in shared memory, or null (then seq_lens is read)
    int64_t pos, hi;
    int b;
    __device__ PieceWalk(const Params& p_, const int32_t* sp_, int64_t lo_, int64_t hi_, const int32_t* lens_ = nullptr)
        : p(p_), sp(sp_), lens(lens_), pos(lo_), hi(hi_), b(0) {
        if (pos < hi) b = find_seq(sp, p.B, pos);
    }
    __device__ bool next(Piece& pc, uint32_t& flags) { return next_impl<false>(pc, flags); }
    // The same step compiled small; needs the cached lengths.
    __device__ bool next_small(Piece& pc, uint32_t& flags) { return next_impl<true>(pc, flags); }
    template <bool SMALL>
    __device__ __forceinline__ bool next_impl(Piece& pc, uint32_t& flags) {
        for (;;) {
            if (pos >= hi) return false;
            while ((int64_t)sp[b + 1] <= pos) ++b;
            if (SMALL) seq_plan_small(p, b, lens[b], pc.sp, flags);
            else if (lens != nullptr) seq_plan_n(p, b, lens[b], pc.sp, flags);
            else seq_plan(p, b, pc.sp, flags);
            const int vg = line_len(p, pc.sp.gt), per = vg + line_len(p, pc.sp.lt);
            const int o = (int)(pos - sp[b]);
            pc.b = b;
            pc.hg = o / per;
            const int o2 = o - pc.hg * per;
            int v0;   // position inside the item
            int64_t item_end;
            if (o2 < vg) {
                pc.kind = 0;
                v0 = o2;
                item_end = pos + (vg - o2);
            } else {
                pc.kind = 1;
                v0 = o2 - vg;
                item_end = pos + (per - o2);
            }
            const int64_t end = item_end < hi ? item_end : hi;
            const int v1 = v0 + (int)(end - pos);
            pos = end;
            pc.t0 = v0 > p.piece_cost ? v0 - p.piece_cost : 0;
            pc.t1 = v1 > p.piece_cost ? v1 - p.piece_cost : 0;
            if (pc.t1 > pc.t0) return true;   // else: only the item's lead-in positions fell to this block
        }
    }
};

__device__ __forceinline__ void note_piece(const Params& p, const Piece& pc, int cta) {
    const int item = item_index(p, pc.b, pc.hg, pc.kind);
    if (pc.t0 == 0) p.item_blocks[2 * item] = cta;
    if (pc.t1 == (pc.kind == 0 ? pc.sp.gt : pc.sp.lt)) p.item_blocks[2 * item + 1] = cta;
}

// Window tile cursor: maps the running tile index of a windows item to (loop, first key in that window).
struct WinCursor {
    int l;      // loop index (0-based), 1..L-1
    int key0;   // first key of the tile inside the window of loop l
    // s.wl[l] picked by compares: an index that is not a constant would put the whole plan into local memory.
    static __device__ __forceinline__ int32_t wl_of(const SeqPlan& s, int l) {
        int32_t v = 0;
#pragma unroll
        for (int k = 1; k < kMaxLoops; ++k)
            if (k == l) v = s.wl[k];
        return v;
    }
    __device__ void seek(const Params& p, const SeqPlan& s, int t) {
        l = 1;
        while (l < p.L - 1) {
            int nt = ceil_div(wl_of(s, l), p.tile_keys);
            if (t < nt) break;
            t -= nt;
            ++l;
        }
        key0 = t * p.tile_keys;
    }
    __device__ void advance(const Params& p, const SeqPlan& s) {
        key0 += p.tile_keys;
        while (key0 >= wl_of(s, l) && l < p.L - 1) {
            ++l;
            key0 = 0;
        }
    }
};

}  // namespace plt
