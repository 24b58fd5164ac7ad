// bf16 split-KV main kernel of the CLP decode attention on the 5th-generation tensor cores
// (tcgen05.mma with accumulators in tensor memory), head dimension 128.
//
// Same tile plan and split-partial format as the other main kernels (y_global and y_local of Algorithm 3 for all
// L loops): one persistent block per SM walks its share of the line of 128-key tiles, one KV head
// per work item. The products are laid out with the KEYS as the M dimension, so that the packed
// query rows (all L loop-queries times all GQA heads of a KV head, R <= 64) form the N dimension
// and nothing is padded up to a 64- or 128-row tile:
//
//   S^T [128 keys x RP]  = K_tile [128 x 128] . Q^T        A = K tile as TMA wrote it (K-major,
//                                                          128-byte swizzle), B = packed query rows
//   O^T [128 dims x RP] += V_tile^T [128 x 128] . P^T      A = V tile as TMA wrote it (MN-major,
//                                                          128-byte swizzle), B = probabilities
//
// RP is R rounded up to 16, 32 or 64. All operands are read from shared memory by the tensor core
// itself, once, whatever R is; the 128 softmax threads own one key each (their tensor-memory lane)
// and the RP scores of that key.
//
// Warp roles: warps 0-3 softmax and epilogue (thread = key / output dimension); warp 4 TMA producer
// of K tiles, warp 6 of V tiles; warp 5 issues the S^T products and owns the tensor-memory
// allocation, warp 7 issues the O^T products. One lane works in each of warps 4-7.
//
// Online softmax with a lazily updated reference maximum per row: probabilities are formed against
// a reference that may lag the true running maximum by up to kSlack powers of two; only when a
// score exceeds that (a vote over the 128 threads) are the true maxima reduced across threads and
// the accumulators in tensor memory rescaled. Every wait on an mbarrier is bounded.
//
// Eight warps run eight different loops here, so the instruction working set decides the speed:
// everything that is not on the per-tile path (waits that actually wait, plan arithmetic, the
// rescale, the epilogue) is kept out of line.
#include <cuda_bf16.h>

#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"
#include "plt_umma_util.cuh"

namespace plt {

namespace {

constexpr int kSlotBytes = UK * UD * 2;  // one K tile or one V tile of one KV head
constexpr int kHalfBytes = UK * 128;     // one 64-element half of a tile: [128 keys][128 bytes]
constexpr int kMaxRing = 3;              // slots per ring (one ring for K tiles, one for V tiles)
constexpr int kUmmaThreads = 256;

// mbarrier indices
constexpr int B_KFULL = 0, B_KEMPTY = 3, B_VFULL = 6, B_VEMPTY = 9, B_SFULL = 12 /* two */, B_SFREE = 14 /* two */,
              B_PFULL = 16, B_PFREE = 17, B_OFULL = 18 /* two */, B_OFREE = 20 /* two */, B_DRAIN = 22 /* two */,
              B_COUNT = 24;

template <int RP>
struct UCfg {
    static constexpr int QLBO = RP * 16 + 16;      // bytes between the 16-byte column chunks of the packed query tile
    static constexpr int QBUF = 16 * QLBO;         // one packed query tile: [16 chunks][RP rows][16 bytes] (+ pad)
    static constexpr int PBUF = RP * 256;          // probabilities: [RP / 8][128 keys][16 bytes]
    // Tensor memory: two S^T buffers (tile parity), then two O^T buffers (piece parity, each with RP spare
    // columns after it), RP columns each; rounded up to a power of two.
    static constexpr int TMEM_COLS = RP == 16 ? 128 : (RP == 32 ? 256 : 512);
    __host__ __device__ static constexpr size_t smem_bytes(int nslot, int max_batch) {
        return 1024 + (size_t)nslot * kSlotBytes + PBUF + 2 * QBUF + B_COUNT * 8 +
               (size_t)RP * 4 * (3 + 4 + 2 + 4) + 64 + (size_t)(2 * max_batch + 4) * 4;
    }
};

// ---- softmax side: per-block context and the pieces of work that are off the per-tile path ----------
struct SmCtx {
    float* negm;       // [RP] minus the reference maximum of each row (1e30 while the row has none)
    float* mref;       // [RP] reference maximum, log2 units
    float* alpha;      // [RP] rescale factors of the slow path
    float* red;        // [4][RP] cross-warp reduction scratch
    float* mfin;       // [2][RP] reference maxima of a finished piece, by O^T buffer
    float* lfin;       // [2][RP] its denominators
    int32_t* lim;      // [RP] keys visible to each row in the current segment
    int32_t* rowloop;  // [RP] loop (0-based) of each packed row
    uint64_t* bars;
    volatile int* abort_flag;
    uint32_t lane_off;  // this warp's lane quarter in a tensor-memory address
    float scale;
    int tid, lane, wid;
};

// Slow path of the online softmax: true maxima of the tile over its 128 keys, new reference maxima, and
// (unless this is the first tile of the piece) the rescale of O^T and of the denominators in tensor memory.
// All 128 softmax threads call it together. `pfree_bar` / `pfree_parity`: completion of the last product
// that accumulated into O^T.
template <int RP>
__device__ __noinline__ bool slow_path(const uint32_t (&sv)[RP], float (&lsum)[RP], const SmCtx& cx, bool rescale,
                                       uint32_t tOb, uint64_t* pfree_bar, uint32_t pfree_parity, bool failed) {
    {
        float v[RP];
#pragma unroll
        for (int r = 0; r < RP; ++r) v[r] = __uint_as_float(sv[r]) * cx.scale;
        warp_reduce_rows<RP, true>(v, cx.lane, cx.red + cx.wid * RP);
    }
    named_barrier_sync(1, kSmThreads);
    if (cx.tid < RP) {
        const int t = cx.tid;
        const float mo = cx.mref[t];
        const float mn = fmaxf(fmaxf(mo, fmaxf(cx.red[t], cx.red[RP + t])), fmaxf(cx.red[2 * RP + t], cx.red[3 * RP + t]));
        cx.alpha[t] = (mo == -INFINITY) ? 1.f : exp2f(mo - mn);
        cx.mref[t] = mn;
        cx.negm[t] = (mn == -INFINITY) ? 1e30f : -mn;
    }
    named_barrier_sync(1, kSmThreads);
    if (rescale) {
        failed = sm_wait(pfree_bar, pfree_parity, cx.abort_flag, failed);
        if (!failed) {
            tc_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < RP / 16; ++c) {
                uint32_t o[16];
                tmem_ld16(tOb + cx.lane_off + c * 16, o);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * cx.alpha[c * 16 + j]);
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

// Epilogue of a finished piece: O^T and the denominators out of tensor memory into the split partial.
template <int RP>
__device__ __noinline__ bool epilogue(const Params& p, const SmCtx& cx, uint32_t tOb, int ob, uint32_t parity,
                                      int64_t prow, bool failed) {
    failed = sm_wait(&cx.bars[B_OFULL + ob], parity, cx.abort_flag, failed);
    // 16 columns (packed rows) at a time, rolled: this runs once per piece and must stay small.
#pragma unroll 1
    for (int c = 0; c < RP / 16; ++c) {
        uint32_t o[16];
        if (!failed) {
            tc_fence_after_sync();
            tmem_ld16(tOb + cx.lane_off + c * 16, o);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (c * 16 + j < p.R) p.part_acc[(prow + c * 16 + j) * UD + cx.tid] = __uint_as_float(o[j]);
        }
    }
    tc_fence_before_sync();
    mbar_arrive(&cx.bars[B_OFREE + ob]);
    if (!failed && cx.tid < p.R)
        *(float2*)(p.part_ml + (prow + cx.tid) * 2) = make_float2(cx.mfin[ob * RP + cx.tid], cx.lfin[ob * RP + cx.tid]);
    return failed;
}

// V rows of a boundary tile that hold no data may contain anything: zero them so that 0 * garbage stays 0.
__device__ __noinline__ bool zero_v_rows(uint8_t* vslot, int nvalid, uint64_t* vfull_bar, uint32_t parity, const SmCtx& cx,
                                         bool failed) {
    failed = sm_wait(vfull_bar, parity, cx.abort_flag, failed);
    if (!failed && cx.tid >= nvalid) {
        uint8_t* row = vslot + cx.tid * 128;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            *(uint4*)(row + i * 16) = make_uint4(0u, 0u, 0u, 0u);
            *(uint4*)(row + kHalfBytes + i * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    return failed;
}

// Start of a piece (shared cache) or of a window inside a windows piece: the visibility limit of each row.
__device__ __noinline__ void set_limits(const Params& p, const SmCtx& cx, const Piece& pc, int RP, int win_loop, int wl,
                                        bool new_piece) {
    // Threads still forming the probabilities of the tile before read negm and lim: nobody rewrites them earlier.
    named_barrier_sync(1, kSmThreads);
    if (cx.tid < RP) {
        const int t = cx.tid;
        if (new_piece) {
            cx.mref[t] = -INFINITY;
            cx.negm[t] = 1e30f;
        }
        int lim = 0;
        if (t < p.R) {
            if (pc.kind == 0) {
#pragma unroll
                for (int l = 0; l < kMaxLoops; ++l)
                    if (l == cx.rowloop[t]) lim = pc.sp.cut[l];
            } else if (cx.rowloop[t] == win_loop) {
                lim = wl;
            }
        }
        cx.lim[t] = lim;
    }
    named_barrier_sync(1, kSmThreads);
}

template <int RP>
__global__ void __launch_bounds__(kUmmaThreads, 1)
plt_decode_main_umma(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmKw, const __grid_constant__ CUtensorMap tmVw,
                     const __grid_constant__ Params p, const UmmaGeom geo) {
    using C = UCfg<RP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int ring = geo.ring;
    uint8_t* kslots = smem;                                // K ring, then V ring
    uint8_t* vslots = smem + (size_t)ring * kSlotBytes;
    uint8_t* pbuf = smem + (size_t)2 * ring * kSlotBytes;
    uint8_t* qbuf = pbuf + C::PBUF;                       // two buffers of QBUF
    uint64_t* bars = (uint64_t*)(qbuf + 2 * C::QBUF);
    float* s_negm = (float*)(bars + B_COUNT);
    float* s_mref = s_negm + RP;
    float* s_alpha = s_mref + RP;
    float* s_red = s_alpha + RP;                          // [4][RP]
    int32_t* s_lim = (int32_t*)(s_red + 4 * RP);
    int32_t* s_rowloop = s_lim + RP;
    float* s_mfin = (float*)(s_rowloop + RP);             // [2][RP]
    float* s_lfin = s_mfin + 2 * RP;                      // [2][RP]
    int32_t* s_ctl = (int32_t*)(s_lfin + 2 * RP);         // [0] abort flag, [1] tensor-memory base, [2] K / [3] V tiles issued
    int32_t* s_prefix = s_ctl + 16;                       // [B + 1] tile prefix
    int32_t* s_len = s_prefix + p.B + 1;                  // [B] clamped sequence lengths
    volatile int* abort_flag = (volatile int*)&s_ctl[0];

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[2] = 0;
        s_ctl[3] = 0;
        for (int s = 0; s < kMaxRing; ++s) {
            mbar_init(&bars[B_KFULL + s], 1);
            mbar_init(&bars[B_KEMPTY + s], 1);
            mbar_init(&bars[B_VFULL + s], 1);
            mbar_init(&bars[B_VEMPTY + s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars[B_SFULL + i], 1);
            mbar_init(&bars[B_SFREE + i], kSmThreads);
            mbar_init(&bars[B_OFULL + i], 1);
            mbar_init(&bars[B_OFREE + i], kSmThreads);
            mbar_init(&bars[B_DRAIN + i], 1);
        }
        mbar_init(&bars[B_PFULL], kSmThreads);
        mbar_init(&bars[B_PFREE], 1);
        mbar_fence_init();
    }
    if (tid < RP) s_rowloop[tid] = tid / p.G;
    // Rows R..RP-1 of both packed-query buffers stay zero for the whole kernel.
    for (int i = tid; i < 2 * C::QBUF / 16; i += kUmmaThreads) *(uint4*)(qbuf + i * 16) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (wid == 5) tmem_alloc((uint32_t*)&s_ctl[1], C::TMEM_COLS);
    grid_launch_dependents();  // the merge kernel may be set up meanwhile; it waits for this grid to complete
    build_prefix(p, s_prefix, flags, s_len, /*small=*/true);  // contains __syncthreads
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = (uint32_t)s_ctl[1];
    // S^T of tile parity g at tS + g RP; O^T of piece parity b at tO + 2 b RP, its denominators RP further
    const uint32_t tS = tmem_base, tO = tmem_base + 2 * RP;

    const int64_t T64 = s_prefix[p.B];
    const int cta = blockIdx.x, nctas = plan_ctas(T64, (int)gridDim.x);
    if (cta == 0)
        for (int b = tid; b <= p.B; b += kUmmaThreads) p.prefix[b] = s_prefix[b];
    const bool in_plan = cta < nctas;
    const int64_t lo = in_plan ? cta_begin(T64, cta, nctas) : 0, hi = in_plan ? cta_begin(T64, cta + 1, nctas) : 0;
    const uint32_t T = (uint32_t)(hi - lo);   // tiles this block streams

    if (wid == 4 || wid == 6) {
        // ========================= TMA producers: warp 4 streams K tiles, warp 6 V tiles ==========
        // Each keeps at most `cap` of its tiles in flight: more outstanding requests make the memory system
        // slower, not faster. (cap <= ring, so the slot of the tile issued `cap` tiles ago has not been refilled
        // and its phase parity is unambiguous.)
        if (lane == 0 && T > 0) {
            const bool is_v = wid == 6;
            uint8_t* slots = is_v ? vslots : kslots;
            uint64_t* full = &bars[is_v ? B_VFULL : B_KFULL];
            uint64_t* empty = &bars[is_v ? B_VEMPTY : B_KEMPTY];
            tma_prefetch_desc(is_v ? &tmV : &tmK);
            if (p.L > 1) tma_prefetch_desc(is_v ? &tmVw : &tmKw);
            bool ok = true;
            uint32_t n = 0;
            Ring cur, old;   // slot of tile n, slot of tile n - cap
            TileSource src(p, s_prefix, lo, hi, s_len);
            TileCoords tc;
            for (; n < T && ok; ++n) {
                src.next(p, geo, tc, flags);
                if (n >= (uint32_t)geo.cap) {
                    ok = wait_or_abort(&full[old.slot], old.parity, abort_flag);
                    old.advance(ring);
                }
                if (ok && n >= (uint32_t)ring) ok = wait_or_abort(&empty[cur.slot], cur.parity ^ 1u, abort_flag);
                if (!ok) break;
                const CUtensorMap* map = tc.window ? (is_v ? &tmVw : &tmKw) : (is_v ? &tmV : &tmK);
                uint8_t* dst = slots + (size_t)cur.slot * kSlotBytes;
                mbar_expect_tx(&full[cur.slot], (uint32_t)(tc.nbox * tc.box_keys * 256));
                for (int i = 0; i < tc.nbox; ++i)
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf)
                        tma_load_4d(dst + hf * kHalfBytes + i * tc.box_keys * 128, map, &full[cur.slot], hf * 64, tc.c1[i],
                                    tc.head, tc.c3[i], l2_evict_first_policy());
                cur.advance(ring);
            }
            s_ctl[is_v ? 3 : 2] = (int32_t)n;
        }
    } else if (wid == 5) {
        // ============ S^T = K Q^T issuer (lane 0 issues); owner of tensor memory ==================
        // The whole warp also copies the packed query rows of each piece into shared memory,
        // [16-byte column chunk c][row r], one piece ahead of the products that read them.
        if (T > 0) {
            constexpr uint32_t idesc_qk = instr_desc(UK, RP, 0, 0);
            const uint32_t qbuf_a = smem_u32(qbuf), kslots_a = smem_u32(kslots);
            const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q;
            auto load_q = [&](const Piece& q_pc, int buf) {
                const uint32_t dst = qbuf_a + buf * C::QBUF;
                for (int id = lane; id < p.R * 16; id += 32) {
                    const int r = id >> 4, c = id & 15;
                    const int l = s_rowloop[r], g = r - l * p.G;
                    const __nv_bfloat16* src = qg + (((int64_t)q_pc.b * p.L + l) * p.Hq + q_pc.hg * p.G + g) * UD + c * 8;
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst + c * C::QLBO + r * 16), "l"(src) : "memory");
                }
            };
            bool ok = true;
            PieceWalk walk(p, s_prefix, lo, hi, s_len);
            Piece pc, npc;
            walk_next(walk, pc, flags);
            load_q(pc, 0);
            int t = pc.t0;
            uint32_t pi = 0;
            Ring kr;
            for (uint32_t g = 0; g < T; ++g) {
                const int sb = (int)(g & 1);           // score buffer
                const uint32_t sph = (g >> 1) & 1;     // parity of this use of it
                if (t == pc.t0) {
                    // this piece's rows have arrived; hand them to the tensor core's view of shared memory
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                if (lane == 0) {
                    if (g >= 2)   // the scores that were in this buffer (two tiles ago) have been read out
                        ok = wait_or_abort(&bars[B_SFREE + sb], sph ^ 1u, abort_flag);
                    if (ok) ok = wait_or_abort(&bars[B_KFULL + kr.slot], kr.parity, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t ks_a = kslots_a + (uint32_t)kr.slot * kSlotBytes;
                        const uint32_t q_a = qbuf_a + (pi & 1) * C::QBUF;
#pragma unroll
                        for (int kk = 0; kk < UD / 16; ++kk)
                            umma_bf16(tS + sb * RP, smem_desc(ks_a + (kk >> 2) * kHalfBytes + (kk & 3) * 32, 16, 1024, 2),
                                      smem_desc(q_a + kk * 2 * C::QLBO, C::QLBO, 128, 0), idesc_qk, kk == 0 ? 0u : 1u);
                        umma_commit(&bars[B_SFULL + sb]);
                        umma_commit(&bars[B_KEMPTY + kr.slot]);
                    }
                }
                kr.advance(ring);
                const bool first = t == pc.t0;
                // The other query buffer was last read by the products of the piece before this one; the last of
                // them (tile g - 1) must have completed before the next piece's rows are fetched into it.
                if (first && lane == 0 && ok && g > 0)
                    ok = wait_or_abort(&bars[B_SFULL + (sb ^ 1)], ((g - 1) >> 1) & 1, abort_flag);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (first && walk_next(walk, npc, flags)) load_q(npc, (pi + 1) & 1);
                if (++t == pc.t1 && g + 1 < T) {
                    pc = npc;
                    t = pc.t0;
                    ++pi;
                }
            }
        }
    } else if (wid == 7) {
        // ================= O^T += V^T P^T and denominators += 1 P^T issuer (one lane) ==============
        if (lane == 0 && T > 0) {
            constexpr uint32_t idesc_pv = instr_desc(UD, RP, 1, 1);
            const uint32_t pbuf_a = smem_u32(pbuf), vslots_a = smem_u32(vslots);
            bool ok = true;
            PieceWalk walk(p, s_prefix, lo, hi, s_len);
            Piece pc;
            walk_next(walk, pc, flags);
            int t = pc.t0;
            uint32_t pi = 0;
            Ring vr;
            for (uint32_t g = 0; g < T && ok; ++g) {
                const bool first = t == pc.t0, last = t == pc.t1 - 1;
                const int ob = (int)(pi & 1);
                if (first && pi >= 2)   // the epilogue of the piece that used this O^T buffer before has read it
                    ok = wait_or_abort(&bars[B_OFREE + ob], ((pi >> 1) & 1) ^ 1u, abort_flag);
                if (ok) ok = wait_or_abort(&bars[B_VFULL + vr.slot], vr.parity, abort_flag);
                if (ok) ok = wait_or_abort(&bars[B_PFULL], g & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t vs = vslots_a + (uint32_t)vr.slot * kSlotBytes;
                const uint32_t tOb = tO + ob * 2 * RP;
#pragma unroll
                for (int ks = 0; ks < UK / 16; ++ks) {
                    const uint64_t pd = smem_desc(pbuf_a + ks * 256, 128, 2048, 0);
                    const uint32_t acc = (first && ks == 0) ? 0u : 1u;
                    umma_bf16(tOb, smem_desc(vs + ks * 2048, kHalfBytes, 1024, 2), pd, idesc_pv, acc);
                }
                umma_commit(&bars[B_PFREE]);
                umma_commit(&bars[B_VEMPTY + vr.slot]);
                if (last) umma_commit(&bars[B_OFULL + ob]);
                vr.advance(ring);
                if (++t == pc.t1 && g + 1 < T) {
                    walk_next(walk, pc, flags);
                    t = pc.t0;
                    ++pi;
                }
            }
        }
    } else {
        // ============================ softmax and epilogue (warps 0-3) ============================
        // Thread tid owns key tid of every tile (tensor-memory lane tid of S^T) and, in the epilogue,
        // output dimension tid (lane tid of O^T).
        SmCtx cx;
        cx.negm = s_negm; cx.mref = s_mref; cx.alpha = s_alpha; cx.red = s_red; cx.mfin = s_mfin; cx.lfin = s_lfin; cx.lim = s_lim;
        cx.rowloop = s_rowloop; cx.bars = bars; cx.abort_flag = abort_flag;
        cx.lane_off = (uint32_t)(wid * 32) << 16;
        cx.scale = p.scale_log2;
        cx.tid = tid; cx.lane = lane; cx.wid = wid;
        const float scale = p.scale_log2;
        bool failed = false;    // a wait of this warp ran out; it stops touching data but keeps the common control flow
        bool aborted = false;   // agreed by all 128 threads

        // The epilogue of a piece runs one piece late, while the next piece is already streaming.
        bool ep_pending = false;
        uint32_t ep_pi = 0;
        int64_t ep_prow = 0;

        uint32_t gt = 0, pi = 0;
        Ring vr;   // V slot of tile gt (only boundary tiles look at it)
        PieceWalk walk(p, s_prefix, lo, hi, s_len);
        Piece pc;
        bool have = walk_next(walk, pc, flags);
        while (have && !aborted) {
            const uint32_t tOb = tO + (pi & 1) * 2 * RP;   // O^T of this piece, its denominators RP columns further
            int cmin = 0x7fffffff;
#pragma unroll
            for (int l = 0; l < kMaxLoops; ++l)
                if (l < p.L) cmin = min(cmin, pc.sp.cut[l]);
            WinCursor cur;
            cur.l = 0;
            cur.key0 = 0;
            int seg_l = -1, wl = 0;
            if (pc.kind == 1) {
                cur.seek(p, pc.sp, pc.t0);
                seg_l = cur.l;
#pragma unroll
                for (int k = 1; k < kMaxLoops; ++k)
                    if (k == cur.l) wl = pc.sp.wl[k];
            }
            set_limits(p, cx, pc, RP, seg_l, wl, true);
            float lsum[RP];   // this key's share of the denominators
#pragma unroll
            for (int r = 0; r < RP; ++r) lsum[r] = 0.f;

            for (int t = pc.t0; t < pc.t1; ++t, ++gt) {
                int kbase, nvalid;
                bool masked;
                if (pc.kind == 0) {
                    kbase = t * UK;
                    nvalid = pc.sp.cmax - kbase;
                    masked = kbase + UK > cmin;
                } else {
                    if (cur.l != seg_l) {   // a new window: only the rows of its loop see it
                        seg_l = cur.l;
#pragma unroll
                        for (int k = 1; k < kMaxLoops; ++k)
                            if (k == cur.l) wl = pc.sp.wl[k];
                        set_limits(p, cx, pc, RP, seg_l, wl, false);
                    }
                    kbase = cur.key0;
                    nvalid = wl - kbase;
                    masked = true;
                }
                // ---- scores of this thread's key ----
                const int sb = (int)(gt & 1);
                failed = sm_wait(&bars[B_SFULL + sb], (gt >> 1) & 1, abort_flag, failed);
                uint32_t sv[RP];
                if (!failed) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < RP / 16; ++c) tmem_ld16(tS + sb * RP + cx.lane_off + c * 16, sv + c * 16);
                    tmem_wait_ld();
                    tc_fence_before_sync();
                } else {
#pragma unroll
                    for (int r = 0; r < RP; ++r) sv[r] = 0xff800000u;
                }
                mbar_arrive(&bars[B_SFREE + sb]);
                if (masked) {
                    const int key = kbase + tid;
#pragma unroll
                    for (int r = 0; r < RP; ++r)
                        if (key >= s_lim[r]) sv[r] = 0xff800000u;   // -inf; also replaces whatever a stale K row gave
                }
                float over = -INFINITY;
#pragma unroll
                for (int r = 0; r < RP; ++r)
                    if (r < p.R) over = fmaxf(over, fmaf(__uint_as_float(sv[r]), scale, s_negm[r]));
                const bool trouble = failed || (*abort_flag != 0);
                if (named_barrier_or(1, kSmThreads, over > kSlack || trouble)) {
                    if (named_barrier_or(1, kSmThreads, trouble)) {
                        aborted = true;
                        break;
                    }
                    // Copies, so that the arrays of the per-tile path stay in registers (the out-of-line call takes
                    // the addresses of its arguments).
                    uint32_t sv_c[RP];
                    float ls_c[RP];
#pragma unroll
                    for (int r = 0; r < RP; ++r) {
                        sv_c[r] = sv[r];
                        ls_c[r] = lsum[r];
                    }
                    failed = slow_path<RP>(sv_c, ls_c, cx, t != pc.t0, tOb, &bars[B_PFREE], (gt - 1) & 1, failed);
#pragma unroll
                    for (int r = 0; r < RP; ++r) lsum[r] = ls_c[r];
                }
                // ---- probabilities (bf16) into shared memory; denominators from the rounded values ----
                if (gt > 0) failed = sm_wait(&bars[B_PFREE], (gt - 1) & 1, abort_flag, failed);
#pragma unroll
                for (int j = 0; j < RP / 8; ++j) {
                    uint32_t w4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int r0 = j * 8 + 2 * q;
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sv[r0]), scale, s_negm[r0]));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sv[r0 + 1]), scale, s_negm[r0 + 1]));
                        w4[q] = pack_bf16x2(p0, p1);
                        lsum[r0] += __uint_as_float(w4[q] << 16);            // the rounded values, as the product uses them
                        lsum[r0 + 1] += __uint_as_float(w4[q] & 0xffff0000u);
                    }
                    if (!failed) *(uint4*)(pbuf + j * 2048 + tid * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                }
                if (masked && nvalid < UK)
                    failed = zero_v_rows(vslots + (size_t)vr.slot * kSlotBytes, nvalid, &bars[B_VFULL + vr.slot], vr.parity, cx,
                                         failed);
                fence_proxy_async_smem();
                mbar_arrive(&bars[B_PFULL]);
                vr.advance(ring);
                if (pc.kind == 1) cur.advance(p, pc.sp);
                if (t == pc.t0 && ep_pending) {
                    // put off so that the pipeline restarts first: the partial of the piece before
                    failed = epilogue<RP>(p, cx, tO + (ep_pi & 1) * 2 * RP, (int)(ep_pi & 1), (ep_pi >> 1) & 1, ep_prow, failed);
                    ep_pending = false;
                }
            }
            if (aborted) break;

            // ---- end of piece: denominators across the 128 keys, parked with the reference maxima; the epilogue
            //      proper runs one piece late ----
            warp_reduce_rows<RP, false>(lsum, lane, s_red + wid * RP);
            named_barrier_sync(1, kSmThreads);
            if (tid < RP) {
                s_lfin[(pi & 1) * RP + tid] = (s_red[tid] + s_red[RP + tid]) + (s_red[2 * RP + tid] + s_red[3 * RP + tid]);
                s_mfin[(pi & 1) * RP + tid] = s_mref[tid];
            }
            ep_pending = true;
            ep_pi = pi;
            ep_prow = slot_of(item_index(p, pc.b, pc.hg, pc.kind), cta) * p.R;   // one KV head per item on this path
            if (tid == 0) note_piece(p, pc, cta);
            have = walk_next(walk, pc, flags);
            ++pi;
        }
        if (ep_pending && !aborted) {
            named_barrier_sync(1, kSmThreads);   // s_mfin of the last piece visible to all
            failed = epilogue<RP>(p, cx, tO + (ep_pi & 1) * 2 * RP, (int)(ep_pi & 1), (ep_pi >> 1) & 1, ep_prow, failed);
        }
    }

    // ---- common exit: nothing of this block may still be in flight when tensor memory is freed ----
    __syncthreads();
    const bool gave_up = *abort_flag != 0;
    if ((wid == 5 || wid == 7) && lane == 0) {
        uint64_t* drain = &bars[wid == 5 ? B_DRAIN : B_DRAIN + 1];
        umma_commit(drain);   // arrives once every product issued by this thread has completed
        mbar_wait_bounded(drain, 0, kUmmaWaitNs);
    }
    if ((wid == 4 || wid == 6) && lane == 0 && gave_up) {
        // give every copy that was issued a bounded chance to land
        const bool is_v = wid == 6;
        const uint32_t issued = (uint32_t)s_ctl[is_v ? 3 : 2];
        for (uint32_t m = issued > (uint32_t)ring ? issued - (uint32_t)ring : 0; m < issued; ++m)
            mbar_wait_bounded(&bars[(is_v ? B_VFULL : B_KFULL) + (int)(m % (uint32_t)ring)], (m / (uint32_t)ring) & 1,
                              kUmmaWaitNs);
    }
    if (gave_up) flags |= kDevWaitTimeout;
    if (flags) atomicOr(p.status, flags);
    tc_fence_before_sync();
    __syncthreads();
    if (wid == 5) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int RP>
cudaError_t umma_prepare(size_t smem, int* blocks_per_sm) {
    auto fn = plt_decode_main_umma<RP>;
    cudaError_t e = allow_max_dynamic_smem((const void*)fn);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, kUmmaThreads, smem);
}

}  // namespace

int main_umma_rows(int R) { return R <= 16 ? 16 : (R <= 32 ? 32 : 64); }

int main_umma_max_slots() { return 2 * kMaxRing; }

size_t main_umma_smem(int R, int nslot, int max_batch) {
    const int rp = main_umma_rows(R);
    return rp == 16 ? UCfg<16>::smem_bytes(nslot, max_batch)
                    : (rp == 32 ? UCfg<32>::smem_bytes(nslot, max_batch) : UCfg<64>::smem_bytes(nslot, max_batch));
}

cudaError_t main_umma_prepare(int R, size_t smem, int* blocks_per_sm) {
    const int rp = main_umma_rows(R);
    return rp == 16 ? umma_prepare<16>(smem, blocks_per_sm)
                    : (rp == 32 ? umma_prepare<32>(smem, blocks_per_sm) : umma_prepare<64>(smem, blocks_per_sm));
}

cudaError_t launch_main_umma(const CUtensorMap maps[4], const Params& p, int grid, size_t smem, int nslot, int kbox,
                             int wbox, int cap, cudaStream_t stream) {
    const UmmaGeom geo{nslot / 2, kbox, wbox, cap < 1 ? 1 : (2 * cap > nslot ? nslot / 2 : cap)};
    const int rp = main_umma_rows(p.R);
    if (rp == 16)
        plt_decode_main_umma<16><<<grid, kUmmaThreads, smem, stream>>>(maps[0], maps[1], maps[2], maps[3], p, geo);
    else if (rp == 32)
        plt_decode_main_umma<32><<<grid, kUmmaThreads, smem, stream>>>(maps[0], maps[1], maps[2], maps[3], p, geo);
    else
        plt_decode_main_umma<64><<<grid, kUmmaThreads, smem, stream>>>(maps[0], maps[1], maps[2], maps[3], p, geo);
    return cudaGetLastError();
}

}  // namespace plt
