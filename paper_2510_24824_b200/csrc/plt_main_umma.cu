// bf16 split-KV main kernel of the CLP decode attention on the 5th-generation tensor cores
// (tcgen05.mma with accumulators in tensor memory), head dimension 128.
//
// Same tile plan and split-partial format as the other main kernels (Algorithm 3 lines 2-3 for all
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
// RP is R rounded up to 16, 32 or 64. Both operands of both products are read from shared memory by
// the tensor core itself, once, whatever R is; the 128 softmax threads own one key each (their
// tensor-memory lane) and the RP scores of that key.
//
// Warp roles: warps 0-3 softmax and epilogue (thread = key / output dimension); warp 4 TMA producer
// of K tiles, warp 6 of V tiles; warp 5 issues the S^T products and owns the tensor-memory
// allocation, warp 7 issues the O^T products. One lane works in each of warps 4-7.
//
// Online softmax with a lazily updated reference maximum per row: probabilities are formed against
// a reference that may lag the true running maximum by up to kSlack powers of two; only when a
// score exceeds that (a vote over the 128 threads) are the true maxima reduced across threads and
// the accumulators in tensor memory rescaled. Every wait on an mbarrier is bounded.
#include <cuda_bf16.h>

#include "plt_common.cuh"
#include "plt_host.h"
#include "plt_ptx.cuh"

namespace plt {

namespace {

constexpr int UK = 128;                  // keys per tile
constexpr int UD = 128;                  // head dimension
constexpr int kSlotBytes = UK * UD * 2;  // one K tile or one V tile of one KV head
constexpr int kHalfBytes = UK * 128;     // one 64-element half of a tile: [128 keys][128 bytes]
constexpr int kMaxSlots = 6;
constexpr int kSmThreads = 128;          // softmax threads
constexpr int kUmmaThreads = 256;
constexpr float kSlack = 8.f;
constexpr uint64_t kUmmaWaitNs = 1000000000ull;

// mbarrier indices
constexpr int B_FULL = 0, B_EMPTY = 8, B_SFULL = 16 /* two */, B_SFREE = 18 /* two */, B_PFULL = 20, B_PFREE = 21,
              B_OFULL = 22 /* two */, B_OFREE = 24 /* two */, B_DRAIN = 26 /* two */, B_COUNT = 28;

template <int RP>
struct UCfg {
    static constexpr int QLBO = RP * 16 + 16;      // bytes between the 16-byte column chunks of the packed query tile
    static constexpr int QBUF = 16 * QLBO;         // one packed query tile: [16 chunks][RP rows][16 bytes] (+ pad)
    static constexpr int PBUF = RP * 256;          // probabilities: [RP / 8][128 keys][16 bytes]
    // Tensor memory: two S^T buffers (tile parity), then per piece parity an O^T buffer followed by the denominators (every lane of
    // the latter holds the same RP row sums), RP columns each; rounded up to a power of two.
    static constexpr int TMEM_COLS = RP == 16 ? 128 : (RP == 32 ? 256 : 512);
    static constexpr int ONES_BYTES = 128 * 32;    // A operand of the denominator product: 128 x 16 ones
    __host__ __device__ static constexpr size_t smem_bytes(int nslot, int max_batch) {
        return 1024 + (size_t)nslot * kSlotBytes + PBUF + 2 * QBUF + ONES_BYTES + B_COUNT * 8 + (size_t)RP * 4 * (3 + 4 + 2 + 2) + 64 +
               (size_t)(2 * max_batch + 4) * 4;
    }
};

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets in
// 16-byte units, descriptor version 1, swizzle mode (0 = none, 2 = 128 bytes).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | ((uint64_t)swizzle << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, majorness (0 = K-major, 1 = MN-major), N / 8, M / 16.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Bounded wait that also gives up as soon as another thread of the block has given up. The slow part is kept
// out of line: this kernel has eight warps in different loops, and its instruction footprint decides its speed.
__device__ __noinline__ bool wait_or_abort_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xffu) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kUmmaWaitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_or_abort_slow(bar, parity, abort_flag);
}
// Out-of-line step of the piece walk (the plan arithmetic is long once unrolled over the loops).
__device__ __noinline__ bool walk_next(PieceWalk& walk, Piece& pc, uint32_t& flags) { return walk.next(pc, flags); }

// Reduces N values per lane across the 32 lanes of a warp with N - 1 (+ a few) shuffles instead of 5 N: each
// step halves the values a lane still carries and doubles the lanes they cover. The result of row r goes to
// dst[r] (shared memory).
template <int N, bool MAX>
__device__ __forceinline__ void warp_reduce_rows(float (&v)[N], int lane, float* dst) {
    static_assert(N == 16 || N == 32 || N == 64, "rows per warp reduction");
    if constexpr (N == 64) {
        float a[32], b[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            a[i] = v[i];
            b[i] = v[32 + i];
        }
        warp_reduce_rows<32, MAX>(a, lane, dst);
        warp_reduce_rows<32, MAX>(b, lane, dst + 32);
    } else {
        int n = N;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (n > 1) {
                const bool up = (lane & o) != 0;
                n >>= 1;
#pragma unroll
                for (int i = 0; i < N / 2; ++i) {
                    if (i < n) {
                        const float keep = up ? v[i + n] : v[i];
                        const float send = up ? v[i] : v[i + n];
                        const float got = __shfl_xor_sync(0xffffffffu, send, o);
                        v[i] = MAX ? fmaxf(keep, got) : keep + got;
                    }
                }
            } else {
                const float got = __shfl_xor_sync(0xffffffffu, v[0], o);
                v[0] = MAX ? fmaxf(v[0], got) : v[0] + got;
            }
        }
        // N = 32: lane l holds row l. N = 16: lanes 2r and 2r + 1 both hold row r.
        if (N == 32) dst[lane] = v[0];
        else if ((lane & 1) == 0) dst[lane >> 1] = v[0];
    }
}

// Launch-time geometry of the TMA boxes (set by the host from the tensor maps it encoded).
struct UmmaGeom {
    int nslot;       // ring slots of kSlotBytes
    int kbox;        // keys per box of the shared cache (min(128, page size or capacity))
    int wbox;        // keys per box of a window (min(128, w))
    int cap;         // tiles each of the two producers keeps in flight (issued, not landed) at most; 2 cap <= nslot
};

// Ring position of the K tile / V tile of the n-th tile a block streams (T tiles in all): K(0), then
// K(n), V(n-1) for n = 1 .. T-1, then V(T-1).
__device__ __forceinline__ uint32_t pos_k(uint32_t n) { return n == 0 ? 0u : 2u * n - 1u; }
__device__ __forceinline__ uint32_t pos_v(uint32_t n, uint32_t T) { return n + 1 == T ? 2u * T - 1u : 2u * n + 2u; }

// TMA boxes of one tile: (key coordinate, outermost coordinate) per box, the same for K and V.
struct TileCoords {
    int nbox, box_keys, head;
    bool window;
    int c1[UK / 16], c3[UK / 16];
};

// Walks the tiles of a block's range in order and yields their box coordinates.
struct TileSource {
    PieceWalk walk;
    Piece pc;
    WinCursor cur;
    int t;
    bool have;
    __device__ TileSource(const Params& p, const int32_t* sp, int64_t lo, int64_t hi, const int32_t* lens)
        : walk(p, sp, lo, hi, lens), t(0), have(false) {
        pc.t0 = pc.t1 = 0;
        cur.l = 0;
        cur.key0 = 0;
    }
    __device__ __noinline__ void next(const Params& p, const UmmaGeom& geo, TileCoords& tc, uint32_t& flags) {
        if (!have || t == pc.t1) {
            have = walk.next(pc, flags);
            t = pc.t0;
            if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
        }
        tc.head = pc.hg;
        tc.window = pc.kind == 1;
        if (pc.kind == 0) {
            const int key0 = t * UK;
            tc.box_keys = geo.kbox;
            if (p.page_size > 0) {
                const int rem = pc.sp.cmax - key0;   // keys that hold data from key0 on (>= 1)
                tc.nbox = (min(rem, UK) + tc.box_keys - 1) / tc.box_keys;
                for (int i = 0; i < tc.nbox; ++i) {
                    const int key = key0 + i * tc.box_keys;
                    int page = p.page_table[(int64_t)pc.b * p.max_pages + key / p.page_size];
                    if (page < 0 || page >= p.num_pool_pages) {
                        flags |= kDevPageIdClamped;
                        page = page < 0 ? 0 : p.num_pool_pages - 1;
                    }
                    tc.c1[i] = key % p.page_size;
                    tc.c3[i] = page;
                }
            } else {
                tc.nbox = 1;
                tc.c1[0] = key0;
                tc.c3[0] = pc.b;
            }
        } else {
            tc.box_keys = geo.wbox;
            tc.nbox = 1;
            tc.c1[0] = cur.key0;
            tc.c3[0] = pc.b * (p.L - 1) + (cur.l - 1);
            cur.advance(p, pc.sp);
        }
        ++t;
    }
};

template <int RP>
__global__ void __launch_bounds__(kUmmaThreads, 1)
plt_decode_main_umma(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmKw, const __grid_constant__ CUtensorMap tmVw,
                     const __grid_constant__ Params p, const UmmaGeom geo) {
    using C = UCfg<RP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int nslot = geo.nslot;
    uint8_t* pbuf = smem + (size_t)nslot * kSlotBytes;
    uint8_t* qbuf = pbuf + C::PBUF;                       // two buffers of QBUF
    uint8_t* ones = qbuf + 2 * C::QBUF;                   // 128 x 16 bf16 ones
    uint64_t* bars = (uint64_t*)(ones + C::ONES_BYTES);
    float* s_negm = (float*)(bars + B_COUNT);             // [RP] minus the reference maximum (1e30 while there is none)
    float* s_mref = s_negm + RP;                          // [RP] reference maximum, log2 units
    float* s_alpha = s_mref + RP;                         // [RP] rescale factors of the slow path
    float* s_red = s_alpha + RP;                          // [4][RP] cross-warp reduction scratch
    int32_t* s_lim = (int32_t*)(s_red + 4 * RP);          // [RP] keys visible to each row in the current segment
    int32_t* s_rowloop = s_lim + RP;                      // [RP] loop (0-based) of each packed row
    float* s_mfin = (float*)(s_rowloop + RP);             // [2][RP] reference maxima of a finished piece, by O^T buffer
    int32_t* s_ctl = (int32_t*)(s_mfin + 2 * RP);         // [0] abort flag, [1] tensor-memory base, [2] fills issued
    int32_t* s_prefix = s_ctl + 16;                       // [B + 1] tile prefix
    int32_t* s_len = s_prefix + p.B + 1;                  // [B] clamped sequence lengths
    volatile int* abort_flag = (volatile int*)&s_ctl[0];

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[2] = 0;
        s_ctl[3] = 0;
        for (int s = 0; s < kMaxSlots; ++s) {
            mbar_init(&bars[B_FULL + s], 1);
            mbar_init(&bars[B_EMPTY + s], 1);
        }
        mbar_init(&bars[B_SFULL], 1);
        mbar_init(&bars[B_SFULL + 1], 1);
        mbar_init(&bars[B_SFREE], kSmThreads);
        mbar_init(&bars[B_SFREE + 1], kSmThreads);
        mbar_init(&bars[B_PFULL], kSmThreads);
        mbar_init(&bars[B_PFREE], 1);
        mbar_init(&bars[B_OFULL], 1);
        mbar_init(&bars[B_OFULL + 1], 1);
        mbar_init(&bars[B_OFREE], kSmThreads);
        mbar_init(&bars[B_OFREE + 1], kSmThreads);
        mbar_init(&bars[B_DRAIN], 1);
        mbar_init(&bars[B_DRAIN + 1], 1);
        mbar_fence_init();
    }
    if (tid < RP) s_rowloop[tid] = tid / p.G;
    for (int i = tid; i < C::ONES_BYTES / 4; i += kUmmaThreads) ((uint32_t*)ones)[i] = 0x3f803f80u;
    // Rows R..RP-1 of both packed-query buffers stay zero for the whole kernel.
    for (int i = tid; i < 2 * C::QBUF / 16; i += kUmmaThreads) *(uint4*)(qbuf + i * 16) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (wid == 5) tmem_alloc((uint32_t*)&s_ctl[1], C::TMEM_COLS);
    grid_launch_dependents();  // the merge kernel may be set up meanwhile; it waits for this grid to complete
    build_prefix(p, s_prefix, flags, s_len);  // contains __syncthreads
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = (uint32_t)s_ctl[1];
    // S^T of tile parity g at tS + g RP; O^T of piece parity b at tO + 2 b RP, its denominators RP further
    const uint32_t tS = tmem_base, tO = tmem_base + 2 * RP;

    const int64_t T = s_prefix[p.B];
    const int cta = blockIdx.x, nctas = plan_ctas(T, (int)gridDim.x);
    if (cta == 0)
        for (int b = tid; b <= p.B; b += kUmmaThreads) p.prefix[b] = s_prefix[b];
    const bool in_plan = cta < nctas;
    const int64_t lo = in_plan ? cta_begin(T, cta, nctas) : 0, hi = in_plan ? cta_begin(T, cta + 1, nctas) : 0;

    if (wid == 4 || wid == 6) {
        // ========================= TMA producers: warp 4 streams K tiles, warp 6 V tiles ==========
        // Ring positions follow the order of use: K(0), then K(n), V(n-1) for n = 1.., then the last V, so a
        // V tile (needed one softmax later than its K tile) does not sit in its slot longer than a K tile.
        // Each producer keeps at most `cap` of its copies in flight: more outstanding requests make the
        // memory system slower, not faster.
        if (lane == 0 && lo < hi) {
            const bool is_v = wid == 6;
            tma_prefetch_desc(is_v ? &tmV : &tmK);
            if (p.L > 1) tma_prefetch_desc(is_v ? &tmVw : &tmKw);
            const uint32_t T = (uint32_t)(hi - lo);
            const uint32_t cap = (uint32_t)geo.cap;
            bool ok = true;
            uint32_t issued = 0;
            TileSource src(p, s_prefix, lo, hi, s_len);
            TileCoords tc;
            for (uint32_t n = 0; n < T && ok; ++n) {
                src.next(p, geo, tc, flags);
                const uint32_t pos = is_v ? pos_v(n, T) : pos_k(n);
                const int slot = (int)(pos % (uint32_t)nslot);
                const uint32_t use = pos / (uint32_t)nslot;
                // The copy issued `cap` tiles ago must have landed. With 2 cap <= slots, the slot of that copy
                // cannot have been refilled and landed again by now, so its phase parity is unambiguous; the one
                // exception, ring position 0 (which the V stream reuses early), is skipped.
                if (n >= cap && (is_v || n > cap)) {
                    const uint32_t q = is_v ? pos_v(n - cap, T) : pos_k(n - cap);
                    ok = wait_or_abort(&bars[B_FULL + (int)(q % (uint32_t)nslot)], (q / (uint32_t)nslot) & 1, abort_flag);
                }
                if (ok && use > 0) ok = wait_or_abort(&bars[B_EMPTY + slot], (use - 1) & 1, abort_flag);
                if (!ok) break;
                const CUtensorMap* map = tc.window ? (is_v ? &tmVw : &tmKw) : (is_v ? &tmV : &tmK);
                uint8_t* dst = smem + (size_t)slot * kSlotBytes;
                mbar_expect_tx(&bars[B_FULL + slot], (uint32_t)(tc.nbox * tc.box_keys * 256));
                for (int i = 0; i < tc.nbox; ++i)
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf)
                        tma_load_4d(dst + hf * kHalfBytes + i * tc.box_keys * 128, map, &bars[B_FULL + slot], hf * 64,
                                    tc.c1[i], tc.head, tc.c3[i]);
                ++issued;
            }
            s_ctl[is_v ? 3 : 2] = (int32_t)issued;
        }
    } else if (wid == 5) {
        // ============ S^T = K Q^T issuer (lane 0 issues); owner of tensor memory ==================
        // The whole warp also copies the packed query rows of each piece into shared memory,
        // [16-byte column chunk c][row r], one piece ahead of the products that read them.
        if (lo < hi) {
            constexpr uint32_t idesc_qk = instr_desc(UK, RP, 0, 0);
            const uint32_t qbuf_a = smem_u32(qbuf), smem_a = smem_u32(smem);
            const uint32_t T = (uint32_t)(hi - lo);
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
            bool nhave = false;
            load_q(pc, 0);
            int t = pc.t0;
            uint32_t pi = 0;
            for (uint32_t g = 0; g < T; ++g) {
                const uint32_t pos = pos_k(g);
                const int slot = (int)(pos % (uint32_t)nslot);
                if (t == pc.t0) {
                    // this piece's rows have arrived; hand them to the tensor core's view of shared memory
                    asm volatile("cp.async.wait_all;" ::: "memory");
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                if (lane == 0) {
                    if (g >= 2)   // the scores that were in this buffer (two tiles ago) have been read out
                        ok = wait_or_abort(&bars[B_SFREE + (g & 1)], ((g >> 1) - 1) & 1, abort_flag);
                    if (ok) ok = wait_or_abort(&bars[B_FULL + slot], (pos / (uint32_t)nslot) & 1, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t ks_a = smem_a + (uint32_t)slot * kSlotBytes;
                        const uint32_t q_a = qbuf_a + (pi & 1) * C::QBUF;
#pragma unroll
                        for (int kk = 0; kk < UD / 16; ++kk)
                            umma_bf16(tS + (g & 1) * RP, smem_desc(ks_a + (kk >> 2) * kHalfBytes + (kk & 3) * 32, 16, 1024, 2),
                                      smem_desc(q_a + kk * 2 * C::QLBO, C::QLBO, 128, 0), idesc_qk, kk == 0 ? 0u : 1u);
                        umma_commit(&bars[B_SFULL + (g & 1)]);
                        umma_commit(&bars[B_EMPTY + slot]);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (t == pc.t0) {
                    // The other buffer was last read by the products of the piece before this one; the last of
                    // them (tile g - 1) must have completed before the next piece's rows are fetched into it.
                    if (lane == 0 && g > 0) ok = wait_or_abort(&bars[B_SFULL + ((g - 1) & 1)], ((g - 1) >> 1) & 1, abort_flag);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    nhave = walk_next(walk, npc, flags);
                    if (nhave) load_q(npc, (pi + 1) & 1);
                }
                if (++t == pc.t1 && g + 1 < T) {
                    pc = npc;
                    t = pc.t0;
                    ++pi;
                }
            }
        }
    } else if (wid == 7) {
        // ================= O^T += V^T P^T and denominators += 1 P^T issuer (one lane) ==============
        if (lane == 0 && lo < hi) {
            constexpr uint32_t idesc_pv = instr_desc(UD, RP, 1, 1);
            constexpr uint32_t idesc_l = instr_desc(128, RP, 0, 1);
            const uint32_t pbuf_a = smem_u32(pbuf), smem_a = smem_u32(smem);
            const uint64_t ones_desc = smem_desc(smem_u32(ones), 2048, 128, 0);   // K-major, no swizzle: all ones anyway
            const uint32_t T = (uint32_t)(hi - lo);
            bool ok = true;
            PieceWalk walk(p, s_prefix, lo, hi, s_len);
            Piece pc;
            walk_next(walk, pc, flags);
            int t = pc.t0;
            uint32_t pi = 0;
            for (uint32_t g = 0; g < T && ok; ++g) {
                const uint32_t pos = pos_v(g, T);
                const int slot = (int)(pos % (uint32_t)nslot);
                const bool first = t == pc.t0, last = t == pc.t1 - 1;
                if (first && pi >= 2)   // the epilogue of the piece that used this O^T buffer before has read it
                    ok = wait_or_abort(&bars[B_OFREE + (pi & 1)], ((pi >> 1) - 1) & 1, abort_flag);
                if (ok) ok = wait_or_abort(&bars[B_FULL + slot], (pos / (uint32_t)nslot) & 1, abort_flag);
                if (ok) ok = wait_or_abort(&bars[B_PFULL], g & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t vs = smem_a + (uint32_t)slot * kSlotBytes;
                const uint32_t tOb = tO + (pi & 1) * 2 * RP;
#pragma unroll
                for (int ks = 0; ks < UK / 16; ++ks) {
                    const uint64_t pd = smem_desc(pbuf_a + ks * 256, 128, 2048, 0);
                    const uint32_t acc = (first && ks == 0) ? 0u : 1u;
                    umma_bf16(tOb, smem_desc(vs + ks * 2048, kHalfBytes, 1024, 2), pd, idesc_pv, acc);
                    umma_bf16(tOb + RP, ones_desc, pd, idesc_l, acc);
                }
                umma_commit(&bars[B_PFREE]);
                umma_commit(&bars[B_EMPTY + slot]);
                if (last) umma_commit(&bars[B_OFULL + (pi & 1)]);
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
        const uint32_t lane_off = (uint32_t)(wid * 32) << 16;
        const float scale = p.scale_log2;
        // `failed`: a wait of this warp ran out; the warp stops touching data but keeps the common control flow.
        // Kept warp-uniform, because the tensor-memory loads and stores are warp-collective.
        bool failed = false;
        auto sm_wait = [&](uint64_t* bar, uint32_t parity) {
            bool bad = false;
            if (!failed) bad = !wait_or_abort(bar, parity, abort_flag);
            failed = __any_sync(0xffffffffu, failed || bad);
        };
        bool aborted = false;   // agreed by all 128 threads

        // Epilogue of a finished piece (its reference maxima are parked in s_mfin): O^T out of
        // tensor memory into the split partial. Runs one piece late, while the next piece is already streaming.
        bool ep_pending = false;
        uint32_t ep_pi = 0;
        int64_t ep_prow = 0;
        auto epilogue = [&]() {
            const int ob = (int)(ep_pi & 1);
            const uint32_t tOb = tO + ob * 2 * RP + lane_off;
            sm_wait(&bars[B_OFULL + ob], (ep_pi >> 1) & 1);
            uint32_t o[RP];
            float lmine = 0.f;   // denominator of row tid: every lane of the denominator buffer holds all RP of them
            if (!failed) {
                tc_fence_after_sync();
#pragma unroll
                for (int c = 0; c < RP / 16; ++c) tmem_ld16(tOb + RP + c * 16, o + c * 16);
                tmem_wait_ld();
#pragma unroll
                for (int r = 0; r < RP; ++r)
                    if (r == tid) lmine = __uint_as_float(o[r]);
#pragma unroll
                for (int c = 0; c < RP / 16; ++c) tmem_ld16(tOb + c * 16, o + c * 16);
                tmem_wait_ld();
                tc_fence_before_sync();
            }
            mbar_arrive(&bars[B_OFREE + ob]);
            if (!failed) {
                if (tid < p.R) *(float2*)(p.part_ml + (ep_prow + tid) * 2) = make_float2(s_mfin[ob * RP + tid], lmine);
#pragma unroll
                for (int r = 0; r < RP; ++r)
                    if (r < p.R) p.part_acc[(ep_prow + r) * UD + tid] = __uint_as_float(o[r]);
            }
            ep_pending = false;
        };

        uint32_t gt = 0, pi = 0;
        PieceWalk walk(p, s_prefix, lo, hi, s_len);
        Piece pc, npc;
        bool have = walk_next(walk, pc, flags);
        while (have && !aborted) {
            const bool nhave = walk_next(walk, npc, flags);
            const uint32_t tOb = tO + (pi & 1) * 2 * RP;   // O^T of this piece, its denominators RP columns further

            // ---- per-piece state ----
            int cmin = 0x7fffffff;
#pragma unroll
            for (int l = 0; l < kMaxLoops; ++l)
                if (l < p.L) cmin = min(cmin, pc.sp.cut[l]);
            if (tid < RP) {
                s_mref[tid] = -INFINITY;
                s_negm[tid] = 1e30f;
                if (pc.kind == 0) {
                    int cut = 0;
#pragma unroll
                    for (int l = 0; l < kMaxLoops; ++l)
                        if (l == s_rowloop[tid]) cut = pc.sp.cut[l];
                    s_lim[tid] = tid < p.R ? cut : 0;
                }
            }
            named_barrier_sync(1, kSmThreads);
            WinCursor cur;
            cur.l = 0;
            cur.key0 = 0;
            if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
            int seg_l = -1, wl = 0;

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
                        if (tid < RP) s_lim[tid] = (tid < p.R && s_rowloop[tid] == cur.l) ? wl : 0;
                        named_barrier_sync(1, kSmThreads);
                    }
                    kbase = cur.key0;
                    nvalid = wl - kbase;
                    masked = true;
                }
                // ---- scores of this thread's key ----
                sm_wait(&bars[B_SFULL + (gt & 1)], (gt >> 1) & 1);
                uint32_t sv[RP];
                if (!failed) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < RP / 16; ++c) tmem_ld16(tS + (gt & 1) * RP + lane_off + c * 16, sv + c * 16);
                    tmem_wait_ld();
                    tc_fence_before_sync();
                } else {
#pragma unroll
                    for (int r = 0; r < RP; ++r) sv[r] = 0xff800000u;
                }
                mbar_arrive(&bars[B_SFREE + (gt & 1)]);
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
                    // ---- slow path: true maxima over the 128 keys, new references, rescale O^T ----
                    {
                        float v[RP];
#pragma unroll
                        for (int r = 0; r < RP; ++r) v[r] = __uint_as_float(sv[r]) * scale;
                        warp_reduce_rows<RP, true>(v, lane, s_red + wid * RP);
                    }
                    named_barrier_sync(1, kSmThreads);
                    if (tid < RP) {
                        const float mo = s_mref[tid];
                        const float mn = fmaxf(fmaxf(mo, fmaxf(s_red[tid], s_red[RP + tid])),
                                               fmaxf(s_red[2 * RP + tid], s_red[3 * RP + tid]));
                        s_alpha[tid] = (mo == -INFINITY) ? 1.f : exp2f(mo - mn);
                        s_mref[tid] = mn;
                        s_negm[tid] = (mn == -INFINITY) ? 1e30f : -mn;
                    }
                    named_barrier_sync(1, kSmThreads);
                    if (t != pc.t0) {
                        // O^T holds the earlier tiles of this piece; their last product must have completed
                        sm_wait(&bars[B_PFREE], (gt - 1) & 1);
                        if (!failed) {
                            tc_fence_after_sync();
#pragma unroll
                            for (int c = 0; c < 2 * RP / 16; ++c) {   // O^T, then the denominators
                                uint32_t o[16];
                                tmem_ld16(tOb + lane_off + c * 16, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    o[j] = __float_as_uint(__uint_as_float(o[j]) * s_alpha[(c * 16 + j) % RP]);
                                tmem_st16(tOb + lane_off + c * 16, o);
                            }
                            tmem_wait_st();
                            tc_fence_before_sync();
                        }
                    }
                }
                // ---- probabilities (bf16) into shared memory; the tensor core sums these rounded values into the denominators ----
                if (gt > 0) sm_wait(&bars[B_PFREE], (gt - 1) & 1);
#pragma unroll
                for (int j = 0; j < RP / 8; ++j) {
                    uint32_t w4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int r0 = j * 8 + 2 * q;
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sv[r0]), scale, s_negm[r0]));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sv[r0 + 1]), scale, s_negm[r0 + 1]));
                        w4[q] = pack_bf16x2(p0, p1);
                    }
                    if (!failed) *(uint4*)(pbuf + j * 2048 + tid * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                }
                if (masked && nvalid < UK) {
                    // V rows that hold no data may contain anything: zero them so that 0 * garbage stays 0
                    const uint32_t fillv = pos_v(gt, (uint32_t)(hi - lo));
                    const int slot = (int)(fillv % (uint32_t)nslot);
                    sm_wait(&bars[B_FULL + slot], (fillv / (uint32_t)nslot) & 1);
                    if (!failed && tid >= nvalid) {
                        uint8_t* row = smem + (size_t)slot * kSlotBytes + tid * 128;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            *(uint4*)(row + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                            *(uint4*)(row + kHalfBytes + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                }
                fence_proxy_async_smem();
                mbar_arrive(&bars[B_PFULL]);
                if (pc.kind == 1) cur.advance(p, pc.sp);
                if (t == pc.t0) {
                    // Work that was put off so that the pipeline restarts first: the partial of the piece before.
                    if (ep_pending) epilogue();
                }
            }
            if (aborted) break;

            // ---- end of piece: park its reference maxima; the epilogue proper runs one piece late ----
            if (tid < RP) s_mfin[(pi & 1) * RP + tid] = s_mref[tid];
            ep_pending = true;
            ep_pi = pi;
            ep_prow = slot_of(item_index(p, pc.b, pc.hg, pc.kind), cta) * p.R;   // hpc == 1 on this path
            pc = npc;
            have = nhave;
            ++pi;
            if (!have) {
                named_barrier_sync(1, kSmThreads);   // s_mfin of the last piece visible to all
                epilogue();
            }
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
        const uint32_t T = (uint32_t)(hi - lo);
        const uint32_t issued = (uint32_t)s_ctl[is_v ? 3 : 2];
        for (uint32_t n = issued > (uint32_t)nslot ? issued - (uint32_t)nslot : 0; n < issued; ++n) {
            const uint32_t pos = is_v ? pos_v(n, T) : pos_k(n);
            mbar_wait_bounded(&bars[B_FULL + (int)(pos % (uint32_t)nslot)], (pos / (uint32_t)nslot) & 1, kUmmaWaitNs);
        }
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
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, fn, kUmmaThreads, smem);
}

}  // namespace

int main_umma_rows(int R) { return R <= 16 ? 16 : (R <= 32 ? 32 : 64); }

int main_umma_max_slots() { return kMaxSlots; }

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
    const UmmaGeom geo{nslot, kbox, wbox, cap < 1 ? 1 : (2 * cap > nslot ? nslot / 2 : cap)};
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
