// bf16 split-KV main kernel of the CLP decode attention (Algorithm 3 lines 2-3 for all L loops).
//
// One persistent thread block owns an equal share of the line of key tiles of all sequences.
// A producer warp streams K/V tiles of the shared first-loop cache (and of the windows of loops
// 2..L) into a shared-memory ring with tiled TMA loads (128-byte swizzle); consumer warps run
// S = Q K^T and acc += P V on the tensor cores with all L loop-queries and all GQA heads of a KV
// head packed as the 16*MT rows of one tile, so every K/V byte is read from HBM once and used by
// every loop. Softmax state is kept online in fp32 per row. Each consumer warp owns one 16-key
// slice of a tile for one KV head and 16 packed rows; slices are merged once per piece.
#pragma once
#include <cuda_bf16.h>
#include "plt_common.cuh"
#include "plt_ptx.cuh"

namespace plt {

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every barrier wait gives up after ~2 s

template <int D, int MT, int HPC, int KW>
struct MainCfg {
    static constexpr int NH = D / 64;               // 64-element (128-byte) halves of a head row
    static constexpr int TK = 16 * KW;              // keys per tile
    static constexpr int NCW = HPC * KW * MT;       // consumer warps
    static constexpr int NTHREADS = (NCW + 1) * 32;
    static constexpr int MIN_BLOCKS = NCW <= 2 ? 4 : (NCW <= 4 ? 2 : 1);  // register budget: blocks per SM aimed at
    static constexpr int BOX_BYTES = 128 * TK * HPC;        // one TMA box: [HPC][TK][64 elements]
    static constexpr int TENSOR_BYTES = NH * BOX_BYTES;     // K (or V) part of a stage
    static constexpr int STAGE_BYTES = 2 * TENSOR_BYTES;
    static constexpr int MROW = D + 8;                      // padded row of the merge buffer (floats)
    static constexpr int MERGE_ACC_FLOATS = KW > 1 ? HPC * MT * 16 * MROW : 0;
    static constexpr int MERGE_ML_FLOATS = KW > 1 ? HPC * MT * KW * 32 : 0;
    static constexpr int kMaxStages = 12;
    __host__ __device__ static constexpr size_t smem_bytes(int stages, int max_batch) {
        return 1024 /* alignment slack */ + (size_t)stages * STAGE_BYTES + 2 * kMaxStages * 8 +
               (size_t)(MERGE_ACC_FLOATS + MERGE_ML_FLOATS) * 4 + (size_t)(max_batch + 4) * 4;
    }
};

template <int D, int MT, int HPC, int KW, bool MASKED>
__device__ __forceinline__ void process_slice(uint32_t sK, uint32_t sV, const uint32_t (&qf)[D / 16][4],
                                              float (&acc)[D / 8][4], float (&m)[2], float (&lsum)[2],
                                              int lim0, int lim1, int nvalid, float scale_log2, int lane,
                                              int kw, int h_local) {
    using C = MainCfg<D, MT, HPC, KW>;
    const int tq = lane & 3;
    // ---- S = Q K^T for this warp's 16 keys -------------------------------------------------------
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    {
        const int key = kw * 16 + ((lane >> 4) << 3) + (lane & 7);
        const int dhalf = (lane >> 3) & 1;
        const uint32_t row = sK + (uint32_t)((h_local * C::TK + key) * 128);
        const int x = key & 7;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int cin = ((ks & 3) * 2 + dhalf) ^ x;
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(row + (uint32_t)((ks >> 2) * C::BOX_BYTES + cin * 16), b0, b1, b2, b3);
            mma_bf16_16816(s[0], qf[ks], b0, b1);
            mma_bf16_16816(s[1], qf[ks], b2, b3);
        }
    }
    // ---- per-loop causal cutoff / window length (only on boundary tiles) --------------------------
    if (MASKED) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int kk = kw * 16 + nt * 8 + 2 * tq + e;
                if (kk >= lim0) s[nt][e] = -INFINITY;
                if (kk >= lim1) s[nt][2 + e] = -INFINITY;
            }
    }
    // ---- online softmax, fp32, rows grp (i = 0) and grp + 8 (i = 1) ------------------------------
    uint32_t pa[4];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float mx = fmaxf(fmaxf(s[0][2 * i], s[0][2 * i + 1]), fmaxf(s[1][2 * i], s[1][2 * i + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m[i], mx * scale_log2);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = fast_exp2(m[i] - m_use);
        m[i] = m_new;
        const float p00 = fast_exp2(fmaf(s[0][2 * i], scale_log2, -m_use));
        const float p01 = fast_exp2(fmaf(s[0][2 * i + 1], scale_log2, -m_use));
        const float p10 = fast_exp2(fmaf(s[1][2 * i], scale_log2, -m_use));
        const float p11 = fast_exp2(fmaf(s[1][2 * i + 1], scale_log2, -m_use));
        pa[i] = pack_bf16x2(p00, p01);       // keys 2tq, 2tq+1
        pa[2 + i] = pack_bf16x2(p10, p11);   // keys 8 + 2tq, 9 + 2tq
        // The denominator sums the probabilities as rounded to bf16, i.e. exactly the weights the P V
        // product uses: numerator and denominator then carry the same rounding, which cancels when a few
        // keys dominate the softmax.
        const float r00 = __uint_as_float(pa[i] << 16), r01 = __uint_as_float(pa[i] & 0xffff0000u);
        const float r10 = __uint_as_float(pa[2 + i] << 16), r11 = __uint_as_float(pa[2 + i] & 0xffff0000u);
        lsum[i] = fmaf(lsum[i], alpha, (r00 + r01) + (r10 + r11));
#pragma unroll
        for (int nd = 0; nd < D / 8; ++nd) {
            acc[nd][2 * i] *= alpha;
            acc[nd][2 * i + 1] *= alpha;
        }
    }
    // ---- acc += P V ------------------------------------------------------------------------------
    {
        const int mi = lane >> 3;
        const int key = kw * 16 + ((mi & 1) << 3) + (lane & 7);
        const uint32_t row = sV + (uint32_t)((h_local * C::TK + key) * 128);
        const int x = key & 7;
        uint32_t mask_lo = 0xffffffffu, mask_hi = 0xffffffffu;
        if (MASKED) {
            // Rows at or beyond nvalid may hold anything (uninitialised cache slots): force them to 0
            // so that 0 * garbage cannot produce NaN.
            const int k0 = kw * 16 + 2 * tq;
            mask_lo = (k0 < nvalid ? 0x0000ffffu : 0u) | (k0 + 1 < nvalid ? 0xffff0000u : 0u);
            mask_hi = (k0 + 8 < nvalid ? 0x0000ffffu : 0u) | (k0 + 9 < nvalid ? 0xffff0000u : 0u);
        }
#pragma unroll
        for (int j = 0; j < D / 16; ++j) {
            const int cin = ((j & 3) * 2 + (mi >> 1)) ^ x;
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(row + (uint32_t)((j >> 2) * C::BOX_BYTES + cin * 16), b0, b1, b2, b3);
            if (MASKED) {
                b0 &= mask_lo;
                b2 &= mask_lo;
                b1 &= mask_hi;
                b3 &= mask_hi;
            }
            mma_bf16_16816(acc[2 * j], pa, b0, b1);
            mma_bf16_16816(acc[2 * j + 1], pa, b2, b3);
        }
    }
}

template <int D, int MT, int HPC, int KW>
__global__ void __launch_bounds__(MainCfg<D, MT, HPC, KW>::NTHREADS, MainCfg<D, MT, HPC, KW>::MIN_BLOCKS)
plt_decode_main_bf16(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmKw, const __grid_constant__ CUtensorMap tmVw,
                     const __grid_constant__ Params p, const int stages) {
    using C = MainCfg<D, MT, HPC, KW>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = (uint64_t*)(smem + (size_t)stages * C::STAGE_BYTES);
    uint64_t* empty_bar = full_bar + C::kMaxStages;
    float* merge_acc = (float*)(empty_bar + C::kMaxStages);
    float* merge_ml = merge_acc + C::MERGE_ACC_FLOATS;
    int32_t* s_ctl = (int32_t*)(merge_ml + C::MERGE_ML_FLOATS);  // [0] abort flag, [1] tiles issued
    int32_t* s_prefix = s_ctl + 2;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t flags = 0;
    bool ok = true;
#ifdef PLT_TIMELINE
    unsigned long long* tl = (unsigned long long*)p.timeline + (size_t)blockIdx.x * 8;
    if (tid == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
        tl[0] = smid;
        tl[1] = global_timer_ns();
    }
#endif

    if (tid == 0) {
        s_ctl[0] = 0;
        s_ctl[1] = 0;
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], C::NCW);
        }
        mbar_fence_init();
    }
    grid_launch_dependents();  // the merge kernel may be set up meanwhile; it waits for this grid to complete
    build_prefix(p, s_prefix, flags);  // contains __syncthreads
    const int64_t T = s_prefix[p.B];
    const int cta = blockIdx.x, nctas = plan_ctas(T, (int)gridDim.x);
    if (cta == 0)
        for (int b = tid; b <= p.B; b += C::NTHREADS) p.prefix[b] = s_prefix[b];
    const bool in_plan = cta < nctas;
    const int64_t lo = in_plan ? cta_begin(T, cta, nctas) : 0, hi = in_plan ? cta_begin(T, cta + 1, nctas) : 0;
#ifdef PLT_TIMELINE
    if (tid == 0) { tl[2] = global_timer_ns(); tl[7] = (unsigned long long)(hi - lo); }
    bool tl_first = true;
#endif

    if (wid == C::NCW) {
        // =========================== producer warp (one lane issues) ==============================
        if (lane == 0 && lo < hi) {
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            if (p.L > 1) {
                tma_prefetch_desc(&tmKw);
                tma_prefetch_desc(&tmVw);
            }
            uint32_t it = 0;
            int stage = 0;
            uint32_t use = 0;  // how many times `stage` has been filled before
            PieceWalk walk(p, s_prefix, lo, hi);
            Piece pc;
            while (walk.next(pc, flags)) {
                const int head0 = pc.hg * HPC;
                WinCursor cur;
                if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
                // Paged cache: the id of the page in use and, loaded one page early so that its latency is off the
                // issue path, the id of the page after it.
                const int32_t* ptab = p.page_table + (int64_t)pc.b * p.max_pages;
                int pg = 0, page_id = 0, page_next = 0;
                if (pc.kind == 0 && p.page_size > 0) {
                    pg = (pc.t0 * C::TK) / p.page_size;
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
                            const int in_page = key0 % p.page_size;
                            if (in_page == 0 && t != pc.t0) {
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
#ifdef PLT_TIMELINE
                    if (tl_first) { tl[3] = global_timer_ns(); tl_first = false; }
#endif
                    if (ok) {
                        uint8_t* dst = smem + (size_t)stage * C::STAGE_BYTES;
                        mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
#pragma unroll
                        for (int hf = 0; hf < C::NH; ++hf) {
                            tma_load_4d(dst + hf * C::BOX_BYTES, mk, &full_bar[stage], hf * 64, c1, head0, c3);
                            tma_load_4d(dst + C::TENSOR_BYTES + hf * C::BOX_BYTES, mv, &full_bar[stage], hf * 64, c1,
                                        head0, c3);
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
        const int h_local = wid / (KW * MT);
        const int mt = (wid % (KW * MT)) / KW;
        const int kw = wid % KW;
        const int grp = lane >> 2, tq = lane & 3;
        const int r0 = mt * 16 + grp, r1 = r0 + 8;
        const int l0 = r0 / p.G, l1 = r1 / p.G;     // loop (0-based) of each row
        const bool v0 = r0 < p.R, v1 = r1 < p.R;
        const __nv_bfloat16* qg = (const __nv_bfloat16*)p.q;

        int stage = 0;
        uint32_t use = 0;
        int q_b = -1, q_hg = -1;   // (sequence, head group) whose query rows are in qf
        uint32_t qf[D / 16][4];
        PieceWalk walk(p, s_prefix, lo, hi);
        Piece pc;
        while (walk.next(pc, flags)) {
            const int kvh = pc.hg * HPC + h_local;
            // ---- packed query rows of this KV head: row r = loop * G + head-in-group --------------
            // (the windows item of a head group follows its shared-cache item: same rows, kept)
            if (pc.b != q_b || pc.hg != q_hg) {
                q_b = pc.b;
                q_hg = pc.hg;
                const int64_t q0 = (((int64_t)pc.b * p.L + l0) * p.Hq + kvh * p.G + (r0 - l0 * p.G)) * D;
                const int64_t q1 = (((int64_t)pc.b * p.L + l1) * p.Hq + kvh * p.G + (r1 - l1 * p.G)) * D;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const int c = ks * 16 + 2 * tq;
                    qf[ks][0] = v0 ? *(const uint32_t*)(qg + q0 + c) : 0u;
                    qf[ks][1] = v1 ? *(const uint32_t*)(qg + q1 + c) : 0u;
                    qf[ks][2] = v0 ? *(const uint32_t*)(qg + q0 + c + 8) : 0u;
                    qf[ks][3] = v1 ? *(const uint32_t*)(qg + q1 + c + 8) : 0u;
                }
            }
            int cut0 = 0, cut1 = 0, cmin = 0x7fffffff;
#pragma unroll
            for (int l = 0; l < kMaxLoops; ++l)
                if (l < p.L) {
                    if (v0 && l == l0) cut0 = pc.sp.cut[l];
                    if (v1 && l == l1) cut1 = pc.sp.cut[l];
                    cmin = min(cmin, pc.sp.cut[l]);
                }
            float acc[D / 8][4];
#pragma unroll
            for (int nd = 0; nd < D / 8; ++nd) acc[nd][0] = acc[nd][1] = acc[nd][2] = acc[nd][3] = 0.f;
            float m[2] = {-INFINITY, -INFINITY}, lsum[2] = {0.f, 0.f};

            WinCursor cur;
            if (pc.kind == 1) cur.seek(p, pc.sp, pc.t0);
            for (int t = pc.t0; t < pc.t1; ++t) {
                if (ok) {
                    ok = mbar_wait_bounded(&full_bar[stage], use & 1, kWaitLimitNs);
                    if (!ok) flags |= kDevWaitTimeout;
                }
#ifdef PLT_TIMELINE
                if (tl_first && tid == 0) { tl[4] = global_timer_ns(); }
                tl_first = false;
#endif
                const uint32_t sK = smem_u32(smem + (size_t)stage * C::STAGE_BYTES);
                const uint32_t sV = sK + C::TENSOR_BYTES;
                if (pc.kind == 0) {
                    const int key0 = t * C::TK;
                    if (ok) {
                        if (key0 + C::TK <= cmin)
                            process_slice<D, MT, HPC, KW, false>(sK, sV, qf, acc, m, lsum, 0, 0, 0, p.scale_log2, lane,
                                                                 kw, h_local);
                        else
                            process_slice<D, MT, HPC, KW, true>(sK, sV, qf, acc, m, lsum, cut0 - key0, cut1 - key0,
                                                                pc.sp.cmax - key0, p.scale_log2, lane, kw, h_local);
                    }
                } else {
                    // Window of loop cur.l: only the rows of that loop take part.
                    const int l = cur.l;
                    int wl = 0;
#pragma unroll
                    for (int k = 1; k < kMaxLoops; ++k)
                        if (k == l) wl = pc.sp.wl[k];
                    const int row_lo = l * p.G, row_hi = row_lo + p.G;
                    const bool any = row_lo < mt * 16 + 16 && row_hi > mt * 16;
                    if (ok && any) {
                        const int n = wl - cur.key0;
                        process_slice<D, MT, HPC, KW, true>(sK, sV, qf, acc, m, lsum, (v0 && l0 == l) ? n : 0,
                                                            (v1 && l1 == l) ? n : 0, n, p.scale_log2, lane, kw,
                                                            h_local);
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
            for (int i = 0; i < 2; ++i) {
                lsum[i] += __shfl_xor_sync(0xffffffffu, lsum[i], 1);
                lsum[i] += __shfl_xor_sync(0xffffffffu, lsum[i], 2);
            }
            const int64_t slot = slot_of(item_index(p, pc.b, pc.hg, pc.kind), cta);
            const int64_t prow = (slot * HPC + h_local) * p.R;
            if (tid == 0) note_piece(p, pc, cta);
            if (KW == 1) {
#pragma unroll
                for (int nd = 0; nd < D / 8; ++nd) {
                    const int c = nd * 8 + 2 * tq;
                    if (v0) *(float2*)(p.part_acc + (prow + r0) * D + c) = make_float2(acc[nd][0], acc[nd][1]);
                    if (v1) *(float2*)(p.part_acc + (prow + r1) * D + c) = make_float2(acc[nd][2], acc[nd][3]);
                }
                if (tq == 0) {
                    if (v0) *(float2*)(p.part_ml + (prow + r0) * 2) = make_float2(m[0], lsum[0]);
                    if (v1) *(float2*)(p.part_ml + (prow + r1) * 2) = make_float2(m[1], lsum[1]);
                }
            } else {
                const int gidx = h_local * MT + mt;
                float* macc = merge_acc + gidx * 16 * C::MROW;
                float* mml = merge_ml + gidx * KW * 32;
                if (tq == 0) {
                    *(float2*)(mml + (kw * 16 + grp) * 2) = make_float2(m[0], lsum[0]);
                    *(float2*)(mml + (kw * 16 + grp + 8) * 2) = make_float2(m[1], lsum[1]);
                }
                named_barrier_sync(1, C::NCW * 32);
                float mstar[2], lstar[2], sc[2];
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    float mm = -INFINITY;
#pragma unroll
                    for (int k = 0; k < KW; ++k) mm = fmaxf(mm, mml[(k * 16 + grp + 8 * i) * 2]);
                    const float ms = (mm == -INFINITY) ? 0.f : mm;
                    float ll = 0.f;
#pragma unroll
                    for (int k = 0; k < KW; ++k) {
                        const float2 v = *(const float2*)(mml + (k * 16 + grp + 8 * i) * 2);
                        ll = fmaf(v.y, fast_exp2(v.x - ms), ll);
                    }
                    mstar[i] = mm;
                    lstar[i] = ll;
                    sc[i] = fast_exp2(m[i] - ms);
                }
#pragma unroll
                for (int k = 0; k < KW; ++k) {
                    if (kw == k) {
#pragma unroll
                        for (int nd = 0; nd < D / 8; ++nd) {
                            float2* a0 = (float2*)(macc + grp * C::MROW + nd * 8 + 2 * tq);
                            float2* a1 = (float2*)(macc + (grp + 8) * C::MROW + nd * 8 + 2 * tq);
                            float2 x0 = make_float2(acc[nd][0] * sc[0], acc[nd][1] * sc[0]);
                            float2 x1 = make_float2(acc[nd][2] * sc[1], acc[nd][3] * sc[1]);
                            if (k > 0) {
                                const float2 y0 = *a0, y1 = *a1;
                                x0.x += y0.x; x0.y += y0.y; x1.x += y1.x; x1.y += y1.y;
                            }
                            *a0 = x0;
                            *a1 = x1;
                        }
                    }
                    named_barrier_sync(1, C::NCW * 32);
                }
                // The KW warps of the group copy the merged rows out, 16 bytes per thread per step.
                for (int i4 = kw * 32 + lane; i4 < 16 * (D / 4); i4 += KW * 32) {
                    const int row = i4 / (D / 4), c = (i4 % (D / 4)) * 4;
                    if (mt * 16 + row < p.R)
                        *(float4*)(p.part_acc + (prow + mt * 16 + row) * D + c) = *(const float4*)(macc + row * C::MROW + c);
                }
                if (kw == 0 && tq == 0) {
                    if (v0) *(float2*)(p.part_ml + (prow + r0) * 2) = make_float2(mstar[0], lstar[0]);
                    if (v1) *(float2*)(p.part_ml + (prow + r1) * 2) = make_float2(mstar[1], lstar[1]);
                }
                named_barrier_sync(1, C::NCW * 32);
            }
        }
    }
#ifdef PLT_TIMELINE
    if (tid == 0) tl[5] = global_timer_ns();
#endif
    if (flags) atomicOr(p.status, flags);
    if (flags & kDevWaitTimeout) s_ctl[0] = 1;
    __syncthreads();
#ifdef PLT_TIMELINE
    if (tid == 0) tl[6] = global_timer_ns();
#endif
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
