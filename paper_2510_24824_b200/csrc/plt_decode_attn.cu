// C ABI of the CLP decode-step attention: argument validation, variant selection, workspace,
// TMA descriptors and the two launches (split-KV main kernel, merge/gate kernel) per run.
#include "../../include/plt_decode_attn.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "plt_host.h"

using namespace plt;

namespace {

thread_local char g_create_error[512] = "";

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapKey {
    const void* base;
    int64_t s1, s2, s3;
    int64_t d1, d2, d3;
    bool operator==(const MapKey& o) const {
        return base == o.base && s1 == o.s1 && s2 == o.s2 && s3 == o.s3 && d1 == o.d1 && d2 == o.d2 && d3 == o.d3;
    }
};

struct Staging {
    void* ptr = nullptr;
    size_t bytes = 0;
};

}  // namespace

struct plt_decode_attn {
    plt_decode_attn_config cfg;
    int32_t delta[kMaxLoops];
    int G, R, Qn = 1;
    bool bf16;
    int sm_count;
    MainVariant var;      // bf16: full variant; fp32: only grid/smem used
    bool umma = false;    // path on tcgen05 / tensor memory (var.HPC = 1, var.KW = 8, var.stages = ring slots)
    bool umma_e4m3 = false;  // ... its kernel for E4M3 caches
    uint8_t* qimg = nullptr;  // that kernel's query images and their scale factors (inside the workspace)
    float* qinv = nullptr;
    int kbox = 0, wbox = 0;  // keys per TMA box of the shared cache / of a window on that path
    int ctas_per_sm;
    int piece_cost = 0;   // Params::piece_cost of the main kernel in use
    float scale_log2;
    // workspace
    float* part_acc = nullptr;
    float* part_ml = nullptr;
    int32_t* prefix = nullptr;
    int32_t* item_blocks = nullptr;
    uint32_t* status = nullptr;
    size_t ws_bytes = 0;
    // TMA descriptors, re-encoded only when a base pointer, stride or extent changes
    EncodeTiledFn encode = nullptr;
    CUtensorMap maps[4];
    MapKey keys[4];
    bool map_valid[4] = {false, false, false, false};
    // device staging for plt_decode_attn_run_host (grow-only)
    Staging st[12];
    cudaEvent_t ev_begin = nullptr, ev_end = nullptr;  // optional, caller-owned
    char err[512];
};

namespace {

plt_status fail(plt_decode_attn_t h, plt_status code, const char* fmt, ...) {
    char* dst = h ? h->err : g_create_error;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(dst, 512, fmt, ap);
    va_end(ap);
    return code;
}

plt_status cuda_fail(plt_decode_attn_t h, const char* what, cudaError_t e) {
    return fail(h, PLT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int elem_size(bool bf16) { return bf16 ? 2 : 4; }

struct Geometry {
    int G, R, Qn;
};

plt_status check_config(const plt_decode_attn_config* c, Geometry* g) {
    if (!c) return fail(nullptr, PLT_ERR_INVALID_ARG, "config is NULL");
    if (c->struct_size != sizeof(plt_decode_attn_config))
        return fail(nullptr, PLT_ERR_INVALID_ARG, "config.struct_size %u != %zu", c->struct_size,
                    sizeof(plt_decode_attn_config));
    if (c->dtype != PLT_F32 && c->dtype != PLT_BF16) return fail(nullptr, PLT_ERR_INVALID_ARG, "unknown dtype %d", c->dtype);
    if (c->max_batch < 1 || c->L < 1 || c->Hq < 1 || c->Hkv < 1 || c->max_seq_len < 1 || c->w < 0 || c->page_size < 0)
        return fail(nullptr, PLT_ERR_INVALID_ARG, "non-positive size in config");
    if (c->max_batch > kMaxBatch) return fail(nullptr, PLT_ERR_UNSUPPORTED, "max_batch %d > %d", c->max_batch, kMaxBatch);
    if (c->L > kMaxLoops) return fail(nullptr, PLT_ERR_UNSUPPORTED, "L %d > %d", c->L, kMaxLoops);
    if (c->Hq % c->Hkv != 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "Hq %d is not a multiple of Hkv %d", c->Hq, c->Hkv);
    if (c->d != 64 && c->d != 128) return fail(nullptr, PLT_ERR_UNSUPPORTED, "head dim %d (supported: 64, 128)", c->d);
    if (c->L > 1 && c->w < 1) return fail(nullptr, PLT_ERR_INVALID_ARG, "w must be >= 1 when L > 1");
    if (c->kv_dtype != PLT_KV_SAME && c->kv_dtype != PLT_KV_E4M3)
        return fail(nullptr, PLT_ERR_INVALID_ARG, "unknown kv_dtype %d", c->kv_dtype);
    if (c->kv_dtype == PLT_KV_E4M3) {
        if (c->dtype != PLT_BF16 || c->d != 128)
            return fail(nullptr, PLT_ERR_UNSUPPORTED, "E4M3 caches need bf16 queries and head dim 128");
    }
    if (c->q_len < 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "q_len %d < 0", c->q_len);
    if (c->typical_seq_len < 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "typical_seq_len %d < 0", c->typical_seq_len);
    g->Qn = c->q_len > 1 ? c->q_len : 1;
    if (g->Qn > 1 && (c->dtype != PLT_BF16 || c->kernel_path == PLT_PATH_TCGEN05))
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "q_len > 1 is served by the warp-level bf16 kernel only");
    g->G = c->Hq / c->Hkv;
    g->R = c->L * g->Qn * g->G;
    if (g->R > kMaxRows)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "L * q_len * Hq/Hkv = %d packed rows > %d", g->R, kMaxRows);
    if (c->kv_dtype == PLT_KV_E4M3 && c->kernel_path == PLT_PATH_TCGEN05 && g->R > 32)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "the tcgen05 path takes E4M3 caches up to 32 packed rows (%d here)", g->R);
    if (c->page_size > 0 && c->page_size % 16 != 0)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "page_size %d is not a multiple of 16", c->page_size);
    if (c->loop_offset)
        for (int l = 0; l < c->L; ++l)
            if (c->loop_offset[l] < 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "loop_offset[%d] < 0", l);
    return PLT_OK;
}

// Picks (rows per warp, heads per block, key slices, stages, blocks per SM) for the warp-level bf16 kernel.
plt_status choose_variant(const plt_decode_attn_config* c, const Geometry& g, MainVariant* v, int* want_ctas_per_sm) {
    v->D = c->d;
    const bool fp8 = c->kv_dtype == PLT_KV_E4M3;
    v->fp8 = fp8;
    int rw = c->row_warps;
    if (rw == 0) rw = g.R > 24 ? 2 : 1;   // 32 rows in one warp leave room for one warp per scheduler only: measured slower
    if (rw != 1 && rw != 2) return fail(nullptr, PLT_ERR_INVALID_ARG, "row_warps %d (supported: 1 or 2)", rw);
    int nt = (g.R + 8 * rw - 1) / (8 * rw);   // 8-row groups per warp
    if (rw == 2 && nt < 2) nt = 2;
    if (nt > 4) return fail(nullptr, PLT_ERR_UNSUPPORTED, "%d packed rows need row_warps = 2", g.R);
    v->NT = nt;
    v->RW = rw;
    // Up to 16 rows per warp the kernel fits 168 registers and two blocks of 4 consumer warps share an SM; above that
    // one block of 4 warps has the SM to itself.
    const bool small = nt <= 2;
    int hpc = c->heads_per_cta, kw = c->key_slices;
    int ks = c->slices_per_warp;
    if (ks == 0) ks = (rw == 2 || fp8) ? 2 : 1;   // two warps per head: 32 keys each per tile (measured 25-35 % faster at 48 and 64 rows)
    if (ks != 1 && ks != 2) return fail(nullptr, PLT_ERR_INVALID_ARG, "slices_per_warp %d (supported: 1 or 2)", ks);
    if (hpc == 0) {
        hpc = 1;
        const int cap = 4 / rw;
        for (int h = cap; h >= 1; h >>= 1)
            if (c->Hkv % h == 0) { hpc = h; break; }
    }
    if (kw == 0) {
        kw = 4 / (hpc * rw);
        if (kw < 1) kw = 1;
    }
    if (c->Hkv % hpc != 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "heads_per_cta %d does not divide Hkv %d", hpc, c->Hkv);
    auto tile = [&]() { return main_bf16_tile_keys(v->D, nt, rw, hpc, kw, ks, fp8); };
    while (c->page_size > 0 && tile() > 0 && c->page_size % tile() != 0 && kw > 1) kw >>= 1;
    if (c->page_size > 0 && tile() > 0 && c->page_size % tile() != 0 && !fp8) ks = 1;
    if (!main_bf16_exists(v->D, nt, rw, hpc, kw, ks, fp8) || (c->page_size > 0 && c->page_size % tile() != 0))
        return fail(nullptr, PLT_ERR_UNSUPPORTED,
                    "no bf16 kernel for heads_per_cta=%d key_slices=%d slices_per_warp=%d row_warps=%d", hpc, kw, ks, rw);
    v->HPC = hpc;
    v->KW = kw;
    v->KS = ks;
    v->tile_keys = tile();
    const int ncw = hpc * kw * rw;
    int cps = c->ctas_per_sm > 0 ? c->ctas_per_sm : (small && ncw <= 4 ? 2 : 1);
    const size_t budget = (size_t)(cps >= 2 ? 227 * 1024 / cps - 1024 : 227 * 1024);
    int stages = c->stages;
    if (stages == 0) {
        // About 128 KB of loads in flight per SM measured fastest on B200; more only delays the first data.
        const size_t stage_bytes = main_bf16_smem(v->D, nt, rw, hpc, kw, ks, 3, c->max_batch, fp8) -
                                   main_bf16_smem(v->D, nt, rw, hpc, kw, ks, 2, c->max_batch, fp8);
        stages = (int)((128 * 1024) / (stage_bytes * (size_t)cps));
        if (stages < 2) stages = 2;
        while (stages > 2 && main_bf16_smem(v->D, nt, rw, hpc, kw, ks, stages, c->max_batch, fp8) > budget) --stages;
        if (stages > 8) stages = 8;
    }
    if (stages < 2 || stages > 12) return fail(nullptr, PLT_ERR_INVALID_ARG, "stages %d outside [2, 12]", stages);
    v->stages = stages;
    v->smem = main_bf16_smem(v->D, nt, rw, hpc, kw, ks, stages, c->max_batch, fp8);
    if (v->smem > 227 * 1024)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "variant needs %zu bytes of shared memory (> 227 KB)", v->smem);
    *want_ctas_per_sm = cps;
    return PLT_OK;
}

// Workspace: split partials, first / last block of every item, tile prefix, status word; for the tcgen05 kernel on
// E4M3 caches also one query image and one scale factor per (sequence, KV head), from a 256-byte boundary on.
size_t workspace_base_bytes(const plt_decode_attn_config* c, int hpc, size_t acc_floats, size_t ml_floats) {
    const size_t items = (size_t)c->max_batch * (c->Hkv / hpc) * 2;
    return (acc_floats + ml_floats) * 4 + items * 8 + (size_t)(c->max_batch + 1) * 4 + 256;
}

size_t workspace_bytes_for(const plt_decode_attn_config* c, const Geometry& g, int hpc, int grid, bool e4m3_images,
                           size_t* acc_floats, size_t* ml_floats) {
    const size_t slots = (size_t)c->max_batch * (c->Hkv / hpc) * 2 + (size_t)grid;
    *acc_floats = slots * hpc * g.R * c->d;
    *ml_floats = slots * hpc * g.R * 2;
    size_t bytes = workspace_base_bytes(c, hpc, *acc_floats, *ml_floats);
    if (e4m3_images) {
        const size_t n = (size_t)c->max_batch * c->Hkv;
        bytes = ((bytes + 255) & ~(size_t)255) + n * main_umma_e4m3_image_bytes(g.R) + n * 4 + 256;
    }
    return bytes;
}

// Points the handle's workspace pointers into `ws` (256-byte aligned, workspace_bytes_for bytes).
void place_workspace(plt_decode_attn* h, const plt_decode_attn_config* c, void* ws, size_t acc_floats, size_t ml_floats) {
    h->part_acc = (float*)ws;
    h->part_ml = h->part_acc + acc_floats;
    h->item_blocks = (int32_t*)(h->part_ml + ml_floats);   // 16-byte aligned: both float counts are multiples of 4
    h->prefix = h->item_blocks + (size_t)c->max_batch * (c->Hkv / h->var.HPC) * 4;
    h->status = (uint32_t*)(h->prefix + c->max_batch + 1);
    h->qimg = nullptr;
    h->qinv = nullptr;
    if (h->umma_e4m3) {
        const size_t base = (workspace_base_bytes(c, h->var.HPC, acc_floats, ml_floats) + 255) & ~(size_t)255;
        h->qimg = (uint8_t*)ws + base;
        h->qinv = (float*)(h->qimg + (size_t)c->max_batch * c->Hkv * main_umma_e4m3_image_bytes(h->R));
    }
}

plt_status encode_map(plt_decode_attn_t h, int idx, const void* base, int es, int D, int64_t d1, int64_t d2, int64_t d3,
                      int64_t s1, int64_t s2, int64_t s3, int box_keys, int box_heads) {
    MapKey key{base, s1, s2, s3, d1, d2, d3};
    if (h->map_valid[idx] && h->keys[idx] == key) return PLT_OK;
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)d1, (cuuint64_t)d2, (cuuint64_t)d3};
    cuuint64_t strides[3] = {(cuuint64_t)(s1 * es), (cuuint64_t)(s2 * es), (cuuint64_t)(s3 * es)};
    cuuint32_t box[4] = {(cuuint32_t)(128 / es), (cuuint32_t)box_keys, (cuuint32_t)box_heads, 1u};   // 128-byte rows
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = h->encode(&h->maps[idx], es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                           estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        h->map_valid[idx] = false;
        return fail(h, PLT_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d for tensor %d", (int)r, idx);
    }
    h->keys[idx] = key;
    h->map_valid[idx] = true;
    return PLT_OK;
}

// Can a tcgen05 kernel take this configuration? (bf16, d = 128, pages that tile or are tiled by 128 keys; with E4M3
// caches at most 32 packed rows, which check_config has already seen to)
bool umma_eligible(const plt_decode_attn_config* c) {
    if (c->dtype != PLT_BF16 || c->d != 128) return false;
    if (c->page_size > 0 && c->page_size % 128 != 0 && 128 % c->page_size != 0) return false;
    return true;
}

// Automatic choice: the warp-level kernel, except
//  - bf16 caches above 48 packed rows on long-context configurations, where the tcgen05 kernel measured 8 % faster
//    (64 rows, N = 16384: 337 vs 368 us); at 48 rows (226 vs 313 us) and on batches of short sequences at any row
//    count (64 rows, N 512-4096: 252 vs 631 us) the warp-level kernel is the faster one;
//  - E4M3 caches, contiguous or in pages of 64 tokens or of a multiple of 128, at 25 to 32 packed rows when sequences
//    can reach 8192 keys, and (pages of 64 left out) at 17 to 24 rows when they can reach 32768: the tcgen05 kernel
//    for E4M3 streams at 6.4 TB/s where the warp-level one is bound by its conversions (4.4 TB/s), but it pays more
//    per work item, and the lengths a batch will really have are not known here. Measured steps, tcgen05 vs
//    warp-level, equal lengths, B = 16: 32 rows 208 vs 292 us at N = 32768, 124 vs 169 us at 16384, 83 vs 106 us at
//    8192, 62 vs 74 us at 4096, 52 vs 56 us at 2048, 48 vs 47 us at 1024, 47 vs 42 us at 512 (B = 4, N = 131072: 200
//    vs 279 us; B = 64, N = 8192: 257 vs 347 us; B = 128, N = 1024: 213 vs 241 us); 24 rows 202 vs 225 us at 32768,
//    119 vs 129 us at 16384, 77 vs 79 us at 8192 (B = 64: 236 vs 259 us), 56 vs 53 us at 4096; 16 rows 177 vs 175 us
//    at 32768 and slower below; pages of 128 or 256 tokens cost nothing (32 rows, N = 32768: 206 us; N = 4096:
//    62 us), pages of 64 tokens (two boxes per tile, in a kernel of their own) 3 us (212 and 65 us). Batches of 256
//    sequences with log-uniform lengths (a serving mix: more than half of them under an eighth of the longest), 32
//    rows: 313 vs 352 us with lengths up to 16384, 232 vs 248 us up to 8192 (B = 64: 75 vs 70 us), 193 vs 183 us up
//    to 4096, 173 vs 143 us up to 2048; 24 rows: 369 vs 389 us up to 32768 (B = 64: 115 vs 115 us), 238 vs 229 us up
//    to 16384 (pages of 64: 255 vs 228 us), 192 vs 162 us up to 8192. The thresholds are where the mixes stop
//    losing; a caller who knows that most sequences reach some length says so (typical_seq_len) and gets the kernel
//    from 2048 tokens at 25 to 32 rows and from 8192 at 17 to 24, where equal-length batches gain up to 15 %. Smaller pages go
//    through the producers' out-of-line path, a dependent page-table read per box, and are left to the warp-level
//    kernel.
// An explicit heads_per_cta / key_slices / ctas_per_sm / row_warps / slices_per_warp asks for the warp-level
// kernel's variants.
bool want_umma(const plt_decode_attn_config* c) {
    if (c->kernel_path == PLT_PATH_WARP_MMA || c->q_len > 1) return false;
    if (c->kernel_path == PLT_PATH_TCGEN05) return true;
    if (c->heads_per_cta != 0 || c->key_slices != 0 || c->ctas_per_sm != 0 || c->row_warps != 0 || c->slices_per_warp != 0)
        return false;
    const int rows = c->L * (c->Hq / c->Hkv);
    if (c->kv_dtype == PLT_KV_E4M3) {
        // With a length the caller expects most sequences to reach, the equal-length figures above decide.
        const int len = c->typical_seq_len < c->max_seq_len ? c->typical_seq_len : c->max_seq_len;
        const bool long32 = len > 0 ? len >= 2048 : c->max_seq_len >= 8192;
        const bool long24 = len > 0 ? len >= 8192 : c->max_seq_len >= 32768;
        return umma_eligible(c) && c->stages == 0 &&
               ((rows > 24 && rows <= 32 && long32 && (c->page_size % 128 == 0 || c->page_size == 64)) ||
                (rows > 16 && rows <= 24 && long24 && c->page_size % 128 == 0));
    }
    const int reach = c->typical_seq_len > 0 && c->typical_seq_len < c->max_seq_len ? c->typical_seq_len : c->max_seq_len;
    return umma_eligible(c) && rows > 48 && reach >= 16384 && (c->stages == 0 || c->stages == 4 || c->stages == 6);
}

// Chooses the kernel path and variant, prepares the kernels (shared-memory attribute, occupancy) and fills
// h->var, h->umma, h->ctas_per_sm. Needs h->bf16, h->sm_count. Errors go to the create-time message.
plt_status setup_kernels(plt_decode_attn* h, const plt_decode_attn_config* config, const Geometry& g) {
    int blocks = 0;
    cudaError_t e;
    h->umma = false;
    h->piece_cost = 0;
    if (config->kernel_path < 0 || config->kernel_path > PLT_PATH_TCGEN05)
        return fail(nullptr, PLT_ERR_INVALID_ARG, "kernel_path %d outside [0, 2]", config->kernel_path);
    if (config->loads_in_flight < 0) return fail(nullptr, PLT_ERR_INVALID_ARG, "loads_in_flight %d < 0", config->loads_in_flight);
    if (config->kernel_path == PLT_PATH_TCGEN05 && !umma_eligible(config))
        return fail(nullptr, PLT_ERR_UNSUPPORTED,
                    "the tcgen05 path needs bf16, d = 128 and a page size that divides or is a multiple of 128");
    h->umma_e4m3 = false;
    if (h->bf16 && want_umma(config) && config->kv_dtype == PLT_KV_E4M3) {
        // Two KV heads per work item when Hkv is even: their tiles of the same keys are fetched one after the other,
        // so that the 128-byte rows of neighbouring heads reach DRAM together (6.4 against 4.5 TB/s measured).
        int hpc = config->heads_per_cta;
        if (hpc == 0) hpc = config->Hkv % 2 == 0 ? 2 : 1;
        if ((hpc != 1 && hpc != 2) || config->Hkv % hpc != 0)
            return fail(nullptr, PLT_ERR_INVALID_ARG, "heads_per_cta %d on the tcgen05 path with E4M3 caches (supported: 1, or 2 when Hkv is even)", hpc);
        // Ring slots of 16 KB (a K or a V tile of one head; 4 hold K tiles, the rest V tiles): as many as fit beside
        // the probability and query buffers.
        int nslot = config->stages;
        if (nslot == 0) {
            nslot = main_umma_e4m3_max_slots();
            while (nslot > main_umma_e4m3_min_slots() && main_umma_e4m3_smem(g.R, hpc, nslot, config->max_batch) > 227 * 1024) --nslot;
        }
        if (nslot < main_umma_e4m3_min_slots() || nslot > main_umma_e4m3_max_slots())
            return fail(nullptr, PLT_ERR_INVALID_ARG, "stages %d on the tcgen05 path with E4M3 caches (supported: %d to %d ring slots)",
                        nslot, main_umma_e4m3_min_slots(), main_umma_e4m3_max_slots());
        const size_t smem = main_umma_e4m3_smem(g.R, hpc, nslot, config->max_batch);
        if (smem > 227 * 1024)
            return fail(nullptr, PLT_ERR_UNSUPPORTED, "tcgen05 path needs %zu bytes of shared memory (> 227 KB)", smem);
        e = main_umma_e4m3_prepare(g.R, hpc, config->page_size == 64, smem, &blocks);
        if (e != cudaSuccess) return cuda_fail(nullptr, "preparing the tcgen05 main kernel for E4M3 caches", e);
        if (blocks < 1) return fail(nullptr, PLT_ERR_UNSUPPORTED, "tcgen05 main kernel does not fit an SM");
        h->umma = true;
        h->umma_e4m3 = true;
        // Starting and finishing a piece costs this kernel more than a tile (plan step, limits, first-tile maxima,
        // end-of-piece reduction, epilogue), and the tiles of a windows item (all masked, a limits update per window)
        // cost more than shared-cache tiles. The plan charges every item a lead-in, so that blocks with more item
        // starts get fewer tiles. Measured per-step times for a lead-in of 0 / 4 / 8 / 14 / 20 tiles: 214.9 / 208.8 /
        // 211.5 / 219.3 / 226.5 us at B = 16, N = 32768; 87.6 / 82.9 / 85.0 / 93.1 / 99.9 us at N = 8192; 208.5 /
        // 200.1 / 199.9 / 201.7 / 203.4 us at B = 4, N = 131072; 260.0 / 257.0 / 259.3 / 262.8 / 267.1 us at B = 64,
        // N = 8192 (3 to 6 tiles within 1 us of one another).
        h->piece_cost = 4;
        h->var = MainVariant{config->d, 0, 0, hpc, 4, 1, 128, nslot, 0, smem, true};
        h->ctas_per_sm = 1;
        h->kbox = config->page_size > 0 ? (config->page_size < 128 ? config->page_size : 128)
                                        : (config->max_seq_len < 128 ? config->max_seq_len : 128);
        h->wbox = config->w < 128 ? (config->w > 0 ? config->w : 1) : 128;
    } else if (h->bf16 && want_umma(config)) {
        // Ring slots: an even number, so that a slot is always refilled by the stream (K or V) that used it before.
        int nslot = config->stages;
        if (nslot == 0) nslot = main_umma_smem(g.R, 6, config->max_batch) <= 227 * 1024 ? 6 : 4;
        if (nslot != 4 && nslot != 6)
            return fail(nullptr, PLT_ERR_INVALID_ARG, "stages %d on the tcgen05 path (supported: 4 or 6 ring slots)", nslot);
        const size_t smem = main_umma_smem(g.R, nslot, config->max_batch);
        if (smem > 227 * 1024)
            return fail(nullptr, PLT_ERR_UNSUPPORTED, "tcgen05 path needs %zu bytes of shared memory (> 227 KB)", smem);
        e = main_umma_prepare(g.R, smem, &blocks);
        if (e != cudaSuccess) return cuda_fail(nullptr, "preparing the tcgen05 main kernel", e);
        if (blocks < 1) return fail(nullptr, PLT_ERR_UNSUPPORTED, "tcgen05 main kernel does not fit an SM");
        h->umma = true;
        h->var = MainVariant{config->d, 0, 0, 1, 8, 1, 128, nslot, 0, smem};
        h->ctas_per_sm = 1;
        h->kbox = config->page_size > 0 ? (config->page_size < 128 ? config->page_size : 128)
                                        : (config->max_seq_len < 128 ? config->max_seq_len : 128);
        h->wbox = config->w < 128 ? (config->w > 0 ? config->w : 1) : 128;
    } else if (h->bf16) {
        int cps = 0;
        plt_status s = choose_variant(config, g, &h->var, &cps);
        if (s != PLT_OK) return s;
        e = main_bf16_prepare(h->var, &blocks);
        if (e != cudaSuccess) return cuda_fail(nullptr, "preparing the bf16 main kernel", e);
        if (blocks < 1) return fail(nullptr, PLT_ERR_UNSUPPORTED, "bf16 main kernel does not fit an SM");
        h->ctas_per_sm = blocks < cps ? blocks : cps;
        // Starting and finishing an item (plan step, query rows, first load latency, partial store) stalls a block for
        // about as long as streaming 192 KB takes it (measured on B200 on a batch of short sequences: 4-5 us);
        // the plan charges every item that much, in tiles, so that blocks with many short items get fewer tiles.
        const size_t stage_bytes = main_bf16_smem(h->var.D, h->var.NT, h->var.RW, h->var.HPC, h->var.KW, h->var.KS, 3, 1, h->var.fp8) -
                                   main_bf16_smem(h->var.D, h->var.NT, h->var.RW, h->var.HPC, h->var.KW, h->var.KS, 2, 1, h->var.fp8);
        h->piece_cost = (int)((192 * 1024) / (stage_bytes * (size_t)h->ctas_per_sm));
        if (h->piece_cost < 1) h->piece_cost = 1;
    } else {
        h->var = MainVariant{config->d, 0, 0, 1, 1, 1, kF32TileKeys, 0, 0, main_f32_smem(config->d, g.R, config->max_batch)};
        e = main_f32_prepare(config->d, g.R, config->max_batch, &blocks);
        if (e != cudaSuccess) return cuda_fail(nullptr, "preparing the fp32 main kernel", e);
        if (blocks < 1) return fail(nullptr, PLT_ERR_UNSUPPORTED, "fp32 main kernel does not fit an SM");
        const int cps = config->ctas_per_sm > 0 ? config->ctas_per_sm : 2;
        h->ctas_per_sm = blocks < cps ? blocks : cps;
    }
    h->var.grid = h->sm_count * h->ctas_per_sm;
    if (h->bf16) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
            return fail(nullptr, PLT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
        h->encode = (EncodeTiledFn)fn;
    }
    // The tile line must fit 31 bits.
    const int tk = h->var.tile_keys;
    const double tiles = (double)config->max_batch * (config->Hkv / h->var.HPC) *
                         ((double)(config->max_seq_len + tk - 1) / tk + (double)(config->L - 1) * ((config->w + tk - 1) / tk));
    if (tiles >= 2147483647.0) return fail(nullptr, PLT_ERR_UNSUPPORTED, "max_batch * max_seq_len too large for the tile plan");
    return PLT_OK;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

#define PLT_API __attribute__((visibility("default")))
extern "C" {

PLT_API plt_status plt_decode_attn_workspace_bytes(const plt_decode_attn_config* config, size_t* out_bytes) {
    Geometry g;
    plt_status s = check_config(config, &g);
    if (s != PLT_OK) return s;
    if (!out_bytes) return fail(nullptr, PLT_ERR_INVALID_ARG, "out_bytes is NULL");
    int sms = 148;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, config->device) == cudaSuccess) sms = prop.multiProcessorCount;
    else (void)cudaGetLastError();
    int hpc = 1, cps = config->ctas_per_sm > 0 ? config->ctas_per_sm : 2;
    bool images = false;
    if (config->dtype == PLT_BF16 && want_umma(config)) {
        cps = 1;
        images = config->kv_dtype == PLT_KV_E4M3;
        if (images) hpc = config->heads_per_cta > 0 ? config->heads_per_cta : (config->Hkv % 2 == 0 ? 2 : 1);
    } else if (config->dtype == PLT_BF16) {
        MainVariant v;
        s = choose_variant(config, g, &v, &cps);
        if (s != PLT_OK) return s;
        hpc = v.HPC;
    }
    size_t a, m;
    *out_bytes = workspace_bytes_for(config, g, hpc, sms * cps, images, &a, &m);
    return PLT_OK;
}

PLT_API plt_status plt_decode_attn_create(const plt_decode_attn_config* config, plt_decode_attn_t* out_handle) {
    if (!out_handle) return fail(nullptr, PLT_ERR_INVALID_ARG, "out_handle is NULL");
    *out_handle = nullptr;
    Geometry g;
    plt_status s = check_config(config, &g);
    if (s != PLT_OK) return s;

    cudaError_t e = cudaSetDevice(config->device);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaSetDevice", e);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, config->device);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDeviceProperties", e);
    if (prop.major != 10)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only",
                    config->device, prop.major, prop.minor);

    plt_decode_attn* h = new (std::nothrow) plt_decode_attn();
    if (!h) return fail(nullptr, PLT_ERR_OUT_OF_MEMORY, "host allocation failed");
    h->cfg = *config;
    h->cfg.loop_offset = nullptr;
    for (int l = 0; l < kMaxLoops; ++l) h->delta[l] = config->loop_offset && l < config->L ? config->loop_offset[l] : l;
    h->G = g.G;
    h->R = g.R;
    h->Qn = g.Qn;
    h->bf16 = config->dtype == PLT_BF16;
    h->sm_count = prop.multiProcessorCount;
    const float scale = config->sm_scale > 0.f ? config->sm_scale : 1.0f / sqrtf((float)config->d);
    h->scale_log2 = scale * 1.4426950408889634f;
    h->err[0] = 0;

    s = setup_kernels(h, config, g);
    if (s != PLT_OK) { delete h; return s; }

    size_t acc_floats, ml_floats;
    h->ws_bytes = workspace_bytes_for(config, g, h->var.HPC, h->var.grid, h->umma_e4m3, &acc_floats, &ml_floats);
    void* ws = nullptr;
    e = cudaMalloc(&ws, h->ws_bytes);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete h;
        return fail(nullptr, PLT_ERR_OUT_OF_MEMORY, "cudaMalloc of %zu workspace bytes failed", h->ws_bytes);
    }
    place_workspace(h, config, ws, acc_floats, ml_floats);
    e = cudaMemset(h->status, 0, 4);
    if (e != cudaSuccess) { cudaFree(ws); delete h; return cuda_fail(nullptr, "cudaMemset", e); }
    *out_handle = h;
    return PLT_OK;
}

namespace {
plt_status run_impl(plt_decode_attn_t h, const plt_decode_attn_args* a, void* cuda_stream,
                    const plt_decode_attn_step_args* step);
plt_decode_attn* no_alloc_handle_of_current_device();
}

PLT_API plt_status plt_decode_attn_run(plt_decode_attn_t h, const plt_decode_attn_args* a, void* cuda_stream) {
    return run_impl(h, a, cuda_stream, nullptr);
}

PLT_API plt_status plt_decode_attn_step(plt_decode_attn_t h, const plt_decode_attn_args* a,
                                        const plt_decode_attn_step_args* step, void* cuda_stream) {
    if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if (!a) return fail(h, PLT_ERR_INVALID_ARG, "args is NULL");
    if (!step) return fail(h, PLT_ERR_INVALID_ARG, "step is NULL");
    if (step->struct_size != sizeof(plt_decode_attn_step_args))
        return fail(h, PLT_ERR_INVALID_ARG, "step.struct_size %u != %zu", step->struct_size, sizeof(plt_decode_attn_step_args));
    if (a->struct_size != sizeof(plt_decode_attn_args))
        return fail(h, PLT_ERR_INVALID_ARG, "args.struct_size %u != %zu", a->struct_size, sizeof(plt_decode_attn_args));
    if (!step->k_new || !step->v_new) return fail(h, PLT_ERR_INVALID_ARG, "k_new and v_new must not be NULL");
    if (!aligned16(step->k_new) || !aligned16(step->v_new))
        return fail(h, PLT_ERR_INVALID_ARG, "k_new and v_new must be 16-byte aligned");
    if (h->cfg.L > 1 && (!step->w_gate || !step->b_gate || !step->gate_logits))
        return fail(h, PLT_ERR_INVALID_ARG, "w_gate, b_gate and gate_logits must not be NULL when L > 1");
    if (a->win_lens) return fail(h, PLT_ERR_INVALID_ARG, "win_lens must be NULL: the ring update fixes wl = min(w, cut)");
    if (h->Qn > 1) return fail(h, PLT_ERR_UNSUPPORTED, "plt_decode_attn_step takes one query token per loop (q_len <= 1)");
    plt_decode_attn_args a2 = *a;
    a2.gate_logits = step->gate_logits;
    return run_impl(h, &a2, cuda_stream, step);
}

namespace {
plt_status run_impl(plt_decode_attn_t h, const plt_decode_attn_args* a, void* cuda_stream,
                    const plt_decode_attn_step_args* step) {
    if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if (!a) return fail(h, PLT_ERR_INVALID_ARG, "args is NULL");
    if (a->struct_size != sizeof(plt_decode_attn_args))
        return fail(h, PLT_ERR_INVALID_ARG, "args.struct_size %u != %zu", a->struct_size, sizeof(plt_decode_attn_args));
    const plt_decode_attn_config& c = h->cfg;
    if (a->batch < 0) return fail(h, PLT_ERR_INVALID_ARG, "batch %d < 0", a->batch);
    if (a->batch > c.max_batch) return fail(h, PLT_ERR_CAPACITY, "batch %d > max_batch %d", a->batch, c.max_batch);
    if (a->batch == 0) return PLT_OK;
    if (!a->q || !a->k_cache || !a->v_cache || !a->seq_lens || !a->out)
        return fail(h, PLT_ERR_INVALID_ARG, "q, k_cache, v_cache, seq_lens and out must not be NULL");
    if (c.L > 1 && (!a->k_win || !a->v_win || !a->gate_logits))
        return fail(h, PLT_ERR_INVALID_ARG, "k_win, v_win and gate_logits must not be NULL when L > 1");
    if (!aligned16(a->q) || !aligned16(a->k_cache) || !aligned16(a->v_cache) || !aligned16(a->out) ||
        (c.L > 1 && (!aligned16(a->k_win) || !aligned16(a->v_win))))
        return fail(h, PLT_ERR_INVALID_ARG, "tensor base pointers must be 16-byte aligned");
    const bool fp8 = h->cfg.kv_dtype == PLT_KV_E4M3;
    const int es = fp8 ? 1 : elem_size(h->bf16);   // element size of the caches and windows
    if (fp8 && (!a->k_scale || !a->v_scale)) return fail(h, PLT_ERR_INVALID_ARG, "k_scale and v_scale must not be NULL with E4M3 caches");
    int64_t sb = a->kv_stride_b, sn = a->kv_stride_n, sh = a->kv_stride_h;
    if (sb == 0 && sn == 0 && sh == 0) {
        sh = c.d;
        sn = (int64_t)c.Hkv * c.d;
        sb = (int64_t)(c.page_size > 0 ? c.page_size : c.max_seq_len) * sn;
    }
    const int64_t unit = 16 / es;
    if (sb <= 0 || sn <= 0 || sh <= 0 || sb % unit || sn % unit || sh % unit)
        return fail(h, PLT_ERR_INVALID_ARG, "kv strides must be positive multiples of %lld elements", (long long)unit);
    if (sh < c.d) return fail(h, PLT_ERR_INVALID_ARG, "kv_stride_h %lld < d", (long long)sh);
    if ((double)sb * es >= 1099511627776.0 || (double)sn * es >= 1099511627776.0)
        return fail(h, PLT_ERR_UNSUPPORTED, "kv stride of 2^40 bytes or more");
    if (c.page_size > 0) {
        if (!a->page_table) return fail(h, PLT_ERR_INVALID_ARG, "page_table is NULL for a paged cache");
        const int need = (c.max_seq_len + c.page_size - 1) / c.page_size;
        if (a->max_pages < need) return fail(h, PLT_ERR_CAPACITY, "max_pages %d < %d", a->max_pages, need);
        if (a->num_pool_pages < 1) return fail(h, PLT_ERR_INVALID_ARG, "num_pool_pages %d < 1", a->num_pool_pages);
    }

    Params p;
    memset(&p, 0, sizeof p);
    p.q = a->q; p.k_cache = a->k_cache; p.v_cache = a->v_cache; p.k_win = a->k_win; p.v_win = a->v_win;
    p.seq_lens = a->seq_lens; p.win_lens = a->win_lens; p.page_table = a->page_table; p.gate_logits = a->gate_logits;
    p.out = a->out;
    p.k_scale = fp8 ? a->k_scale : nullptr;
    p.v_scale = fp8 ? a->v_scale : nullptr;
    p.part_acc = h->part_acc; p.part_ml = h->part_ml; p.prefix = h->prefix; p.item_blocks = h->item_blocks;
    p.status = h->status;
    p.kv_stride_b = sb; p.kv_stride_n = sn; p.kv_stride_h = sh;
    p.B = a->batch; p.L = c.L; p.Hq = c.Hq; p.Hkv = c.Hkv; p.G = h->G; p.R = h->R; p.d = c.d; p.w = c.w;
    p.Qn = h->Qn;
    p.max_seq_len = c.max_seq_len; p.page_size = c.page_size; p.max_pages = a->max_pages;
    p.num_pool_pages = a->num_pool_pages;
    p.hpc = h->var.HPC;
    p.tile_keys = h->var.tile_keys;
    p.piece_cost = h->piece_cost;
    p.num_ctas = h->var.grid;
    p.scale_log2 = h->scale_log2;
    for (int l = 0; l < kMaxLoops; ++l) p.delta[l] = h->delta[l];

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (step) {
        e = launch_prestep(p, h->bf16, step->k_new, step->v_new, step->w_gate, step->b_gate, step->gate_logits, stream);
        if (e != cudaSuccess) return cuda_fail(h, "launching the pre-step kernel", e);
    }
    if (h->bf16) {
        // keys and heads per TMA box: the warp-level kernel loads [heads per block][tile keys], the tcgen05 kernel
        // [1 head][up to 128 keys]
        const int tk = h->umma ? h->kbox : h->var.tile_keys;
        const int tkw = h->umma ? h->wbox : h->var.tile_keys;
        const int bh = h->umma ? 1 : h->var.HPC;
        plt_status s;
        if (c.page_size > 0) {
            s = encode_map(h, 0, a->k_cache, es, c.d, c.page_size, c.Hkv, a->num_pool_pages, sn, sh, sb, tk, bh);
            if (s == PLT_OK)
                s = encode_map(h, 1, a->v_cache, es, c.d, c.page_size, c.Hkv, a->num_pool_pages, sn, sh, sb, tk, bh);
        } else {
            s = encode_map(h, 0, a->k_cache, es, c.d, c.max_seq_len, c.Hkv, a->batch, sn, sh, sb, tk, bh);
            if (s == PLT_OK)
                s = encode_map(h, 1, a->v_cache, es, c.d, c.max_seq_len, c.Hkv, a->batch, sn, sh, sb, tk, bh);
        }
        if (s != PLT_OK) return s;
        if (c.L > 1) {
            const int64_t wn = (int64_t)c.Hkv * c.d, wb = (int64_t)c.w * wn;
            s = encode_map(h, 2, a->k_win, es, c.d, c.w, c.Hkv, (int64_t)a->batch * (c.L - 1), wn, c.d, wb, tkw, bh);
            if (s == PLT_OK)
                s = encode_map(h, 3, a->v_win, es, c.d, c.w, c.Hkv, (int64_t)a->batch * (c.L - 1), wn, c.d, wb, tkw, bh);
            if (s != PLT_OK) return s;
        } else {
            h->maps[2] = h->maps[0];
            h->maps[3] = h->maps[1];
        }
        if (h->umma_e4m3) {
            e = launch_pack_q_e4m3(p, h->qimg, h->qinv, stream);
            if (e != cudaSuccess) return cuda_fail(h, "launching the query pack kernel", e);
        }
        if (h->ev_begin) cudaEventRecord(h->ev_begin, stream);
        if (h->umma_e4m3)
            e = launch_main_umma_e4m3(h->maps, p, h->var.grid, h->var.smem, h->var.stages, h->kbox, h->wbox,
                                      c.loads_in_flight > 0 ? c.loads_in_flight : 4, h->qimg, h->qinv, stream);
        else if (h->umma)
            e = launch_main_umma(h->maps, p, h->var.grid, h->var.smem, h->var.stages, h->kbox, h->wbox,
                                 c.loads_in_flight > 0 ? c.loads_in_flight : 2, stream);
        else
            e = launch_main_bf16(h->var, h->maps, p, /*overlap=*/true, stream);
    } else {
        if (h->ev_begin) cudaEventRecord(h->ev_begin, stream);
        e = launch_main_f32(p, h->var.grid, h->var.smem, stream);
    }
    if (e != cudaSuccess) return cuda_fail(h, "launching the main kernel", e);
    if (h->ev_end) cudaEventRecord(h->ev_end, stream);
    // The merge kernel may set up while the main kernel drains, unless an event sits between the two launches.
    e = launch_reduce(p, h->bf16, /*overlap=*/h->ev_end == nullptr, stream);
    if (e != cudaSuccess) return cuda_fail(h, "launching the merge kernel", e);
    return PLT_OK;
}
}  // namespace

static plt_status stage_in(plt_decode_attn_t h, int idx, const void* host, size_t bytes, cudaStream_t stream,
                           const void** dev) {
    *dev = nullptr;
    if (!host || bytes == 0) return PLT_OK;
    Staging& s = h->st[idx];
    if (s.bytes < bytes) {
        if (s.ptr) cudaFree(s.ptr);
        s.ptr = nullptr;
        s.bytes = 0;
        cudaError_t e = cudaMalloc(&s.ptr, bytes);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return fail(h, PLT_ERR_OUT_OF_MEMORY, "cudaMalloc of %zu staging bytes failed", bytes);
        }
        s.bytes = bytes;
    }
    cudaError_t e = cudaMemcpyAsync(s.ptr, host, bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(h, "cudaMemcpyAsync (host to device)", e);
    *dev = s.ptr;
    return PLT_OK;
}

PLT_API plt_status plt_decode_attn_run_host(plt_decode_attn_t h, const plt_decode_attn_args* a, void* cuda_stream) {
    if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if (!a) return fail(h, PLT_ERR_INVALID_ARG, "args is NULL");
    if (a->struct_size != sizeof(plt_decode_attn_args))
        return fail(h, PLT_ERR_INVALID_ARG, "args.struct_size %u != %zu", a->struct_size, sizeof(plt_decode_attn_args));
    const plt_decode_attn_config& c = h->cfg;
    if (a->batch < 0) return fail(h, PLT_ERR_INVALID_ARG, "batch %d < 0", a->batch);
    if (a->batch > c.max_batch) return fail(h, PLT_ERR_CAPACITY, "batch %d > max_batch %d", a->batch, c.max_batch);
    if (a->batch == 0) return PLT_OK;
    if (a->kv_stride_b || a->kv_stride_n || a->kv_stride_h)
        return fail(h, PLT_ERR_UNSUPPORTED, "run_host takes dense shared caches only (strides must be 0)");
    if (h->Qn > 1) return fail(h, PLT_ERR_UNSUPPORTED, "run_host takes one query token per loop (q_len <= 1)");
    if (!a->q || !a->k_cache || !a->v_cache || !a->seq_lens || !a->out)
        return fail(h, PLT_ERR_INVALID_ARG, "q, k_cache, v_cache, seq_lens and out must not be NULL");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const bool fp8 = c.kv_dtype == PLT_KV_E4M3;
    if (fp8 && (!a->k_scale || !a->v_scale)) return fail(h, PLT_ERR_INVALID_ARG, "k_scale and v_scale must not be NULL with E4M3 caches");
    const size_t es = elem_size(h->bf16), B = (size_t)a->batch;
    const size_t row = (size_t)c.Hkv * c.d * (fp8 ? 1 : es);   // K (or V) of one token, all KV heads, as stored
    size_t kv_bytes;
    if (c.page_size > 0) {
        if (a->num_pool_pages < 1 || (size_t)a->num_pool_pages > (size_t)c.max_batch * (size_t)(a->max_pages > 0 ? a->max_pages : 0))
            return fail(h, PLT_ERR_CAPACITY, "num_pool_pages %d outside [1, max_batch * max_pages]", a->num_pool_pages);
        kv_bytes = (size_t)a->num_pool_pages * c.page_size * row;
    } else {
        kv_bytes = B * c.max_seq_len * row;
    }
    const size_t qo_bytes = B * c.L * c.Hq * c.d * es;
    const size_t win_bytes = c.L > 1 ? B * (c.L - 1) * c.w * row : 0;
    plt_decode_attn_args d = *a;
    plt_status s;
    const void* ptr;
#define PLT_STAGE(idx, field, bytes)                                                   \
    s = stage_in(h, idx, a->field, bytes, stream, &ptr);                               \
    if (s != PLT_OK) return s;                                                         \
    d.field = (decltype(d.field))ptr;
    PLT_STAGE(0, q, qo_bytes)
    PLT_STAGE(1, k_cache, kv_bytes)
    PLT_STAGE(2, v_cache, kv_bytes)
    PLT_STAGE(3, seq_lens, B * 4)
    PLT_STAGE(4, page_table, c.page_size > 0 ? B * (size_t)a->max_pages * 4 : 0)
    PLT_STAGE(5, k_win, win_bytes)
    PLT_STAGE(6, v_win, win_bytes)
    PLT_STAGE(7, win_lens, c.L > 1 ? B * (c.L - 1) * 4 : 0)
    PLT_STAGE(8, gate_logits, c.L > 1 ? B * (c.L - 1) * c.Hq * 4 : 0)
    PLT_STAGE(10, k_scale, fp8 ? (size_t)c.Hkv * 4 : 0)
    PLT_STAGE(11, v_scale, fp8 ? (size_t)c.Hkv * 4 : 0)
#undef PLT_STAGE
    Staging& so = h->st[9];
    if (so.bytes < qo_bytes) {
        if (so.ptr) cudaFree(so.ptr);
        so.ptr = nullptr;
        so.bytes = 0;
        if (cudaMalloc(&so.ptr, qo_bytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return fail(h, PLT_ERR_OUT_OF_MEMORY, "cudaMalloc of %zu staging bytes failed", qo_bytes);
        }
        so.bytes = qo_bytes;
    }
    d.out = so.ptr;
    s = plt_decode_attn_run(h, &d, cuda_stream);
    if (s != PLT_OK) return s;
    cudaError_t e = cudaMemcpyAsync(a->out, so.ptr, qo_bytes, cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return cuda_fail(h, "cudaMemcpyAsync (device to host)", e);
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(h, "cudaStreamSynchronize", e);
    return PLT_OK;
}

PLT_API plt_status plt_decode_attn_check(plt_decode_attn_t h, void* cuda_stream, uint32_t* out_bits) {
    if (!h) {
        // No handle: the status word of the allocation-free entry point on the current device.
        h = no_alloc_handle_of_current_device();
        if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL and plt_decode_attn_run_no_alloc has not run on the current device");
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    uint32_t bits = 0;
    cudaError_t e = cudaMemcpyAsync(&bits, h->status, 4, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->status, 0, 4, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(h, "reading the device status word", e);
    if (out_bits) *out_bits = bits;
    if (bits == 0) return PLT_OK;
    return fail(h, PLT_ERR_DEVICE_CHECK, "device status 0x%x:%s%s%s%s", bits,
                (bits & PLT_DEV_SEQ_LEN_CLAMPED) ? " seq_lens entry out of range (clamped)" : "",
                (bits & PLT_DEV_PAGE_ID_CLAMPED) ? " page id out of range (clamped)" : "",
                (bits & PLT_DEV_WAIT_TIMEOUT) ? " a bounded wait ran out (output invalid)" : "",
                (bits & PLT_DEV_WIN_LEN_CLAMPED) ? " win_lens entry out of range (clamped)" : "");
}

PLT_API plt_status plt_decode_attn_destroy(plt_decode_attn_t h) {
    if (!h) return PLT_OK;
    if (h->part_acc) cudaFree(h->part_acc);
    for (Staging& s : h->st)
        if (s.ptr) cudaFree(s.ptr);
    delete h;
    return PLT_OK;
}

PLT_API const char* plt_decode_attn_last_error(plt_decode_attn_t h) { return h ? h->err : g_create_error; }

PLT_API plt_status plt_decode_attn_set_profile_events(plt_decode_attn_t h, void* ev_main_begin, void* ev_main_end) {
    if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if ((ev_main_begin == nullptr) != (ev_main_end == nullptr))
        return fail(h, PLT_ERR_INVALID_ARG, "pass both events or neither");
    h->ev_begin = (cudaEvent_t)ev_main_begin;
    h->ev_end = (cudaEvent_t)ev_main_end;
    return PLT_OK;
}

PLT_API plt_status plt_decode_attn_launch_info(plt_decode_attn_t h, int32_t* kernels_per_run, int32_t* heads_per_cta,
                                       int32_t* key_slices, int32_t* stages, int32_t* ctas_per_sm, int32_t* grid,
                                       int32_t* kernel_path) {
    if (!h) return fail(nullptr, PLT_ERR_INVALID_ARG, "handle is NULL");
    if (kernels_per_run) *kernels_per_run = h->umma_e4m3 ? 3 : 2;   // (query pack,) main, merge
    if (heads_per_cta) *heads_per_cta = h->var.HPC;
    if (key_slices) *key_slices = h->var.KW;
    if (stages) *stages = h->var.stages;
    if (ctas_per_sm) *ctas_per_sm = h->ctas_per_sm;
    if (grid) *grid = h->var.grid;
    if (kernel_path) *kernel_path = h->umma ? PLT_PATH_TCGEN05 : PLT_PATH_WARP_MMA;
    return PLT_OK;
}

}  // extern "C"


// ===================================================================================================
// Allocation-free entry point.
//
// Some callers are not allowed to allocate device memory at the moment they need this attention:
// code that runs inside a memory-budgeted serving process whose allocator has handed every byte of
// HBM to the KV cache, code called from a context where cudaMalloc's implicit device synchronisation
// is unacceptable, or a plug-in that is given tensors but no right to create any. For them the split
// partials, the tile prefix and the status word live in one file-scope device array of fixed size,
// which every process that loads this library holds on each GPU it uses until it exits.
// ===================================================================================================
namespace {

constexpr size_t kNoAllocScratchBytes = PLT_NO_ALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_no_alloc_scratch[kNoAllocScratchBytes];

constexpr int kNoAllocMaxDevices = 64;

struct NoAllocDevice {
    bool ready = false;          // set-up done for this device
    void* scratch = nullptr;     // DEVICE address of g_no_alloc_scratch on this device
    int sm_count = 0;
    EncodeTiledFn encode = nullptr;
    bool have_handle = false;    // `handle` is prepared for `cfg`
    plt_decode_attn_config cfg;
    int32_t offsets[kMaxLoops];
    plt_decode_attn handle;      // host-side state only; its workspace pointers point into `scratch`
};

NoAllocDevice g_no_alloc[kNoAllocMaxDevices];

// Once per device, with that device current: take the device address of the scratch array. In host
// code the array's name is only a stand-in for the symbol; a kernel must be given this address.
plt_status no_alloc_setup(NoAllocDevice& dv, int device) {
    if (dv.ready) return PLT_OK;
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_no_alloc_scratch);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetSymbolAddress(scratch)", e);
    if (ptr == nullptr || ((uintptr_t)ptr & 255u) != 0)
        return fail(nullptr, PLT_ERR_CUDA, "scratch symbol address %p is null or not 256-byte aligned", ptr);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDeviceProperties", e);
    if (prop.major != 10)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", device,
                    prop.major, prop.minor);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
        return fail(nullptr, PLT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    dv.scratch = ptr;
    dv.sm_count = prop.multiProcessorCount;
    dv.encode = (EncodeTiledFn)fn;
    dv.ready = true;
    return PLT_OK;
}

// Field by field: the struct has padding after its last member, which a caller's stack copy leaves undefined.
bool same_config(const NoAllocDevice& dv, const plt_decode_attn_config* c) {
    const plt_decode_attn_config& a = dv.cfg;
    if (a.struct_size != c->struct_size || a.dtype != c->dtype || a.max_batch != c->max_batch || a.L != c->L ||
        a.Hq != c->Hq || a.Hkv != c->Hkv || a.d != c->d || a.max_seq_len != c->max_seq_len || a.w != c->w ||
        a.page_size != c->page_size || memcmp(&a.sm_scale, &c->sm_scale, sizeof(float)) != 0 || a.device != c->device ||
        a.heads_per_cta != c->heads_per_cta || a.key_slices != c->key_slices || a.stages != c->stages ||
        a.ctas_per_sm != c->ctas_per_sm || a.kernel_path != c->kernel_path || a.loads_in_flight != c->loads_in_flight ||
        a.slices_per_warp != c->slices_per_warp || a.row_warps != c->row_warps || a.kv_dtype != c->kv_dtype ||
        a.q_len != c->q_len || a.typical_seq_len != c->typical_seq_len)
        return false;
    for (int l = 0; l < c->L; ++l)
        if ((c->loop_offset ? c->loop_offset[l] : l) != dv.offsets[l]) return false;
    return true;
}

plt_decode_attn* no_alloc_handle_of_current_device() {
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current < 0 || current >= kNoAllocMaxDevices) return nullptr;
    NoAllocDevice& dv = g_no_alloc[current];
    return dv.ready && dv.have_handle ? &dv.handle : nullptr;
}

}  // namespace

extern "C" PLT_API plt_status plt_decode_attn_run_no_alloc(const plt_decode_attn_config* config,
                                                           const plt_decode_attn_args* args, void* cuda_stream) {
    Geometry g;
    plt_status s = check_config(config, &g);
    if (s != PLT_OK) return s;
    int current = -1;
    cudaError_t e = cudaGetDevice(&current);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDevice", e);
    if (current != config->device)
        return fail(nullptr, PLT_ERR_INVALID_ARG, "config.device %d is not the current device %d", config->device, current);
    if (current < 0 || current >= kNoAllocMaxDevices)
        return fail(nullptr, PLT_ERR_UNSUPPORTED, "device ordinal %d beyond %d", current, kNoAllocMaxDevices - 1);
    NoAllocDevice& dv = g_no_alloc[current];
    s = no_alloc_setup(dv, current);
    if (s != PLT_OK) return s;

    plt_decode_attn* h = &dv.handle;
    if (!dv.have_handle || !same_config(dv, config)) {
        // Prepare the host-side state for this configuration: the same choices create makes, minus cudaMalloc.
        dv.have_handle = false;
        h->cfg = *config;
        h->cfg.loop_offset = nullptr;
        for (int l = 0; l < kMaxLoops; ++l) h->delta[l] = config->loop_offset && l < config->L ? config->loop_offset[l] : l;
        h->G = g.G;
        h->R = g.R;
        h->Qn = g.Qn;
        h->bf16 = config->dtype == PLT_BF16;
        h->sm_count = dv.sm_count;
        const float scale = config->sm_scale > 0.f ? config->sm_scale : 1.0f / sqrtf((float)config->d);
        h->scale_log2 = scale * 1.4426950408889634f;
        h->err[0] = 0;
        for (bool& v : h->map_valid) v = false;
        s = setup_kernels(h, config, g);
        if (s != PLT_OK) return s;
        size_t acc_floats, ml_floats;
        h->ws_bytes = workspace_bytes_for(config, g, h->var.HPC, h->var.grid, h->umma_e4m3, &acc_floats, &ml_floats);
        if (h->ws_bytes > kNoAllocScratchBytes)
            return fail(nullptr, PLT_ERR_CAPACITY,
                        "this configuration needs %zu bytes of scratch but the built-in array holds %zu: lower max_batch "
                        "(scratch grows with max_batch * Hkv * L * Hq/Hkv * d) or use plt_decode_attn_create",
                        h->ws_bytes, kNoAllocScratchBytes);
        place_workspace(h, config, dv.scratch, acc_floats, ml_floats);
        dv.cfg = *config;
        for (int l = 0; l < kMaxLoops; ++l) dv.offsets[l] = h->delta[l];
        dv.have_handle = true;
    }
    // The array keeps whatever the previous call left. Partials and the prefix are rewritten before they are
    // read; only the status word must start at zero.
    e = cudaMemsetAsync(h->status, 0, 4, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(nullptr, "cudaMemsetAsync(status)", e);
    s = plt_decode_attn_run(h, args, cuda_stream);
    if (s != PLT_OK) {
        snprintf(g_create_error, sizeof g_create_error, "%s", h->err);
        return s;
    }
    return PLT_OK;
}
