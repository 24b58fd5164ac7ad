/*
 * plt_decode_attn.h - C ABI of the Cross-Loop-Parallel (CLP) decode-step
 * attention of the Parallel Loop Transformer, for NVIDIA B200 (sm_100a).
 *
 * One call computes, for a batch of B sequences, the attention of ONE layer at
 * ONE decode step for all L loops at once (the paper's displaced micro-batch,
 * Algorithm 1 and the "Inference" paragraph of Sec. 2.2.1): loop l
 * (1-indexed) serves token i-l+1, so its query may see the first
 * cut(b,l) = max(0, N_b - delta_l) entries of the single shared first-loop KV
 * cache (delta_l = l-1 unless overridden).  Every loop attends that one cache
 * (the first-loop KV sharing of Sec. 2.2.2, y_global of Algorithm 3),
 * which the kernels read from HBM once per sequence, not once per loop.
 * Loops 2..L additionally attend their private window of their newest
 * <= w entries (y_local of Algorithm 3) and the two normalised results are mixed
 * with a per-head sigmoid gate (Algorithm 3, Eq. 2):
 *
 *   y_global = softmax(sm_scale * q K_share[0:cut]^T) V_share[0:cut]
 *   y_local  = softmax(sm_scale * q K_win[0:wl]^T)    V_win[0:wl]
 *   g        = sigmoid(gate_logit)
 *   O        = g * y_local + (1 - g) * y_global        (loops 2..L)
 *   O        = y_global                                (loop 1)
 *
 * Rows whose loop has no token yet (cut == 0) are written as zeros.  With
 * cut > 0 and wl == 0, y_local is taken as 0.  Query head h reads KV head
 * h / (Hq / Hkv).
 *
 * All tensor pointers are DEVICE pointers owned by the caller unless a comment
 * says "host".  No exception crosses this boundary; every function returns a
 * plt_status.  There is no CPU fallback: without a CUDA device every call that
 * needs one fails with PLT_ERR_CUDA.
 */
#ifndef PLT_DECODE_ATTN_H
#define PLT_DECODE_ATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct plt_decode_attn* plt_decode_attn_t; /* opaque; owned by the library */

typedef enum {
    PLT_OK = 0,
    PLT_ERR_INVALID_ARG = 1,  /* null pointer, bad size, misaligned base, struct_size mismatch */
    PLT_ERR_UNSUPPORTED = 2,  /* shape outside what the kernels implement (never a silent fallback) */
    PLT_ERR_OUT_OF_MEMORY = 3,
    PLT_ERR_CUDA = 4,         /* a CUDA runtime/driver call failed; see plt_decode_attn_last_error */
    PLT_ERR_CAPACITY = 5,     /* batch > max_batch, or a table smaller than the configuration needs */
    PLT_ERR_DEVICE_CHECK = 6  /* plt_decode_attn_check: a kernel clamped a device-resident value or gave up a wait */
} plt_status;

typedef enum { PLT_F32 = 0, PLT_BF16 = 1 } plt_dtype;

/* Storage of the shared cache and the windows (plt_decode_attn_config.kv_dtype). */
typedef enum {
    PLT_KV_SAME = 0,   /* like q and out (config.dtype) */
    PLT_KV_E4M3 = 1    /* 8-bit E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities) with one
                          fp32 scale per KV head for K and one for V: value = code value * scale.  The attention is the
                          same definition on those dequantised values (the paper's efficiency runs use FP8 attention,
                          Sec. 3.2).  Needs dtype = PLT_BF16 and d = 128; q and out stay bf16; softmax and
                          accumulation stay fp32.  Served by the warp-level kernel (codes converted to f16
                          in registers) or, up to 32 packed rows, by a tcgen05 kernel whose products take the
                          codes as they are (queries and probabilities split into sums of E4M3 terms);
                          plt_decode_attn_step quantises the rows it appends. */
} plt_kv_dtype;

/* Which main kernel streams the caches (plt_decode_attn_config.kernel_path). */
typedef enum {
    PLT_PATH_AUTO = 0,      /* the library chooses: tcgen05 above 48 packed rows (L * Hq / Hkv) when max_seq_len >= 16384
                               (bf16 caches), or on E4M3 caches at 25 to 32 packed rows when max_seq_len >= 8192 (contiguous,
                               or in pages of 64 tokens or of a multiple of 128) and at 17 to 24 rows when max_seq_len >= 32768
                               (contiguous, or in pages of a multiple of 128 tokens), and it applies; else the warp-level
                               kernel. With E4M3 caches at 17 to 32 rows, batches whose sequences are all longer than about
                               2048 (25-32 rows) or 8192 (17-24 rows) tokens gain from the tcgen05 kernel below these limits
                               too: say so with config.typical_seq_len, or ask for PLT_PATH_TCGEN05 */
    PLT_PATH_WARP_MMA = 1,  /* warp-level tensor-core products (mma.sync); fp32 inputs always use SIMT fp32 */
    PLT_PATH_TCGEN05 = 2    /* tcgen05.mma with accumulators in tensor memory: bf16 queries, d = 128, pages that divide
                               or are a multiple of 128 tokens, q_len <= 1, with E4M3 caches at most 32 packed rows;
                               anything else is refused with PLT_ERR_UNSUPPORTED */
} plt_kernel_path;

/* Bits of the device status word reported by plt_decode_attn_check. */
#define PLT_DEV_SEQ_LEN_CLAMPED 1u  /* a seq_lens entry was outside [0, max_seq_len] */
#define PLT_DEV_PAGE_ID_CLAMPED 2u  /* a page id was outside [0, num_pool_pages) */
#define PLT_DEV_WAIT_TIMEOUT 4u     /* a bounded wait inside a kernel ran out; the output is not valid */
#define PLT_DEV_WIN_LEN_CLAMPED 8u  /* a win_lens entry was outside [0, w] */

/*
 * Fixed at create.  struct_size = sizeof(plt_decode_attn_config) (versioning).
 * Supported: d in {64, 128}; Hq % Hkv == 0; L * q_len * (Hq / Hkv) <= 64 packed
 * query rows per KV head; L <= 8; paged caches need page_size % 16 == 0.
 */
typedef struct {
    uint32_t struct_size;
    int32_t dtype;        /* plt_dtype of Q, K, V, Kwin, Vwin and O; gate logits are always fp32 */
    int32_t max_batch;    /* largest batch any run may pass (<= 4096) */
    int32_t L;            /* loops computed in parallel (CLP micro-batch size), >= 1 */
    int32_t Hq, Hkv, d;   /* query heads, KV heads, head dimension */
    int32_t max_seq_len;  /* capacity of the shared cache per sequence, in tokens */
    int32_t w;            /* window capacity in tokens (G-SWA, Sec. 2.2.2); may be 0 only if L == 1 */
    int32_t page_size;    /* 0: contiguous shared cache; > 0: tokens per page */
    float sm_scale;       /* score scale; <= 0 selects 1/sqrt(d) */
    int32_t device;       /* CUDA device ordinal */
    const int32_t* loop_offset; /* host, L entries delta_l >= 0; NULL: delta_l = l-1. Copied at create. */
    /* Launch tuning, 0 = automatic. Results do not depend on these beyond rounding order. */
    int32_t heads_per_cta; /* KV heads one thread block streams together (bf16 path; divides Hkv) */
    int32_t key_slices;    /* warps that split the keys of a pipeline tile (bf16 path; 1, 2, 4 or 8) */
    int32_t stages;        /* depth of the shared-memory pipeline (bf16 path) */
    int32_t ctas_per_sm;   /* persistent thread blocks per SM */
    int32_t kernel_path;   /* plt_kernel_path. On PLT_PATH_TCGEN05, `stages` counts 32 KB ring slots (4 or 6) and
                              heads_per_cta, key_slices and ctas_per_sm are ignored (1 head, 128-key tiles, 1 block).
                              With E4M3 caches on that path: `stages` counts 16 KB slots (7 or 8: 4 for K tiles, the
                              rest for V tiles) and heads_per_cta is 1 or 2 (KV heads of one work item, whose tiles of
                              the same keys take turns; 2 needs an even Hkv and is the default then) */
    int32_t loads_in_flight; /* PLT_PATH_TCGEN05: K tiles (and likewise V tiles) kept in flight at most, clamped to the
                              ring of each; 0 = automatic */
    int32_t slices_per_warp; /* PLT_PATH_WARP_MMA: 16-key slices each of those warps takes per tile (1 or 2); a tile holds
                              16 * key_slices * slices_per_warp keys */
    int32_t row_warps;     /* PLT_PATH_WARP_MMA: warps that split the L * Hq/Hkv packed rows of a KV head (1 or 2; each
                              takes at most 32 rows) */
    int32_t kv_dtype;      /* plt_kv_dtype of k_cache, v_cache, k_win, v_win; strides are then in bytes (= elements) */
    int32_t q_len;         /* query tokens per loop in one step (multi-token / speculative decode); 0 or 1: one.
                              With q_len = Qn > 1 (bf16, PLT_PATH_WARP_MMA only; L * Qn * Hq/Hkv <= 64): q and out are
                              [B, L, Qn, Hq, d] and gate_logits [B, L-1, Qn, Hq], token j = 0..Qn-1 oldest first; the
                              caller has appended all Qn tokens of the step (N_b counts them; each window holds its
                              loop's newest entries IN AGE ORDER, oldest in slot 0). Token j of loop l is served as it
                              would have been Qn-1-j steps earlier: it sees the first cut(b,l) - (Qn-1-j) entries of the
                              shared cache and the first wl - (Qn-1-j) slots of its loop's window (the loops are
                              displaced by whole tokens, Sec. 2.2.1, so the causal cutoff moves by one per token).
                              plt_decode_attn_step and plt_decode_attn_run_host take q_len <= 1 only. */
    int32_t typical_seq_len; /* a length most sequences of a run will reach, if the caller knows one; 0: unknown. Only the
                              automatic choice of the kernel path reads it (results do not depend on it): the lengths
                              of a batch live on the device, so without it PLT_PATH_AUTO judges by max_seq_len and is
                              cautious. With E4M3 caches the tcgen05 kernel is then taken at 25 to 32 packed rows from
                              typical_seq_len >= 2048 and at 17 to 24 rows from >= 8192; with bf16 caches above 48 rows
                              it stands in for max_seq_len in the rule. < 0 is an error; values above max_seq_len count
                              as max_seq_len. */
} plt_decode_attn_config;

/*
 * Per call.  struct_size = sizeof(plt_decode_attn_args).  Every tensor base
 * must be 16-byte aligned.  Inputs are read-only; `out` is fully overwritten
 * for sequences [0, batch).
 */
typedef struct {
    uint32_t struct_size;
    int32_t batch;                 /* B, 0 <= B <= max_batch */
    const void* q;                 /* [B, L, Hq, d] contiguous */
    const void* k_cache;           /* shared first-loop keys: contiguous [B, N, Hkv, d] (strides below) */
    const void* v_cache;           /*   or page pool [num_pool_pages, page_size, Hkv, d] */
    int64_t kv_stride_b;           /* elements between sequences (contiguous) or between pages (paged) */
    int64_t kv_stride_n;           /* elements between tokens */
    int64_t kv_stride_h;           /* elements between KV heads; the head dimension itself is dense */
                                   /* all three 0: dense layout as written above. Each a multiple of 8 (bf16) / 4 (fp32). */
    const int32_t* seq_lens;       /* [B]; N_b counts the current token; values outside [0, max_seq_len] are clamped */
    const int32_t* page_table;     /* [B, max_pages] page ids (paged only; else NULL) */
    int32_t max_pages;             /* row length of page_table; >= ceil(max_seq_len / page_size) */
    int32_t num_pool_pages;        /* pages in the pool */
    const void* k_win;             /* [B, L-1, w, Hkv, d] contiguous; slots [0, wl) are attended (any order) */
    const void* v_win;             /*   (both NULL allowed when L == 1) */
    const int32_t* win_lens;       /* optional [B, L-1]; NULL: wl = min(w, cut(b,l)) */
    const float* gate_logits;      /* [B, L-1, Hq] pre-sigmoid; +-inf allowed (NULL allowed when L == 1) */
    void* out;                     /* [B, L, Hq, d], same dtype as q */
    const float* k_scale;          /* PLT_KV_E4M3 only: [Hkv] fp32 scales of the K codes (cache and windows); else ignored */
    const float* v_scale;          /* PLT_KV_E4M3 only: [Hkv] fp32 scales of the V codes */
} plt_decode_attn_args;

/*
 * Validates the configuration, selects the kernel variant and allocates the
 * handle's workspace on config->device (split partials, plan, status word).
 * This is the only call that allocates device memory for plt_decode_attn_run.
 */
plt_status plt_decode_attn_create(const plt_decode_attn_config* config, plt_decode_attn_t* out_handle);

/*
 * Enqueues one decode-step attention (Algorithm 3 from y_global to the gate mix, for all L loops of
 * all B sequences) on `cuda_stream` (a cudaStream_t; NULL = default stream).
 * Asynchronous: no allocation and no host synchronisation.  Host-visible
 * arguments are validated first and nothing is launched on error.  Two kernels
 * are launched: the split-KV main kernel and the merge/gate kernel.
 * Calls on the same handle must be stream-ordered (they share the workspace).  Once a first call has seen the
 * tensor addresses (it encodes the TMA descriptors on the host), calls with the same addresses do no host work
 * besides the launches and can be captured in a CUDA graph.
 * The main kernel is launched with programmatic stream serialisation: its set-up reads seq_lens and win_lens while
 * the kernel before it in the stream finishes, everything else after that kernel has completed.  A kernel of yours
 * that writes seq_lens or win_lens right before this call must therefore not release its programmatic dependents
 * early (kernels that never call griddepcontrol.launch_dependents release them when they end: nothing to do).
 * The same holds after the call: the merge kernel releases its programmatic dependents at its start, while it still
 * reads seq_lens, win_lens and gate_logits and before it writes `out`.  A kernel of yours that is enqueued after this
 * call WITH programmatic stream serialisation may therefore touch those arrays, the caches and `out` only after its own
 * griddepcontrol.wait (an ordinary launch waits for the whole call: nothing to do).
 */
plt_status plt_decode_attn_run(plt_decode_attn_t handle, const plt_decode_attn_args* args, void* cuda_stream);

/*
 * Same computation with every tensor pointer in `args` pointing to HOST memory
 * (pinned memory makes the copies asynchronous).  Copies the inputs into
 * device staging buffers owned by the handle (allocated on the first call,
 * sized for max_batch), runs, copies `out` back and synchronises the stream.
 * Shared-cache strides must be 0 (dense); a paged pool must have
 * num_pool_pages <= max_batch * max_pages.
 */
plt_status plt_decode_attn_run_host(plt_decode_attn_t handle, const plt_decode_attn_args* host_args, void* cuda_stream);

/*
 * What one decode step hands to plt_decode_attn_step besides plt_decode_attn_args: the K and V rows that f_qkv of
 * Algorithm 3 produced for this step, and the head-wise gate linear f_gate of that algorithm (Sec. 2.2.2: one
 * scalar per head).  All pointers are device memory; k_new / v_new 16-byte aligned.
 */
typedef struct {
    uint32_t struct_size;
    const void* k_new;        /* [B, L, Hkv, d], dtype of q: row l-1 = keys of the token loop l handles now.  With
                                 PLT_KV_E4M3 the rows are stored as round-to-nearest-even codes of x / scale[head]
                                 (fp32 division, clamped to the largest finite magnitude 448) */
    const void* v_new;        /* [B, L, Hkv, d] */
    const float* w_gate;      /* [Hq, d] fp32 (ignored when L == 1) */
    const float* b_gate;      /* [Hq] fp32 */
    float* gate_logits;       /* [B, L-1, Hq] fp32, written by the call and then used by the attention */
} plt_decode_attn_step_args;

/*
 * One whole decode step of the path: the pre-step and then the attention of plt_decode_attn_run, three launches.
 * Pre-step (one kernel), with cut(b,l) = max(0, N_b - delta_l) and N_b counting the current token:
 *   - loop 1: k_new/v_new[b, 0] are stored at position cut(b,1) - 1 of the shared cache (Algorithm 1: the
 *     step returns the updated cache);
 *   - loops 2..L: k_new/v_new[b, l-1] are stored in slot (cut(b,l) - 1) mod w of that loop's window, so that the window
 *     holds the w newest entries of that loop (Sec. 2.2.2); nothing is written where cut(b,l) = 0;
 *   - step->gate_logits[b, l-2, h] = sum_j w_gate[h, j] * q[b, l-1, h, j] + b_gate[h]  (fp32 accumulation).
 * This call therefore WRITES through args->k_cache, v_cache, k_win and v_win although the struct declares them
 * const; args->gate_logits is ignored and args->win_lens must be NULL (the window length is min(w, cut)).  Errors and
 * stream semantics as plt_decode_attn_run; out-of-range page ids are clamped and flagged in the status word.
 */
plt_status plt_decode_attn_step(plt_decode_attn_t handle, const plt_decode_attn_args* args,
                                const plt_decode_attn_step_args* step, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the device status word and clears it.
 * PLT_OK if it was 0; else PLT_ERR_DEVICE_CHECK with *out_bits (optional) = PLT_DEV_* bits.
 * handle == NULL reads the status word of plt_decode_attn_run_no_alloc on the calling thread's current device (that
 * entry point clears the word at the start of every call, so this reports the most recent call only). */
plt_status plt_decode_attn_check(plt_decode_attn_t handle, void* cuda_stream, uint32_t* out_bits);

/* Frees the workspace. NULL is accepted. The caller makes sure no run is in flight. */
plt_status plt_decode_attn_destroy(plt_decode_attn_t handle);

/* Message for the last non-OK status of this handle (or of the last failed create when handle == NULL).
 * Owned by the library; valid until the next call on the same handle / thread. */
const char* plt_decode_attn_last_error(plt_decode_attn_t handle);

/* Device bytes plt_decode_attn_create would allocate for this configuration (no device needed for the arithmetic,
 * but the SM count of config->device is queried when a device is present; 148 is assumed otherwise). */
plt_status plt_decode_attn_workspace_bytes(const plt_decode_attn_config* config, size_t* out_bytes);

/* Number of kernels one plt_decode_attn_run launches, and the variant chosen at create
 * (heads_per_cta, key_slices = warps along the keys of a tile as in the configuration, stages, ctas_per_sm, grid size,
 * plt_kernel_path actually used); any pointer may be NULL. */
plt_status plt_decode_attn_launch_info(plt_decode_attn_t handle, int32_t* kernels_per_run, int32_t* heads_per_cta,
                                       int32_t* key_slices, int32_t* stages, int32_t* ctas_per_sm, int32_t* grid,
                                       int32_t* kernel_path);

/* Measurement aid: when both are non-NULL (cudaEvent_t created by the caller, with timing enabled), every later
 * plt_decode_attn_run records ev_main_begin just before and ev_main_end just after the split-KV main kernel on
 * the run's stream, so that the caller can time that kernel apart from the merge kernel. NULL, NULL switches it off. */
plt_status plt_decode_attn_set_profile_events(plt_decode_attn_t handle, void* ev_main_begin, void* ev_main_end);

/*
 * plt_decode_attn_run_no_alloc - the same decode-step attention for callers that cannot allocate device memory.
 * (An addition of this library; the paper has no counterpart.)
 *
 * Who needs it: a serving process that has given every byte of HBM to its KV cache and has no allocator left to
 * ask, code that must not trigger the device-wide synchronisation a cudaMalloc implies, or a plug-in that is
 * handed tensors without the right to create device buffers. Such callers skip plt_decode_attn_create: this call
 * takes the configuration and the per-call arguments together and keeps its scratch (split partials, tile prefix,
 * status word) in a device array compiled into the library, PLT_NO_ALLOC_SCRATCH_BYTES large, which every
 * process that loads the library holds on each GPU it touches until the process exits.
 *
 * - It never calls cudaMalloc, cudaFree or any allocating routine. `args` is as for plt_decode_attn_run
 *   (device pointers owned by the caller; `out` fully overwritten); `config` as for plt_decode_attn_create.
 * - config->device must be the current device of the calling thread.
 * - A configuration whose scratch (it grows with max_batch * Hkv * L * Hq/Hkv * d; ask
 *   plt_decode_attn_workspace_bytes) exceeds the array is refused with PLT_ERR_CAPACITY and a message that states
 *   both sizes. Set max_batch to the batch actually used.
 * - The first call on a device looks up the array's device address and prepares the kernels; make that first
 *   call outside any stream capture. Later calls with the same configuration reuse the prepared state.
 * - All calls on one device share the one array, which keeps what the previous call left. The call clears the
 *   part that must start at zero (the status word) itself. Two calls whose GPU work overlaps (different streams,
 *   or different host threads) race on the partials: keep calls on a device stream-ordered and issue them from
 *   one thread at a time.
 * - Errors are reported like those of create: plt_decode_attn_last_error(NULL) holds the message.
 * - Clamped lengths or page ids and a wait that ran out are flagged in a status word inside the array, which
 *   plt_decode_attn_check(NULL, stream, &bits) reads for the current device.
 */
#define PLT_NO_ALLOC_SCRATCH_BYTES (16u << 20)
plt_status plt_decode_attn_run_no_alloc(const plt_decode_attn_config* config, const plt_decode_attn_args* args,
                                        void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PLT_DECODE_ATTN_H */
