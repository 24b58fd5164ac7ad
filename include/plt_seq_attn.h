/*
 * plt_seq_attn.h - C ABI of the sequence-shaped attention of the Parallel Loop Transformer, for NVIDIA B200 (sm_100a).
 *
 * The attention of a prefill or training-forward pass: what plt_decode_attn_run computes for ONE decode step, for
 * every step of a sequence at once (Algorithm 2 "Training for PLT", whose non-first loops use the attention of
 * Algorithm 3, and the prefill line of Algorithm 1).  Row t (0-indexed) of loop l (1-indexed) is the query that loop
 * holds at decode step t: the l-th loop of token t - delta_l, delta_l = l - 1 (Sec. 2.2.1 "Inference"); delta = 0
 * for every loop gives the reading of Algorithm 2, where the shifted states sit at their own positions.  Per sequence
 * b of length n_b, loop l, row t < n_b and query head h (KV head h / (Hq / Hkv)):
 *
 *   cut      = max(0, t + 1 - delta_l)
 *   y_global = softmax(sm_scale * q K_share[0:cut]^T) V_share[0:cut]                        (Algorithm 3, global)
 *   y_local  = softmax(sm_scale * q K_l[lo:t+1]^T) V_l[lo:t+1],  lo = max(delta_l, t+1-w)    (Algorithm 3, SWA)
 *   O        = sigmoid(gate) * y_local + (1 - sigmoid(gate)) * y_global   (l >= 2);   O = y_global   (l = 1)   (Eq. 2)
 *
 * K_share, V_share are the first loop's keys and values, shared by all loops (Sec. 2.2.2); K_l, V_l are loop l's own
 * (row t' = what the loop produced at step t'), of which a row sees its w newest including its own.  Rows with
 * cut = 0 and rows t >= n_b are written as zeros.
 *
 * All tensor pointers are DEVICE pointers owned by the caller, bf16, 16-byte aligned; head dimension 128.  No
 * exception crosses this boundary; errors are plt_status codes (plt_decode_attn.h).  There is no CPU fallback.
 */
#ifndef PLT_SEQ_ATTN_H
#define PLT_SEQ_ATTN_H

#include "plt_decode_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct plt_seq_attn* plt_seq_attn_t; /* opaque; owned by the library */

/* Fixed at create.  struct_size = sizeof(plt_seq_attn_config).  Supported: bf16, d = 128, Hq % Hkv == 0, L <= 8. */
typedef struct {
    uint32_t struct_size;
    int32_t max_batch;    /* largest batch any run may pass */
    int32_t L;            /* loops, >= 1 */
    int32_t Hq, Hkv, d;   /* query heads, KV heads, head dimension (128) */
    int32_t max_seq_len;  /* T: rows per sequence in every tensor (the padded length) */
    int32_t w;            /* window of the sliding-window attention in tokens (Sec. 2.2.2); may be 0 only if L == 1 */
    float sm_scale;       /* score scale; <= 0 selects 1/sqrt(d) */
    int32_t device;       /* CUDA device ordinal */
    const int32_t* loop_offset; /* host, L entries delta_l >= 0; NULL: delta_l = l - 1.  Copied at create. */
} plt_seq_attn_config;

/* Per call.  struct_size = sizeof(plt_seq_attn_args).  Inputs are read-only; `out` is fully overwritten for
 * sequences [0, batch), rows [0, T).  Rows of K/V at or beyond n_b may hold anything. */
typedef struct {
    uint32_t struct_size;
    int32_t batch;              /* B, 0 <= B <= max_batch */
    const void* q;              /* [B, L, T, Hq, d] */
    const void* k_share;        /* [B, T, Hkv, d]  first-loop keys */
    const void* v_share;        /* [B, T, Hkv, d] */
    const void* k_loc;          /* [B, L-1, T, Hkv, d]  own keys of loops 2..L (NULL allowed when L == 1) */
    const void* v_loc;          /* [B, L-1, T, Hkv, d] */
    const float* gate_logits;   /* [B, L-1, T, Hq] fp32, pre-sigmoid; +-inf allowed (NULL allowed when L == 1) */
    const int32_t* seq_lens;    /* [B] n_b; values outside [0, T] are clamped and flagged in the status word */
    void* out;                  /* [B, L, T, Hq, d] bf16 */
} plt_seq_attn_args;

/* Validates the configuration and allocates the handle's device state (a status word). */
plt_status plt_seq_attn_create(const plt_seq_attn_config* config, plt_seq_attn_t* out_handle);

/* Enqueues the attention of Algorithm 2 / Algorithm 3 over whole sequences on `cuda_stream` (cudaStream_t; NULL =
 * default stream).  One kernel (tcgen05.mma with accumulators in tensor memory, K/V tiles by TMA, the pass over
 * the shared K/V and the banded pass over the loop's own K/V fused).  Asynchronous: no allocation, no host
 * synchronisation; host-visible arguments are validated first and nothing is launched on error. */
plt_status plt_seq_attn_run(plt_seq_attn_t handle, const plt_seq_attn_args* args, void* cuda_stream);

/* Synchronises `cuda_stream`, reads the device status word (PLT_DEV_* bits of plt_decode_attn.h) and clears it. */
plt_status plt_seq_attn_check(plt_seq_attn_t handle, void* cuda_stream, uint32_t* out_bits);

/* Frees the handle.  NULL is accepted. */
plt_status plt_seq_attn_destroy(plt_seq_attn_t handle);

/* Message for the last non-OK status of this handle (or of the last failed create when handle == NULL). */
const char* plt_seq_attn_last_error(plt_seq_attn_t handle);

#ifdef __cplusplus
}
#endif
#endif /* PLT_SEQ_ATTN_H */
