/*
 * speckv.h -- C ABI of libspeckv, the sm_100a implementation of one SpecKV speculation
 * step's pass over vocabulary-sized logits.
 *
 * What the library computes, per batch row b with gamma_b drafted positions:
 *   - draft signals (paper Sec. 4.2): H_i = -sum_v q_i(v) log q_i(v) and c_i = max_v q_i(v) for
 *     the draft distribution q_i = softmax(draft logits / T_b) at every drafted position i,
 *     and the step signals: mean H, mean c, max H, min c;
 *   - the gamma controller (paper Sec. 4.3): context vector -> 16 hidden ReLU units -> one
 *     predicted acceptance rate per candidate gamma; Eq. 1 score E = a_hat * gamma + 1;
 *     gamma* = argmax over the candidates {2,4,6,8};
 *   - verification of the draft against the target logits: the greedy rule of paper Sec. 3.1
 *     for rows with temperature 0, and for temperature > 0 the lossless speculative-sampling
 *     rule the paper builds on (Sec. 1, 2.1): accept x_i while u_i < min(1, p_i(x_i)/q_i(x_i)),
 *     resample the first rejected position from norm(max(0, p - q)), and draw a bonus token
 *     from p when every drafted token is accepted.  Tokens per step = accepted + 1 (Sec. 3.1).
 *
 * Conventions
 *   - Every data pointer is DEVICE memory owned by the caller.  The struct arguments
 *     themselves (speckv_batch, speckv_mlp) are HOST structs holding device pointers.
 *   - Logit tensors are row-major with the vocabulary dimension contiguous; strides are
 *     counted in ELEMENTS.  The fast path needs 16-byte aligned base pointers and row strides
 *     that are multiples of 16 bytes; anything else takes a slower element-wise path.
 *   - The library allocates nothing and never synchronises; work is enqueued on the
 *     caller's stream (a cudaStream_t passed as void*).  Scratch memory comes from the
 *     caller: speckv_workspace_size() bytes,
 *     256-byte aligned, arbitrary contents, not shared between calls that may overlap.
 *   - The return code covers what the host can check (NULL or inconsistent arguments,
 *     unsupported sizes, workspace too small, launch failure).  Data-dependent problems are
 *     reported per row in row_status[b]; such a row gets n_accepted = 0, out_tokens = -1,
 *     gamma_next = 0 and zeros in its float outputs.  No kernel traps; every wait inside a
 *     kernel is bounded and ends in SPECKV_ROW_TIMEOUT on the row at hand.
 *   - Logits below -2^100 are treated as -inf (probability 0).  NaN or +inf anywhere in a used
 *     logit row, or a used row without any finite entry, flags the row.  Used rows are the draft
 *     rows of all gamma_b drafted positions and the target rows up to the stop position (the first
 *     position that is rejected, or gamma_b); target rows behind it are not part of the step
 *     (Sec. 3.1) and flag nothing.
 *   - Temperature: 0 selects the greedy rule (and T = 1 for that row's signals); otherwise
 *     finite and >= 1e-6.
 */
#ifndef SPECKV_H
#define SPECKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPECKV_OK = 0,
    SPECKV_ERR_INVALID_ARG = 1,
    SPECKV_ERR_UNSUPPORTED = 2,
    SPECKV_ERR_WORKSPACE = 3,
    SPECKV_ERR_CUDA = 4,
    SPECKV_ERR_STATIC_LIMIT = 5 /* batch needs more scratch than the built-in array holds */
} speckv_status;

typedef enum { SPECKV_F32 = 0, SPECKV_BF16 = 1 } speckv_dtype;

/* bits of row_status[b] */
enum {
    SPECKV_ROW_OK = 0,
    SPECKV_ROW_BAD_GAMMA = 1,       /* gamma_b outside 1..gamma_max                       */
    SPECKV_ROW_BAD_TOKEN = 2,       /* a used draft token outside 0..V-1                  */
    SPECKV_ROW_NONFINITE = 4,       /* NaN / +inf / all -inf in a used logit row          */
    SPECKV_ROW_BAD_TEMPERATURE = 8, /* negative, NaN or infinite temperature              */
    SPECKV_ROW_TIMEOUT = 16         /* a bounded wait inside a kernel ran out              */
};

#define SPECKV_MAX_GAMMA 16  /* gamma_max <= 16                                           */
#define SPECKV_MAX_HIDDEN 32 /* controller: n_hidden <= 32, n_in <= 8, n_out <= 8         */

typedef struct {
    int32_t B;         /* rows in the batch (>= 0)                                        */
    int32_t gamma_max; /* drafted positions stored per row (1..SPECKV_MAX_GAMMA)          */
    int32_t V;         /* vocabulary size (>= 1)                                          */
    speckv_dtype dtype;
    const void* draft_logits; /* [B, gamma_max, V]                                        */
    int64_t draft_stride_b, draft_stride_pos;
    const void* target_logits; /* [B, gamma_max+1, V]; not read by speckv_signals         */
    int64_t target_stride_b, target_stride_pos;
    const int32_t* draft_tokens; /* [B, gamma_max]; not read by speckv_signals            */
    const int32_t* gamma;        /* [B] in 1..gamma_max; NULL => gamma_max for every row  */
    const float* temperature;    /* [B]; NULL => temperature_scalar                       */
    float temperature_scalar;
    const float* uniforms;   /* [B, gamma_max+1, 2] in [0,1): [b,i,0] accept test at i,   */
                             /* [b,n,1] resample at the stop position n (bonus: n=gamma_b) */
    int32_t entropy_in_bits; /* 0: nats; 1: bits (the paper's log2)                       */
    int32_t flags;           /* SPECKV_* flags below, 0 for the defaults                  */
} speckv_batch;

/* speckv_batch.flags (verification calls; ignored by the others) */
enum {
    /* Read every target row 0..gamma_b of every batch row.  By default a target row behind a position
     * that is already known to be rejected is left out: Sec. 3.1 discards what the target produced
     * behind the first mismatch, so such a row changes no output.  Results are the same either way. */
    SPECKV_READ_ALL_TARGET_ROWS = 1,
    /* Scheduling hint (results are the same either way): take the sliced sweep whatever the batch size
     * and the logit type (fp32 batches of a few hundred rows otherwise take the bulk-copy ring sweep).
     * The value 2 is not in use: a batch that sets it is rejected with SPECKV_ERR_INVALID_ARG.          */
    SPECKV_SCHEDULE_SLICED = 4
};

typedef struct {
    int32_t n_in, n_hidden, n_out; /* 5, 16, 4 in the primary form                        */
    const float* W1;               /* [n_hidden, n_in]  device                            */
    const float* b1;               /* [n_hidden]        device                            */
    const float* W2;               /* [n_out, n_hidden] device                            */
    const float* b2;               /* [n_out]           device                            */
    int32_t gamma_choices[8];      /* candidate gammas, first n_out used ({2,4,6,8})      */
    int32_t feature_layout;        /* 0: x = [Hbar, cbar, cmin, comp0, comp1]             */
                                   /* 1: x = [Hbar, cbar, Hmax, cmin, comp0] (Sec. 4.3)   */
                                   /* 2: the predictor exactly as Sec. 4.3 writes it,      */
                                   /*    a_hat = f([Hbar, cbar, Hmax, cmin, comp.., gamma_j]): one */
                                   /*    output (W2 [1,n_hidden], b2 [1]) evaluated for each of the */
                                   /*    n_out candidate gammas; n_hidden = 0 makes it the linear  */
                                   /*    (Ridge) predictor with W2 [1,n_in], W1 and b1 unused      */
    int32_t score_transform;       /* 0: E_j = o_j * gamma_j + 1 (Eq. 1); 1: E_j = o_j    */
} speckv_mlp;

/* Scratch bytes needed by speckv_signals / speckv_verify / speckv_step for this batch
 * shape (depends on B, gamma_max, V and dtype only).                                      */
speckv_status speckv_workspace_size(const speckv_batch* batch, size_t* bytes);

/* Draft signals (paper Sec. 4.2).  H, C: [B, gamma_max] fp32 (0 at i >= gamma_b);
 * feat: [B,4] fp32 = mean H, mean c, max H, min c.  Any of H, C, feat, row_status may be
 * NULL.  Reads only the draft logits, gamma and temperature.                              */
speckv_status speckv_signals(const speckv_batch* batch, float* H, float* C, float* feat,
                             int32_t* row_status, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);

/* Controller (paper Sec. 4.3, Eq. 1).  feat: [B,4] as written by speckv_signals;
 * comp: [B, n_in-3] (layout 0), [B, n_in-4] (layout 1) or [B, n_in-5] (layout 2) fp32, NULL => zeros;
 * scores: [B, n_out] fp32 (may be NULL); gamma_next: [B] int32.  Ties go to the
 * lowest candidate index.                                                                 */
speckv_status speckv_select_gamma(int32_t B, const float* feat, const float* comp,
                                  const speckv_mlp* mlp, float* scores, int32_t* gamma_next,
                                  void* cuda_stream);

/* Verification (paper Sec. 3.1; speculative sampling for T > 0).  n_accepted: [B];
 * out_tokens: [B, gamma_max+1] = the accepted draft tokens, then the fresh token
 * (resampled, bonus, or the target's argmax), then -1; row_status: [B] (may be NULL).     */
speckv_status speckv_verify(const speckv_batch* batch, int32_t* n_accepted, int32_t* out_tokens,
                            int32_t* row_status, void* workspace, size_t workspace_bytes,
                            void* cuda_stream);

/* Drafting (paper Sec. 3.1: the draft model proposes gamma tokens): tokens[b,i] for i < gamma_b is
 * drawn from softmax(draft_logits[b,i] / T_b) by inverse CDF in vocabulary order at
 * uniforms[b,i] (the convention of the verification draws); T_b = 0 takes the argmax (lowest
 * index).  tokens: [B, gamma_max] int32, -1 at i >= gamma_b and in flagged rows; uniforms:
 * [B, gamma_max] fp32 in [0,1); row_status may be NULL.  Reads only the draft logits, gamma and
 * temperature.  Needs its own scratch size (one resample slot per drafted position).          */
speckv_status speckv_sample_workspace_size(const speckv_batch* batch, size_t* bytes);
speckv_status speckv_sample_draft(const speckv_batch* batch, const float* uniforms, int32_t* tokens,
                                  int32_t* row_status, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream);

/* One fused step: signals, controller and verification from a single pass over the logits
 * (plus a second look at the stop position's two rows for the residual / bonus draw, taken
 * while those rows are still in L2 where the batch is large enough for the stream kernel).
 * gamma_next[b] is the controller's choice for the NEXT step of row b; this step verifies
 * with the gamma given in the batch.  H, C, scores may be NULL.                            */
speckv_status speckv_step(const speckv_batch* batch, const float* comp, const speckv_mlp* mlp,
                          float* H, float* C, float* feat, float* scores, int32_t* gamma_next,
                          int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* speckv_signals for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for deployment reasons only.)
 *
 * Some hosts of this library may not call cudaMalloc once they are running: an inference server
 * whose framework has already claimed all device memory for its own pool, a plug-in that is only
 * allowed to touch buffers handed to it, a latency-critical decode loop where an allocation's
 * implicit device synchronisation would stall every stream.  Such a caller has nowhere to get
 * the workspace that speckv_signals asks for.  This variant brings its own: a fixed array of
 * SPECKV_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the
 * library holds that much memory until the process exits.  The caller still owns and passes the
 * inputs and the outputs; arguments, results and row_status are exactly those of speckv_signals.
 *
 *   - A batch whose speckv_workspace_size() exceeds SPECKV_STATIC_SCRATCH_BYTES is refused with
 *     SPECKV_ERR_STATIC_LIMIT before anything is enqueued (B = 256, gamma_max = 8, V = 128256
 *     needs 2.7 MB).
 *   - The call allocates and frees nothing.  The first call on each device looks up the
 *     array's device address (cudaGetSymbolAddress with that device current) and remembers it;
 *     make that first call outside any stream capture.
 *   - All calls on one device share the one array.  The parts that must start from zero are
 *     cleared on the caller's stream at the start of each call; the rest keeps whatever the
 *     previous call left.  Two calls that can overlap on the GPU (different streams without an
 *     ordering between them) race on it: order them, or use speckv_signals with separate
 *     workspaces.                                                                             */
#define SPECKV_STATIC_SCRATCH_BYTES (4u << 20)
speckv_status speckv_signals_static(const speckv_batch* batch, float* H, float* C, float* feat,
                                    int32_t* row_status, void* cuda_stream);

/* ---- Vocabulary-sharded step (the verification of Sec. 3.1 and the signals of Sec. 4.1 when the
 * vocabulary axis of the logits is split over n_shards devices, as a tensor-parallel output
 * projection leaves them).  Shard r holds columns [v_begin_r, v_begin_r + V_r) of every logit row:
 * `local` is an ordinary speckv_batch whose V is V_r and whose logit pointers and strides describe
 * the local slice; draft_tokens, gamma, temperature and uniforms are the full batch's, identical
 * on every shard.  All shards but the last have the same width (shard_width); the last may be
 * narrower.  The results equal those of speckv_step on the concatenated logits (same tolerance,
 * same near-tie caveats).  The four calls run on every shard, in this order, with two small
 * exchanges and one reduction between them that the caller performs (any all-gather will do):
 *
 *   speckv_shard_sweep      local slice -> shard_state [B, 2*gamma_max+1, 4] fp32, shard_tokl [B, gamma_max, 2] fp32
 *      -- all-gather both over the shards, in shard order: all_state [n_shards, B, 2*gamma_max+1, 4],
 *         all_tokl [n_shards, B, gamma_max, 2]
 *   speckv_shard_finish     every output of speckv_step except the fresh token of sampled rows (its
 *                           slot holds -1), and row_info (SPECKV_ROW_INFO_BYTES per row, opaque,
 *                           16-byte aligned) for the next two calls; identical on every shard
 *   speckv_shard_draw_sums  local slice -> shard_weight [B, 2] fp64
 *      -- all-gather: all_weight [n_shards, B, 2]
 *   speckv_shard_draw_pick  the shard that holds the drawn token writes it into out_tokens[b, n_accepted[b]]
 *      -- element-wise maximum of out_tokens over the shards.
 *
 * The workspace (speckv_shard_workspace_size(local) bytes, 256-byte aligned) is the shard's own;
 * its contents must survive from speckv_shard_draw_sums to speckv_shard_draw_pick.  All pointers are
 * device pointers; n_shards <= 32.  mlp may be NULL (no controller: scores and gamma_next untouched). */
#define SPECKV_ROW_INFO_BYTES 32
speckv_status speckv_shard_workspace_size(const speckv_batch* local, size_t* bytes);
speckv_status speckv_shard_sweep(const speckv_batch* local, int64_t v_begin, float* shard_state, float* shard_tokl,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);
speckv_status speckv_shard_finish(const speckv_batch* local, int32_t n_shards, int32_t shard_width, int32_t V_total,
                                  const float* all_state, const float* all_tokl, const float* comp,
                                  const speckv_mlp* mlp, float* H, float* C, float* feat, float* scores,
                                  int32_t* gamma_next, int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status,
                                  void* row_info, void* cuda_stream);
speckv_status speckv_shard_draw_sums(const speckv_batch* local, const void* row_info, double* shard_weight,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream);
speckv_status speckv_shard_draw_pick(const speckv_batch* local, int64_t v_begin, int32_t rank, int32_t n_shards,
                                     const void* row_info, const double* all_weight, int32_t* out_tokens,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream);

const char* speckv_status_string(speckv_status s);
int speckv_version(void);

#ifdef __cplusplus
}
#endif
#endif
