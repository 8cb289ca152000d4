/*
 * SpecKV oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision CPU statement of what one SpecKV speculation
 * step computes from draft and target logits: the draft signals (paper Sec. 4.2),
 * the gamma controller (paper Sec. 4.3, Eq. 1) and the verification of the draft
 * (paper Sec. 3.1 for the greedy rule; the lossless speculative-sampling rule of
 * Leviathan et al. / Chen et al., which the paper cites in Sec. 1 and 2.1, for
 * temperature > 0).
 *
 * Nothing in the product may import, link or call this library.  It shares no
 * code, header, table or helper with the CUDA path.  Only tests, the smoke
 * check and the cpu_baseline / reference legs of the benchmark use it.
 *
 * All pointers are HOST pointers.  Logit tensors are row-major with V
 * contiguous; strides are counted in elements.
 */
#ifndef SPECKV_ORACLE_H
#define SPECKV_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element type of the logit tensors */
#define ORACLE_DT_F32 0
#define ORACLE_DT_BF16 1 /* raw 16-bit patterns, upper half of an IEEE float */

/* per-row status bits */
#define ORACLE_ROW_OK 0
#define ORACLE_ROW_BAD_GAMMA 1
#define ORACLE_ROW_BAD_TOKEN 2
#define ORACLE_ROW_NONFINITE 4
#define ORACLE_ROW_BAD_TEMPERATURE 8

/* per-row near-tie bits (rows where a comparison is closer than the stated margin) */
#define ORACLE_NEAR_ACCEPT 1 /* |u - p(x)/q(x)| < 1e-6 at a tested position            */
#define ORACLE_NEAR_CDF 2    /* inverse-CDF threshold within 1e-6*W of a boundary        */
#define ORACLE_NEAR_GREEDY 4 /* (unused for exact ties: those resolve by lowest index)   */
#define ORACLE_NEAR_GAMMA 8  /* best and second-best controller score within 1e-5 rel.   */
#define ORACLE_NEAR_SMALL_RESIDUAL 16 /* rejected position whose residual mass is below 1e-5 */
#define ORACLE_NEAR_CDF_ABS 32        /* residual draw: threshold within 1e-6 of a boundary in units of probability
                                         (not of the residual's own mass W, which bit 2 measures)            */

typedef struct {
    int32_t B;         /* rows (sequences) in the batch                                  */
    int32_t gamma_max; /* drafted positions stored per row                               */
    int32_t V;         /* vocabulary size                                                */
    int32_t dtype;     /* ORACLE_DT_*                                                    */
    const void* draft; /* [B, gamma_max, V]                                              */
    int64_t draft_stride_row, draft_stride_pos;
    const void* target; /* [B, gamma_max+1, V]; may be NULL for signals                  */
    int64_t target_stride_row, target_stride_pos;
    const int32_t* draft_tokens; /* [B, gamma_max]; may be NULL for signals              */
    const int32_t* gamma;        /* [B] in 1..gamma_max; NULL => gamma_max               */
    const float* temperature;    /* [B]; NULL => temperature_scalar; 0 => greedy         */
    float temperature_scalar;
    const float* uniforms;   /* [B, gamma_max+1, 2]; [..,0] accept, [..,1] resample      */
    int32_t entropy_in_bits; /* 0: nats, 1: bits (the paper's log2)                      */
    int32_t n_threads;       /* rows are split over this many std::threads (>=1)         */
} oracle_batch;

typedef struct {
    int32_t n_in, n_hidden, n_out; /* 5, 16, 4 in the primary form                       */
    const float* W1;               /* [n_hidden, n_in]                                    */
    const float* b1;               /* [n_hidden]                                          */
    const float* W2;               /* [n_out, n_hidden]                                   */
    const float* b2;               /* [n_out]                                             */
    int32_t gamma_choices[8];      /* first n_out entries used                            */
    int32_t feature_layout;        /* 0: [Hbar,cbar,cmin,flag0,flag1]; 1: [Hbar,cbar,Hmax,cmin,comp];
                                      2: the paper's f(x, gamma): [Hbar,cbar,Hmax,cmin,comp..,gamma_j], one
                                         output (W2 [1,n_hidden], b2 [1]) evaluated for each of the n_out
                                         candidates; n_hidden = 0: linear predictor, W2 [1,n_in]        */
    int32_t score_transform;       /* 0: E_j = o_j*gamma_j + 1 (Eq. 1); 1: E_j = o_j      */
} oracle_mlp;

/* Draft signals.  H, C: [B, gamma_max] (entries at i >= gamma_b are 0);
 * feat: [B,4] = Hbar, cbar, Hmax, cmin.  Outputs are double.                 */
int oracle_signals(const oracle_batch* bt, double* H, double* C, double* feat, int32_t* row_status);

/* Controller.  feat: [B,4] doubles, comp: [B, n_comp] floats (n_comp = 2 for layout 0,
 * 1 for layout 1).  scores: [B, n_out] doubles, gamma_next: [B], near: [B] or NULL.  */
int oracle_select_gamma(int32_t B, const double* feat, const float* comp, const oracle_mlp* mlp,
                        double* scores, int32_t* gamma_next, int32_t* near);

/* Verification.  n_accepted: [B]; out_tokens: [B, gamma_max+1]; near: [B] or NULL. */
int oracle_verify(const oracle_batch* bt, int32_t* n_accepted, int32_t* out_tokens,
                  int32_t* row_status, int32_t* near);

/* Drafting: tokens[b,i] ~ softmax(draft[b,i] / T_b) for i < gamma_b by inverse CDF at
 * uniforms[b,i] (vocabulary order); argmax for T_b = 0; -1 at i >= gamma_b and in flagged rows.
 * uniforms: [B, gamma_max] floats.  tokens: [B, gamma_max].  near: [B] or NULL.             */
int oracle_sample_draft(const oracle_batch* bt, const float* uniforms, int32_t* tokens,
                        int32_t* row_status, int32_t* near);

/* Whole step = signals -> controller -> verification on one batch. */
int oracle_step(const oracle_batch* bt, const float* comp, const oracle_mlp* mlp, double* H,
                double* C, double* feat, double* scores, int32_t* gamma_next,
                int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status, int32_t* near);

/* Building blocks exposed so that tests can pin them one by one. */
/* softmax of one logit row at temperature T (T > 0) into prob[V]; returns 0, or
 * ORACLE_ROW_NONFINITE when the row holds NaN / +inf or is -inf throughout.   */
int oracle_softmax_row(const void* row, int32_t dtype, int32_t V, double T, double* prob);
/* -sum q ln q with 0 ln 0 = 0 */
double oracle_entropy_nats(const double* prob, int32_t V);
/* smallest v with cumulative weight > u * sum(w); falls back to the last v with w>0.
 * *near_boundary (may be NULL) is set when the threshold lies within 1e-6*sum(w) of
 * the chosen token's upper or lower cumulative boundary.  Returns -1 if sum(w) <= 0. */
int32_t oracle_inverse_cdf(const double* w, int32_t V, double u, int32_t* near_boundary);
/* lowest index attaining the row maximum */
int32_t oracle_argmax_row(const void* row, int32_t dtype, int32_t V);

#ifdef __cplusplus
}
#endif
#endif
