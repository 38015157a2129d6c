/*
 * adasd.h - C ABI of the AdaSD hot path for NVIDIA B200 (sm_100a).
 *
 * The library computes, for every draft and candidate position of a speculative
 * decoding round, the full-vocabulary softmax statistics, the token entropy H(q_i)
 * that drives the adaptive draft-stop check (Sec. 4.3), the Jensen-Shannon distance
 * between the target row p_i and the draft row q_i (Sec. 2.2), the KDE/Bayes
 * acceptance probability P(A|d_i) and the first-rejection accept scan (Sec. 4.4,
 * Algorithm 1), the update of the three lists L_E^R, L_D^A, L_D^R and of the
 * generation threshold T_G (Algorithm 1, step 3), and vanilla speculative sampling
 * (Sec. 2.1.3) as the comparison mode; also greedy decoding (Sec. 2.1.3), the ablation
 * variants of Sec. 5, and the adjusted distribution of Sec. 2.1.1 (temperature, top-k,
 * top-p) ahead of all of it.
 *
 * Conventions
 *   - Every pointer named *_dev is a DEVICE pointer owned by the caller; the library
 *     neither frees nor keeps it beyond the call.  Pointers without the suffix are
 *     host pointers.  `stream` is a cudaStream_t passed as void* (NULL = default).
 *   - Hot calls (draft_entropy, verify, update_thresholds, vanilla_verify, greedy_verify,
 *     gen_only_update, get_thresholds, reset) only enqueue kernels on `stream`: they never allocate,
 *     free or synchronise.  create/destroy/state_export/state_import/status do.
 *   - Logits are row-major with contiguous vocabulary; strides are in ELEMENTS.
 *     bf16 or fp32 as fixed at create time.  Rows whose base address and stride are
 *     multiples of 16 bytes take the vectorised path; anything else still works
 *     through a scalar path.
 *   - Uniforms are fp32 in [0,1), supplied by the caller (the library draws nothing).
 *   - Entropy, log-sum-exp and the JS divergence are in nats; the JS distance is
 *     sqrt(D_JS / ln 2), i.e. in [0,1].
 *   - Return value: ADASD_OK or a negative ADASD_ERR_* code.  Errors detectable on
 *     the host launch nothing.  Conditions found on the device (list capacity
 *     exhausted, NaN / all -inf rows, a bounded wait that expired) set sticky bits
 *     in a status word read with adasd_status(); the call never traps or hangs.
 *   - A context is bound to one device and must be used from one stream at a time.
 *     The hot calls launch on the calling thread's current device: when that is not the
 *     context's device they return ADASD_ERR_DEVICE and launch nothing (create, destroy,
 *     state_export/import and status switch to the context's device themselves).
 *   - Conditions only the device can see never become return codes: a NaN row, a full
 *     list or an expired wait is reported through the status word alone.
 */
#ifndef ADASD_H
#define ADASD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ADASD_OK 0
#define ADASD_ERR_NULL (-1)      /* a required pointer is NULL */
#define ADASD_ERR_ALIGN (-2)     /* a pointer is not aligned to its element type (4 bytes for float /
                                    int32 arrays, 2 or 4 for logits); nothing is launched */
#define ADASD_ERR_SHAPE (-3)     /* a size, stride or window is out of range */
#define ADASD_ERR_DTYPE (-4)     /* unknown dtype / rule */
#define ADASD_ERR_CAPACITY (-5)  /* size beyond a stated maximum */
#define ADASD_ERR_CUDA (-7)      /* a CUDA runtime call failed */
#define ADASD_ERR_DEVICE (-9)    /* the calling thread's current device is not the context's device */

/* bits of the sticky device status word */
#define ADASD_STATUS_CAPACITY 1u /* an append was skipped: list full */
#define ADASD_STATUS_TIMEOUT 2u  /* a bounded wait expired; outputs of that row are NaN */
#define ADASD_STATUS_NAN 4u      /* a row held NaN or no finite logit */

#define ADASD_BF16 0
#define ADASD_FP32 1

#define ADASD_KMAX_LIMIT 32      /* largest window supported (the paper uses W = 20) */

/* limits of adasd_vanilla_verify_static (its scratch is a fixed array of about 132 KB) */
#define ADASD_STATIC_MAX_B 1024            /* sequences per call */
#define ADASD_STATIC_MAX_POSITIONS 16384   /* B * (Kmax + 1) per call */

/* flags of adasd_verify */
#define ADASD_FUSE_UPDATE 1u     /* run the list appends and the T_G update in the same launch */

typedef struct adasd_ctx adasd_ctx; /* opaque; owns the per-sequence adaptive state */

typedef struct {
    int32_t B;               /* sequences, each with its own T_G and lists */
    int32_t V;               /* vocabulary size */
    int32_t Kmax;            /* largest window, 1..ADASD_KMAX_LIMIT */
    int32_t dtype;           /* ADASD_BF16 or ADASD_FP32 */
    int32_t list_capacity;   /* max entries of each of L_E^R, L_D^A, L_D^R per sequence */
    int32_t kde_bandwidth;   /* 0: Silverman factor (3n/4)^(-1/5); 1: Scott n^(-1/5) */
    int32_t reject_rule;     /* 0: Bernoulli, reject iff u >= P(A|d); 1: reject iff P(A|d) < 1/2 */
    int32_t min_kde_samples; /* below this many entries in either list P(A|d) := 0 (>= 2) */
    int32_t cluster_size;    /* 0 = choose automatically; else 1..8 CTAs per row / position */
    int32_t device;          /* CUDA device ordinal */
} adasd_config;

/*
 * Per-position results of one round (all device arrays; any may be NULL in
 * adasd_verify, in which case it is not written).  Entries of positions at or
 * beyond a sequence's window are left untouched.
 */
typedef struct {
    float* H_d;          /* [B,Kmax]   H(q_i), nats */
    float* H_t;          /* [B,Kmax+1] H(p_i), nats */
    float* lse_d;        /* [B,Kmax]   log-sum-exp of draft rows */
    float* lse_t;        /* [B,Kmax+1] */
    float* jsd;          /* [B,Kmax]   D_JS(p_i||q_i), nats */
    float* dist;         /* [B,Kmax]   d_i in [0,1] */
    float* p_acc;        /* [B,Kmax]   P(A|d_i) with d_1..d_{i-1} of this round counted as accepted */
    int32_t* y;          /* [B,Kmax+1] y_i ~ p_i */
    int32_t* draft_len;  /* [B] window K_t the round used */
    int32_t* accept_len; /* [B] */
    int32_t* rejected;   /* [B] 1 if the accept scan stopped at a rejection */
} adasd_round_record;

/* Allocates the context and its device state: T_G = 0, all lists empty (Algorithm 1,
 * initialisation).  Synchronises. */
int adasd_create(adasd_ctx** out, const adasd_config* cfg);
int adasd_destroy(adasd_ctx* ctx);

/* Back to the initial state for the n sequences listed in seq_ids_dev (NULL: all). */
int adasd_reset(adasd_ctx* ctx, const int32_t* seq_ids_dev, int32_t n, void* stream);

/*
 * One draft step for every active sequence (Algorithm 1, generation loop body;
 * Sec. 4.3; entropy as in Appendix A).  For row b of logits_dev [B,V]:
 *   H_out[b]   = H(q)             lse_out[b] = log-sum-exp (nullable)
 *   token_out[b] = inverse-CDF sample of q in index order with uniform u_dev[b];
 *                  with u_dev NULL and token_out_dev given: the most probable token
 *                  argmax q (greedy drafting, Sec. 2.1.3; lowest index among equal maxima);
 *                  both NULL: no token
 *   stop_out[b]  = 1 iff H(q) > T_G[b]   (strict; the token stays in the window)
 *   draft_len_inout[b] += 1               (nullable)
 * active_inout_dev (nullable): rows with 0 are skipped and their outputs left
 * untouched; a row whose stop flag is raised gets its entry cleared, so the next
 * draft step skips it without host involvement.
 */
int adasd_draft_entropy(adasd_ctx* ctx, const void* logits_dev, int64_t row_stride,
                        const float* u_dev, uint8_t* active_inout_dev, float* H_out_dev,
                        float* lse_out_dev, int32_t* token_out_dev, uint8_t* stop_out_dev,
                        int32_t* draft_len_inout_dev, void* stream);

/*
 * Verification of one round for every sequence (Algorithm 1, step 2; Sec. 4.4;
 * JS divergence/distance as in Sec. 2.2).
 *   draft_logits_dev  [B,Kmax,V]   row (b,i) at b*d_seq_stride + i*d_row_stride
 *   target_logits_dev [B,Kmax+1,V] row (b,i) at b*t_seq_stride + i*t_row_stride;
 *                                  row K_t of a sequence is its bonus row
 *   draft_tokens_dev  [B,Kmax]     x_i
 *   draft_len_dev     [B]          K_t in 0..Kmax (NULL: Kmax for all)
 *   u_target_dev      [B,Kmax+1]   uniforms for y_i ~ p_i
 *   u_accept_dev      [B,Kmax]     uniforms for the accept draw
 *   accept_len_dev    [B]          number of accepted draft tokens
 *   next_token_dev    [B]          y_{accept_len+1}
 *   record            host struct of device arrays to receive per-position values
 *                     (NULL: none)
 * Candidate i is rejected iff x_i != y_i and Reject(P(A|d_i)); the scan stops at the
 * first rejection.  With ADASD_FUSE_UPDATE the same launch appends to the lists and
 * recomputes T_G = mean(L_E^R); without it the state is left unchanged and
 * adasd_update_thresholds() applies the update from a record.
 */
int adasd_verify(adasd_ctx* ctx, const void* draft_logits_dev, const void* target_logits_dev,
                 int64_t d_seq_stride, int64_t d_row_stride, int64_t t_seq_stride,
                 int64_t t_row_stride, const int32_t* draft_tokens_dev,
                 const int32_t* draft_len_dev, const float* u_target_dev,
                 const float* u_accept_dev, int32_t* accept_len_dev, int32_t* next_token_dev,
                 const adasd_round_record* record, uint32_t flags, void* stream);

/*
 * List appends and threshold update of one round from a record (Algorithm 1, the
 * append lines of step 2 and step 3): accepted d_i with 0 < d_i < 1 go to L_D^A; at a
 * rejection H(q_i) goes to L_E^R and d_i (if 0 < d_i < 1) to L_D^R; T_G = mean(L_E^R).
 * The record must carry H_d, dist, draft_len, accept_len and rejected.
 * A rejected candidate whose entropy is not finite (its row held NaN or no finite logit;
 * ADASD_STATUS_NAN is already set) is not recorded, so T_G stays finite.  An append to a
 * list that already holds list_capacity entries is skipped whole (L_E^R too: T_G stays the
 * mean of what the list holds) and sets ADASD_STATUS_CAPACITY.
 */
int adasd_update_thresholds(adasd_ctx* ctx, const adasd_round_record* record, void* stream);

/*
 * Vanilla speculative sampling on the same inputs (Sec. 2.1.3): accept x_i iff
 * u_accept[b,i] < min(1, p_i(x_i)/q_i(x_i)); at the first rejection the next token is
 * drawn from norm(max(0, p_i - q_i)) with u_resample[b] (from p_i if that has no
 * mass); with no rejection it is drawn from the bonus row with u_resample[b].
 * The adaptive state is neither read nor written.  alpha_out_dev [B,Kmax] nullable.
 */
int adasd_vanilla_verify(adasd_ctx* ctx, const void* draft_logits_dev,
                         const void* target_logits_dev, int64_t d_seq_stride,
                         int64_t d_row_stride, int64_t t_seq_stride, int64_t t_row_stride,
                         const int32_t* draft_tokens_dev, const int32_t* draft_len_dev,
                         const float* u_accept_dev, const float* u_resample_dev,
                         int32_t* accept_len_dev, int32_t* next_token_dev, float* alpha_out_dev,
                         void* stream);

/*
 * Greedy verification of one round (Sec. 2.1.3, greedy decoding): candidate x_i is accepted
 * only if it equals the target's own choice argmax p_i (lowest index among equal maxima); the
 * scan stops at the first mismatch; next_token is the target's choice at that position, the
 * bonus row's after a full match.  Only the target rows are read.  The adaptive state is
 * neither read nor written.
 *   target_logits_dev [B,Kmax+1,V], draft_tokens_dev [B,Kmax], draft_len_dev [B] (NULL: Kmax)
 *   argmax_out_dev    [B,Kmax+1] nullable: the target's choices of rows 0..K_t
 * A target row with NaN or without a finite logit has no choice (-1): it matches nothing and
 * sets ADASD_STATUS_NAN.
 */
int adasd_greedy_verify(adasd_ctx* ctx, const void* target_logits_dev, int64_t t_seq_stride,
                        int64_t t_row_stride, const int32_t* draft_tokens_dev,
                        const int32_t* draft_len_dev, int32_t* accept_len_dev, int32_t* next_token_dev,
                        int32_t* argmax_out_dev, void* stream);

/*
 * Feedback of the generation component on its own (Sec. 5, ablation variant "Gen-Only": the
 * entropy stop check of Sec. 4.3 with vanilla verification).  Where vanilla verification
 * rejected a candidate (accept_len[b] < draft_len[b]) the entropy H(q) of that candidate, as
 * adasd_draft_entropy reported it, joins L_E^R and T_G[b] becomes the mean of the list; the
 * distance lists are not touched.  H_draft_dev [B,Kmax]: entropy of draft step i of sequence b.
 *
 * The paper's variants as sequences of calls:
 *   AdaSD        draft_entropy (stop on H > T_G) ... ; verify (ADASD_FUSE_UPDATE)
 *   Gen-Only     draft_entropy (stop on H > T_G) ... ; vanilla_verify ; gen_only_update
 *   Verify-Only  five draft_entropy calls, stop flags ignored ; verify (ADASD_FUSE_UPDATE)
 *   Vanilla      five draft_entropy calls ; vanilla_verify
 *   greedy       draft_entropy with u_dev = NULL (argmax q) ... ; greedy_verify
 */
int adasd_gen_only_update(adasd_ctx* ctx, const float* H_draft_dev, const int32_t* draft_len_dev,
                          const int32_t* accept_len_dev, void* stream);

/*
 * The adjusted distribution tokens are sampled from (Sec. 2.1.1: temperature scaling, top-k
 * sampling, top-p sampling).  Host-side setting of the context; every later
 * adasd_draft_entropy, adasd_verify and adasd_vanilla_verify on it works on the adjusted
 * rows: entropies, log-sum-exps, JS distances, accept ratios and every sampled token are
 * those of softmax(adjust(z)), for draft and target rows alike.
 *
 *   temperature   > 0; logits are divided by it.
 *   top_k         the k most probable tokens stay, tokens whose logit equals the k-th largest
 *                 stay with it (ties are never split); <= 0 or >= V: off.
 *   top_p         in (0, 1]; of what top-k left, a token stays iff the tokens strictly more
 *                 probable than it hold less than top_p of the mass (the smallest
 *                 most-probable set whose mass reaches top_p, ties at its edge included);
 *                 1: off.
 * Applied in that order.  (1, 0, 1) is the default and changes nothing, bit for bit.
 * Greedy selection (adasd_greedy_verify, argmax drafting) is unaffected: the most probable
 * token always stays.  adasd_vanilla_verify_static takes no context and applies none.
 *
 * Cost: temperature is a constant in the row passes.  With top-k or top-p on, each call first
 * finds one cutoff logit per row (row_cutoff_kernel: one more read of the rows), and the row
 * passes read logits below it as -inf.  Rows without a usable maximum are not cut and are
 * reported by the row pass (ADASD_STATUS_NAN).
 * The values are read when a call is issued (or captured in a graph), not when it runs.
 * Returns ADASD_ERR_SHAPE for a temperature that is not a positive finite number or a top_p
 * outside (0, 1].
 */
int adasd_set_warpers(adasd_ctx* ctx, float temperature, int32_t top_k, float top_p);

/*
 * Vanilla verification for callers that must not allocate device memory.  (The paper has
 * no counterpart: this is a packaging variant of adasd_vanilla_verify, same inputs, same
 * outputs, same arithmetic.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving engine
 * that has handed the whole GPU to its own memory pool, in a plugin or callback that is
 * forbidden to touch the allocator, or in a process that may not grow its footprint after
 * start-up.  Such a caller cannot use adasd_create(), which allocates the context's
 * state.  This entry point needs no context: the few words of scratch the kernel uses
 * between its blocks (per-candidate accept flags, per-position candidate tokens, per-
 * sequence arrival counters, a status word) live in a fixed array inside the library
 * image.  It calls neither cudaMalloc nor cudaFree nor any routine that does.
 *
 *   B, V, Kmax, dtype   as in adasd_config; B <= ADASD_STATIC_MAX_B and
 *                       B * (Kmax + 1) <= ADASD_STATIC_MAX_POSITIONS, else
 *                       ADASD_ERR_CAPACITY is returned and nothing is launched
 *   logits, strides, draft_tokens_dev, draft_len_dev, u_accept_dev, u_resample_dev,
 *   accept_len_dev, next_token_dev, alpha_out_dev      as in adasd_vanilla_verify
 *   status_out_dev      nullable device word: receives the ADASD_STATUS_* bits of this
 *                       call (cleared first)
 *
 * The device used is the calling thread's current device.  The first call on each device
 * looks up the device address of the scratch array (one cudaGetSymbolAddress, no
 * allocation); make that first call outside any stream capture.  Every GPU that loads the
 * library holds the array (about 132 KB) until the process exits.  All calls on a device
 * share it, and it keeps the previous call's contents: each call clears the counters and
 * the status word it needs on `stream` before its kernel.  Two calls that overlap on the
 * same GPU (different streams, different threads) race on the array and give wrong
 * results: serialise them on one stream.
 */
int adasd_vanilla_verify_static(int32_t B, int32_t V, int32_t Kmax, int32_t dtype,
                                const void* draft_logits_dev, const void* target_logits_dev,
                                int64_t d_seq_stride, int64_t d_row_stride, int64_t t_seq_stride,
                                int64_t t_row_stride, const int32_t* draft_tokens_dev,
                                const int32_t* draft_len_dev, const float* u_accept_dev,
                                const float* u_resample_dev, int32_t* accept_len_dev,
                                int32_t* next_token_dev, float* alpha_out_dev,
                                uint32_t* status_out_dev, void* stream);

/* Copies T_G and the list sizes |L_E^R|, |L_D^A|, |L_D^R| to caller arrays [B] (each nullable). */
int adasd_get_thresholds(adasd_ctx* ctx, float* T_G_dev, int32_t* nE_dev, int32_t* nA_dev,
                         int32_t* nR_dev, void* stream);

/*
 * Checkpoint of ONE sequence's adaptive state to / from HOST memory (a whole context is
 * saved sequence by sequence; per-sequence is what resuming or migrating a single request
 * needs).  Layout:
 *   int32 nE, nA, nR, pad; float T_G, pad; then nE + nA + nR floats (L_E^R, L_D^A, L_D^R).
 * Export: call with host_buf = NULL to get the size in *bytes.  Both synchronise the
 * device.  Import recomputes the running sums from the lists.
 */
int adasd_state_export(adasd_ctx* ctx, int32_t seq, void* host_buf, size_t* bytes);
int adasd_state_import(adasd_ctx* ctx, int32_t seq, const void* host_buf, size_t bytes);

/*
 * Self-test of the failure detection of the device code (the paper has no counterpart).  Every
 * wait in the kernels is bounded: a warp whose wait runs out sets ADASD_STATUS_TIMEOUT, stops
 * waiting and copying, publishes NaN / -1 for what it could not compute and lets the kernel
 * end.  This call runs one draft step (as adasd_draft_entropy with no active mask) in which
 * one warp working on row `row` never asks for its first chunk of the row and waits for it
 * only briefly: the wait runs out with nothing in flight.  Afterwards adasd_status() reports
 * ADASD_STATUS_TIMEOUT, H_out[row] is NaN and token_out[row] is -1, every other row is as
 * usual, and the context is fit for further calls.  Needs the streaming draft kernel (bf16
 * rows of a multiple of 8 logits, V >= 8192, 16-byte aligned), else ADASD_ERR_SHAPE.
 */
int adasd_selftest_expired_wait(adasd_ctx* ctx, const void* logits_dev, int64_t row_stride, int32_t row,
                                const float* u_dev, float* H_out_dev, int32_t* token_out_dev, void* stream);

/* Reads and clears the sticky status word (ADASD_STATUS_* bits).  Synchronises. */
int adasd_status(adasd_ctx* ctx, uint32_t* status_out);

const char* adasd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ADASD_H */
