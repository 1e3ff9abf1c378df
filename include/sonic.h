/*
 * sonic — fused LLM sampling and speculative verification on one B200 (sm_100a).
 *
 * C ABI of the library.  Every array pointer in the argument structs is a
 * DEVICE pointer owned by the caller; the library reads the inputs, writes the
 * outputs and the workspace, allocates nothing and never synchronises with the
 * host, so each call can be captured in a CUDA Graph (pointers are baked at
 * capture, contents may change between replays).  The argument structs
 * themselves are HOST memory and are only read during the call.
 *
 * All functions return SONIC_OK (0) or a negative error code; the text of the
 * last error of the calling thread is available from sonic_last_error().
 *
 * Mode bits of a request (paper Section 3.5, bit-level indicator table):
 *   0x001 grammar bit-mask      0x002 repetition penalty   0x004 frequency penalty
 *   0x008 presence penalty      0x010 logit bias           0x020 temperature
 *   0x040 greedy selection      0x080 top-k                0x100 top-p
 *   0x200 min-p                 0x400 top-k log-probabilities (reserved, ignored)
 * A parameter array may be NULL when no request sets the bit that reads it.
 * Parameter domains: tau > 0 finite; k >= 0 (0: no top-k); p, theta in (0, 1] (p = 1: no top-p truncation); rep_penalty alpha > 0 finite (the paper states
 * alpha >= 1), freq_penalty and pres_penalty finite (the paper states >= 0); a set bit with a parameter outside
 * its domain gives SONIC_FLAG_BADPARAM for that row (greedy rows too, for tau and the penalty coefficients).
 * Bias values and logits must not be NaN or +inf (a precondition, not checked; -inf logits are masked entries).
 */
#ifndef SONIC_H
#define SONIC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SONIC_OK           0
#define SONIC_EINVAL      -1   /* null / misaligned pointer, bad struct size, bad scalar argument */
#define SONIC_ESHAPE      -2   /* unsupported B, V, K, k, dtype or stride */
#define SONIC_EWORKSPACE  -3   /* workspace too small or not initialised for this size */
#define SONIC_ECUDA       -4   /* a CUDA runtime call or launch failed */

#define SONIC_DTYPE_F32    0
#define SONIC_DTYPE_BF16   1

#define SONIC_MAX_VOCAB    262144   /* largest supported V (2^18) */
#define SONIC_MAX_TOPK     4096     /* largest k of sonic_topk */

/* per-row output flags */
#define SONIC_FLAG_NO_TOKEN  0x1u   /* no finite processed logit: token is -1 */
#define SONIC_FLAG_BADPARAM  0x2u   /* tau <= 0, p or theta outside (0,1], k < 0, list id out of range: token is -1 */
#define SONIC_FLAG_FALLBACK  0x4u   /* diagnostic: the row was finished by the cluster kernel (top-k beyond the streaming
                                       path, or a row no other path could finish) */
#define SONIC_FLAG_DENSE     0x8u   /* diagnostic: top-k off, the row was finished by the full-vocabulary histogram passes */
#define SONIC_FLAG_TIMEOUT   0x10u  /* a bounded wait inside the streaming kernel expired: token is -1 (see sonic_workspace_init) */

/* Bytes of workspace that serve every call over at most max_rows logit rows (B for sonic_sample / sonic_topk,
 * B*(K+1) for sonic_verify) of at most max_vocab entries each, and every sonic_topk call with k <= max_topk.  Pure
 * host arithmetic.  Per row: 1.3 KB of control words, 8 bytes per candidate slot (min(32768, V rounded up to 8192);
 * twice as many for sonic_topk with k > 2048), and for sampling and verification 4 bytes per vocabulary entry (the
 * processed logits of rows with top-k off as ordered keys) plus 58 KB of histogram and lists. */
size_t sonic_workspace_bytes(int max_rows, int max_vocab, int max_topk);

/* Zeroes the workspace header (the first 512 bytes: work counters and the sticky error word) once after allocation
 * (a memset enqueued on `stream`, a cudaStream_t passed as void*).  The kernels put the counters back to zero
 * at the end of every call and initialise every other word they read themselves, so replays need no
 * re-initialisation and one workspace serves calls of different shapes.  Two calls that use the same workspace
 * must not overlap on the device.
 *
 * Error word: 32-bit word 0 of the workspace is sticky; bit 0 is set when a bounded wait of the streaming kernel
 * (a tile copy that never completed) ran out.  Every row of such a call, and of later calls on that workspace,
 * reports SONIC_FLAG_TIMEOUT with token -1 until the workspace is initialised again with this function.
 *
 * Streams: a call's kernels are ordered on the caller's `stream` (everything enqueued before the call precedes
 * them, everything after follows them).  Per host thread and device the library keeps ONE internal non-blocking stream
 * and two events, created by this function or by the thread's first sampling call outside a stream capture:
 * sonic_sample / sonic_verify fork it from `stream` behind their first kernel and join it back before their last
 * one, so that rows with and without top-k are finished side by side.  Under stream capture the fork is captured
 * with the caller's stream (one graph, no dependency outside it).  Whenever the internal stream cannot be used -
 * it does not exist yet and the caller is capturing, or it still belongs to another capture that is open - the
 * call runs all of its kernels on `stream` alone: same results, about a third slower on mixed batches.  So: call
 * this function (or one eager sampling call) on a thread before that thread captures, and do not keep two captures
 * open on one thread at the same time if both should get the two-stream schedule.  sonic_topk uses no other stream. */
int sonic_workspace_init(void *workspace, size_t bytes, void *stream);

/*
 * Singular mode (standard decode or one draft step): one token per row.
 * Paper: Algorithm "Stage 1" (prologue: grammar mask -> repetition/frequency/presence
 * penalties -> logit bias -> temperature, then per-tile candidate selection),
 * Algorithm "Stage 2" (cross-tile merge, TopK -> TopP -> MinP epilogue, token
 * selection), Appendix "Detailed Formulation" for each operator.  Ties go to the
 * lowest index (Section 3.4).  The draw is one Philox4x32-10 uniform per row,
 * key = seed[b], counter = (offset[b], b, 0), inverted through the CDF of the
 * truncated renormalised distribution taken in vocabulary-index order.
 */
typedef struct sonic_sample_args {
    uint32_t struct_size;            /* sizeof(sonic_sample_args) */
    int32_t  B, V;                   /* rows, vocabulary size (1 <= V <= SONIC_MAX_VOCAB) */
    const void *logits;              /* [B, row_stride] fp32 or bf16; rows 16-byte aligned */
    int32_t  dtype;                  /* SONIC_DTYPE_* */
    int64_t  row_stride;             /* elements; multiple of 4 (fp32) or 8 (bf16), >= V; the buffer holds B*row_stride elements */
    const uint32_t *mode;            /* [B] mode bits */
    const uint32_t *bitmask;         /* [B, bitmask_stride] words; bit (i&31) of word (i>>5) set = token i allowed */
    int64_t  bitmask_stride;         /* words, >= ceil(V/32) */
    const float *temperature;        /* [B] tau > 0 */
    const int32_t *top_k;            /* [B] k >= 0 (0 = off) */
    const float *top_p;              /* [B] p in (0,1] */
    const float *min_p;              /* [B] theta in (0,1] */
    const float *rep_penalty;        /* [B] alpha */
    const float *freq_penalty;       /* [B] beta */
    const float *pres_penalty;       /* [B] gamma */
    const int32_t *hist_ids;         /* [B, hist_stride] distinct token ids seen so far */
    const int32_t *hist_counts;      /* [B, hist_stride] their occurrence counts (entries with count <= 0 are skipped) */
    const int32_t *hist_len;         /* [B] valid entries per row */
    int32_t  hist_stride;
    const int32_t *bias_ids;         /* [B, bias_stride] distinct token ids */
    const float *bias_vals;          /* [B, bias_stride] finite additive biases */
    const int32_t *bias_len;         /* [B] */
    int32_t  bias_stride;
    const uint64_t *seed;            /* [B] Philox key */
    const uint64_t *offset;          /* [B] Philox counter (position) */
    int32_t *out_token;              /* [B] selected token, -1 if none */
    float   *out_prob;               /* [B] probability of the selected token under the final distribution (1 for greedy) */
    uint32_t *out_flags;             /* [B] SONIC_FLAG_* */
    int32_t *out_support;            /* [B] or NULL: size of the final support (1 for greedy) */
} sonic_sample_args;

int sonic_sample(const sonic_sample_args *args, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Multistep mode (speculative verification).  Paper: Section "Speculative
 * Verification" (background and appendix): draft token d_l is accepted iff
 * u * q(d_l) <= p(d_l); at the first rejection a token is drawn from
 * normalise(max(0, p - q)); if all K drafts are accepted a bonus token is drawn
 * from the last target row.  p is the target distribution after the full
 * pipeline with the request's parameters, q the draft distribution as passed
 * in.  Greedy requests accept while the draft equals the argmax.  Position l of
 * request b uses Philox counter (offset[b] + l, b, 0): word 0 for the accept
 * test, word 1 for the draw.
 */
typedef struct sonic_verify_args {
    uint32_t struct_size;            /* sizeof(sonic_verify_args) */
    int32_t  K;                      /* draft length, 0 <= K <= 15 */
    sonic_sample_args s;             /* per-request arrays are [B]; logits is [B, K+1, V] with row_stride between
                                        consecutive positions (row index b*(K+1)+l); bitmask, if used, is per logit
                                        row [B*(K+1), bitmask_stride]; out_token/out_prob/out_support are ignored */
    const int32_t *draft_tokens;     /* [B, K] */
    const float *draft_probs;        /* [B, K, V] fp32, dense draft distribution q */
    int32_t *out_tokens;             /* [B, K+1]: accepted drafts, then the correction or bonus token, then -1 */
    int32_t *out_accept_len;         /* [B] in 0..K */
    float   *out_p_draft;            /* [B, K] or NULL: p_l(d_l) */
} sonic_verify_args;

int sonic_verify(const sonic_verify_args *args, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Standalone hierarchical top-k (the selection primitive of Section 3.4 on its
 * own): the k largest logits of every row, sorted descending, ties to the
 * lowest index.  1 <= k <= min(V, SONIC_MAX_TOPK).  out_vals/out_idx are [B, k].
 */
int sonic_topk(const void *logits, int dtype, int B, int V, int64_t row_stride, int k,
               float *out_vals, int32_t *out_idx, void *workspace, size_t workspace_bytes, void *stream);

/*
 * sonic_topk without a caller-provided workspace and without any allocation.
 * (The paper has no counterpart: this entry point exists for callers of this library
 * that are not allowed to allocate device memory -- plugins handed a fixed memory
 * budget by their host engine, processes whose device memory pool was sized once at
 * start-up, and latency-critical serving loops in which a cudaMalloc would synchronise
 * the whole device.)
 *
 * Same inputs, outputs and results as sonic_topk, for at most SONIC_STATIC_MAX_ROWS rows
 * per call; larger B is rejected with SONIC_ESHAPE.  The scratch memory is a fixed array
 * of about 4.2 MB inside the library image (SONIC_STATIC_MAX_ROWS rows of candidate
 * slots and control words); every GPU that loads the library holds it until the process
 * exits.  The function calls no cudaMalloc, cudaFree or other allocating routine, and
 * all of its kernels go to `stream`.
 *
 * The first call on each device resolves the array's device address and configures the
 * kernels; that first call should come before any stream capture is begun.  All calls on a device share
 * the one array, which keeps the contents of the previous call: each call first clears
 * the control words it needs at zero (a memset enqueued on `stream`), and two calls that
 * overlap on the device (different streams, or graphs replayed concurrently) race on it.
 */
#define SONIC_STATIC_MAX_ROWS 8
int sonic_topk_static(const void *logits, int dtype, int B, int V, int64_t row_stride, int k,
                      float *out_vals, int32_t *out_idx, void *stream);

/* Text of the calling thread's last error ("" if none).  Never NULL. */
const char *sonic_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SONIC_H */
