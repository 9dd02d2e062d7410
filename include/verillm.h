/*
 * verillm.h - C ABI of the B200 (sm_100a) verifier-prefill library.
 *
 * The library recomputes a served sequence [prompt || output] of a Llama-style decoder in one
 * causal pass, compares the per-layer hidden states at the checked positions against the
 * states the prover committed, and emits per-position and per-sequence accept/reject verdicts
 * (VeriLLM, "Full-Sequence Prefill for Parallel Verification", Eq. 1; "Verification Scheme";
 * "Comparison, Sampling, and On-Chain Adjudication").
 *
 * Conventions
 *  - Every pointer says whether it is HOST or DEVICE memory.  The caller owns every buffer it
 *    passes and the CUDA stream; the library owns the model handle, its copies of the weights
 *    and one workspace sized at load time from max_tokens / max_checks / max_batch.
 *  - All calls enqueue work on the given stream and return without synchronising unless stated;
 *    results are valid once the caller has synchronised the stream.  Host arrays passed to a call
 *    may be reused as soon as the call returns, whether they are pageable or pinned: the library
 *    copies them into memory of its own before it queues the transfer.
 *  - A handle serves one call at a time: its workspace, staging arrays and counters are shared by
 *    all calls, so calls on one handle must not overlap, neither from several threads nor on several
 *    streams.  Different handles are independent.
 *  - The projections over more than 128 rows split the last, partly filled round of output tiles
 *    along K over otherwise idle SM pairs, and a later part waits for the earlier part of the same
 *    tile, which runs on another SM pair of the same launch.  The parts are dealt so that a part
 *    never waits for a pair with a higher index, and the wait is bounded: if the GPU is shared with
 *    other kernels to the point that the producing pair is not scheduled within about two seconds,
 *    the call ends with VERILLM_DEV_WAIT_TIMEOUT in the status word instead of hanging.
 *  - Return value: 0 on success, a negative VERILLM_E_* code otherwise; nothing is launched when
 *    an argument is rejected.  Problems only the device can see (a token id >= vocab) clamp the
 *    offending index, set *report.status to a positive VERILLM_DEV_* code and force a reject.
 *  - Matrices are row-major; every projection weight is [out_features][in_features] bf16.
 *  - Model conventions: pre-norm blocks, RMSNorm (x * rsqrt(mean x^2 + eps) * gain), rotary
 *    embedding with half-split pairing (element i rotates with i + head_dim/2, angle
 *    pos * rope_base^(-2i/head_dim)), grouped-query causal attention scaled by 1/sqrt(head_dim)
 *    (query head g reads key/value head g * n_kv_heads / n_heads), SwiGLU feed-forward
 *    (silu(x W_gate^T) * (x W_up^T)) W_down^T, no biases.
 *  - The "hidden state of layer l" is the residual stream after block l (l = 0 .. n_layers-1),
 *    one d_model vector per position, before the final norm.
 */
#ifndef VERILLM_H
#define VERILLM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VERILLM_NSTAT 16
/* order of the VERILLM_NSTAT floats reported per (check slot, layer) */
enum {
    VERILLM_STAT_REL_L2 = 0,      /* ||h - c||_2 / max(||c||_2, 1e-30) */
    VERILLM_STAT_MAX_ABS = 1,     /* max |h - c| */
    VERILLM_STAT_MAE = 2,         /* phi: mean |h - c| */
    VERILLM_STAT_MEAN_SIGNED = 3, /* e: mean (h - c) */
    VERILLM_STAT_P_E = 4,         /* fraction of exponent-field mismatches */
    VERILLM_STAT_P_M = 5,         /* among mismatches: fraction with |mantissa field difference| > e_m (1 if none) */
    VERILLM_STAT_P_W = 6,         /* among matches: fraction with significand difference <= e_w * 2^mantissa_bits (1 if none) */
    VERILLM_STAT_Q_SMALL = 7,     /* fraction with |h - c| <= 1e-5 */
    VERILLM_STAT_Z_LARGE = 8,     /* fraction with |h - c| > tau_large */
    VERILLM_STAT_N_EXP_MISMATCH = 9,
    VERILLM_STAT_N_MANT_LARGE = 10,
    VERILLM_STAT_N_MANT_SMALL = 11,
    VERILLM_STAT_N_EXACT = 12,    /* bit-identical after rounding to the commit dtype */
    VERILLM_STAT_N_NONFINITE = 13,
    VERILLM_STAT_L2_DELTA = 14,
    VERILLM_STAT_L2_REF = 15
};

enum {
    VERILLM_OK = 0,
    VERILLM_E_INVAL = -1, /* null pointer, bad enum, negative size */
    VERILLM_E_SHAPE = -2, /* shape the kernels do not support, or larger than the handle was sized for */
    VERILLM_E_RANGE = -3, /* sequence index / position / cu_seqlens out of range */
    VERILLM_E_NOMEM = -4, /* device allocation failed */
    VERILLM_E_CUDA = -5,  /* a CUDA call failed */
    VERILLM_E_ARCH = -6   /* current device is not compute capability 10.x */
};

/* positive codes written to the device status word */
enum {
    VERILLM_DEV_OK = 0,
    VERILLM_DEV_TOKEN_RANGE = 1, /* token id outside [0, vocab): clamped */
    VERILLM_DEV_WAIT_TIMEOUT = 2 /* a pipeline wait inside a kernel gave up; results are invalid */
};

enum { VERILLM_BF16 = 0, VERILLM_F32 = 1 };

#define VERILLM_TOL_BIT_AWARE 1u /* enable the P_e / P_m / P_w / e tests in the verdict */

typedef struct verillm_model verillm_model; /* opaque */

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float rope_base, rms_eps;
    int32_t max_tokens; /* largest total number of tokens (all sequences of a call together) */
    int32_t max_checks; /* largest number of checked positions in one call */
    int32_t max_batch;  /* largest number of sequences in one call */
} verillm_config;

/* Weights of one layer; all bf16, HOST or DEVICE as the enclosing call says.
 * attn_norm, ffn_norm: [d_model]; wq: [n_heads*head_dim][d_model]; wk, wv: [n_kv_heads*head_dim][d_model];
 * wo: [d_model][n_heads*head_dim]; w_gate, w_up: [d_ffn][d_model]; w_down: [d_model][d_ffn]. */
typedef struct {
    const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
} verillm_layer_weights;

typedef struct {
    const void *embed;      /* [vocab][d_model] bf16 */
    const void *final_norm; /* [d_model] bf16 (kept for the tail check; unused by the hidden-state path) */
    const verillm_layer_weights *layers; /* HOST array [n_layers], or NULL to load layers later one by one */
    int32_t on_device;      /* 1: the weight pointers are DEVICE memory, 0: HOST memory */
} verillm_weights;

/* Tolerances of the verdict (Comparison paragraph: b = 1[T_v <= tau]; bit-aware statistical comparison;
 * offline battery T_off).  A float test whose threshold is <= 0 is disabled; z_large_max < 0 disables it.
 * Float thresholds accept at equality; the bit-aware tests use the paper's strict directions
 * (P_e < pe_max, P_m > pm_min, P_w > pw_min, |e| <= e_abs_max) and run only with VERILLM_TOL_BIT_AWARE. */
typedef struct {
    float rel_l2, max_abs, mae;
    float pe_max, pm_min, pw_min, e_abs_max;
    float e_w;     /* relative significand step counted as "small" inside an exponent match */
    int32_t e_m;   /* mantissa-field distance above which an exponent mismatch counts as "large" */
    float tau_large, z_large_max, q_small_min;
    uint32_t flags;
} verillm_tol;

/* Caller-allocated DEVICE outputs.  hidden_out may be NULL. */
typedef struct {
    float *stats;             /* [n_check][n_layers][VERILLM_NSTAT] */
    uint8_t *pos_ok;          /* [n_check] 1 = accept */
    int32_t *first_bad_layer; /* [n_check] smallest failing layer, -1 if none */
    uint8_t *seq_ok;          /* [batch] 1 = every checked position of the sequence accepted (1 if none checked) */
    float *seq_score;         /* [batch] T_v = mean over the sequence's checked positions and layers of MAE (0 if none) */
    float *hidden_out;        /* optional [n_layers][n_check][d_model]: the recomputed states at the checked positions */
    int32_t *status;          /* one word, VERILLM_DEV_*; the library zeroes it at the start of the call */
} verillm_report;

/* Fills *tol with the defaults: rel_l2 = 5e-2 enabled, every other float test disabled, the paper's
 * off-chain bit-aware thresholds (P_e < 0.05, P_m > 0.75, P_w > 0.80, |e| <= 0.01, e_w = 1e-2, e_m = 7)
 * present but not enabled. */
void verillm_default_tol(verillm_tol *tol);

/* Creates a handle on the current device: allocates the weight copies (re-laid out for the kernels:
 * q/k/v rows concatenated, gate/up rows interleaved in blocks of 128) and the workspace, builds the
 * rotary table and the TMA descriptors.  weights->layers may be NULL (or the whole of `weights`), in
 * which case layers are supplied afterwards with verillm_load_layer.  Synchronises the device.
 * Errors: E_INVAL, E_SHAPE (needs head_dim in {64,128}, d_model % 64 == 0, d_ffn % 128 == 0,
 * n_heads % n_kv_heads == 0), E_ARCH, E_NOMEM, E_CUDA.  (S_{i+1} = F_i(S_i; W_i): the W_i.) */
int verillm_load_weights(const verillm_config *cfg, const verillm_weights *weights, verillm_model **out);

/* Copies one layer's weights into the handle (HOST or DEVICE source per on_device).  Synchronous.
 * The source buffers can be released when the call returns, so a model larger than half the
 * device memory can be handed over layer by layer. */
int verillm_load_layer(verillm_model *model, int32_t layer, const verillm_layer_weights *w, int32_t on_device);

/* Same for the embedding table and the final norm gain. */
int verillm_load_globals(verillm_model *model, const void *embed, const void *final_norm, int32_t on_device);

/* The verifier: one causal pass over the packed batch, fused gather-and-compare at the checked
 * positions, verdict (Eq. 1; Prefill Computation; Comparison and On-Chain Commitment).
 *  tokens           DEVICE int32 [cu_seqlens[batch]], sequences packed back to back (prompt || output)
 *  cu_seqlens       HOST int32 [batch+1], cu_seqlens[0] = 0, non-decreasing
 *  committed_hidden DEVICE [n_layers][n_check][d_model] in commit_dtype: the prover's states S
 *  check_seq/pos    HOST int32 [n_check]: sequence index and 0-based position inside it (input-token
 *                   index; prompt positions are allowed); any order, duplicates allowed
 * Allocates nothing.  Errors: E_INVAL, E_SHAPE (more tokens / checks / sequences than the handle was
 * sized for), E_RANGE, E_CUDA. */
int verillm_verify_prefill(verillm_model *model, const int32_t *tokens, const int32_t *cu_seqlens, int32_t batch,
                           const void *committed_hidden, int32_t commit_dtype, const int32_t *check_seq,
                           const int32_t *check_pos, int32_t n_check, const verillm_tol *tol,
                           const verillm_report *report, void *cuda_stream);

/* Segment-local verification (Verification Scheme, segment-local recompute; T_verify ~ T_prefill / L): blocks
 * layer_begin .. layer_end-1 are recomputed for all positions from the recorded states entering block
 * layer_begin, and compared at the checked positions with the committed outputs of those blocks.
 *  input_states     DEVICE [cu_seqlens[batch]][d_model] in input_dtype (BF16 / F32): the residual stream entering
 *                   block layer_begin at every position (the output of block layer_begin-1, or the embeddings)
 *  committed_hidden DEVICE [layer_end - layer_begin][n_check][d_model]
 * The report arrays have layer_end - layer_begin layers and their layer indices count from layer_begin; all else
 * as verillm_verify_prefill.  Extra errors: E_RANGE for an empty or out-of-range layer interval.
 * The recorded states come from another party: an entry that is NaN, infinite or beyond 1e15 in magnitude is
 * read as 0 and its sequence is rejected as a whole (seq_ok = 0, every checked position of it pos_ok = 0 with
 * first_bad_layer = 0), as an exact recomputation would: one such entry makes every state of its sequence
 * non-finite.  The other sequences of the batch are unaffected. */
int verillm_verify_segment(verillm_model *model, const void *input_states, int32_t input_dtype, int32_t layer_begin,
                           int32_t layer_end, const int32_t *cu_seqlens, int32_t batch, const void *committed_hidden,
                           int32_t commit_dtype, const int32_t *check_seq, const int32_t *check_pos, int32_t n_check,
                           const verillm_tol *tol, const verillm_report *report, void *cuda_stream);

/* The prover's side, for generating traces: teacher-forced token-by-token decode with a bf16
 * key/value cache (the decode loop of the Inference Scheme), after an optional parallel pass over the
 * first n_prefill tokens of every sequence.  Writes the layer-output states at the requested
 * positions to committed_out (DEVICE, [n_layers][n_check][d_model], commit_dtype).  The first call
 * allocates the cache and a staging buffer inside the handle; the call synchronises the stream.
 * status: optional DEVICE word as in verillm_report. */
int verillm_decode_commit(verillm_model *model, const int32_t *tokens, const int32_t *cu_seqlens, int32_t batch,
                          int32_t n_prefill, const int32_t *check_seq, const int32_t *check_pos, int32_t n_check,
                          void *committed_out, int32_t commit_dtype, int32_t *status, void *cuda_stream);

/* Tail token check (the TokenMatch equation; token-state cross-check of the forged-output analysis): the
 * last-layer states at the checked positions go through the final RMSNorm and the output
 * head, and the arg-max token of each row is compared with the token the prover claims to have emitted there.
 *  verillm_load_lm_head: output head [vocab][d_model] bf16 (HOST or DEVICE per on_device); the first call also
 *                        allocates the scratch of the check inside the handle.  vocab % 32 == 0 (else E_SHAPE).
 *  last_hidden  DEVICE float32 [n_check][d_model]: e.g. the last layer of verify_prefill's hidden_out
 *  claimed      HOST int32 [n_check]: the next token the prover reported for that position
 *  argmax_out   DEVICE int32 [n_check]; match_out DEVICE uint8 [n_check] (1 = equal);
 *  margin_out   DEVICE float [n_check]: best logit minus runner-up (a small margin marks a row whose arg-max
 *               rounding noise may flip).  Ties resolve to the lowest token id.
 * Allocates nothing per call.  Errors: E_INVAL (also when no output head was loaded), E_SHAPE (n_check >
 * max_checks). */
int verillm_load_lm_head(verillm_model *model, const void *lm_head, int32_t on_device);
int verillm_token_match(verillm_model *model, const float *last_hidden, const int32_t *claimed, int32_t n_check,
                        int32_t *argmax_out, uint8_t *match_out, float *margin_out, void *cuda_stream);

/* Comparison and verdict alone, on states the caller already holds (Delta = S_hat - S, phi, Psi, b):
 *  hidden    DEVICE float32 [n_layers][n_check][d_model]
 *  committed DEVICE [n_layers][n_check][d_model] in commit_dtype
 *  check_seq HOST int32 [n_check]
 * report->hidden_out is ignored.  Scratch for the partial sums is taken from the stream-ordered
 * allocator (cudaMallocAsync) and returned to it. */
int verillm_compare(const float *hidden, const void *committed, int32_t commit_dtype, int32_t n_layers,
                    int32_t n_check, int32_t d_model, const int32_t *check_seq, int32_t batch,
                    const verillm_tol *tol, const verillm_report *report, void *cuda_stream);

/* Same computation, arguments and results as verillm_compare, for callers that must not allocate device
 * memory while they run: code inside a latency-critical serving loop where cudaMalloc would synchronise
 * the device, processes that handed their whole memory budget to a pool at start-up, and hosts that run
 * under an allocator they cannot re-enter.  (The paper has no counterpart; this is a packaging variant.)
 * Its scratch (the partial sums and the slot-to-sequence map) is a fixed array of about 3.3 MB inside the
 * library, held by every GPU that loads the library until the process exits.  Limits: n_check <= 65536
 * and n_layers * n_check <= 65536, otherwise VERILLM_E_SHAPE and nothing is launched.  The call makes no
 * cudaMalloc / cudaFree and uses no allocating library routine.  The first call on each device looks up
 * the array's device address (cudaGetSymbolAddress); make that first call outside any stream capture.
 * All calls share the one array, which keeps whatever the previous call left there (the part a call reads
 * is cleared first): two calls that overlap on the GPU, on different streams or from different threads,
 * race on it and must be serialised by the caller. */
int verillm_compare_noalloc(const float *hidden, const void *committed, int32_t commit_dtype, int32_t n_layers,
                            int32_t n_check, int32_t d_model, const int32_t *check_seq, int32_t batch,
                            const verillm_tol *tol, const verillm_report *report, void *cuda_stream);

/* Relaxed spot check on sampled scalar entries (on-chain value matching: Delta_j = |v_j - V_j| <= eps,
 * agreement rate p_hat = (1/n) sum 1[Delta_j <= eps], positive verdict iff p_hat >= theta).
 *  hidden      DEVICE float32 [n_rows][d_model]: the verifier's states (e.g. one layer of hidden_out)
 *  sample_row / sample_col  HOST int32 [n_samples]: the sampled entries; reference HOST float32 [n_samples]: V_j
 *  agree_out   DEVICE uint8 [n_samples]; p_hat_out DEVICE float [1]; verdict_out DEVICE uint8 [1]
 * The comparison is made in float32; a NaN never agrees.  Staging memory comes from the stream-ordered
 * allocator.  Errors: E_INVAL, E_RANGE (an index outside the matrix). */
int verillm_spot_check(const float *hidden, int32_t n_rows, int32_t d_model, const int32_t *sample_row,
                       const int32_t *sample_col, const float *reference, int32_t n_samples, float eps, float theta,
                       uint8_t *agree_out, float *p_hat_out, uint8_t *verdict_out, void *cuda_stream);

/* Threshold sensitivity of the offline tests (appendix Threshold Sensitivity Analysis: one threshold varies, the
 * others stay at their selected values, and the false-positive / false-negative rates are read off honest and
 * attack traces).  The tests of the verdict are applied to statistics reported by an earlier verify / compare call.
 *  stats      DEVICE float32 [n_cells][VERILLM_NSTAT]: one row per (position, layer) cell, as written to report.stats
 *  is_attack  DEVICE uint8 [n_cells]: 0 = the cell comes from an honest trace, non-zero = from an attack trace
 *  variants   HOST verillm_tol [n_variants], 1 <= n_variants <= 64 (E_SHAPE beyond): the tolerance sets to evaluate;
 *             tau_large, e_w and e_m are not used (they shaped the statistics when these were produced)
 *  counts_out DEVICE int32 [n_variants][4], zeroed by the call: honest accepted, honest rejected, attack accepted,
 *             attack rejected.  FPR = honest rejected / honest, FNR = attack accepted / attack.
 * A cell with a non-finite element is rejected by every variant.  Allocates nothing. */
int verillm_threshold_sweep(const float *stats, const uint8_t *is_attack, int32_t n_cells, const verillm_tol *variants,
                            int32_t n_variants, int32_t *counts_out, void *cuda_stream);

/* Merkle commitment of hidden states (Inference Scheme, commitment step: a tree over all scalar entries of the
 * serialised output tensor, whose root is submitted; canonical float32 leaves, SHA-256): one root per vector.
 *  states    DEVICE float32 [n_vec][d_model]; roots_out DEVICE uint8 [n_vec][32]
 * Leaf j = SHA-256(4 bytes of entry j, little-endian IEEE-754 float32); node = SHA-256(left || right); an odd
 * node at the end of a level is paired with itself; a single entry's leaf is its own root.
 * Errors: E_INVAL, E_SHAPE (d_model > 12800), E_ARCH, E_CUDA. */
int verillm_merkle_roots(const float *states, int32_t n_vec, int32_t d_model, uint8_t *roots_out, void *cuda_stream);

/* Single steps of the path, exposed for testing against the oracle.  All pointers DEVICE. */

/* C[M][N] = A[M][K] * B[N][K]^T, bf16 inputs, fp32 accumulation on the tensor cores; out_f32 selects a
 * float32 or bf16 C.  K % 8 == 0, N % 32 == 0. */
int verillm_op_gemm(const void *a, const void *b, void *c, int32_t m, int32_t n, int32_t k, int32_t out_f32,
                    int32_t *status, void *cuda_stream);
/* y[M][d] (bf16) = RMSNorm(x[M][d] float32; gain[d] bf16, eps). */
int verillm_op_rmsnorm(const float *x, const void *gain, void *y, int32_t m, int32_t d, float eps, void *cuda_stream);
/* Causal grouped-query attention over packed sequences.  qkv: bf16 [M][(n_heads + 2 n_kv_heads) head_dim]
 * (q heads, then k heads, then v heads; q and k already rotated); cu_seqlens: DEVICE int32 [batch+1];
 * out: bf16 [M][n_heads*head_dim]. */
int verillm_op_attention(const void *qkv, const int32_t *cu_seqlens, int32_t batch, int32_t max_seqlen, int32_t m,
                         int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void *out, void *cuda_stream);

/* Per-kernel timing of verify_prefill, for the roofline report (measurement aid, not part of the method).
 * While enabled, every verify_prefill call records one CUDA event after each launch on the caller's
 * stream; verillm_profile_read waits for the last call and returns, per class below, the summed
 * milliseconds and the number of launches (HOST arrays of VERILLM_PROF_NCLASS entries).  Enabling creates
 * the events once (not on the hot path); the events add a few microseconds per launch. */
enum {
    VERILLM_PROF_SETUP = 0,       /* index maps, slot lists, embedding gather */
    VERILLM_PROF_RMSNORM = 1,
    VERILLM_PROF_GEMM_QKV = 2,    /* + rotary epilogue */
    VERILLM_PROF_ATTENTION = 3,
    VERILLM_PROF_GEMM_O = 4,      /* + residual */
    VERILLM_PROF_GEMM_GATE_UP = 5,/* + SwiGLU */
    VERILLM_PROF_GEMM_DOWN = 6,   /* + residual + gather-and-compare */
    VERILLM_PROF_VERDICT = 7,
    VERILLM_PROF_NCLASS = 8
};
int verillm_profile_enable(verillm_model *model, int32_t on);
int verillm_profile_read(verillm_model *model, float *ms, int32_t *launches);

/* Exercise of the bounded wait that every pipeline of the library uses (failure detection; the paper has no
 * counterpart): one thread waits, for at most limit_cycles SM clock cycles (1 .. 2e9), on a barrier that nothing
 * signals, holding no copy in flight and no tensor memory.  *status (DEVICE) receives VERILLM_DEV_WAIT_TIMEOUT and
 * *gave_up (DEVICE, optional) 1; the context stays usable.  The waits inside the real kernels use the same code
 * with a limit of about two seconds. */
int verillm_selftest_wait_timeout(int64_t limit_cycles, int32_t *status, int32_t *gave_up, void *cuda_stream);

void verillm_free(verillm_model *model);
const char *verillm_strerror(int code);
/* Number of kernel launches the last verify_prefill call on this handle enqueued. */
int32_t verillm_last_launch_count(const verillm_model *model);

#ifdef __cplusplus
}
#endif
#endif /* VERILLM_H */
