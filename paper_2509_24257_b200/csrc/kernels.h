// Host-side launch interface between the C-ABI driver and the kernel translation units.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "compare.cuh"

namespace vl {

// ------------------------------------------------------------------ tensor-core GEMM
enum GemmEpilogue {
    EPI_STORE_BF16 = 0,      // C bf16
    EPI_STORE_F32 = 1,       // C fp32
    EPI_QKV_ROPE = 2,        // C bf16, rotary embedding on the q and k head columns
    EPI_RESID_ADD = 3,       // resid fp32 += acc (in place)
    EPI_SWIGLU = 4,          // tile holds 128 gate columns then 128 up columns: out bf16 = silu(g) * u
    EPI_RESID_ADD_COMPARE = 5,  // resid += acc, then gather-and-compare on the checked rows
    EPI_ARGMAX = 6              // no matrix output: per row and column tile (best value, its column, runner-up)
};

constexpr int kGemmBM = 128;
constexpr int kGemmBN = 256;
constexpr int kGemmBK = 64;

struct GemmParams {
    int M, N, K;
    void* out;  // bf16 / fp32 matrix or the fp32 residual stream
    int ldo;    // leading dimension of out, elements
    int group_m;  // tile-rows per band of the tile walk (0: default)
    int pair;     // 1: CTA-pair kernel (256 x 256 tile over two SMs; B map encoded with 128-row boxes)
    // EPI_QKV_ROPE
    const float2* rope_cs;    // [position][head_dim/2] (cos, sin)
    const int* pos_of_token;  // [M]
    int head_dim;
    int rope_cols;  // columns [0, rope_cols) hold heads that are rotated (q and k); the rest (v) are not
    // EPI_ARGMAX: `out` is float [M][n_tiles][4] = (best, column as int bits, runner-up, unused)
    // EPI_RESID_ADD_COMPARE (slabs of the current layer)
    const int* slot_first;  // [M] first check slot of a token row, -1 if none
    const int* slot_next;   // [n_check] next slot on the same row, -1 terminates
    int n_check;
    const void* committed;  // [n_check][N]
    float* partials;        // [n_check][n_tiles_n][kNPart]
    float* hidden_out;      // optional [n_check][N]
    CmpParams cmp;
    // RMSNorm folded into the neighbouring projections (x * rsqrt(mean x^2 + eps) * gain = rstd * (x * gain)).
    // Producer, EPI_RESID_ADD(_COMPARE) of the CTA-pair kernel: with norm_gain set, the epilogue also writes
    // xg_out[M][N] = bf16(residual * gain) and sumsq_out[M][n_tiles] = sum of squares of its row segment.
    const void* norm_gain;  // bf16 [N]
    void* xg_out;           // bf16 [M][N]
    float* sumsq_out;       // [M][ceil(N / 256)]
    // Consumer, EPI_QKV_ROPE and EPI_SWIGLU: with sumsq_in set, row m of the accumulator is multiplied by
    // rsqrt(sum_k sumsq_in[m][k] * norm_inv_d + norm_eps) (parts added in index order) before the epilogue proper.
    const float* sumsq_in;  // [M][n_parts]
    int n_parts;
    float norm_eps, norm_inv_d;
    // CTA-pair kernel with an additive epilogue: per-tile counters (one int per pair of SMs) that order the K
    // parts of the last, partly filled round of tiles; nullptr: no K split.  pairs_total is set by the launcher.
    int* split_flags;
    int pairs_total;
    // 1: launch with programmatic stream serialisation, so that the kernel's prologue (barriers, tensor memory,
    // descriptor prefetch) runs under the tail of the kernel before it in the stream; the kernel waits for that
    // kernel's completion before it reads or writes any global memory.
    int overlap_prologue;
    // 1: split_flags points at zeroed counters that belong to this launch alone (cleared before the chain of
    // kernels started), so the launcher queues no clearing between the kernels.
    int split_prezeroed;
    int* status;
};

// Maps are encoded for a box of 64 (K) x 128 rows (A) and 64 x 256 rows (B), 128-byte swizzle.
int make_tmap_bf16_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld_elems,
                      uint32_t box_rows);
cudaError_t launch_gemm(int epilogue, const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const GemmParams& p,
                        int num_sms, cudaStream_t stream);
cudaError_t gemm_init();  // raises the dynamic shared memory limit of every instantiation

// ------------------------------------------------------------------ attention
// tmap_q / tmap_kv are 64-column boxes of 128 / 64 rows over the same [tokens][(H+2KV)dh] buffer.
// overlap_prologue as in GemmParams; cu_seqlens_dev must not be written by the kernel just before in the stream.
cudaError_t launch_attention_tc(const CUtensorMap& tmap_q, const CUtensorMap& tmap_kv, const int* cu_seqlens_dev,
                                int batch, int max_seqlen, int n_heads, int n_kv_heads, int head_dim, void* out,
                                int* status, int num_sms, int overlap_prologue, cudaStream_t stream);
cudaError_t attention_tc_init();

// ------------------------------------------------------------------ small kernels
cudaError_t launch_token_maps(const int* cu_seqlens_dev, int batch, int n_tokens, int* pos_of_token,
                              int* seq_of_token, cudaStream_t stream);
cudaError_t launch_slot_lists(const int* tok_of_slot, int n_check, int n_tokens, int* slot_first, int* slot_next,
                              cudaStream_t stream);
cudaError_t launch_embed(const int* tokens, const void* table, int n_tokens, int d_model, int vocab, float* resid,
                         int* status, cudaStream_t stream);
// resid[n] (fp32) = recorded states in `dtype` (VERILLM_BF16 / VERILLM_F32): input of a segment-local pass.
// Values that are not finite or beyond 1e15 in magnitude become 0 and mark their sequence in seq_flags[batch].
cudaError_t launch_load_states(const void* src, int dtype, size_t n, int d_model, const int* seq_of_token,
                               int* seq_flags, float* resid, cudaStream_t stream);
cudaError_t launch_rmsnorm(const float* x, const void* gain, void* y, int rows, int d, float eps,
                           cudaStream_t stream);
// The producer half of a folded norm as a kernel of its own (first layer of a pass, small batches):
// y = bf16(x * gain), sumsq[row][0] = sum of squares of the row, sumsq[row][1 .. n_parts) = 0.
cudaError_t launch_prenorm(const float* x, const void* gain, void* y, float* sumsq, int n_parts, int rows, int d,
                           cudaStream_t stream);
cudaError_t launch_compare_rows(const float* hidden, const void* committed, int n_rows, int d, const CmpParams& cmp,
                                float* partials, cudaStream_t stream);
struct TolDev {
    float rel_l2, max_abs, mae, pe_max, pm_min, pw_min, e_abs_max, z_large_max, q_small_min;
    int bit_aware;
};
// partials: [n_layers][n_check][n_tiles][kNPart] -> stats [n_check][n_layers][NSTAT], pos_ok, first_bad_layer
// seq_flags (optional, with seq_of_slot): sequences whose input was malformed; all their positions are rejected.
cudaError_t launch_verdict(const float* partials, int n_layers, int n_check, int n_tiles, int d, const TolDev& tol,
                           const int* status, const int* seq_of_slot, const int* seq_flags, float* stats,
                           uint8_t* pos_ok, int* first_bad_layer, cudaStream_t stream);
// status / seq_flags (both optional): a non-zero status word rejects every sequence, a flag its sequence.
cudaError_t launch_seq_verdict(const float* stats, const uint8_t* pos_ok, const int* seq_of_slot, int n_check,
                               int n_layers, int batch, const int* status, const int* seq_flags, uint8_t* seq_ok,
                               float* seq_score, cudaStream_t stream);

// Threshold sensitivity: counts[v][4] += (honest accepted, honest rejected, attack accepted, attack rejected)
// over the cells' reported statistics [n_cells][VERILLM_NSTAT] for each of n_variants tolerance sets.
constexpr int kSweepMaxVariants = 64;
struct TolSet {
    TolDev v[kSweepMaxVariants];
};
cudaError_t launch_threshold_sweep(const float* stats, const uint8_t* is_attack, int n_cells, const TolSet& tols,
                                   int n_variants, int* counts, cudaStream_t stream);

// Tail token check: reduces the per-tile argmax records of the output-head product [rows][n_tiles][4] (fixed order,
// lowest column wins ties), compares with the claimed tokens.
cudaError_t launch_argmax_reduce(const float* records, int rows, int n_tiles, const int* claimed, int* argmax_out,
                                 uint8_t* match_out, float* margin_out, cudaStream_t stream);

// Sampled value matching: agree[j] = |hidden[row_j][col_j] - ref_j| <= eps; p_hat = mean(agree); ok = p_hat >= theta.
cudaError_t launch_spot_check(const float* hidden, int d, const int* rows, const int* cols, const float* ref, int n,
                              float eps, float theta, uint8_t* agree, float* p_hat, uint8_t* ok, cudaStream_t stream);

// Merkle roots (SHA-256 over little-endian float32 leaves), one 32-byte root per vector of d entries.
cudaError_t merkle_init();  // derives the SHA-256 constants and uploads them (once per device)
cudaError_t launch_merkle_roots(const float* states, int n_vec, int d, uint8_t* roots, cudaStream_t stream);

// ------------------------------------------------------------------ decode (prover side)
// out[rows][n] (fp32) = x[rows][k] (bf16) * w[n][k]^T, rows <= 8 per launch group; optional in-place add.
cudaError_t launch_skinny_gemm(const void* x, const void* w, float* out, int rows, int n, int k, int accumulate,
                               cudaStream_t stream);
cudaError_t launch_decode_rope_append(const float* qkv, const int* tok_index, const int* positions, int rows,
                                      int n_heads, int n_kv_heads, int head_dim, const float2* rope_cs, void* q_out,
                                      void* kv_cache_layer, cudaStream_t stream);
cudaError_t launch_decode_attention(const void* q, const void* kv_cache_layer, const int* seq_start,
                                    const int* positions, int rows, int n_heads, int n_kv_heads, int head_dim,
                                    int max_keys, void* out, cudaStream_t stream);
cudaError_t launch_swiglu_rows(const float* gu, void* out, int rows, int d_ffn, cudaStream_t stream);
cudaError_t launch_gather_rows(const float* resid, const int* row_of_slot, const int* slots, int n_slots, int d,
                               float* hidden_layer, cudaStream_t stream);
cudaError_t launch_scatter_kv(const void* qkv, const int* dst_row, int rows, int n_heads, int n_kv_heads,
                              int head_dim, void* kv_cache_layer, cudaStream_t stream);
cudaError_t launch_convert_states(const float* src, void* dst, size_t n, int commit_dtype, cudaStream_t stream);
// One thread waits on a barrier nobody signals, for at most limit_cycles: *status receives
// VERILLM_DEV_WAIT_TIMEOUT, *gave_up 1.
cudaError_t launch_wait_probe(long long limit_cycles, int* status, int* gave_up, cudaStream_t stream);
cudaError_t launch_gather_tokens(const int* tokens, const int* src_index, int n, int* out, cudaStream_t stream);

}  // namespace vl
