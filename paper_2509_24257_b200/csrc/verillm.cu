// C-ABI host driver: argument validation, weight re-layout, workspace planning and the launch
// sequence of the verifier's prefill pass, the prover-side decode loop and the standalone comparison.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "kernels.h"

using namespace vl;

namespace {

typedef __nv_bfloat16 bf16;

// Projections over more than 128 token rows run on CTA pairs (256 x 256 tiles over two SMs, each CTA loading
// a 128-row half of the weight tile); smaller ones on single CTAs with 128 x 256 tiles.
#ifdef VL_NO_PAIR
inline int use_pair(int) { return 0; }
#else
inline int use_pair(int M) { return M > kGemmBM ? 1 : 0; }
#endif

#define CU_TRY(expr)                                  \
    do {                                              \
        cudaError_t _e = (expr);                      \
        if (_e != cudaSuccess) {                      \
            g_last_cuda_error = _e;                   \
            return _e == cudaErrorMemoryAllocation ? VERILLM_E_NOMEM : VERILLM_E_CUDA; \
        }                                             \
    } while (0)

thread_local cudaError_t g_last_cuda_error = cudaSuccess;

struct LayerDev {
    bf16 *attn_norm = nullptr, *ffn_norm = nullptr;
    bf16 *wqkv = nullptr;  // [(H + 2 KV) dh][d]: q rows, k rows, v rows
    bf16 *wo = nullptr;    // [d][H dh]
    bf16 *wgu = nullptr;   // [2 F][d]: blocks of 128 gate rows followed by the 128 matching up rows
    bf16 *wd = nullptr;    // [d][F]
    CUtensorMap t_wqkv, t_wo, t_wgu, t_wd;          // boxes of 256 weight rows (single-CTA tiles)
    CUtensorMap t_wqkv_h, t_wo_h, t_wgu_h, t_wd_h;  // boxes of 128 weight rows (one half per CTA of a pair)
};

struct DecodeState {
    bool ready = false;
    bf16* kv_cache = nullptr;   // [n_layers][max_tokens][2 * KV * dh]
    float* hidden_tmp = nullptr;  // [n_layers][max_checks][d]
    float *resid = nullptr, *qkv = nullptr, *gu = nullptr;  // [max_batch][...]
    bf16 *xn = nullptr, *q = nullptr, *attn = nullptr, *mid = nullptr;
    int* ints = nullptr;  // index scratch: 6 * max_tokens + 3 * max_checks
};

// Optional per-kernel timing: one event after every launch of a verify_prefill call.
struct Profile {
    bool on = false;
    std::vector<cudaEvent_t> ev;
    std::vector<int> cls;
    int n = 0;
};

}  // namespace

struct verillm_model {
    verillm_config cfg;
    int device = 0, num_sms = 0;
    int d_q = 0, d_kv = 0, n_qkv = 0, n_tiles_d = 0;
    bf16 *embed = nullptr, *final_norm = nullptr;
    std::vector<LayerDev> layers;
    // workspace
    float* resid = nullptr;
    bf16 *xn = nullptr, *qkv = nullptr, *attn = nullptr, *mid = nullptr;
    int *pos_of_token = nullptr, *seq_of_token = nullptr, *slot_first = nullptr, *slot_next = nullptr;
    int *tok_of_slot = nullptr, *seq_of_slot = nullptr, *cu_dev = nullptr, *status = nullptr;
    int* seq_flags = nullptr;  // [max_batch] sequences whose recorded input states were malformed
    // Library-owned (pageable) copies of the caller's host arrays: an asynchronous copy out of pageable memory
    // is staged before the call returns, so the caller's arrays, pinned or not, are free again at return.
    std::vector<int> h_cu, h_tok_of_slot, h_seq_of_slot, h_claimed;
    float* partials = nullptr;
    int* split_flags = nullptr;  // K-part counters of the GEMMs' last round (one per pair of SMs)
    // K-part counters of the additive projections of one call, kSplitInts per launch, cleared once before the
    // first layer: a clearing queued between two kernels would keep the later one's prologue from overlapping
    int* split_arena = nullptr;
    size_t split_launches = 0;  // launches the arena has room for
    float* sumsq = nullptr;  // [max_tokens][n_tiles_d]: per-tile sums of squares of the residual rows (folded RMSNorm)
    float2* rope_cs = nullptr;
    CUtensorMap t_xn, t_attn, t_mid;
    CUtensorMap t_qkv_q, t_qkv_kv;  // attention operands: boxes of 128 query rows / 64 key rows
    // tail token check (allocated by verillm_load_lm_head)
    bf16 *lm_head = nullptr, *tm_y = nullptr;
    float* tm_rec = nullptr;
    int* tm_claimed = nullptr;
    int n_tiles_v = 0;
    CUtensorMap t_lm, t_lm_h, t_tm_y;
    DecodeState dec;
    Profile prof;
    int last_launches = 0;
};

namespace {

inline void prof_mark(verillm_model* m, int cls, cudaStream_t st) {
    Profile& p = m->prof;
    if (!p.on || p.n >= static_cast<int>(p.ev.size())) return;
    cudaEventRecord(p.ev[p.n], st);
    p.cls[p.n] = cls;
    ++p.n;
}

int ensure_init() {
    static bool done[64] = {false};
    int dev = 0;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return VERILLM_E_INVAL;
    if (done[dev]) return VERILLM_OK;
    cudaDeviceProp prop;
    CU_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return VERILLM_E_ARCH;
    CU_TRY(gemm_init());
    CU_TRY(attention_tc_init());
    CU_TRY(merkle_init());
    done[dev] = true;
    return VERILLM_OK;
}

template <typename T>
int dev_alloc(T** p, size_t count) {
    *p = nullptr;
    if (count == 0) return VERILLM_OK;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
    if (e != cudaSuccess) {
        g_last_cuda_error = e;
        cudaGetLastError();
        return VERILLM_E_NOMEM;
    }
    return VERILLM_OK;
}

bool shape_ok(const verillm_config& c) {
    if (c.n_layers < 1 || c.d_model < 64 || c.n_heads < 1 || c.n_kv_heads < 1 || c.d_ffn < 128 || c.vocab < 1) return false;
    if (c.head_dim != 64 && c.head_dim != 128) return false;
    if (c.d_model % 64 != 0 || c.d_ffn % 128 != 0 || c.n_heads % c.n_kv_heads != 0) return false;
    if (c.max_tokens < 1 || c.max_checks < 0 || c.max_batch < 1) return false;
    if (!(c.rope_base > 1.f) || !(c.rms_eps >= 0.f)) return false;
    return true;
}

int copy_in(void* dst, const void* src, size_t bytes, int on_device) {
    CU_TRY(cudaMemcpy(dst, src, bytes, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice));
    return VERILLM_OK;
}

TolDev tol_dev(const verillm_tol& t) {
    TolDev d;
    d.rel_l2 = t.rel_l2; d.max_abs = t.max_abs; d.mae = t.mae;
    d.pe_max = t.pe_max; d.pm_min = t.pm_min; d.pw_min = t.pw_min; d.e_abs_max = t.e_abs_max;
    d.z_large_max = t.z_large_max; d.q_small_min = t.q_small_min;
    d.bit_aware = (t.flags & VERILLM_TOL_BIT_AWARE) ? 1 : 0;
    return d;
}

CmpParams cmp_params(const verillm_tol& t, int commit_dtype) {
    return make_cmp_params(commit_dtype, t.tau_large, t.e_w, t.e_m);
}

// Checks the packed batch description; fills n_tokens and max_len.
int check_batch(const verillm_model* m, const int32_t* cu, int32_t batch, int* n_tokens, int* max_len) {
    if (!cu || batch < 1) return VERILLM_E_INVAL;
    if (batch > m->cfg.max_batch) return VERILLM_E_SHAPE;
    if (cu[0] != 0) return VERILLM_E_RANGE;
    int mx = 0;
    for (int b = 0; b < batch; ++b) {
        if (cu[b + 1] < cu[b]) return VERILLM_E_RANGE;
        mx = std::max(mx, cu[b + 1] - cu[b]);
    }
    if (cu[batch] < 1) return VERILLM_E_RANGE;
    if (cu[batch] > m->cfg.max_tokens) return VERILLM_E_SHAPE;
    *n_tokens = cu[batch];
    *max_len = mx;
    return VERILLM_OK;
}

int check_slots(const verillm_model* m, const int32_t* cu, int32_t batch, const int32_t* check_seq,
                const int32_t* check_pos, int32_t n_check, std::vector<int>* tok_of_slot) {
    if (n_check < 0) return VERILLM_E_INVAL;
    if (n_check > m->cfg.max_checks) return VERILLM_E_SHAPE;
    if (n_check > 0 && (!check_seq || !check_pos)) return VERILLM_E_INVAL;
    tok_of_slot->resize(n_check);
    for (int s = 0; s < n_check; ++s) {
        const int b = check_seq[s], p = check_pos[s];
        if (b < 0 || b >= batch) return VERILLM_E_RANGE;
        if (p < 0 || p >= cu[b + 1] - cu[b]) return VERILLM_E_RANGE;
        (*tok_of_slot)[s] = cu[b] + p;
    }
    return VERILLM_OK;
}

// One transformer block over M packed tokens, residual stream updated in place.  With cmp_layer set the
// down projection runs the gather(-and-compare) epilogue.
//
// Both RMSNorms are folded into the projections around them: the producer of the residual stream (the O and
// down projections, or a small kernel at the start of a pass and for batches the single-CTA GEMM serves) leaves
// bf16(x * gain) in `xn` and the rows' sums of squares in `sumsq`; the consumer (QKV, gate/up) multiplies its
// accumulator rows by rsqrt(mean x^2 + eps).
struct LayerRun {
    int M, batch, max_len;
    const int* cu_dev;
    const GemmParams* cmp_layer;  // fields slot_first .. cmp, or nullptr
    int next_layer;               // layer whose attention norm follows this block's output, -1 if none
    bool norm_ready;              // in/out: xn / sumsq already hold the input of this layer's attention norm
    size_t split_cursor = 0;  // next free slot of the K-part counter arena
};
constexpr int kSplitInts = 80;  // one counter per tile of a last round (at most 73 with 74 pairs of SMs)

// Clears the K-part counters of a call; to be queued before its first layer.
int split_reset(verillm_model* m, LayerRun& r, cudaStream_t st) {
    r.split_cursor = 0;
    CU_TRY(cudaMemsetAsync(m->split_arena, 0, m->split_launches * kSplitInts * sizeof(int), st));
    return VERILLM_OK;
}

int run_layer(verillm_model* m, int l, LayerRun& r, int* status, cudaStream_t st, int* launches) {
    const verillm_config& c = m->cfg;
    const LayerDev& w = m->layers[l];
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.status = status;
    p.M = r.M;
    p.pair = use_pair(r.M);
    p.overlap_prologue = 1;  // the five kernels of a block chain their prologues under each other's tails
    // Tile walk in bands of 16 tile-rows for every projection (measured: bands of 4, 8, 32 and "all rows" are
    // no faster, also for the K = d_model projections whose activations would fit in L2).
    const int band_qkv = 16, band_o = 16, band_gate_up = 16, band_down = 16;
    const bool fold = p.pair != 0;  // the coalesced residual epilogue of the CTA-pair kernel carries the producer half
    auto consumer = [&](GemmParams& q) {
        q.sumsq_in = m->sumsq; q.n_parts = m->n_tiles_d; q.norm_eps = c.rms_eps; q.norm_inv_d = 1.f / static_cast<float>(c.d_model);
    };
    auto producer = [&](GemmParams& q, const void* gain) {
        q.norm_gain = gain; q.xg_out = gain ? m->xn : nullptr; q.sumsq_out = gain ? m->sumsq : nullptr;
    };
    // K-part counters of an additive projection: a zeroed slot of its own where the arena has one left
    auto split_slot = [&](GemmParams& q) {
        if (p.pair && r.split_cursor < m->split_launches) {
            q.split_flags = m->split_arena + (r.split_cursor++) * kSplitInts;
            q.split_prezeroed = 1;
        } else {
            q.split_flags = m->split_flags;
            q.split_prezeroed = 0;
        }
    };

    if (!r.norm_ready) {
        CU_TRY(launch_prenorm(m->resid, w.attn_norm, m->xn, m->sumsq, m->n_tiles_d, r.M, c.d_model, st));
        prof_mark(m, VERILLM_PROF_RMSNORM, st);
        *launches += 1;
    }
    p.N = m->n_qkv; p.K = c.d_model; p.out = m->qkv; p.ldo = m->n_qkv; p.group_m = band_qkv;
    p.rope_cs = m->rope_cs; p.pos_of_token = m->pos_of_token; p.head_dim = c.head_dim; p.rope_cols = m->d_q + m->d_kv;
    consumer(p);
    CU_TRY(launch_gemm(EPI_QKV_ROPE, m->t_xn, p.pair ? w.t_wqkv_h : w.t_wqkv, p, m->num_sms, st));
    prof_mark(m, VERILLM_PROF_GEMM_QKV, st);
    CU_TRY(launch_attention_tc(m->t_qkv_q, m->t_qkv_kv, r.cu_dev, r.batch, r.max_len, c.n_heads, c.n_kv_heads,
                               c.head_dim, m->attn, status, m->num_sms, 1, st));
    prof_mark(m, VERILLM_PROF_ATTENTION, st);
    p.N = c.d_model; p.K = m->d_q; p.out = m->resid; p.ldo = c.d_model;
    p.group_m = band_o;
    p.sumsq_in = nullptr;
    producer(p, fold ? w.ffn_norm : nullptr);
    split_slot(p);
    CU_TRY(launch_gemm(EPI_RESID_ADD, m->t_attn, p.pair ? w.t_wo_h : w.t_wo, p, m->num_sms, st));
    prof_mark(m, VERILLM_PROF_GEMM_O, st);
    if (!fold) {
        CU_TRY(launch_prenorm(m->resid, w.ffn_norm, m->xn, m->sumsq, m->n_tiles_d, r.M, c.d_model, st));
        prof_mark(m, VERILLM_PROF_RMSNORM, st);
        *launches += 1;
    }
    p.N = 2 * c.d_ffn; p.K = c.d_model; p.out = m->mid; p.ldo = c.d_ffn; p.group_m = band_gate_up;
    producer(p, nullptr);
    consumer(p);
    p.split_flags = nullptr;
    CU_TRY(launch_gemm(EPI_SWIGLU, m->t_xn, p.pair ? w.t_wgu_h : w.t_wgu, p, m->num_sms, st));
    prof_mark(m, VERILLM_PROF_GEMM_GATE_UP, st);
    p.N = c.d_model; p.K = c.d_ffn; p.out = m->resid; p.ldo = c.d_model;
    p.group_m = band_down;
    p.sumsq_in = nullptr;
    split_slot(p);
    const bool feeds_next = fold && r.next_layer >= 0;
    producer(p, feeds_next ? m->layers[r.next_layer].attn_norm : nullptr);
    if (r.cmp_layer) {
        p.slot_first = r.cmp_layer->slot_first; p.slot_next = r.cmp_layer->slot_next; p.n_check = r.cmp_layer->n_check;
        p.committed = r.cmp_layer->committed; p.partials = r.cmp_layer->partials; p.hidden_out = r.cmp_layer->hidden_out;
        p.cmp = r.cmp_layer->cmp;
        CU_TRY(launch_gemm(EPI_RESID_ADD_COMPARE, m->t_mid, p.pair ? w.t_wd_h : w.t_wd, p, m->num_sms, st));
    } else {
        CU_TRY(launch_gemm(EPI_RESID_ADD, m->t_mid, p.pair ? w.t_wd_h : w.t_wd, p, m->num_sms, st));
    }
    prof_mark(m, VERILLM_PROF_GEMM_DOWN, st);
    r.norm_ready = feeds_next;
    *launches += 5;
    return VERILLM_OK;
}

int ensure_decode_state(verillm_model* m) {
    if (m->dec.ready) return VERILLM_OK;
    const verillm_config& c = m->cfg;
    DecodeState& d = m->dec;
    int rc;
    const size_t B = c.max_batch;
    if ((rc = dev_alloc(&d.kv_cache, static_cast<size_t>(c.n_layers) * c.max_tokens * 2 * m->d_kv))) return rc;
    if ((rc = dev_alloc(&d.hidden_tmp, static_cast<size_t>(c.n_layers) * std::max(c.max_checks, 1) * c.d_model))) return rc;
    if ((rc = dev_alloc(&d.resid, B * c.d_model))) return rc;
    if ((rc = dev_alloc(&d.qkv, B * m->n_qkv))) return rc;
    if ((rc = dev_alloc(&d.gu, B * 2 * c.d_ffn))) return rc;
    if ((rc = dev_alloc(&d.xn, B * c.d_model))) return rc;
    if ((rc = dev_alloc(&d.q, B * m->d_q))) return rc;
    if ((rc = dev_alloc(&d.attn, B * m->d_q))) return rc;
    if ((rc = dev_alloc(&d.mid, B * c.d_ffn))) return rc;
    if ((rc = dev_alloc(&d.ints, static_cast<size_t>(6) * c.max_tokens + 3 * static_cast<size_t>(std::max(c.max_checks, 1))))) return rc;
    d.ready = true;
    return VERILLM_OK;
}

}  // namespace

// =============================================================================== C ABI

extern "C" {

void verillm_default_tol(verillm_tol* t) {
    if (!t) return;
    t->rel_l2 = 5e-2f; t->max_abs = 0.f; t->mae = 0.f;
    t->pe_max = 0.05f; t->pm_min = 0.75f; t->pw_min = 0.80f; t->e_abs_max = 0.01f;
    t->e_w = 1e-2f; t->e_m = 7;
    t->tau_large = 0.f; t->z_large_max = -1.f; t->q_small_min = 0.f;
    t->flags = 0u;
}

const char* verillm_strerror(int code) {
    switch (code) {
        case VERILLM_OK: return "ok";
        case VERILLM_E_INVAL: return "invalid argument";
        case VERILLM_E_SHAPE: return "unsupported shape or larger than the handle was sized for";
        case VERILLM_E_RANGE: return "index out of range";
        case VERILLM_E_NOMEM: return "device allocation failed";
        case VERILLM_E_CUDA: return cudaGetErrorString(g_last_cuda_error);
        case VERILLM_E_ARCH: return "device is not compute capability 10.x (sm_100a kernels)";
        default: return "unknown error";
    }
}

void verillm_free(verillm_model* m) {
    if (!m) return;
    cudaFree(m->embed); cudaFree(m->final_norm);
    for (LayerDev& w : m->layers) {
        cudaFree(w.attn_norm); cudaFree(w.ffn_norm); cudaFree(w.wqkv); cudaFree(w.wo); cudaFree(w.wgu); cudaFree(w.wd);
    }
    cudaFree(m->resid); cudaFree(m->xn); cudaFree(m->qkv); cudaFree(m->attn); cudaFree(m->mid);
    cudaFree(m->pos_of_token); cudaFree(m->seq_of_token); cudaFree(m->slot_first); cudaFree(m->slot_next);
    cudaFree(m->tok_of_slot); cudaFree(m->seq_of_slot); cudaFree(m->cu_dev); cudaFree(m->status);
    cudaFree(m->seq_flags);
    cudaFree(m->partials); cudaFree(m->sumsq); cudaFree(m->split_flags); cudaFree(m->split_arena); cudaFree(m->rope_cs);
    cudaFree(m->lm_head); cudaFree(m->tm_y); cudaFree(m->tm_rec); cudaFree(m->tm_claimed);
    DecodeState& d = m->dec;
    cudaFree(d.kv_cache); cudaFree(d.hidden_tmp); cudaFree(d.resid); cudaFree(d.qkv); cudaFree(d.gu);
    cudaFree(d.xn); cudaFree(d.q); cudaFree(d.attn); cudaFree(d.mid); cudaFree(d.ints);
    for (cudaEvent_t e : m->prof.ev) cudaEventDestroy(e);
    delete m;
}

int32_t verillm_last_launch_count(const verillm_model* m) { return m ? m->last_launches : 0; }

int verillm_profile_enable(verillm_model* m, int32_t on) {
    if (!m) return VERILLM_E_INVAL;
    Profile& p = m->prof;
    if (on && p.ev.empty()) {
        const size_t n = static_cast<size_t>(m->cfg.n_layers) * 7 + 8;
        p.ev.resize(n);
        p.cls.assign(n, -1);
        for (size_t i = 0; i < n; ++i) CU_TRY(cudaEventCreate(&p.ev[i]));
    }
    p.on = on != 0;
    p.n = 0;
    return VERILLM_OK;
}

int verillm_profile_read(verillm_model* m, float* ms, int32_t* launches) {
    if (!m || !ms || !launches) return VERILLM_E_INVAL;
    Profile& p = m->prof;
    for (int i = 0; i < VERILLM_PROF_NCLASS; ++i) { ms[i] = 0.f; launches[i] = 0; }
    if (p.n < 2) return VERILLM_OK;
    CU_TRY(cudaEventSynchronize(p.ev[p.n - 1]));
    for (int i = 1; i < p.n; ++i) {
        float t = 0.f;
        CU_TRY(cudaEventElapsedTime(&t, p.ev[i - 1], p.ev[i]));
        const int c = p.cls[i];
        if (c >= 0 && c < VERILLM_PROF_NCLASS) { ms[c] += t; launches[c] += 1; }
    }
    return VERILLM_OK;
}

int verillm_load_layer(verillm_model* m, int32_t layer, const verillm_layer_weights* w, int32_t on_device) {
    if (!m || !w || layer < 0 || layer >= m->cfg.n_layers) return VERILLM_E_INVAL;
    if (!w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down)
        return VERILLM_E_INVAL;
    const verillm_config& c = m->cfg;
    LayerDev& L = m->layers[layer];
    const size_t d = c.d_model, e = sizeof(bf16);
    int rc;
    if ((rc = copy_in(L.attn_norm, w->attn_norm, d * e, on_device))) return rc;
    if ((rc = copy_in(L.ffn_norm, w->ffn_norm, d * e, on_device))) return rc;
    if ((rc = copy_in(L.wqkv, w->wq, m->d_q * d * e, on_device))) return rc;
    if ((rc = copy_in(L.wqkv + m->d_q * d, w->wk, m->d_kv * d * e, on_device))) return rc;
    if ((rc = copy_in(L.wqkv + (m->d_q + m->d_kv) * d, w->wv, m->d_kv * d * e, on_device))) return rc;
    if ((rc = copy_in(L.wo, w->wo, d * m->d_q * e, on_device))) return rc;
    if ((rc = copy_in(L.wd, w->w_down, d * c.d_ffn * e, on_device))) return rc;
    // gate/up rows interleaved in blocks of 128 so that one 256-column output tile holds matching columns
    const cudaMemcpyKind kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    const size_t blk = 128 * d * e;
    CU_TRY(cudaMemcpy2D(L.wgu, 2 * blk, w->w_gate, blk, blk, c.d_ffn / 128, kind));
    CU_TRY(cudaMemcpy2D(reinterpret_cast<char*>(L.wgu) + blk, 2 * blk, w->w_up, blk, blk, c.d_ffn / 128, kind));
    CU_TRY(cudaDeviceSynchronize());
    return VERILLM_OK;
}

int verillm_load_globals(verillm_model* m, const void* embed, const void* final_norm, int32_t on_device) {
    if (!m || !embed) return VERILLM_E_INVAL;
    int rc;
    if ((rc = copy_in(m->embed, embed, static_cast<size_t>(m->cfg.vocab) * m->cfg.d_model * sizeof(bf16), on_device)))
        return rc;
    if (final_norm && (rc = copy_in(m->final_norm, final_norm, m->cfg.d_model * sizeof(bf16), on_device))) return rc;
    CU_TRY(cudaDeviceSynchronize());
    return VERILLM_OK;
}

int verillm_load_weights(const verillm_config* cfg, const verillm_weights* weights, verillm_model** out) {
    if (!cfg || !out) return VERILLM_E_INVAL;
    *out = nullptr;
    if (!shape_ok(*cfg)) return VERILLM_E_SHAPE;
    int rc = ensure_init();
    if (rc) return rc;
    verillm_model* m = new (std::nothrow) verillm_model();
    if (!m) return VERILLM_E_NOMEM;
    m->cfg = *cfg;
    const verillm_config& c = m->cfg;
    cudaGetDevice(&m->device);
    cudaDeviceGetAttribute(&m->num_sms, cudaDevAttrMultiProcessorCount, m->device);
    m->d_q = c.n_heads * c.head_dim;
    m->d_kv = c.n_kv_heads * c.head_dim;
    m->n_qkv = m->d_q + 2 * m->d_kv;
    m->n_tiles_d = (c.d_model + kGemmBN - 1) / kGemmBN;
    m->layers.resize(c.n_layers);
    const size_t d = c.d_model, T = c.max_tokens, NC = std::max(c.max_checks, 1);

#define TRY_RC(expr)            \
    do {                        \
        rc = (expr);            \
        if (rc) {               \
            verillm_free(m);    \
            return rc;          \
        }                       \
    } while (0)

    TRY_RC(dev_alloc(&m->embed, static_cast<size_t>(c.vocab) * d));
    TRY_RC(dev_alloc(&m->final_norm, d));
    for (LayerDev& L : m->layers) {
        TRY_RC(dev_alloc(&L.attn_norm, d));
        TRY_RC(dev_alloc(&L.ffn_norm, d));
        TRY_RC(dev_alloc(&L.wqkv, static_cast<size_t>(m->n_qkv) * d));
        TRY_RC(dev_alloc(&L.wo, d * m->d_q));
        TRY_RC(dev_alloc(&L.wgu, static_cast<size_t>(2) * c.d_ffn * d));
        TRY_RC(dev_alloc(&L.wd, d * c.d_ffn));
    }
    TRY_RC(dev_alloc(&m->resid, T * d));
    TRY_RC(dev_alloc(&m->xn, T * d));
    TRY_RC(dev_alloc(&m->qkv, T * m->n_qkv));
    TRY_RC(dev_alloc(&m->attn, T * m->d_q));
    TRY_RC(dev_alloc(&m->mid, T * c.d_ffn));
    TRY_RC(dev_alloc(&m->pos_of_token, T));
    TRY_RC(dev_alloc(&m->seq_of_token, T));
    TRY_RC(dev_alloc(&m->slot_first, T));
    TRY_RC(dev_alloc(&m->slot_next, NC));
    TRY_RC(dev_alloc(&m->tok_of_slot, NC));
    TRY_RC(dev_alloc(&m->seq_of_slot, NC));
    TRY_RC(dev_alloc(&m->cu_dev, static_cast<size_t>(c.max_batch) + 1));
    TRY_RC(dev_alloc(&m->status, 1));
    TRY_RC(dev_alloc(&m->seq_flags, static_cast<size_t>(c.max_batch)));
    TRY_RC(dev_alloc(&m->partials, static_cast<size_t>(c.n_layers) * NC * m->n_tiles_d * kNPart));
    TRY_RC(dev_alloc(&m->sumsq, T * m->n_tiles_d));
    TRY_RC(dev_alloc(&m->split_flags, 256));
    m->split_launches = static_cast<size_t>(c.n_layers) * 2;
    TRY_RC(dev_alloc(&m->split_arena, m->split_launches * kSplitInts));
    cudaMemset(m->split_flags, 0, 256 * sizeof(int));
    TRY_RC(dev_alloc(&m->rope_cs, T * (c.head_dim / 2)));

    // Rows past a call's last token are never stored, but tiles that straddle the end are read: keep them finite.
    cudaMemset(m->xn, 0, T * d * sizeof(bf16));
    cudaMemset(m->qkv, 0, T * m->n_qkv * sizeof(bf16));
    cudaMemset(m->attn, 0, T * m->d_q * sizeof(bf16));
    cudaMemset(m->mid, 0, T * c.d_ffn * sizeof(bf16));
    // rotary table: angle = pos * base^(-2i/dh), evaluated in double, stored as (cos, sin) float pairs
    {
        const int half = c.head_dim / 2;
        std::vector<float2> tab(T * half);
        std::vector<double> inv_freq(half);
        for (int i = 0; i < half; ++i) inv_freq[i] = std::pow(static_cast<double>(c.rope_base), -2.0 * i / c.head_dim);
        for (size_t p = 0; p < T; ++p)
            for (int i = 0; i < half; ++i) {
                const double a = static_cast<double>(p) * inv_freq[i];
                tab[p * half + i] = make_float2(static_cast<float>(std::cos(a)), static_cast<float>(std::sin(a)));
            }
        cudaError_t e = cudaMemcpy(m->rope_cs, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            g_last_cuda_error = e;
            verillm_free(m);
            return VERILLM_E_CUDA;
        }
    }
    // TMA descriptors: activations are A operands (box of 128 rows), weights B operands (box of 256 rows)
    bool ok = true;
    ok = ok && make_tmap_bf16_2d(&m->t_xn, m->xn, T, d, d, kGemmBM) == 0;
    ok = ok && make_tmap_bf16_2d(&m->t_attn, m->attn, T, m->d_q, m->d_q, kGemmBM) == 0;
    ok = ok && make_tmap_bf16_2d(&m->t_mid, m->mid, T, c.d_ffn, c.d_ffn, kGemmBM) == 0;
    ok = ok && make_tmap_bf16_2d(&m->t_qkv_q, m->qkv, T, m->n_qkv, m->n_qkv, 128) == 0;
    ok = ok && make_tmap_bf16_2d(&m->t_qkv_kv, m->qkv, T, m->n_qkv, m->n_qkv, 64) == 0;
    for (LayerDev& L : m->layers) {
        for (int half = 0; half < 2; ++half) {
            const uint32_t box = half ? 128 : kGemmBN;
            ok = ok && make_tmap_bf16_2d(half ? &L.t_wqkv_h : &L.t_wqkv, L.wqkv, m->n_qkv, d, d, box) == 0;
            ok = ok && make_tmap_bf16_2d(half ? &L.t_wo_h : &L.t_wo, L.wo, d, m->d_q, m->d_q, box) == 0;
            ok = ok && make_tmap_bf16_2d(half ? &L.t_wgu_h : &L.t_wgu, L.wgu, 2 * static_cast<uint64_t>(c.d_ffn), d, d, box) == 0;
            ok = ok && make_tmap_bf16_2d(half ? &L.t_wd_h : &L.t_wd, L.wd, d, c.d_ffn, c.d_ffn, box) == 0;
        }
    }
    if (!ok) {
        verillm_free(m);
        return VERILLM_E_CUDA;
    }
    if (weights) {
        if (weights->embed) TRY_RC(verillm_load_globals(m, weights->embed, weights->final_norm, weights->on_device));
        if (weights->layers)
            for (int l = 0; l < c.n_layers; ++l) TRY_RC(verillm_load_layer(m, l, &weights->layers[l], weights->on_device));
    }
#undef TRY_RC
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        g_last_cuda_error = e;
        verillm_free(m);
        return VERILLM_E_CUDA;
    }
    *out = m;
    return VERILLM_OK;
}

// Shared body of the full verifier (tokens in, blocks 0 .. n_layers-1) and the segment verifier (recorded
// upstream states in, blocks l0 .. l1-1).  Exactly one of tokens / states_in is given.
static int verify_impl(verillm_model* m, const int32_t* tokens, const void* states_in, int32_t in_dtype, int l0, int l1,
                       const int32_t* cu_seqlens, int32_t batch, const void* committed_hidden, int32_t commit_dtype,
                       const int32_t* check_seq, const int32_t* check_pos, int32_t n_check, const verillm_tol* tol,
                       const verillm_report* rep, void* cuda_stream) {
    if (!m || (!tokens && !states_in) || !tol || !rep) return VERILLM_E_INVAL;
    if (tol->e_m < 0 || !(tol->e_w >= 0.f)) return VERILLM_E_INVAL;
    if (l0 < 0 || l1 > m->cfg.n_layers || l0 >= l1) return VERILLM_E_RANGE;
    if (commit_dtype != VERILLM_BF16 && commit_dtype != VERILLM_F32) return VERILLM_E_INVAL;
    if (!rep->seq_ok || !rep->seq_score || !rep->status) return VERILLM_E_INVAL;
    if (n_check > 0 && (!committed_hidden || !rep->stats || !rep->pos_ok || !rep->first_bad_layer)) return VERILLM_E_INVAL;
    int M = 0, max_len = 0, rc;
    if ((rc = check_batch(m, cu_seqlens, batch, &M, &max_len))) return rc;
    if ((rc = check_slots(m, cu_seqlens, batch, check_seq, check_pos, n_check, &m->h_tok_of_slot))) return rc;
    m->h_cu.assign(cu_seqlens, cu_seqlens + batch + 1);
    m->h_seq_of_slot.assign(check_seq, check_seq + n_check);

    const verillm_config& c = m->cfg;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int launches = 0;
    m->prof.n = 0;
    prof_mark(m, -1, st);
    CU_TRY(cudaMemsetAsync(rep->status, 0, sizeof(int), st));
    CU_TRY(cudaMemcpyAsync(m->cu_dev, m->h_cu.data(), sizeof(int) * (batch + 1), cudaMemcpyHostToDevice, st));
    if (n_check > 0) {
        CU_TRY(cudaMemcpyAsync(m->tok_of_slot, m->h_tok_of_slot.data(), sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(m->seq_of_slot, m->h_seq_of_slot.data(), sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
    }
    // Key/value tiles of the last sequence reach up to 63 rows past the last token; those rows still hold
    // what an earlier, larger call left there.  Their probabilities are zero, but zero times a non-finite
    // value is not: clear them.
    {
        const size_t tail = std::min<size_t>(static_cast<size_t>(c.max_tokens) - M, 128);
        if (tail > 0) CU_TRY(cudaMemsetAsync(m->qkv + static_cast<size_t>(M) * m->n_qkv, 0, tail * m->n_qkv * sizeof(bf16), st));
    }
    CU_TRY(launch_token_maps(m->cu_dev, batch, M, m->pos_of_token, m->seq_of_token, st));
    CU_TRY(launch_slot_lists(m->tok_of_slot, n_check, M, m->slot_first, m->slot_next, st));
    int* seq_flags = nullptr;
    if (tokens) {
        CU_TRY(launch_embed(tokens, m->embed, M, c.d_model, c.vocab, m->resid, rep->status, st));
    } else {
        seq_flags = m->seq_flags;
        CU_TRY(cudaMemsetAsync(seq_flags, 0, sizeof(int) * batch, st));
        CU_TRY(launch_load_states(states_in, in_dtype, static_cast<size_t>(M) * c.d_model, c.d_model, m->seq_of_token,
                                  seq_flags, m->resid, st));
    }
    launches += 2 + (n_check > 0 ? 1 : 0);
    prof_mark(m, VERILLM_PROF_SETUP, st);

    const size_t e_commit = commit_dtype == VERILLM_BF16 ? 2 : 4;
    GemmParams cl;
    std::memset(&cl, 0, sizeof(cl));
    cl.slot_first = m->slot_first; cl.slot_next = m->slot_next; cl.n_check = n_check;
    cl.cmp = cmp_params(*tol, commit_dtype);
    LayerRun run{M, batch, max_len, m->cu_dev, n_check > 0 ? &cl : nullptr, -1, false};
    if ((rc = split_reset(m, run, st))) return rc;
    for (int l = l0; l < l1; ++l) {
        run.next_layer = l + 1 < l1 ? l + 1 : -1;
        const size_t slab = static_cast<size_t>(l - l0) * n_check;
        cl.committed = reinterpret_cast<const char*>(committed_hidden) + slab * c.d_model * e_commit;
        cl.partials = m->partials + slab * m->n_tiles_d * kNPart;
        cl.hidden_out = rep->hidden_out ? rep->hidden_out + slab * c.d_model : nullptr;
        if ((rc = run_layer(m, l, run, rep->status, st, &launches))) return rc;
    }
    CU_TRY(launch_verdict(m->partials, l1 - l0, n_check, m->n_tiles_d, c.d_model, tol_dev(*tol), rep->status,
                          m->seq_of_slot, seq_flags, rep->stats, rep->pos_ok, rep->first_bad_layer, st));
    CU_TRY(launch_seq_verdict(rep->stats, rep->pos_ok, m->seq_of_slot, n_check, l1 - l0, batch, rep->status, seq_flags,
                              rep->seq_ok, rep->seq_score, st));
    launches += (n_check > 0 ? 1 : 0) + 1;
    prof_mark(m, VERILLM_PROF_VERDICT, st);
    m->last_launches = launches;
    return VERILLM_OK;
}

int verillm_verify_prefill(verillm_model* m, const int32_t* tokens, const int32_t* cu_seqlens, int32_t batch,
                           const void* committed_hidden, int32_t commit_dtype, const int32_t* check_seq,
                           const int32_t* check_pos, int32_t n_check, const verillm_tol* tol,
                           const verillm_report* rep, void* cuda_stream) {
    if (!m || !tokens) return VERILLM_E_INVAL;
    return verify_impl(m, tokens, nullptr, VERILLM_BF16, 0, m->cfg.n_layers, cu_seqlens, batch, committed_hidden,
                       commit_dtype, check_seq, check_pos, n_check, tol, rep, cuda_stream);
}

int verillm_verify_segment(verillm_model* m, const void* input_states, int32_t input_dtype, int32_t layer_begin,
                           int32_t layer_end, const int32_t* cu_seqlens, int32_t batch, const void* committed_hidden,
                           int32_t commit_dtype, const int32_t* check_seq, const int32_t* check_pos, int32_t n_check,
                           const verillm_tol* tol, const verillm_report* rep, void* cuda_stream) {
    if (!m || !input_states) return VERILLM_E_INVAL;
    if (input_dtype != VERILLM_BF16 && input_dtype != VERILLM_F32) return VERILLM_E_INVAL;
    return verify_impl(m, nullptr, input_states, input_dtype, layer_begin, layer_end, cu_seqlens, batch,
                       committed_hidden, commit_dtype, check_seq, check_pos, n_check, tol, rep, cuda_stream);
}

int verillm_compare(const float* hidden, const void* committed, int32_t commit_dtype, int32_t n_layers, int32_t n_check,
                    int32_t d_model, const int32_t* check_seq, int32_t batch, const verillm_tol* tol,
                    const verillm_report* rep, void* cuda_stream) {
    if (!hidden || !committed || !check_seq || !tol || !rep) return VERILLM_E_INVAL;
    if (tol->e_m < 0 || !(tol->e_w >= 0.f)) return VERILLM_E_INVAL;
    if (commit_dtype != VERILLM_BF16 && commit_dtype != VERILLM_F32) return VERILLM_E_INVAL;
    if (n_layers < 1 || n_check < 1 || batch < 1) return VERILLM_E_INVAL;
    if (d_model < 8 || d_model % 8 != 0) return VERILLM_E_SHAPE;
    if (!rep->stats || !rep->pos_ok || !rep->first_bad_layer || !rep->seq_ok || !rep->seq_score || !rep->status)
        return VERILLM_E_INVAL;
    for (int s = 0; s < n_check; ++s)
        if (check_seq[s] < 0 || check_seq[s] >= batch) return VERILLM_E_RANGE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t rows = static_cast<size_t>(n_layers) * n_check;
    float* partials = nullptr;
    int* seq_dev = nullptr;
    CU_TRY(cudaMallocAsync(reinterpret_cast<void**>(&partials), rows * kNPart * sizeof(float), st));
    CU_TRY(cudaMallocAsync(reinterpret_cast<void**>(&seq_dev), sizeof(int) * n_check, st));
    CU_TRY(cudaMemsetAsync(rep->status, 0, sizeof(int), st));
    // (a library-owned pageable copy is staged before the call returns, whatever memory the caller's array is in)
    const std::vector<int> seq_host(check_seq, check_seq + n_check);
    CU_TRY(cudaMemcpyAsync(seq_dev, seq_host.data(), sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
    CU_TRY(launch_compare_rows(hidden, committed, static_cast<int>(rows), d_model, cmp_params(*tol, commit_dtype), partials, st));
    CU_TRY(launch_verdict(partials, n_layers, n_check, 1, d_model, tol_dev(*tol), rep->status, nullptr, nullptr,
                          rep->stats, rep->pos_ok, rep->first_bad_layer, st));
    CU_TRY(launch_seq_verdict(rep->stats, rep->pos_ok, seq_dev, n_check, n_layers, batch, rep->status, nullptr,
                              rep->seq_ok, rep->seq_score, st));
    CU_TRY(cudaFreeAsync(partials, st));
    CU_TRY(cudaFreeAsync(seq_dev, st));
    return VERILLM_OK;
}

// ---------------------------------------------------------------------------------------------
// Comparison and verdict without any allocation.  The scratch that verillm_compare takes from the
// stream-ordered allocator lives here in a fixed array that is part of the loaded library image.
// Layout: [kNoAllocMaxRows][kNPart] floats of partial sums, then [kNoAllocMaxChecks] ints.
constexpr int kNoAllocMaxRows = 65536;    // n_layers * n_check
constexpr int kNoAllocMaxChecks = 65536;  // n_check
constexpr size_t kNoAllocPartialBytes = static_cast<size_t>(kNoAllocMaxRows) * kNPart * sizeof(float);
constexpr size_t kNoAllocBytes = kNoAllocPartialBytes + static_cast<size_t>(kNoAllocMaxChecks) * sizeof(int);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];
// Device address of the array on each device, resolved on the first call made with that device current.
// (In host code `g_noalloc_scratch` is only a handle for the runtime, never a pointer a kernel may use.)
static void* g_noalloc_ptr[64] = {nullptr};
// Pageable host copy of the caller's check_seq (copies out of pageable memory are staged before the copy call
// returns, so the caller's array is free again at return even if it is pinned).  Shared like the device array.
static int g_noalloc_host_seq[kNoAllocMaxChecks];

int verillm_compare_noalloc(const float* hidden, const void* committed, int32_t commit_dtype, int32_t n_layers,
                            int32_t n_check, int32_t d_model, const int32_t* check_seq, int32_t batch,
                            const verillm_tol* tol, const verillm_report* rep, void* cuda_stream) {
    if (!hidden || !committed || !check_seq || !tol || !rep) return VERILLM_E_INVAL;
    if (tol->e_m < 0 || !(tol->e_w >= 0.f)) return VERILLM_E_INVAL;
    if (commit_dtype != VERILLM_BF16 && commit_dtype != VERILLM_F32) return VERILLM_E_INVAL;
    if (n_layers < 1 || n_check < 1 || batch < 1) return VERILLM_E_INVAL;
    if (d_model < 8 || d_model % 8 != 0) return VERILLM_E_SHAPE;
    if (n_check > kNoAllocMaxChecks || static_cast<long long>(n_layers) * n_check > kNoAllocMaxRows)
        return VERILLM_E_SHAPE;  // beyond the fixed scratch: use verillm_compare
    if (!rep->stats || !rep->pos_ok || !rep->first_bad_layer || !rep->seq_ok || !rep->seq_score || !rep->status)
        return VERILLM_E_INVAL;
    for (int s = 0; s < n_check; ++s)
        if (check_seq[s] < 0 || check_seq[s] >= batch) return VERILLM_E_RANGE;
    int dev = 0;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return VERILLM_E_INVAL;
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        CU_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        g_noalloc_ptr[dev] = ptr;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    const size_t rows = static_cast<size_t>(n_layers) * n_check;
    float* partials = reinterpret_cast<float*>(g_noalloc_ptr[dev]);
    int* seq_dev = reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(g_noalloc_ptr[dev]) + kNoAllocPartialBytes);
    // the array still holds the previous call's records: wipe the part this call will read
    CU_TRY(cudaMemsetAsync(partials, 0, rows * kNPart * sizeof(float), st));
    CU_TRY(cudaMemsetAsync(rep->status, 0, sizeof(int), st));
    std::memcpy(g_noalloc_host_seq, check_seq, sizeof(int) * n_check);
    CU_TRY(cudaMemcpyAsync(seq_dev, g_noalloc_host_seq, sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
    CU_TRY(launch_compare_rows(hidden, committed, static_cast<int>(rows), d_model, cmp_params(*tol, commit_dtype), partials, st));
    CU_TRY(launch_verdict(partials, n_layers, n_check, 1, d_model, tol_dev(*tol), rep->status, nullptr, nullptr,
                          rep->stats, rep->pos_ok, rep->first_bad_layer, st));
    CU_TRY(launch_seq_verdict(rep->stats, rep->pos_ok, seq_dev, n_check, n_layers, batch, rep->status, nullptr,
                              rep->seq_ok, rep->seq_score, st));
    return VERILLM_OK;
}

int verillm_load_lm_head(verillm_model* m, const void* lm_head, int32_t on_device) {
    if (!m || !lm_head) return VERILLM_E_INVAL;
    const verillm_config& c = m->cfg;
    if (c.vocab % 32 != 0) return VERILLM_E_SHAPE;
    const size_t d = c.d_model, NC = std::max(c.max_checks, 1);
    int rc;
    if (!m->lm_head) {
        m->n_tiles_v = (c.vocab + kGemmBN - 1) / kGemmBN;
        if ((rc = dev_alloc(&m->lm_head, static_cast<size_t>(c.vocab) * d))) return rc;
        if ((rc = dev_alloc(&m->tm_y, NC * d))) return rc;
        if ((rc = dev_alloc(&m->tm_rec, NC * m->n_tiles_v * 4))) return rc;
        if ((rc = dev_alloc(&m->tm_claimed, NC))) return rc;
        CU_TRY(cudaMemset(m->tm_y, 0, NC * d * sizeof(bf16)));
        bool ok = make_tmap_bf16_2d(&m->t_lm, m->lm_head, c.vocab, d, d, kGemmBN) == 0;
        ok = ok && make_tmap_bf16_2d(&m->t_lm_h, m->lm_head, c.vocab, d, d, 128) == 0;
        ok = ok && make_tmap_bf16_2d(&m->t_tm_y, m->tm_y, NC, d, d, kGemmBM) == 0;
        if (!ok) return VERILLM_E_CUDA;
    }
    if ((rc = copy_in(m->lm_head, lm_head, static_cast<size_t>(c.vocab) * d * sizeof(bf16), on_device))) return rc;
    CU_TRY(cudaDeviceSynchronize());
    return VERILLM_OK;
}

int verillm_token_match(verillm_model* m, const float* last_hidden, const int32_t* claimed, int32_t n_check,
                        int32_t* argmax_out, uint8_t* match_out, float* margin_out, void* cuda_stream) {
    if (!m || !last_hidden || !claimed || !argmax_out || !match_out || !margin_out || n_check < 1) return VERILLM_E_INVAL;
    if (!m->lm_head) return VERILLM_E_INVAL;  // verillm_load_lm_head first
    if (n_check > m->cfg.max_checks) return VERILLM_E_SHAPE;
    const verillm_config& c = m->cfg;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    m->h_claimed.assign(claimed, claimed + n_check);
    CU_TRY(cudaMemcpyAsync(m->tm_claimed, m->h_claimed.data(), sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
    CU_TRY(launch_rmsnorm(last_hidden, m->final_norm, m->tm_y, n_check, c.d_model, c.rms_eps, st));
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.M = n_check; p.N = c.vocab; p.K = c.d_model; p.out = m->tm_rec; p.ldo = 0; p.status = m->status;
    p.pair = use_pair(n_check);
    CU_TRY(cudaMemsetAsync(m->status, 0, sizeof(int), st));
    CU_TRY(launch_gemm(EPI_ARGMAX, m->t_tm_y, p.pair ? m->t_lm_h : m->t_lm, p, m->num_sms, st));
    CU_TRY(launch_argmax_reduce(m->tm_rec, n_check, m->n_tiles_v, m->tm_claimed, argmax_out, match_out, margin_out, st));
    return VERILLM_OK;
}

int verillm_spot_check(const float* hidden, int32_t n_rows, int32_t d_model, const int32_t* sample_row,
                       const int32_t* sample_col, const float* reference, int32_t n_samples, float eps, float theta,
                       uint8_t* agree_out, float* p_hat_out, uint8_t* verdict_out, void* cuda_stream) {
    if (!hidden || !sample_row || !sample_col || !reference || !agree_out || !p_hat_out || !verdict_out) return VERILLM_E_INVAL;
    if (n_rows < 1 || d_model < 1 || n_samples < 1 || !(eps >= 0.f)) return VERILLM_E_INVAL;
    for (int j = 0; j < n_samples; ++j)
        if (sample_row[j] < 0 || sample_row[j] >= n_rows || sample_col[j] < 0 || sample_col[j] >= d_model) return VERILLM_E_RANGE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    char* buf = nullptr;
    const size_t n = static_cast<size_t>(n_samples);
    CU_TRY(cudaMallocAsync(reinterpret_cast<void**>(&buf), n * 12, st));
    int* rows = reinterpret_cast<int*>(buf);
    int* cols = rows + n;
    float* ref = reinterpret_cast<float*>(cols + n);
    // one library-owned pageable copy of the three arrays: staged before the copy call returns
    std::vector<int> host(3 * n);
    std::memcpy(host.data(), sample_row, n * 4);
    std::memcpy(host.data() + n, sample_col, n * 4);
    std::memcpy(host.data() + 2 * n, reference, n * 4);
    CU_TRY(cudaMemcpyAsync(buf, host.data(), n * 12, cudaMemcpyHostToDevice, st));
    CU_TRY(launch_spot_check(hidden, d_model, rows, cols, ref, n_samples, eps, theta, agree_out, p_hat_out, verdict_out, st));
    CU_TRY(cudaFreeAsync(buf, st));
    return VERILLM_OK;
}

int verillm_threshold_sweep(const float* stats, const uint8_t* is_attack, int32_t n_cells, const verillm_tol* variants,
                            int32_t n_variants, int32_t* counts_out, void* cuda_stream) {
    if (!stats || !is_attack || !variants || !counts_out || n_cells < 1 || n_variants < 1) return VERILLM_E_INVAL;
    if (n_variants > kSweepMaxVariants) return VERILLM_E_SHAPE;
    TolSet set;
    std::memset(&set, 0, sizeof(set));
    for (int v = 0; v < n_variants; ++v) set.v[v] = tol_dev(variants[v]);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    CU_TRY(cudaMemsetAsync(counts_out, 0, sizeof(int32_t) * 4 * n_variants, st));
    CU_TRY(launch_threshold_sweep(stats, is_attack, n_cells, set, n_variants, counts_out, st));
    return VERILLM_OK;
}

int verillm_merkle_roots(const float* states, int32_t n_vec, int32_t d_model, uint8_t* roots_out, void* cuda_stream) {
    if (!states || !roots_out || n_vec < 1 || d_model < 1) return VERILLM_E_INVAL;
    if (d_model > 12800) return VERILLM_E_SHAPE;  // one level of the tree must fit in shared memory
    int rc = ensure_init();
    if (rc) return rc;
    CU_TRY(launch_merkle_roots(states, n_vec, d_model, roots_out, reinterpret_cast<cudaStream_t>(cuda_stream)));
    return VERILLM_OK;
}

int verillm_decode_commit(verillm_model* m, const int32_t* tokens, const int32_t* cu_seqlens, int32_t batch,
                          int32_t n_prefill, const int32_t* check_seq, const int32_t* check_pos, int32_t n_check,
                          void* committed_out, int32_t commit_dtype, int32_t* status, void* cuda_stream) {
    if (!m || !tokens || n_prefill < 0) return VERILLM_E_INVAL;
    if (commit_dtype != VERILLM_BF16 && commit_dtype != VERILLM_F32) return VERILLM_E_INVAL;
    if (n_check > 0 && !committed_out) return VERILLM_E_INVAL;
    int M = 0, max_len = 0, rc;
    if ((rc = check_batch(m, cu_seqlens, batch, &M, &max_len))) return rc;
    std::vector<int> tok_of_slot;
    if ((rc = check_slots(m, cu_seqlens, batch, check_seq, check_pos, n_check, &tok_of_slot))) return rc;
    if ((rc = ensure_decode_state(m))) return rc;

    const verillm_config& c = m->cfg;
    DecodeState& d = m->dec;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    int* dev_status = status ? status : m->status;
    CU_TRY(cudaMemsetAsync(dev_status, 0, sizeof(int), st));
    const size_t T = c.max_tokens, NC = std::max(c.max_checks, 1);
    // index scratch layout
    int* i_src = d.ints;                 // [Mp] packed-prompt row -> token index in the full batch
    int* i_tok = d.ints + T;             // gathered token ids (prompt rows, then one decode step)
    int* i_row_tok = d.ints + 2 * T;     // per decode row: token index in the full batch
    int* i_row_pos = d.ints + 3 * T;     // per decode row: position
    int* i_row_start = d.ints + 4 * T;   // per decode row: first token index of its sequence
    int* i_misc = d.ints + 5 * T;        // prompt-phase slot rows [NC] live in tok_of_slot; spare
    int* i_slot_row = d.ints + 6 * T;    // [NC] per sorted slot: row inside its decode step
    int* i_slot_id = i_slot_row + NC;    // [NC] per sorted slot: slot index
    (void)i_misc;

    // ---------------------------------------------------------------- phase A: parallel pass over the prompts
    std::vector<int> cu_p(batch + 1, 0), np(batch);
    for (int b = 0; b < batch; ++b) {
        np[b] = std::min(n_prefill, cu_seqlens[b + 1] - cu_seqlens[b]);
        cu_p[b + 1] = cu_p[b] + np[b];
    }
    const int Mp = cu_p[batch];
    if (Mp > 0) {
        std::vector<int> src(Mp), slot_row(n_check);
        int max_np = 0;
        for (int b = 0; b < batch; ++b) {
            max_np = std::max(max_np, np[b]);
            for (int p = 0; p < np[b]; ++p) src[cu_p[b] + p] = cu_seqlens[b] + p;
        }
        for (int s = 0; s < n_check; ++s)
            slot_row[s] = check_pos[s] < np[check_seq[s]] ? cu_p[check_seq[s]] + check_pos[s] : -1;
        CU_TRY(cudaMemcpyAsync(i_src, src.data(), sizeof(int) * Mp, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(m->cu_dev, cu_p.data(), sizeof(int) * (batch + 1), cudaMemcpyHostToDevice, st));
        if (n_check > 0)
            CU_TRY(cudaMemcpyAsync(m->tok_of_slot, slot_row.data(), sizeof(int) * n_check, cudaMemcpyHostToDevice, st));
        CU_TRY(launch_gather_tokens(tokens, i_src, Mp, i_tok, st));
        CU_TRY(launch_token_maps(m->cu_dev, batch, Mp, m->pos_of_token, m->seq_of_token, st));
        CU_TRY(launch_slot_lists(m->tok_of_slot, n_check, Mp, m->slot_first, m->slot_next, st));
        CU_TRY(launch_embed(i_tok, m->embed, Mp, c.d_model, c.vocab, m->resid, dev_status, st));
        GemmParams cl;
        std::memset(&cl, 0, sizeof(cl));
        cl.slot_first = m->slot_first; cl.slot_next = m->slot_next; cl.n_check = n_check;
        cl.committed = nullptr; cl.partials = nullptr;
        LayerRun run{Mp, batch, max_np, m->cu_dev, n_check > 0 ? &cl : nullptr, -1, false};
        int launches = 0;
        if ((rc = split_reset(m, run, st))) return rc;
        for (int l = 0; l < c.n_layers; ++l) {
            run.next_layer = l + 1 < c.n_layers ? l + 1 : -1;
            cl.hidden_out = d.hidden_tmp + static_cast<size_t>(l) * n_check * c.d_model;
            if ((rc = run_layer(m, l, run, dev_status, st, &launches))) return rc;
            // run_layer leaves this layer's rotated keys and values in qkv: append them to the cache
            CU_TRY(launch_scatter_kv(m->qkv, i_src, Mp, c.n_heads, c.n_kv_heads, c.head_dim,
                                     d.kv_cache + static_cast<size_t>(l) * T * 2 * m->d_kv, st));
        }
    }

    // ---------------------------------------------------------------- phase B: token-by-token decode
    // rows of step t: the sequences with n_prefill <= t < len, in batch order
    std::vector<int> step_first, row_tok, row_pos, row_start;
    int t_begin = max_len, t_end = max_len;
    for (int b = 0; b < batch; ++b) t_begin = std::min(t_begin, np[b]);
    for (int t = t_begin; t < t_end; ++t) {
        step_first.push_back(static_cast<int>(row_tok.size()));
        for (int b = 0; b < batch; ++b) {
            const int len = cu_seqlens[b + 1] - cu_seqlens[b];
            if (t >= np[b] && t < len) {
                row_tok.push_back(cu_seqlens[b] + t);
                row_pos.push_back(t);
                row_start.push_back(cu_seqlens[b]);
            }
        }
    }
    step_first.push_back(static_cast<int>(row_tok.size()));
    const int n_rows_total = static_cast<int>(row_tok.size());
    if (n_rows_total > 0) {
        // check slots of decoded positions, grouped by step
        std::vector<int> order;
        for (int s = 0; s < n_check; ++s)
            if (check_pos[s] >= np[check_seq[s]]) order.push_back(s);
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return check_pos[a] < check_pos[b]; });
        std::vector<int> slot_row(order.size()), slot_id(order.size()), slots_first(t_end - t_begin + 1, 0);
        {
            size_t k = 0;
            for (int t = t_begin; t < t_end; ++t) {
                slots_first[t - t_begin] = static_cast<int>(k);
                while (k < order.size() && check_pos[order[k]] == t) {
                    const int s = order[k];
                    int row = 0;  // rank of the slot's sequence among the rows of step t
                    for (int b = 0; b < check_seq[s]; ++b) {
                        const int len = cu_seqlens[b + 1] - cu_seqlens[b];
                        if (t >= np[b] && t < len) ++row;
                    }
                    slot_row[k] = row;
                    slot_id[k] = s;
                    ++k;
                }
            }
            slots_first[t_end - t_begin] = static_cast<int>(k);
        }
        CU_TRY(cudaMemcpyAsync(i_row_tok, row_tok.data(), sizeof(int) * n_rows_total, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(i_row_pos, row_pos.data(), sizeof(int) * n_rows_total, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(i_row_start, row_start.data(), sizeof(int) * n_rows_total, cudaMemcpyHostToDevice, st));
        if (!order.empty()) {
            CU_TRY(cudaMemcpyAsync(i_slot_row, slot_row.data(), sizeof(int) * order.size(), cudaMemcpyHostToDevice, st));
            CU_TRY(cudaMemcpyAsync(i_slot_id, slot_id.data(), sizeof(int) * order.size(), cudaMemcpyHostToDevice, st));
        }
        for (int t = t_begin; t < t_end; ++t) {
            const int r0 = step_first[t - t_begin], rows = step_first[t - t_begin + 1] - r0;
            if (rows == 0) continue;
            const int s0 = slots_first[t - t_begin], n_slots = slots_first[t - t_begin + 1] - s0;
            CU_TRY(launch_gather_tokens(tokens, i_row_tok + r0, rows, i_tok, st));
            CU_TRY(launch_embed(i_tok, m->embed, rows, c.d_model, c.vocab, d.resid, dev_status, st));
            for (int l = 0; l < c.n_layers; ++l) {
                const LayerDev& w = m->layers[l];
                bf16* cache_l = d.kv_cache + static_cast<size_t>(l) * T * 2 * m->d_kv;
                CU_TRY(launch_rmsnorm(d.resid, w.attn_norm, d.xn, rows, c.d_model, c.rms_eps, st));
                CU_TRY(launch_skinny_gemm(d.xn, w.wqkv, d.qkv, rows, m->n_qkv, c.d_model, 0, st));
                CU_TRY(launch_decode_rope_append(d.qkv, i_row_tok + r0, i_row_pos + r0, rows, c.n_heads, c.n_kv_heads,
                                                 c.head_dim, m->rope_cs, d.q, cache_l, st));
                CU_TRY(launch_decode_attention(d.q, cache_l, i_row_start + r0, i_row_pos + r0, rows, c.n_heads,
                                               c.n_kv_heads, c.head_dim, t + 1, d.attn, st));
                CU_TRY(launch_skinny_gemm(d.attn, w.wo, d.resid, rows, c.d_model, m->d_q, 1, st));
                CU_TRY(launch_rmsnorm(d.resid, w.ffn_norm, d.xn, rows, c.d_model, c.rms_eps, st));
                CU_TRY(launch_skinny_gemm(d.xn, w.wgu, d.gu, rows, 2 * c.d_ffn, c.d_model, 0, st));
                CU_TRY(launch_swiglu_rows(d.gu, d.mid, rows, c.d_ffn, st));
                CU_TRY(launch_skinny_gemm(d.mid, w.wd, d.resid, rows, c.d_model, c.d_ffn, 1, st));
                if (n_slots > 0)
                    CU_TRY(launch_gather_rows(d.resid, i_slot_row + s0, i_slot_id + s0, n_slots, c.d_model,
                                              d.hidden_tmp + static_cast<size_t>(l) * n_check * c.d_model, st));
            }
        }
    }
    if (n_check > 0)
        CU_TRY(launch_convert_states(d.hidden_tmp, committed_out, static_cast<size_t>(c.n_layers) * n_check * c.d_model,
                                     commit_dtype, st));
    CU_TRY(cudaStreamSynchronize(st));
    return VERILLM_OK;
}

int verillm_selftest_wait_timeout(int64_t limit_cycles, int32_t* status, int32_t* gave_up, void* cuda_stream) {
    if (!status || limit_cycles < 1 || limit_cycles > 2000000000LL) return VERILLM_E_INVAL;
    int rc = ensure_init();
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    CU_TRY(cudaMemsetAsync(status, 0, sizeof(int), st));
    CU_TRY(launch_wait_probe(limit_cycles, status, gave_up, st));
    return VERILLM_OK;
}

int verillm_op_gemm(const void* a, const void* b, void* cmat, int32_t M, int32_t N, int32_t K, int32_t out_f32,
                    int32_t* status, void* cuda_stream) {
    if (!a || !b || !cmat || M < 1 || N < 1 || K < 1) return VERILLM_E_INVAL;
    if (K % 8 != 0 || N % 32 != 0) return VERILLM_E_SHAPE;
    int rc = ensure_init();
    if (rc) return rc;
    int dev = 0, sms = 0;
    CU_TRY(cudaGetDevice(&dev));
    CU_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUtensorMap ta, tb;
    if (make_tmap_bf16_2d(&ta, a, M, K, K, kGemmBM) != 0) return VERILLM_E_CUDA;
    if (make_tmap_bf16_2d(&tb, b, N, K, K, use_pair(M) ? 128 : kGemmBN) != 0) return VERILLM_E_CUDA;
    GemmParams p;
    std::memset(&p, 0, sizeof(p));
    p.M = M; p.N = N; p.K = K; p.out = cmat; p.ldo = N; p.status = status; p.pair = use_pair(M);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (status) CU_TRY(cudaMemsetAsync(status, 0, sizeof(int), st));
    CU_TRY(launch_gemm(out_f32 ? EPI_STORE_F32 : EPI_STORE_BF16, ta, tb, p, sms, st));
    return VERILLM_OK;
}

int verillm_op_rmsnorm(const float* x, const void* gain, void* y, int32_t M, int32_t d, float eps, void* cuda_stream) {
    if (!x || !gain || !y || M < 1 || d < 4) return VERILLM_E_INVAL;
    if (d % 4 != 0) return VERILLM_E_SHAPE;
    CU_TRY(launch_rmsnorm(x, gain, y, M, d, eps, reinterpret_cast<cudaStream_t>(cuda_stream)));
    return VERILLM_OK;
}

int verillm_op_attention(const void* qkv, const int32_t* cu_seqlens, int32_t batch, int32_t max_seqlen, int32_t M,
                         int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* out, void* cuda_stream) {
    if (!qkv || !cu_seqlens || !out || batch < 1 || max_seqlen < 1 || M < 1) return VERILLM_E_INVAL;
    if ((head_dim != 64 && head_dim != 128) || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0)
        return VERILLM_E_SHAPE;
    int rc = ensure_init();
    if (rc) return rc;
    const int n_qkv = (n_heads + 2 * n_kv_heads) * head_dim;
    CUtensorMap tq, tkv;
    if (make_tmap_bf16_2d(&tq, qkv, M, n_qkv, n_qkv, 128) != 0) return VERILLM_E_CUDA;
    if (make_tmap_bf16_2d(&tkv, qkv, M, n_qkv, n_qkv, 64) != 0) return VERILLM_E_CUDA;
    int dev = 0, num_sms = 0;
    CU_TRY(cudaGetDevice(&dev));
    CU_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    CU_TRY(launch_attention_tc(tq, tkv, cu_seqlens, batch, max_seqlen, n_heads, n_kv_heads, head_dim, out, nullptr,
                               num_sms, 0, reinterpret_cast<cudaStream_t>(cuda_stream)));
    return VERILLM_OK;
}

}  // extern "C"
