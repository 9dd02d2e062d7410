// The memory-bound steps of the verifier path (index maps, embedding gather, RMSNorm, standalone
// comparison, verdict reductions) and the CUDA-core kernels of the prover-side decode loop.
#include "kernels.h"

namespace vl {

namespace {

// ------------------------------------------------------------------ index maps
__global__ void token_maps_kernel(const int* __restrict__ cu, int batch, int n_tokens, int* __restrict__ pos_of_token,
                                  int* __restrict__ seq_of_token) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_tokens) return;
    int lo = 0, hi = batch;  // largest s with cu[s] <= i
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= i) lo = mid; else hi = mid;
    }
    pos_of_token[i] = i - cu[lo];
    seq_of_token[i] = lo;
}

// Each check slot pushes itself on the list of its token row; the list order is arbitrary, every
// slot is compared independently.
__global__ void slot_lists_kernel(const int* __restrict__ tok_of_slot, int n_check, int n_tokens,
                                  int* __restrict__ slot_first, int* __restrict__ slot_next) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n_check) return;
    const int t = tok_of_slot[s];
    if (t < 0 || t >= n_tokens) {
        slot_next[s] = -1;
        return;
    }
    slot_next[s] = atomicExch(&slot_first[t], s);
}

// ------------------------------------------------------------------ embedding gather: S_1 = Embed(x)
__global__ void embed_kernel(const int* __restrict__ tokens, const __nv_bfloat16* __restrict__ table, int d_model,
                             int vocab, float* __restrict__ resid, int* status) {
    const int row = blockIdx.x;
    int tok = tokens[row];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, VERILLM_DEV_TOKEN_RANGE);
        tok = tok < 0 ? 0 : vocab - 1;
    }
    const uint4* src = reinterpret_cast<const uint4*>(table + static_cast<size_t>(tok) * d_model);
    float4* dst = reinterpret_cast<float4*>(resid + static_cast<size_t>(row) * d_model);
    for (int i = threadIdx.x; i < d_model / 8; i += blockDim.x) {
        const uint4 v = __ldg(src + i);
        dst[2 * i] = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
        dst[2 * i + 1] = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
    }
}

// ------------------------------------------------------------------ RMSNorm: x * rsqrt(mean x^2 + eps) * gain
constexpr int kNormThreads = 256;
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ y,
               int d, float eps) {
    const int row = blockIdx.x;
    const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(row) * d);
    float ss = 0.f;
    for (int i = threadIdx.x; i < d / 4; i += kNormThreads) {
        const float4 v = xr[i];
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    __shared__ float warp_part[kNormThreads / 32];
    __shared__ float s_rstd;
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < kNormThreads / 32; ++w) t += warp_part[w];
        s_rstd = rsqrtf(t / static_cast<float>(d) + eps);
    }
    __syncthreads();
    const float rstd = s_rstd;
    uint2* yr = reinterpret_cast<uint2*>(y + static_cast<size_t>(row) * d);
    const uint2* g2 = reinterpret_cast<const uint2*>(gain);
    for (int i = threadIdx.x; i < d / 4; i += kNormThreads) {
        const float4 v = xr[i];
        const uint2 g = __ldg(g2 + i);
        uint2 o;
        o.x = pack_bf16(v.x * rstd * bf16_lo(g.x), v.y * rstd * bf16_hi(g.x));
        o.y = pack_bf16(v.z * rstd * bf16_lo(g.y), v.w * rstd * bf16_hi(g.y));
        yr[i] = o;
    }
}

// Unnormalised half of a folded norm: y = bf16(x * gain) and the row's sum of squares (see GemmParams).
__global__ void __launch_bounds__(kNormThreads)
prenorm_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain, __nv_bfloat16* __restrict__ y,
               float* __restrict__ sumsq, int n_parts, int d) {
    const int row = blockIdx.x;
    const float4* xr = reinterpret_cast<const float4*>(x + static_cast<size_t>(row) * d);
    uint2* yr = reinterpret_cast<uint2*>(y + static_cast<size_t>(row) * d);
    const uint2* g2 = reinterpret_cast<const uint2*>(gain);
    float ss = 0.f;
    for (int i = threadIdx.x; i < d / 4; i += kNormThreads) {
        const float4 v = xr[i];
        const uint2 g = __ldg(g2 + i);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        uint2 o;
        o.x = pack_bf16(v.x * bf16_lo(g.x), v.y * bf16_hi(g.x));
        o.y = pack_bf16(v.z * bf16_lo(g.y), v.w * bf16_hi(g.y));
        yr[i] = o;
    }
    __shared__ float warp_part[kNormThreads / 32];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < kNormThreads / 32; ++w) t += warp_part[w];
        sumsq[static_cast<size_t>(row) * n_parts] = t;
    }
    for (int k = 1 + threadIdx.x; k < n_parts; k += kNormThreads) sumsq[static_cast<size_t>(row) * n_parts + k] = 0.f;
}

// ------------------------------------------------------------------ standalone comparison
// One pass of a lane over its share of a row (16-byte loads, lanes interleaved).
template <bool kChecked>
__device__ __forceinline__ void compare_row_pass(CmpAcc& a, const float* __restrict__ h, const void* __restrict__ committed,
                                                 size_t row, int d, int lane, const CmpParams& cmp) {
    if (cmp.commit_dtype == VERILLM_BF16) {
        const uint4* c4 = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(committed) + row * d);
        if constexpr (kChecked) {
            for (int j = lane * 8; j < d; j += 256) {
                const uint4 cv = __ldg(c4 + j / 8);
                const float4 h0 = __ldg(reinterpret_cast<const float4*>(h + j));
                const float4 h1 = __ldg(reinterpret_cast<const float4*>(h + j + 4));
                a.add_bf16x2<true>(h0.x, h0.y, cv.x, cmp);
                a.add_bf16x2<true>(h0.z, h0.w, cv.y, cmp);
                a.add_bf16x2<true>(h1.x, h1.y, cv.z, cmp);
                a.add_bf16x2<true>(h1.z, h1.w, cv.w, cmp);
            }
        } else {
            float2 ss2 = make_float2(0.f, 0.f), rr2 = ss2, sg2 = ss2, sa2 = ss2;
            for (int j = lane * 8; j < d; j += 256) {
                const uint4 cv = __ldg(c4 + j / 8);
                const float4 h0 = __ldg(reinterpret_cast<const float4*>(h + j));
                const float4 h1 = __ldg(reinterpret_cast<const float4*>(h + j + 4));
                a.add_bf16x2_packed(h0.x, h0.y, cv.x, cmp, ss2, rr2, sg2, sa2);
                a.add_bf16x2_packed(h0.z, h0.w, cv.y, cmp, ss2, rr2, sg2, sa2);
                a.add_bf16x2_packed(h1.x, h1.y, cv.z, cmp, ss2, rr2, sg2, sa2);
                a.add_bf16x2_packed(h1.z, h1.w, cv.w, cmp, ss2, rr2, sg2, sa2);
            }
            a.fold(ss2, rr2, sg2, sa2);
        }
    } else {
        const uint4* c4 = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(committed) + row * d);
        for (int j = lane * 4; j < d; j += 128) {
            const uint4 cv = __ldg(c4 + j / 4);
            const float4 h0 = __ldg(reinterpret_cast<const float4*>(h + j));
            a.add_f32<kChecked>(h0.x, cv.x, cmp);
            a.add_f32<kChecked>(h0.y, cv.y, cmp);
            a.add_f32<kChecked>(h0.z, cv.z, cmp);
            a.add_f32<kChecked>(h0.w, cv.w, cmp);
        }
    }
}

// One warp per (layer, slot) row: coalesced 16-byte loads of both operands, per-lane accumulation,
// fixed-order shuffle reduction, one partial record per row.
__global__ void compare_rows_kernel(const float* __restrict__ hidden, const void* __restrict__ committed, int n_rows,
                                    int d, CmpParams cmp, float* __restrict__ partials) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    const float* h = hidden + static_cast<size_t>(row) * d;
    CmpAcc a;
    a.clear();
    // first pass without the per-element test for non-finite operands; any such operand leaves the sum
    // of |h - c| non-finite, and the lane then repeats its share with the test
    compare_row_pass<false>(a, h, committed, static_cast<size_t>(row), d, lane, cmp);
    if (!(a.sa < INFINITY)) {
        a.clear();
        compare_row_pass<true>(a, h, committed, static_cast<size_t>(row), d, lane, cmp);
    }
    a.ss = warp_sum(a.ss);
    a.rr = warp_sum(a.rr);
    a.sa = warp_sum(a.sa);
    a.sg = warp_sum(a.sg);
    a.mx = warp_max(a.mx);
    a.n_mis = warp_sum_u32(a.n_mis);
    a.n_large_m = warp_sum_u32(a.n_large_m);
    a.n_small_w = warp_sum_u32(a.n_small_w);
    a.n_exact = warp_sum_u32(a.n_exact);
    a.n_qsmall = warp_sum_u32(a.n_qsmall);
    a.n_zlarge = warp_sum_u32(a.n_zlarge);
    a.n_nonfinite = warp_sum_u32(a.n_nonfinite);
    if (lane == 0) a.store(partials + static_cast<size_t>(row) * kNPart);
}

// ------------------------------------------------------------------ verdict
// One warp per check slot, lanes over layers: each lane sums the column-tile partials of its layers in
// a fixed order, derives the reported statistics and applies the enabled tests (b = 1[T_v <= tau]; a
// non-finite value, a device-side error or a sequence marked as malformed rejects); the first failing layer is
// the minimum over lanes.
__global__ void verdict_kernel(const float* __restrict__ partials, int n_layers, int n_check, int n_tiles, int d,
                               TolDev tol, const int* __restrict__ status, const int* __restrict__ seq_of_slot,
                               const int* __restrict__ seq_flags, float* __restrict__ stats,
                               uint8_t* __restrict__ pos_ok, int* __restrict__ first_bad_layer) {
    const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (slot >= n_check) return;
    // a device-side error rejects everything; malformed recorded states reject their sequence
    const bool dev_error = (status != nullptr && *status != 0) ||
                           (seq_flags != nullptr && seq_flags[seq_of_slot[slot]] != 0);
    int first_bad = 0x7FFFFFFF;
    const float inv_d = 1.f / static_cast<float>(d);
    for (int l = lane; l < n_layers; l += 32) {
        const float* rec = partials + (static_cast<size_t>(l) * n_check + slot) * n_tiles * kNPart;
        float ss = 0.f, rr = 0.f, sa = 0.f, sg = 0.f, mx = 0.f;
        uint32_t n_mis = 0, n_large = 0, n_small = 0, n_exact = 0, n_q = 0, n_z = 0, n_nf = 0;
        for (int t = 0; t < n_tiles; ++t) {
            const float4 a = *reinterpret_cast<const float4*>(rec + t * kNPart);
            const float4 b = *reinterpret_cast<const float4*>(rec + t * kNPart + 4);
            const float4 c = *reinterpret_cast<const float4*>(rec + t * kNPart + 8);
            ss += a.x; rr += a.y; sa += a.z; sg += a.w;
            mx = fmaxf(mx, b.x);
            n_mis += __float_as_uint(b.y); n_large += __float_as_uint(b.z); n_small += __float_as_uint(b.w);
            n_exact += __float_as_uint(c.x); n_q += __float_as_uint(c.y); n_z += __float_as_uint(c.z);
            n_nf += __float_as_uint(c.w);
        }
        const float l2d = sqrtf(ss), l2r = sqrtf(rr);
        const float rel = l2d / fmaxf(l2r, 1e-30f);
        const float mae = sa * inv_d, mean_signed = sg * inv_d;
        const uint32_t n_match = static_cast<uint32_t>(d) - n_nf - n_mis;
        const float p_e = static_cast<float>(n_mis) * inv_d;
        const float p_m = n_mis > 0 ? static_cast<float>(n_large) / static_cast<float>(n_mis) : 1.f;
        const float p_w = n_match > 0 ? static_cast<float>(n_small) / static_cast<float>(n_match) : 1.f;
        const float q_small = static_cast<float>(n_q) * inv_d, z_large = static_cast<float>(n_z) * inv_d;

        bool ok = (n_nf == 0) && !dev_error;
        if (tol.rel_l2 > 0.f) ok = ok && (rel <= tol.rel_l2);
        if (tol.max_abs > 0.f) ok = ok && (mx <= tol.max_abs);
        if (tol.mae > 0.f) ok = ok && (mae <= tol.mae);
        if (tol.z_large_max >= 0.f) ok = ok && (z_large <= tol.z_large_max);
        if (tol.q_small_min > 0.f) ok = ok && (q_small >= tol.q_small_min);
        if (tol.bit_aware) {
            ok = ok && (p_e < tol.pe_max) && (p_m > tol.pm_min) && (p_w > tol.pw_min) &&
                 (fabsf(mean_signed) <= tol.e_abs_max);
        }
        if (!ok && l < first_bad) first_bad = l;

        float4* o = reinterpret_cast<float4*>(stats + (static_cast<size_t>(slot) * n_layers + l) * VERILLM_NSTAT);
        o[0] = make_float4(rel, mx, mae, mean_signed);                       // REL_L2, MAX_ABS, MAE, MEAN_SIGNED
        o[1] = make_float4(p_e, p_m, p_w, q_small);                          // P_E, P_M, P_W, Q_SMALL
        o[2] = make_float4(z_large, static_cast<float>(n_mis), static_cast<float>(n_large),
                           static_cast<float>(n_small));                     // Z_LARGE, N_EXP_MISMATCH, N_MANT_LARGE, N_MANT_SMALL
        o[3] = make_float4(static_cast<float>(n_exact), static_cast<float>(n_nf), l2d, l2r);  // N_EXACT, N_NONFINITE, L2_*
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) first_bad = min(first_bad, __shfl_xor_sync(0xFFFFFFFFu, first_bad, o));
    if (lane == 0) {
        pos_ok[slot] = first_bad == 0x7FFFFFFF ? 1 : 0;
        first_bad_layer[slot] = first_bad == 0x7FFFFFFF ? -1 : first_bad;
    }
}

// ------------------------------------------------------------------ threshold sensitivity
// The tests of verdict_kernel applied to statistics that were reported earlier: one thread per (position,
// layer) cell reads its VERILLM_NSTAT floats once and evaluates every tolerance variant; per variant the block
// counts accepted / rejected cells of the honest and of the attack class (warp ballots, integer atomics).
__device__ __forceinline__ bool stats_pass(const float4& s0, const float4& s1, const float4& s2, const float4& s3,
                                           const TolDev& tol) {
    bool ok = s3.y == 0.f;  // no non-finite element
    if (tol.rel_l2 > 0.f) ok = ok && (s0.x <= tol.rel_l2);
    if (tol.max_abs > 0.f) ok = ok && (s0.y <= tol.max_abs);
    if (tol.mae > 0.f) ok = ok && (s0.z <= tol.mae);
    if (tol.z_large_max >= 0.f) ok = ok && (s2.x <= tol.z_large_max);
    if (tol.q_small_min > 0.f) ok = ok && (s1.w >= tol.q_small_min);
    if (tol.bit_aware)
        ok = ok && (s1.x < tol.pe_max) && (s1.y > tol.pm_min) && (s1.z > tol.pw_min) && (fabsf(s0.w) <= tol.e_abs_max);
    return ok;
}

__global__ void __launch_bounds__(256)
threshold_sweep_kernel(const float* __restrict__ stats, const uint8_t* __restrict__ is_attack, int n_cells,
                       const __grid_constant__ TolSet tols, int n_variants, int* __restrict__ counts) {
    const int cell = blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = cell < n_cells;
    float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0, s2 = s0, s3 = s0;
    bool attack = false;
    if (live) {
        const float4* p = reinterpret_cast<const float4*>(stats + static_cast<size_t>(cell) * VERILLM_NSTAT);
        s0 = __ldg(p);
        s1 = __ldg(p + 1);
        s2 = __ldg(p + 2);
        s3 = __ldg(p + 3);
        attack = is_attack[cell] != 0;
    }
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (int v = 0; v < n_variants; ++v) {
        const bool ok = stats_pass(s0, s1, s2, s3, tols.v[v]);
        const uint32_t ha = __ballot_sync(0xFFFFFFFFu, live && !attack && ok);
        const uint32_t hr = __ballot_sync(0xFFFFFFFFu, live && !attack && !ok);
        const uint32_t aa = __ballot_sync(0xFFFFFFFFu, live && attack && ok);
        const uint32_t ar = __ballot_sync(0xFFFFFFFFu, live && attack && !ok);
        if (lane == 0) {
            if (ha) atomicAdd(counts + 4 * v + 0, __popc(ha));
            if (hr) atomicAdd(counts + 4 * v + 1, __popc(hr));
            if (aa) atomicAdd(counts + 4 * v + 2, __popc(aa));
            if (ar) atomicAdd(counts + 4 * v + 3, __popc(ar));
        }
    }
}

// One block per sequence, threads over check slots: accept iff all its checked positions were accepted (one
// deviation above tolerance suffices to fail, and so does a device-side error or malformed input of that
// sequence); score = mean MAE over its (slot, layer) cells.  Per-thread
// double sums are combined by a fixed shuffle tree and then in warp order, so the result is reproducible.
constexpr int kSeqThreads = 1024;
__global__ void __launch_bounds__(kSeqThreads)
seq_verdict_kernel(const float* __restrict__ stats, const uint8_t* __restrict__ pos_ok,
                   const int* __restrict__ seq_of_slot, int n_check, int n_layers, int batch,
                   const int* __restrict__ status, const int* __restrict__ seq_flags,
                   uint8_t* __restrict__ seq_ok, float* __restrict__ seq_score) {
    const int b = blockIdx.x;
    // a device-side error invalidates every result of the call, also for sequences without a checked position
    int bad = ((status != nullptr && *status != 0) || (seq_flags != nullptr && seq_flags[b] != 0)) ? 1 : 0;
    int cells = 0;
    double sum = 0.0;
    for (int s = threadIdx.x; s < n_check; s += kSeqThreads) {
        if (seq_of_slot[s] != b) continue;
        bad |= (pos_ok[s] == 0) ? 1 : 0;
        const float* mae = stats + static_cast<size_t>(s) * n_layers * VERILLM_NSTAT + VERILLM_STAT_MAE;
        float part = 0.f;
        int l = 0;
        for (; l + 4 <= n_layers; l += 4)  // four independent loads in flight
            part += (mae[(l + 0) * VERILLM_NSTAT] + mae[(l + 1) * VERILLM_NSTAT]) +
                    (mae[(l + 2) * VERILLM_NSTAT] + mae[(l + 3) * VERILLM_NSTAT]);
        for (; l < n_layers; ++l) part += mae[l * VERILLM_NSTAT];
        sum += static_cast<double>(part);
        cells += n_layers;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        bad |= __shfl_xor_sync(0xFFFFFFFFu, bad, o);
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        cells += __shfl_xor_sync(0xFFFFFFFFu, cells, o);
    }
    __shared__ double w_sum[kSeqThreads / 32];
    __shared__ int w_bad[kSeqThreads / 32], w_cells[kSeqThreads / 32];
    if ((threadIdx.x & 31) == 0) {
        w_sum[threadIdx.x >> 5] = sum;
        w_bad[threadIdx.x >> 5] = bad;
        w_cells[threadIdx.x >> 5] = cells;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        int bd = 0, c = 0;
        for (int w = 0; w < kSeqThreads / 32; ++w) {
            t += w_sum[w];
            bd |= w_bad[w];
            c += w_cells[w];
        }
        seq_ok[b] = bd ? 0 : 1;
        seq_score[b] = c > 0 ? static_cast<float>(t / static_cast<double>(c)) : 0.f;
    }
}

// ------------------------------------------------------------------ tail token check
// One warp per row: lanes take column tiles in a strided order, records are merged with "larger value, then
// lower column" so the result does not depend on the merge order; match = (argmax == claimed token).
struct Top2 {
    float best, second;
    int col;
};
__device__ __forceinline__ Top2 top2_merge(const Top2& a, const Top2& b) {
    const bool a_wins = a.best > b.best || (a.best == b.best && a.col < b.col);
    Top2 r;
    r.best = a_wins ? a.best : b.best;
    r.col = a_wins ? a.col : b.col;
    r.second = fmaxf(fmaxf(a.second, b.second), a_wins ? b.best : a.best);
    return r;
}
__global__ void argmax_reduce_kernel(const float4* __restrict__ records, int rows, int n_tiles,
                                     const int* __restrict__ claimed, int* __restrict__ argmax_out,
                                     uint8_t* __restrict__ match_out, float* __restrict__ margin_out) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    Top2 t = {-INFINITY, -INFINITY, 0x7FFFFFFF};
    for (int i = lane; i < n_tiles; i += 32) {
        const float4 r = records[static_cast<size_t>(row) * n_tiles + i];
        const Top2 u = {r.x, r.z, __float_as_int(r.y)};
        t = top2_merge(t, u);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 u;
        u.best = __shfl_xor_sync(0xFFFFFFFFu, t.best, o);
        u.second = __shfl_xor_sync(0xFFFFFFFFu, t.second, o);
        u.col = __shfl_xor_sync(0xFFFFFFFFu, t.col, o);
        t = top2_merge(t, u);
    }
    if (lane == 0) {
        argmax_out[row] = t.col;
        match_out[row] = (t.col == claimed[row]) ? 1 : 0;
        margin_out[row] = t.best - t.second;
    }
}

// ------------------------------------------------------------------ sampled value matching
// One block: threads stride over the samples, agreement counts are integers, so the reduction order is free.
__global__ void __launch_bounds__(256)
spot_check_kernel(const float* __restrict__ hidden, int d, const int* __restrict__ rows, const int* __restrict__ cols,
                  const float* __restrict__ ref, int n, float eps, float theta, uint8_t* __restrict__ agree,
                  float* __restrict__ p_hat, uint8_t* __restrict__ ok) {
    uint32_t cnt = 0;
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
        const float v = hidden[static_cast<size_t>(rows[j]) * d + cols[j]];
        const bool a = fabsf(v - ref[j]) <= eps;  // false for NaN
        agree[j] = a ? 1 : 0;
        cnt += a ? 1u : 0u;
    }
    __shared__ uint32_t part[8];
    cnt = warp_sum_u32(cnt);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int w = 0; w < 8; ++w) t += part[w];
        const float p = static_cast<float>(t) / static_cast<float>(n);
        *p_hat = p;
        *ok = p >= theta ? 1 : 0;
    }
}

// ------------------------------------------------------------------ decode-side kernels
// out[r][n] (+)= sum_k x[r][k] * w[n][k] for up to 8 rows: one warp per output column streams the
// weight row once (16-byte loads) and keeps one accumulator per row.
constexpr int kSkinnyRows = 8;
__global__ void __launch_bounds__(256)
skinny_gemm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w, float* __restrict__ out,
                   int rows, int n, int k, int accumulate) {
    const int col = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (col >= n) return;
    float acc[kSkinnyRows];
#pragma unroll
    for (int r = 0; r < kSkinnyRows; ++r) acc[r] = 0.f;
    const uint4* wr = reinterpret_cast<const uint4*>(w + static_cast<size_t>(col) * k);
    for (int j = lane; j < k / 8; j += 32) {
        const uint4 wv = __ldg(wr + j);
        const float w0 = bf16_lo(wv.x), w1 = bf16_hi(wv.x), w2 = bf16_lo(wv.y), w3 = bf16_hi(wv.y);
        const float w4 = bf16_lo(wv.z), w5 = bf16_hi(wv.z), w6 = bf16_lo(wv.w), w7 = bf16_hi(wv.w);
#pragma unroll
        for (int r = 0; r < kSkinnyRows; ++r) {
            if (r < rows) {
                const uint4 xv = *(reinterpret_cast<const uint4*>(x + static_cast<size_t>(r) * k) + j);
                float a = acc[r];
                a = fmaf(bf16_lo(xv.x), w0, a); a = fmaf(bf16_hi(xv.x), w1, a);
                a = fmaf(bf16_lo(xv.y), w2, a); a = fmaf(bf16_hi(xv.y), w3, a);
                a = fmaf(bf16_lo(xv.z), w4, a); a = fmaf(bf16_hi(xv.z), w5, a);
                a = fmaf(bf16_lo(xv.w), w6, a); a = fmaf(bf16_hi(xv.w), w7, a);
                acc[r] = a;
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kSkinnyRows; ++r) {
        const float s = warp_sum(acc[r]);
        if (lane == 0 && r < rows) {
            float* o = out + static_cast<size_t>(r) * n + col;
            *o = accumulate ? *o + s : s;
        }
    }
}

// Rotates the q and k heads of one decoded token, rounds to bf16, writes q and appends k/v to the cache.
// Cache row layout: [n_kv_heads*head_dim keys | n_kv_heads*head_dim values].
__global__ void decode_rope_append_kernel(const float* __restrict__ qkv, const int* __restrict__ tok_index,
                                          const int* __restrict__ positions, int n_heads, int n_kv_heads, int head_dim,
                                          const float2* __restrict__ rope_cs, __nv_bfloat16* __restrict__ q_out,
                                          __nv_bfloat16* __restrict__ kv_cache) {
    const int r = blockIdx.x;
    const int dq = n_heads * head_dim, dkv = n_kv_heads * head_dim, half = head_dim / 2;
    const float* src = qkv + static_cast<size_t>(r) * (dq + 2 * dkv);
    const int pos = positions[r];
    __nv_bfloat16* cache_row = kv_cache + static_cast<size_t>(tok_index[r]) * (2 * dkv);
    const float2* cs = rope_cs + static_cast<size_t>(pos) * half;
    for (int i = threadIdx.x; i < (dq + dkv) / 2; i += blockDim.x) {  // one rotation pair per iteration
        const int head = i / half, j = i - head * half;
        const int c0 = head * head_dim + j;
        const float a = src[c0], b = src[c0 + half];
        const float2 t = cs[j];
        const float lo = a * t.x - b * t.y, hi = b * t.x + a * t.y;
        if (c0 < dq) {
            q_out[static_cast<size_t>(r) * dq + c0] = __float2bfloat16_rn(lo);
            q_out[static_cast<size_t>(r) * dq + c0 + half] = __float2bfloat16_rn(hi);
        } else {
            cache_row[c0 - dq] = __float2bfloat16_rn(lo);
            cache_row[c0 - dq + half] = __float2bfloat16_rn(hi);
        }
    }
    for (int i = threadIdx.x; i < dkv; i += blockDim.x) cache_row[dkv + i] = __float2bfloat16_rn(src[dq + dkv + i]);
}

// One block per (decoded token, query head): scores against the cached keys of its sequence, softmax,
// weighted sum of the cached values.
__global__ void __launch_bounds__(128)
decode_attention_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kv_cache,
                        const int* __restrict__ seq_start, const int* __restrict__ positions, int n_heads,
                        int n_kv_heads, int head_dim, __nv_bfloat16* __restrict__ out) {
    extern __shared__ float sh[];  // [head_dim] query, then [pos+1] scores
    const int r = blockIdx.x, h = blockIdx.y;
    const int kvh = h * n_kv_heads / n_heads;
    const int dkv = n_kv_heads * head_dim;
    const int n_keys = positions[r] + 1;
    float* qs = sh;
    float* sc = sh + head_dim;
    for (int i = threadIdx.x; i < head_dim; i += blockDim.x)
        qs[i] = __bfloat162float(q[(static_cast<size_t>(r) * n_heads + h) * head_dim + i]);
    __syncthreads();
    const __nv_bfloat16* base = kv_cache + static_cast<size_t>(seq_start[r]) * (2 * dkv) + kvh * head_dim;
    const float scale = rsqrtf(static_cast<float>(head_dim));
    float lmax = -INFINITY;
    for (int t = threadIdx.x; t < n_keys; t += blockDim.x) {
        const uint4* kr = reinterpret_cast<const uint4*>(base + static_cast<size_t>(t) * (2 * dkv));
        float s = 0.f;
        for (int j = 0; j < head_dim / 8; ++j) {
            const uint4 kv = kr[j];
            const float* qq = qs + 8 * j;
            s += qq[0] * bf16_lo(kv.x) + qq[1] * bf16_hi(kv.x) + qq[2] * bf16_lo(kv.y) + qq[3] * bf16_hi(kv.y) +
                 qq[4] * bf16_lo(kv.z) + qq[5] * bf16_hi(kv.z) + qq[6] * bf16_lo(kv.w) + qq[7] * bf16_hi(kv.w);
        }
        s *= scale;
        sc[t] = s;
        lmax = fmaxf(lmax, s);
    }
    __shared__ float red[4];
    __shared__ float s_max, s_sum;
    lmax = warp_max(lmax);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = lmax;
    __syncthreads();
    if (threadIdx.x == 0) s_max = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    const float m = s_max;
    float lsum = 0.f;
    for (int t = threadIdx.x; t < n_keys; t += blockDim.x) {
        const float e = __expf(sc[t] - m);
        sc[t] = e;
        lsum += e;
    }
    lsum = warp_sum(lsum);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = lsum;
    __syncthreads();
    if (threadIdx.x == 0) s_sum = red[0] + red[1] + red[2] + red[3];
    __syncthreads();
    const float inv = 1.f / s_sum;
    for (int j = threadIdx.x; j < head_dim; j += blockDim.x) {
        const __nv_bfloat16* vcol = base + dkv + j;
        float o = 0.f;
        for (int t = 0; t < n_keys; ++t) o = fmaf(sc[t], __bfloat162float(vcol[static_cast<size_t>(t) * (2 * dkv)]), o);
        out[(static_cast<size_t>(r) * n_heads + h) * head_dim + j] = __float2bfloat16_rn(o * inv);
    }
}

// gate/up outputs arrive interleaved in blocks of 128 columns (gate block, up block, ...).
__global__ void swiglu_rows_kernel(const float* __restrict__ gu, __nv_bfloat16* __restrict__ out, int d_ffn) {
    const int r = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_ffn) return;
    const float* row = gu + static_cast<size_t>(r) * 2 * d_ffn;
    const int blk = j >> 7, in = j & 127;
    const float g = row[blk * 256 + in], u = row[blk * 256 + 128 + in];
    out[static_cast<size_t>(r) * d_ffn + j] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
}

__global__ void gather_rows_kernel(const float* __restrict__ resid, const int* __restrict__ row_of_slot,
                                   const int* __restrict__ slots, int d, float* __restrict__ hidden_layer) {
    const int i = blockIdx.x;
    const float4* src = reinterpret_cast<const float4*>(resid + static_cast<size_t>(row_of_slot[i]) * d);
    float4* dst = reinterpret_cast<float4*>(hidden_layer + static_cast<size_t>(slots[i]) * d);
    for (int j = threadIdx.x; j < d / 4; j += blockDim.x) dst[j] = src[j];
}

// Copies the (already rotated) k heads and the v heads of a prefilled token into its cache row.
__global__ void scatter_kv_kernel(const __nv_bfloat16* __restrict__ qkv, const int* __restrict__ dst_row, int dq,
                                  int dkv, __nv_bfloat16* __restrict__ kv_cache) {
    const int r = blockIdx.x;
    const uint4* src = reinterpret_cast<const uint4*>(qkv + static_cast<size_t>(r) * (dq + 2 * dkv) + dq);
    uint4* dst = reinterpret_cast<uint4*>(kv_cache + static_cast<size_t>(dst_row[r]) * (2 * dkv));
    for (int j = threadIdx.x; j < (2 * dkv) / 8; j += blockDim.x) dst[j] = src[j];
}

__global__ void convert_states_kernel(const float* __restrict__ src, void* __restrict__ dst, size_t n, int dtype) {
    const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (dtype == VERILLM_BF16) reinterpret_cast<__nv_bfloat16*>(dst)[i] = __float2bfloat16_rn(src[i]);
    else reinterpret_cast<float*>(dst)[i] = src[i];
}

// Recorded states entering a segment come from another party.  A value that is not finite, or so large that
// the first norm could overflow (|x| > kStateLimit), is replaced by zero and its sequence is marked in
// seq_flags: such a sequence is rejected as a whole, and nothing non-finite reaches the packed buffers that
// neighbouring sequences' attention tiles read.
constexpr float kStateLimit = 1e15f;
__global__ void load_states_kernel(const void* __restrict__ src, int dtype, size_t n, int d_model,
                                   const int* __restrict__ seq_of_token, int* __restrict__ seq_flags,
                                   float* __restrict__ dst) {
    const size_t i = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;  // n is a multiple of 4 (d_model % 64 == 0)
    float4 v;
    if (dtype == VERILLM_BF16) {
        const uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(src) + i);
        v = make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
    } else {
        v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(src) + i);
    }
    const bool ok0 = fabsf(v.x) <= kStateLimit, ok1 = fabsf(v.y) <= kStateLimit;  // false for NaN
    const bool ok2 = fabsf(v.z) <= kStateLimit, ok3 = fabsf(v.w) <= kStateLimit;
    if (!(ok0 && ok1 && ok2 && ok3)) {
        v.x = ok0 ? v.x : 0.f; v.y = ok1 ? v.y : 0.f; v.z = ok2 ? v.z : 0.f; v.w = ok3 ? v.w : 0.f;
        if (seq_flags != nullptr) atomicOr(seq_flags + seq_of_token[i / static_cast<size_t>(d_model)], 1);
    }
    *reinterpret_cast<float4*>(dst + i) = v;
}

// Exercise of the bounded wait every pipeline uses: one thread waits, with a short limit, on a barrier that
// nothing will ever signal (no copy in flight, no tensor memory held), and returns with the timeout recorded.
__global__ void wait_probe_kernel(long long limit_cycles, int* status, int* gave_up) {
    __shared__ __align__(8) uint64_t bar_word;
    if (threadIdx.x == 0) {
        const uint32_t bar = smem_u32(&bar_word);
        mbar_init(bar, 1);
        fence_mbar_init();
        const bool done = mbar_wait_limit(bar, 0u, status, limit_cycles);
        if (gave_up) *gave_up = done ? 0 : 1;
    }
}

__global__ void gather_tokens_kernel(const int* __restrict__ tokens, const int* __restrict__ src_index, int n,
                                     int* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = tokens[src_index[i]];
}

}  // namespace

// ------------------------------------------------------------------ launchers
cudaError_t launch_token_maps(const int* cu, int batch, int n_tokens, int* pos_of_token, int* seq_of_token,
                              cudaStream_t s) {
    if (n_tokens <= 0) return cudaSuccess;
    token_maps_kernel<<<(n_tokens + 255) / 256, 256, 0, s>>>(cu, batch, n_tokens, pos_of_token, seq_of_token);
    return cudaGetLastError();
}

cudaError_t launch_slot_lists(const int* tok_of_slot, int n_check, int n_tokens, int* slot_first, int* slot_next,
                              cudaStream_t s) {
    cudaError_t e = cudaMemsetAsync(slot_first, 0xFF, sizeof(int) * static_cast<size_t>(n_tokens), s);
    if (e != cudaSuccess || n_check <= 0) return e;
    slot_lists_kernel<<<(n_check + 255) / 256, 256, 0, s>>>(tok_of_slot, n_check, n_tokens, slot_first, slot_next);
    return cudaGetLastError();
}

cudaError_t launch_embed(const int* tokens, const void* table, int n_tokens, int d_model, int vocab, float* resid,
                         int* status, cudaStream_t s) {
    if (n_tokens <= 0) return cudaSuccess;
    embed_kernel<<<n_tokens, 128, 0, s>>>(tokens, reinterpret_cast<const __nv_bfloat16*>(table), d_model, vocab, resid,
                                          status);
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(const float* x, const void* gain, void* y, int rows, int d, float eps, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    rmsnorm_kernel<<<rows, kNormThreads, 0, s>>>(x, reinterpret_cast<const __nv_bfloat16*>(gain),
                                                 reinterpret_cast<__nv_bfloat16*>(y), d, eps);
    return cudaGetLastError();
}

cudaError_t launch_prenorm(const float* x, const void* gain, void* y, float* sumsq, int n_parts, int rows, int d,
                           cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    prenorm_kernel<<<rows, kNormThreads, 0, s>>>(x, reinterpret_cast<const __nv_bfloat16*>(gain),
                                                 reinterpret_cast<__nv_bfloat16*>(y), sumsq, n_parts, d);
    return cudaGetLastError();
}

cudaError_t launch_compare_rows(const float* hidden, const void* committed, int n_rows, int d, const CmpParams& cmp,
                                float* partials, cudaStream_t s) {
    if (n_rows <= 0) return cudaSuccess;
    compare_rows_kernel<<<(n_rows + 7) / 8, 256, 0, s>>>(hidden, committed, n_rows, d, cmp, partials);
    return cudaGetLastError();
}

cudaError_t launch_verdict(const float* partials, int n_layers, int n_check, int n_tiles, int d, const TolDev& tol,
                           const int* status, const int* seq_of_slot, const int* seq_flags, float* stats,
                           uint8_t* pos_ok, int* first_bad_layer, cudaStream_t s) {
    if (n_check <= 0) return cudaSuccess;
    verdict_kernel<<<(n_check + 3) / 4, 128, 0, s>>>(partials, n_layers, n_check, n_tiles, d, tol, status, seq_of_slot,
                                                      seq_flags, stats, pos_ok, first_bad_layer);
    return cudaGetLastError();
}

cudaError_t launch_seq_verdict(const float* stats, const uint8_t* pos_ok, const int* seq_of_slot, int n_check,
                               int n_layers, int batch, const int* status, const int* seq_flags, uint8_t* seq_ok,
                               float* seq_score, cudaStream_t s) {
    if (batch <= 0) return cudaSuccess;
    seq_verdict_kernel<<<batch, kSeqThreads, 0, s>>>(stats, pos_ok, seq_of_slot, n_check, n_layers, batch, status,
                                                        seq_flags, seq_ok, seq_score);
    return cudaGetLastError();
}

cudaError_t launch_threshold_sweep(const float* stats, const uint8_t* is_attack, int n_cells, const TolSet& tols,
                                   int n_variants, int* counts, cudaStream_t s) {
    if (n_cells <= 0 || n_variants <= 0) return cudaSuccess;
    threshold_sweep_kernel<<<(n_cells + 255) / 256, 256, 0, s>>>(stats, is_attack, n_cells, tols, n_variants, counts);
    return cudaGetLastError();
}

cudaError_t launch_argmax_reduce(const float* records, int rows, int n_tiles, const int* claimed, int* argmax_out,
                                 uint8_t* match_out, float* margin_out, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    argmax_reduce_kernel<<<(rows + 3) / 4, 128, 0, s>>>(reinterpret_cast<const float4*>(records), rows, n_tiles, claimed,
                                                       argmax_out, match_out, margin_out);
    return cudaGetLastError();
}

cudaError_t launch_spot_check(const float* hidden, int d, const int* rows, const int* cols, const float* ref, int n,
                              float eps, float theta, uint8_t* agree, float* p_hat, uint8_t* ok, cudaStream_t s) {
    if (n <= 0) return cudaErrorInvalidValue;
    spot_check_kernel<<<1, 256, 0, s>>>(hidden, d, rows, cols, ref, n, eps, theta, agree, p_hat, ok);
    return cudaGetLastError();
}

cudaError_t launch_skinny_gemm(const void* x, const void* w, float* out, int rows, int n, int k, int accumulate,
                               cudaStream_t s) {
    const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(x);
    for (int r0 = 0; r0 < rows; r0 += kSkinnyRows) {
        const int nr = rows - r0 < kSkinnyRows ? rows - r0 : kSkinnyRows;
        skinny_gemm_kernel<<<(n + 7) / 8, 256, 0, s>>>(xb + static_cast<size_t>(r0) * k,
                                                      reinterpret_cast<const __nv_bfloat16*>(w),
                                                      out + static_cast<size_t>(r0) * n, nr, n, k, accumulate);
    }
    return cudaGetLastError();
}

cudaError_t launch_decode_rope_append(const float* qkv, const int* tok_index, const int* positions, int rows,
                                      int n_heads, int n_kv_heads, int head_dim, const float2* rope_cs, void* q_out,
                                      void* kv_cache_layer, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    decode_rope_append_kernel<<<rows, 256, 0, s>>>(qkv, tok_index, positions, n_heads, n_kv_heads, head_dim, rope_cs,
                                                   reinterpret_cast<__nv_bfloat16*>(q_out),
                                                   reinterpret_cast<__nv_bfloat16*>(kv_cache_layer));
    return cudaGetLastError();
}

cudaError_t launch_decode_attention(const void* q, const void* kv_cache_layer, const int* seq_start,
                                    const int* positions, int rows, int n_heads, int n_kv_heads, int head_dim,
                                    int max_keys, void* out, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    const size_t smem = sizeof(float) * (static_cast<size_t>(head_dim) + static_cast<size_t>(max_keys));
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    // the attribute belongs to the (function, device) pair: remember what each device was given
    static size_t configured[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (smem > 48 * 1024 && smem > configured[dev]) {
        e = cudaFuncSetAttribute(decode_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        configured[dev] = smem;
    }
    decode_attention_kernel<<<dim3(rows, n_heads), 128, smem, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(q), reinterpret_cast<const __nv_bfloat16*>(kv_cache_layer), seq_start,
        positions, n_heads, n_kv_heads, head_dim, reinterpret_cast<__nv_bfloat16*>(out));
    return cudaGetLastError();
}

cudaError_t launch_swiglu_rows(const float* gu, void* out, int rows, int d_ffn, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    swiglu_rows_kernel<<<dim3((d_ffn + 255) / 256, rows), 256, 0, s>>>(gu, reinterpret_cast<__nv_bfloat16*>(out), d_ffn);
    return cudaGetLastError();
}

cudaError_t launch_gather_rows(const float* resid, const int* row_of_slot, const int* slots, int n_slots, int d,
                               float* hidden_layer, cudaStream_t s) {
    if (n_slots <= 0) return cudaSuccess;
    gather_rows_kernel<<<n_slots, 128, 0, s>>>(resid, row_of_slot, slots, d, hidden_layer);
    return cudaGetLastError();
}

cudaError_t launch_scatter_kv(const void* qkv, const int* dst_row, int rows, int n_heads, int n_kv_heads, int head_dim,
                              void* kv_cache_layer, cudaStream_t s) {
    if (rows <= 0) return cudaSuccess;
    scatter_kv_kernel<<<rows, 128, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(qkv), dst_row, n_heads * head_dim,
                                           n_kv_heads * head_dim, reinterpret_cast<__nv_bfloat16*>(kv_cache_layer));
    return cudaGetLastError();
}

cudaError_t launch_convert_states(const float* src, void* dst, size_t n, int commit_dtype, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    convert_states_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, s>>>(src, dst, n, commit_dtype);
    return cudaGetLastError();
}

cudaError_t launch_load_states(const void* src, int dtype, size_t n, int d_model, const int* seq_of_token,
                               int* seq_flags, float* resid, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    load_states_kernel<<<static_cast<unsigned>((n / 4 + 255) / 256), 256, 0, s>>>(src, dtype, n, d_model, seq_of_token,
                                                                                  seq_flags, resid);
    return cudaGetLastError();
}

cudaError_t launch_wait_probe(long long limit_cycles, int* status, int* gave_up, cudaStream_t s) {
    wait_probe_kernel<<<1, 32, 0, s>>>(limit_cycles, status, gave_up);
    return cudaGetLastError();
}

cudaError_t launch_gather_tokens(const int* tokens, const int* src_index, int n, int* out, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    gather_tokens_kernel<<<(n + 255) / 256, 256, 0, s>>>(tokens, src_index, n, out);
    return cudaGetLastError();
}

}  // namespace vl
