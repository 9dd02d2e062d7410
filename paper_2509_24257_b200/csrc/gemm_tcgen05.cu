// bf16 GEMM on the fifth-generation tensor cores: C[M][N] = A[M][K] * B[N][K]^T with fp32 accumulation
// in tensor memory, and the fused epilogues of the verifier's layer (rotary embedding, residual add,
// SwiGLU, gather-and-compare).  These are the projections inside F_i of S_{i+1} = F_i(S_i; W_i).
//
// Two kernels share the epilogues.  For M > 128 rows, clusters of two CTAs on neighbouring SMs share one
// 256 x 256 output tile (tcgen05.mma.cta_group::2; see gemm_bf16_tcgen05_pair below); for M <= 128 one
// persistent CTA per SM walks 128 x 256 tiles.  In both, warp 0 feeds a ring of shared-memory tiles with TMA
// (128-byte swizzle), warp 1 issues tcgen05.mma (one thread) into one of two 256-column TMEM accumulators,
// warps 2-5 drain the other accumulator (tcgen05.ld, one output row per thread) and run the epilogue, so the
// epilogue of a tile overlaps the main loop of the next.  Every mbarrier wait is bounded; a wait that runs out
// records VERILLM_DEV_WAIT_TIMEOUT and the CTA falls through to its tail, which frees the tensor memory.
#include "kernels.h"

namespace vl {

namespace {

constexpr int BM = kGemmBM, BN = kGemmBN, BK = kGemmBK;
constexpr int STAGES = 4;
constexpr int UMMA_K = 16;
constexpr int A_STAGE_BYTES = BM * BK * 2;  // 16 KiB
constexpr int B_STAGE_BYTES = BN * BK * 2;  // 32 KiB
constexpr int TILE_BYTES = STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);
constexpr int BAR_BYTES = 256;
constexpr int GEMM_SMEM = TILE_BYTES + BAR_BYTES + 1024;  // + slack for the 1024-byte alignment
constexpr int GEMM_THREADS = 192;
constexpr int TMEM_COLS = 512;  // two fp32 accumulators of 128 lanes x 256 columns

struct TileCoord {
    int m_idx, n_idx;
};

// Tiles are walked in bands of `group_m` tile-rows, row index fastest, so that the CTAs of a wave share
// weight tiles through L2 and a band's activation rows stay L2-resident across its column tiles.
__device__ __forceinline__ TileCoord tile_coord(int tile, int num_m, int num_n, int group_m) {
    const int per_group = group_m * num_n;
    const int g = tile / per_group;
    const int r = tile - g * per_group;
    const int m_first = g * group_m;
    const int gm = min(group_m, num_m - m_first);
    TileCoord c;
    c.n_idx = r / gm;
    c.m_idx = m_first + (r - c.n_idx * gm);
    return c;
}

__device__ __forceinline__ float silu_f(float z) { return z / (1.f + __expf(-z)); }

// Stores 32 consecutive fp32 accumulators of one row as bf16 (64 bytes, 16-byte vectors).
__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* dst, const float (&v)[32]) {
    uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint4 u;
        u.x = pack_bf16(v[8 * i + 0], v[8 * i + 1]);
        u.y = pack_bf16(v[8 * i + 2], v[8 * i + 3]);
        u.z = pack_bf16(v[8 * i + 4], v[8 * i + 5]);
        u.w = pack_bf16(v[8 * i + 6], v[8 * i + 7]);
        d4[i] = u;
    }
}

__device__ __forceinline__ void load_acc(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    __syncwarp();  // tcgen05.ld is warp-collective: lanes that skipped a store rejoin here
    tmem_ld32(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Factor of a folded RMSNorm for one row: rsqrt(mean x^2 + eps) from the producer's per-tile sums of squares,
// added in index order (1 when the projection's input was normalised beforehand).
__device__ __forceinline__ float row_rstd(const GemmParams& p, int row, bool row_ok) {
    if (p.sumsq_in == nullptr || !row_ok) return 1.f;
    const float* s = p.sumsq_in + static_cast<size_t>(row) * p.n_parts;
    float t = 0.f;
    for (int k = 0; k < p.n_parts; ++k) t += s[k];
    return rsqrtf(t * p.norm_inv_d + p.norm_eps);
}

// Epilogue of one tile for one thread (= one output row).  `trow` is the TMEM address of the thread's
// lane at column 0 of the accumulator.  tcgen05.ld is warp-collective: every branch that contains one
// is uniform across the warp (it depends on the tile only); row validity only predicates memory traffic.
template <int EPI>
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, uint32_t trow, int row, int n0, int n_idx) {
    const bool row_ok = row < p.M;

    if constexpr (EPI == EPI_ARGMAX) {
        // largest and second largest accumulator of the row inside this column tile (first column wins ties)
        float best = -INFINITY, second = -INFINITY;
        int best_col = n0;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            const int col = n0 + c * 32;
            if (col >= p.N) break;
            float v[32];
            load_acc(trow + c * 32, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float x = v[i];
                if (x > best) {
                    second = best;
                    best = x;
                    best_col = col + i;
                } else {
                    second = fmaxf(second, x);
                }
            }
        }
        if (row_ok && n0 < p.N) {
            const int n_tiles = (p.N + BN - 1) / BN;
            float4* rec = reinterpret_cast<float4*>(p.out) + static_cast<size_t>(row) * n_tiles + n_idx;
            *rec = make_float4(best, __int_as_float(best_col), second, 0.f);
        }
    } else if constexpr (EPI == EPI_STORE_BF16 || EPI == EPI_STORE_F32) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            const int col = n0 + c * 32;
            if (col >= p.N) break;
            float v[32];
            load_acc(trow + c * 32, v);
            if (!row_ok) continue;
            if constexpr (EPI == EPI_STORE_BF16) {
                store_bf16x32(reinterpret_cast<__nv_bfloat16*>(p.out) + static_cast<size_t>(row) * p.ldo + col, v);
            } else {
                float4* d4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) +
                                                       static_cast<size_t>(row) * p.ldo + col);
#pragma unroll
                for (int i = 0; i < 8; ++i) d4[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
        }
    } else if constexpr (EPI == EPI_RESID_ADD || EPI == EPI_RESID_ADD_COMPARE) {
        // in-place fp32 read-modify-write of the thread's row; the reads of the next 32-column chunk are
        // issued before the current chunk is combined, so their latency overlaps the TMEM load and the stores
        float* rrow = reinterpret_cast<float*>(p.out) + static_cast<size_t>(row_ok ? row : 0) * p.ldo + n0;
        const int n_chunks = min(BN, p.N - n0) / 32;
        float4 nxt[8];
        if (row_ok && n_chunks > 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) nxt[i] = reinterpret_cast<const float4*>(rrow)[i];
        }
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
            float4 cur[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) cur[i] = nxt[i];
            if (row_ok && c + 1 < n_chunks) {
#pragma unroll
                for (int i = 0; i < 8; ++i) nxt[i] = reinterpret_cast<const float4*>(rrow + (c + 1) * 32)[i];
            }
            float v[32];
            load_acc(trow + c * 32, v);
            if (!row_ok) continue;
            float4* d4 = reinterpret_cast<float4*>(rrow + c * 32);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 r = cur[i];
                r.x += v[4 * i];
                r.y += v[4 * i + 1];
                r.z += v[4 * i + 2];
                r.w += v[4 * i + 3];
                d4[i] = r;
            }
        }
    } else if constexpr (EPI == EPI_QKV_ROPE) {
        // heads of head_dim columns; inside a rotated head column i pairs with i + head_dim/2
        const int dh = p.head_dim;
        const int half_chunks = dh / 64;  // 32-column chunks per half head: 1 (dh 64) or 2 (dh 128)
        const int pos = row_ok ? p.pos_of_token[row] : 0;
        const float rs = row_rstd(p, row, row_ok);
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.out) + static_cast<size_t>(row_ok ? row : 0) * p.ldo;
#pragma unroll 1
        for (int hb = 0; hb < BN; hb += dh) {
            const int col0 = n0 + hb;
            if (col0 >= p.N) break;
            const bool rotate = col0 < p.rope_cols;
#pragma unroll 1
            for (int j = 0; j < half_chunks; ++j) {
                float lo[32], hi[32];
                load_acc(trow + hb + j * 32, lo);
                load_acc(trow + hb + dh / 2 + j * 32, hi);
                if (!row_ok) continue;
                if (rotate) {
                    const float2* cs = p.rope_cs + static_cast<size_t>(pos) * (dh / 2) + j * 32;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float2 t = __ldg(cs + i);
                        const float a = lo[i] * rs, b = hi[i] * rs;
                        lo[i] = a * t.x - b * t.y;
                        hi[i] = b * t.x + a * t.y;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        lo[i] *= rs;
                        hi[i] *= rs;
                    }
                }
                store_bf16x32(orow + col0 + j * 32, lo);
                store_bf16x32(orow + col0 + dh / 2 + j * 32, hi);
            }
        }
    } else if constexpr (EPI == EPI_SWIGLU) {
        // weight rows were interleaved in blocks of 128: tile columns [0,128) gate, [128,256) up
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.out) + static_cast<size_t>(row_ok ? row : 0) * p.ldo +
                              static_cast<size_t>(n_idx) * (BN / 2);
        if (n0 < p.N) {
            const float rs = row_rstd(p, row, row_ok);
#pragma unroll 1
            for (int c = 0; c < BN / 64; ++c) {
                float g[32], u[32];
                load_acc(trow + c * 32, g);
                load_acc(trow + BN / 2 + c * 32, u);
                if (!row_ok) continue;
#pragma unroll
                for (int i = 0; i < 32; ++i) g[i] = silu_f(g[i] * rs) * (u[i] * rs);
                store_bf16x32(orow + c * 32, g);
            }
        }
    }
}

constexpr int EPI_STAGE_BYTES = 4 * 32 * 32 * 4;  // pair kernel: one 32 x 32 fp32 block per epilogue warp

// Residual add of one tile with coalesced global traffic: each 32 x 32 block of the accumulator (one
// row per lane) is transposed through a swizzled shared-memory block so that eight lanes cover the 128
// contiguous bytes of one residual row.  `row0` is the first row of the warp's 32, `stage` its block.
__device__ __forceinline__ void epilogue_resid_staged(const GemmParams& p, uint32_t trow, int row0, int n0, int lane,
                                                      float4* stage, int n_idx, int n_tiles, bool final_part) {
    const int n_chunks = min(BN, p.N - n0) / 32;
    const int sub = lane >> 3, c4 = lane & 7;
    float* gbase = reinterpret_cast<float*>(p.out) + static_cast<size_t>(row0) * p.ldo + n0 + c4 * 4;
    // folded RMSNorm of the stream just updated: bf16(x * gain) beside it, and per row the sum of squares of
    // this tile's columns (lanes that share a row combine theirs at the end)
    const bool norm = p.norm_gain != nullptr && final_part;  // only the last K part of a tile holds final values
    const __nv_bfloat16* gain = reinterpret_cast<const __nv_bfloat16*>(p.norm_gain) + n0 + c4 * 4;
    __nv_bfloat16* xg = reinterpret_cast<__nv_bfloat16*>(p.xg_out) + static_cast<size_t>(row0) * p.N + n0 + c4 * 4;
    float ssq[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) ssq[it] = 0.f;
    float4 nxt[8];
    auto fetch = [&](int c, float4 (&dst)[8]) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int r = it * 4 + sub;
            // (read around L1: another SM may have added an earlier K part of this tile)
            if (row0 + r < p.M) dst[it] = __ldcg(reinterpret_cast<const float4*>(gbase + static_cast<size_t>(r) * p.ldo + c * 32));
        }
    };
    if (n_chunks > 0) fetch(0, nxt);
#pragma unroll 1
    for (int c = 0; c < n_chunks; ++c) {
        float4 cur[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) cur[i] = nxt[i];
        if (c + 1 < n_chunks) fetch(c + 1, nxt);
        float v[32];
        load_acc(trow + c * 32, v);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            stage[lane * 8 + (i ^ (lane & 7))] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        __syncwarp();
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
        if (norm) {
            const uint2 gv = __ldg(reinterpret_cast<const uint2*>(gain + c * 32));
            g0 = bf16_lo(gv.x); g1 = bf16_hi(gv.x); g2 = bf16_lo(gv.y); g3 = bf16_hi(gv.y);
        }
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int r = it * 4 + sub;
            const float4 a = stage[r * 8 + (c4 ^ (r & 7))];
            if (row0 + r < p.M) {
                float4 x = cur[it];
                x.x += a.x; x.y += a.y; x.z += a.z; x.w += a.w;
                *reinterpret_cast<float4*>(gbase + static_cast<size_t>(r) * p.ldo + c * 32) = x;
                if (norm) {
                    ssq[it] += (x.x * x.x + x.y * x.y) + (x.z * x.z + x.w * x.w);
                    uint2 o;
                    o.x = pack_bf16(x.x * g0, x.y * g1);
                    o.y = pack_bf16(x.z * g2, x.w * g3);
                    *reinterpret_cast<uint2*>(xg + static_cast<size_t>(r) * p.N + c * 32) = o;
                }
            }
        }
        __syncwarp();
    }
    if (norm) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            float s = ssq[it];
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 1);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 2);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 4);
            const int r = it * 4 + sub;
            if (c4 == 0 && row0 + r < p.M) p.sumsq_out[static_cast<size_t>(row0 + r) * n_tiles + n_idx] = s;
        }
    }
}

// Gather-and-compare on the rows of this tile that carry check slots: the thread re-reads the 256
// residual values it has just written, streams the committed values of each slot on the row
// (16-byte loads) and leaves one partial record per (slot, column tile).
__device__ __forceinline__ void compare_row(const GemmParams& p, int row, int n0, int n_idx, int n_tiles) {
    int slot = p.slot_first[row];
    const int ncols = min(BN, p.N - n0);
    const float* hrow = reinterpret_cast<const float*>(p.out) + static_cast<size_t>(row) * p.ldo + n0;
#pragma unroll 1
    for (int it = 0; slot >= 0 && it < p.n_check; ++it) {
        CmpAcc acc;
        acc.clear();
        float* hout = p.hidden_out ? p.hidden_out + static_cast<size_t>(slot) * p.N + n0 : nullptr;
        if (p.committed == nullptr) {
            // gather only (trace generation): copy the row segment, no statistics
            if (hout)
                for (int j = 0; j < ncols; j += 4)
                    *reinterpret_cast<float4*>(hout + j) = *reinterpret_cast<const float4*>(hrow + j);
            slot = p.slot_next[slot];
            continue;
        }
        if (p.cmp.commit_dtype == VERILLM_BF16) {
            const uint4* c4 = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.committed) +
                                                             static_cast<size_t>(slot) * p.N + n0);
#pragma unroll 1
            for (int j = 0; j < ncols; j += 8) {
                const uint4 cv = __ldg(c4 + j / 8);
                const float4 h0 = *reinterpret_cast<const float4*>(hrow + j);
                const float4 h1 = *reinterpret_cast<const float4*>(hrow + j + 4);
                acc.add_bf16x2(h0.x, h0.y, cv.x, p.cmp);
                acc.add_bf16x2(h0.z, h0.w, cv.y, p.cmp);
                acc.add_bf16x2(h1.x, h1.y, cv.z, p.cmp);
                acc.add_bf16x2(h1.z, h1.w, cv.w, p.cmp);
                if (hout) {
                    *reinterpret_cast<float4*>(hout + j) = h0;
                    *reinterpret_cast<float4*>(hout + j + 4) = h1;
                }
            }
        } else {
            const uint4* c4 = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(p.committed) +
                                                             static_cast<size_t>(slot) * p.N + n0);
#pragma unroll 1
            for (int j = 0; j < ncols; j += 4) {
                const uint4 cv = __ldg(c4 + j / 4);
                const float4 h0 = *reinterpret_cast<const float4*>(hrow + j);
                acc.add_f32(h0.x, cv.x, p.cmp);
                acc.add_f32(h0.y, cv.y, p.cmp);
                acc.add_f32(h0.z, cv.z, p.cmp);
                acc.add_f32(h0.w, cv.w, p.cmp);
                if (hout) *reinterpret_cast<float4*>(hout + j) = h0;
            }
        }
        acc.store(p.partials + (static_cast<size_t>(slot) * n_tiles + n_idx) * kNPart);
        slot = p.slot_next[slot];
    }
}

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    const uint32_t a_base = base;
    const uint32_t b_base = base + STAGES * A_STAGE_BYTES;
    const uint32_t bar_base = base + TILE_BYTES;
    // barrier words (8 bytes each): full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (base - raw) + TILE_BYTES + 8 * (2 * STAGES + 4));
    __shared__ int s_failed;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_m = (p.M + BM - 1) / BM;
    const int num_n = (p.N + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_kb = (p.K + BK - 1) / BK;
    const int group_m = p.group_m > 0 ? p.group_m : 16;

    if (threadIdx.x == 0) {
        s_failed = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full_bar(a), 1);
            mbar_init(acc_empty_bar(a), 4);  // one arrival per epilogue warp
        }
        fence_mbar_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    // everything above touched only this CTA's own resources: it may run under the previous kernel's tail
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const TileCoord tc = tile_coord(tile, num_m, num_n, group_m);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.status)) {
                        ok = false;
                        break;
                    }
                    mbar_arrive_expect_tx(full_bar(stage), A_STAGE_BYTES + B_STAGE_BYTES);
                    tma_load_2d(a_base + stage * A_STAGE_BYTES, &tmap_a, kb * BK, tc.m_idx * BM, full_bar(stage));
                    tma_load_2d(b_base + stage * B_STAGE_BYTES, &tmap_b, kb * BK, tc.n_idx * BN, full_bar(stage));
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) s_failed = 1;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, p.status)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t a_desc = umma_desc_k_sw128(a_base + stage * A_STAGE_BYTES);
                    const uint64_t b_desc = umma_desc_k_sw128(b_base + stage * B_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
                        umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(empty_bar(stage));  // the stage is free once these MMAs have read it
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(acc_full_bar(acc));
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
            if (!ok) s_failed = 1;
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps 2..5
        const int quarter = warp & 3;  // the TMEM lane quarter this warp may read
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const TileCoord tc = tile_coord(tile, num_m, num_n, group_m);
            if (!mbar_wait(acc_full_bar(acc), acc_phase, p.status)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const int row = tc.m_idx * BM + quarter * 32 + lane;
            const int n0 = tc.n_idx * BN;
            const uint32_t trow = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(acc * BN);
            epilogue_tile<EPI>(p, trow, row, n0, tc.n_idx);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(acc));  // accumulator may be overwritten
            if constexpr (EPI == EPI_RESID_ADD_COMPARE) {
                if (row < p.M && p.slot_first != nullptr) compare_row(p, row, n0, tc.n_idx, num_n);
                __syncwarp();
            }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
        if (!ok) s_failed = 1;
    }

    // ---------------------------------------------------------------- tail
    tc_fence_before();
    __syncthreads();
    if (s_failed) {
        // a wait gave up: let copies and MMAs still in flight land before the CTA's memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant: two CTAs on neighbouring SMs (a cluster of two) share one 256 x 256 output tile.
// Each CTA stages only its 128 rows of A and its 128-row half of B per K step (32 KiB instead of 48),
// the leader's MMA thread issues tcgen05.mma.cta_group::2 over both CTAs' shared memory and each CTA's
// TMEM receives its own 128 rows of the accumulator.  Per unit of math this cuts the L2 -> SM traffic
// by a third and leaves room for a 6-stage ring.  Barrier protocol: both CTAs' TMA loads count on the
// leader's full barrier; the leader's tcgen05.commit releases the stage / publishes the accumulator in
// both CTAs; the epilogue warps of both CTAs report the accumulator drained on the leader's barrier.
constexpr int P_STAGES = 6;
constexpr int P_B_STAGE_BYTES = 128 * BK * 2;  // half of the B tile
constexpr int P_STAGE_BYTES = A_STAGE_BYTES + P_B_STAGE_BYTES;
constexpr int P_TILE_BYTES = P_STAGES * P_STAGE_BYTES;
constexpr int P_GEMM_SMEM = P_TILE_BYTES + BAR_BYTES + EPI_STAGE_BYTES + 1024;

// Bounded wait until a global counter has reached `target` (written with atomicAdd by other CTAs of this launch).
__device__ __forceinline__ bool wait_counter(const int* counter, int target, int* status) {
    const volatile int* c = counter;
    const long long t0 = clock64();
    while (*c < target) {
        if (clock64() - t0 > kWaitLimitCycles) {
            if (status) atomicCAS(status, 0, VERILLM_DEV_WAIT_TIMEOUT);
            return false;
        }
    }
    return true;
}

// Work of one CTA pair.  Tiles are dealt round robin over `pairs_total` pairs; the last, partly filled round
// of a projection whose epilogue is additive (residual += accumulator) is cut along K into `split` parts so
// that it occupies all pairs: part q of a tile adds its partial product to the residual after part q-1 has
// (a per-tile counter in global memory orders them, so the sum is formed in a fixed order), and only the
// last part runs what needs the final values (folded norm, gather-and-compare).
struct SplitPlan {
    int full, rem, split;
};
__host__ __device__ inline SplitPlan split_plan(int num_tiles, int pairs_total, int num_kb, bool additive) {
    SplitPlan s;
    s.full = num_tiles / pairs_total;
    s.rem = num_tiles % pairs_total;
    s.split = 1;
    if (additive && s.rem > 0) {
        int sp = pairs_total / s.rem;
        if (sp > 4) sp = 4;
        if (sp > num_kb / 16) sp = num_kb / 16;  // parts of at least 16 K steps
        if (sp > 1) s.split = sp;
    }
    return s;
}
struct PairItem {
    int tile, kb0, kb1, part, n_parts, rem_idx;
};
// k-th item of pair x; false past the end.
__device__ __forceinline__ bool pair_item(const SplitPlan& s, int pairs_total, int num_kb, int x, int k, PairItem& it) {
    it.kb0 = 0; it.kb1 = num_kb; it.part = 0; it.n_parts = 1; it.rem_idx = -1;
    if (k < s.full) {
        it.tile = x + k * pairs_total;
        return true;
    }
    if (k > s.full || x >= s.rem * s.split) return false;
    it.rem_idx = x % s.rem;
    it.part = x / s.rem;
    it.n_parts = s.split;
    it.tile = s.full * pairs_total + it.rem_idx;
    it.kb0 = it.part * num_kb / s.split;
    it.kb1 = (it.part + 1) * num_kb / s.split;
    return true;
}

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_tcgen05_pair(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                       const __grid_constant__ GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t a_base = base;
    const uint32_t b_base = base + P_STAGES * A_STAGE_BYTES;
    const uint32_t bar_base = base + P_TILE_BYTES;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (P_STAGES + s); };
    auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * P_STAGES + a); };
    auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * P_STAGES + 2 + a); };
    const uint32_t tmem_slot = bar_base + 8u * (2 * P_STAGES + 4);
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (base - raw) + P_TILE_BYTES + 8 * (2 * P_STAGES + 4));
    __shared__ int s_failed;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: leader (issues the MMAs), 1: peer
    const int pair_id = blockIdx.x >> 1;
    const int num_m = (p.M + 2 * BM - 1) / (2 * BM);  // tile-rows of 256
    const int num_n = (p.N + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_kb = (p.K + BK - 1) / BK;
    const int group_m = p.group_m > 0 ? p.group_m : 8;
    constexpr bool kAdditive = EPI == EPI_RESID_ADD || EPI == EPI_RESID_ADD_COMPARE;
    const SplitPlan plan = split_plan(num_tiles, p.pairs_total, num_kb, kAdditive && p.split_flags != nullptr);
    PairItem item;

    if (threadIdx.x == 0) {
        s_failed = 0;
        for (int s = 0; s < P_STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full_bar(a), 1);
            mbar_init(acc_empty_bar(a), 8);  // four epilogue warps in each CTA of the pair
        }
        fence_mbar_init();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive();  // both CTAs' barriers exist before anyone signals across the pair
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    // everything above touched only the pair's own resources: it may run under the previous kernel's tail
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (each CTA its own tiles)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int k = 0; ok && pair_item(plan, p.pairs_total, num_kb, pair_id, k, item); ++k) {
                const TileCoord tc = tile_coord(item.tile, num_m, num_n, group_m);
                const int a_row = tc.m_idx * 2 * BM + static_cast<int>(rank) * BM;
                const int b_row = tc.n_idx * BN + static_cast<int>(rank) * 128;
                for (int kb = item.kb0; kb < item.kb1; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * P_STAGE_BYTES);  // both CTAs' bytes
                    tma_load_2d_pair(a_base + stage * A_STAGE_BYTES, &tmap_a, kb * BK, a_row, leader_full);
                    tma_load_2d_pair(b_base + stage * P_B_STAGE_BYTES, &tmap_b, kb * BK, b_row, leader_full);
                    if (++stage == P_STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) s_failed = 1;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int k = 0; ok && pair_item(plan, p.pairs_total, num_kb, pair_id, k, item); ++k) {
                if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, p.status)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
                for (int kb = item.kb0; kb < item.kb1; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t a_desc = umma_desc_k_sw128(a_base + stage * A_STAGE_BYTES);
                    const uint64_t b_desc = umma_desc_k_sw128(b_base + stage * P_B_STAGE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk)
                        umma_bf16_pair(d_tmem, a_desc + 2u * kk, b_desc + 2u * kk, idesc, (kb != item.kb0 || kk != 0) ? 1u : 0u);
                    umma_commit_pair(empty_bar(stage));  // frees the stage in both CTAs
                    if (++stage == P_STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(acc_full_bar(acc));  // accumulator ready in both CTAs
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
            if (!ok) s_failed = 1;
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps 2..5 (both CTAs)
        const int quarter = warp & 3;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int k = 0; ok && pair_item(plan, p.pairs_total, num_kb, pair_id, k, item); ++k) {
            const TileCoord tc = tile_coord(item.tile, num_m, num_n, group_m);
            if (!mbar_wait(acc_full_bar(acc), acc_phase, p.status)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const int row = tc.m_idx * 2 * BM + static_cast<int>(rank) * BM + quarter * 32 + lane;
            const int n0 = tc.n_idx * BN;
            const uint32_t trow = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(acc * BN);
            const bool final_part = item.part == item.n_parts - 1;
            if constexpr (kAdditive) {
                if (item.part > 0) {
                    // the earlier parts of this tile (eight epilogue warps each) must have added theirs
                    uint32_t done = 1u;
                    if (lane == 0) done = wait_counter(p.split_flags + item.rem_idx, 8 * item.part, p.status) ? 1u : 0u;
                    if (__shfl_sync(0xFFFFFFFFu, done, 0) == 0u) {
                        ok = false;
                        break;
                    }
                    __threadfence();
                }
                float4* stage = reinterpret_cast<float4*>(smem_raw + (base - raw) + P_TILE_BYTES + BAR_BYTES) + quarter * 256;
                epilogue_resid_staged(p, trow, row - lane, n0, lane, stage, tc.n_idx, num_n, final_part);
            } else {
                epilogue_tile<EPI>(p, trow, row, n0, tc.n_idx);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(acc), 0));  // the leader collects all 8
            if constexpr (kAdditive) {
                if (!final_part) {  // publish this warp's share of the partial sum
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) atomicAdd(p.split_flags + item.rem_idx, 1);
                }
            }
            if constexpr (EPI == EPI_RESID_ADD_COMPARE) {
                if (final_part && row < p.M && p.slot_first != nullptr) compare_row(p, row, n0, tc.n_idx, num_n);
                __syncwarp();
            }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
        if (!ok) s_failed = 1;
    }

    // ---------------------------------------------------------------- tail: neither CTA leaves while the other may
    // still read its shared memory or signal its barriers
    tc_fence_before();
    __syncthreads();
    if (s_failed) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {
        }
        __syncthreads();
    }
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

template <int EPI>
cudaError_t launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int num_sms,
                        cudaStream_t stream) {
    const int num_tiles = ((p.M + 2 * BM - 1) / (2 * BM)) * ((p.N + BN - 1) / BN);
    if (num_tiles <= 0) return cudaSuccess;
    GemmParams q = p;
    q.pairs_total = num_sms / 2;
    constexpr bool additive = EPI == EPI_RESID_ADD || EPI == EPI_RESID_ADD_COMPARE;
    const SplitPlan plan = split_plan(num_tiles, q.pairs_total, (p.K + BK - 1) / BK, additive && p.split_flags != nullptr);
    if (plan.split > 1) {  // the per-tile part counters of the last round start at zero
        if (!p.split_prezeroed) {
            const cudaError_t e = cudaMemsetAsync(p.split_flags, 0, sizeof(int) * plan.rem, stream);
            if (e != cudaSuccess) return e;
        }
    } else {
        q.split_flags = nullptr;
    }
    const int pairs = plan.full > 0 ? q.pairs_total : plan.rem * plan.split;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = P_GEMM_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap_prologue ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, gemm_bf16_tcgen05_pair<EPI>, ta, tb, q);
}

template <int EPI>
cudaError_t init_pair() {
    return cudaFuncSetAttribute(gemm_bf16_tcgen05_pair<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_GEMM_SMEM);
}

template <int EPI>
cudaError_t launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int num_sms,
                       cudaStream_t stream) {
    const int num_tiles = ((p.M + BM - 1) / BM) * ((p.N + BN - 1) / BN);
    if (num_tiles <= 0) return cudaSuccess;
    const int grid = num_tiles < num_sms ? num_tiles : num_sms;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = GEMM_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap_prologue ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_bf16_tcgen05<EPI>, ta, tb, p);
}

template <int EPI>
cudaError_t init_one() {
    return cudaFuncSetAttribute(gemm_bf16_tcgen05<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

}  // namespace

cudaError_t gemm_init() {
    cudaError_t e;
    if ((e = init_one<EPI_STORE_BF16>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_STORE_F32>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_QKV_ROPE>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_RESID_ADD>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_SWIGLU>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_RESID_ADD_COMPARE>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_STORE_BF16>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_STORE_F32>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_QKV_ROPE>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_RESID_ADD>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_SWIGLU>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_RESID_ADD_COMPARE>()) != cudaSuccess) return e;
    if ((e = init_one<EPI_ARGMAX>()) != cudaSuccess) return e;
    if ((e = init_pair<EPI_ARGMAX>()) != cudaSuccess) return e;
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    return cudaSuccess;
}

int make_tmap_bf16_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld_elems,
                      uint32_t box_rows) {
    if (!g_encode) return -1;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || (ld_elems * 2) % 16 != 0) return -2;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld_elems * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -3;
}

cudaError_t launch_gemm(int epilogue, const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int num_sms,
                        cudaStream_t stream) {
    if (p.pair) {  // tb must then be encoded with 128-row boxes (each CTA loads half of the B tile)
        switch (epilogue) {
            case EPI_STORE_BF16: return launch_pair<EPI_STORE_BF16>(ta, tb, p, num_sms, stream);
            case EPI_STORE_F32: return launch_pair<EPI_STORE_F32>(ta, tb, p, num_sms, stream);
            case EPI_QKV_ROPE: return launch_pair<EPI_QKV_ROPE>(ta, tb, p, num_sms, stream);
            case EPI_RESID_ADD: return launch_pair<EPI_RESID_ADD>(ta, tb, p, num_sms, stream);
            case EPI_SWIGLU: return launch_pair<EPI_SWIGLU>(ta, tb, p, num_sms, stream);
            case EPI_RESID_ADD_COMPARE: return launch_pair<EPI_RESID_ADD_COMPARE>(ta, tb, p, num_sms, stream);
            case EPI_ARGMAX: return launch_pair<EPI_ARGMAX>(ta, tb, p, num_sms, stream);
            default: return cudaErrorInvalidValue;
        }
    }
    switch (epilogue) {
        case EPI_STORE_BF16: return launch_one<EPI_STORE_BF16>(ta, tb, p, num_sms, stream);
        case EPI_STORE_F32: return launch_one<EPI_STORE_F32>(ta, tb, p, num_sms, stream);
        case EPI_QKV_ROPE: return launch_one<EPI_QKV_ROPE>(ta, tb, p, num_sms, stream);
        case EPI_RESID_ADD: return launch_one<EPI_RESID_ADD>(ta, tb, p, num_sms, stream);
        case EPI_SWIGLU: return launch_one<EPI_SWIGLU>(ta, tb, p, num_sms, stream);
        case EPI_RESID_ADD_COMPARE: return launch_one<EPI_RESID_ADD_COMPARE>(ta, tb, p, num_sms, stream);
        case EPI_ARGMAX: return launch_one<EPI_ARGMAX>(ta, tb, p, num_sms, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace vl
