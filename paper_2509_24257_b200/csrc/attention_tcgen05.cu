// Causal grouped-query attention over packed sequences on the fifth-generation tensor cores:
// softmax(q k^T / sqrt(dh) + causal mask) v, flash style ("a single forward pass under the causal mask").
//
// One CTA owns 128 query rows of one (sequence, query head) and walks the key/value tiles of 64 positions
// up to the diagonal.  Warp 4 (one thread) drives everything asynchronous: TMA loads of Q and of separate
// key (3 tiles) and value (2 tiles) rings (128-byte swizzle), S = Q K^T and O += P V as tcgen05.mma.
// Warps 0-3 own one query row per thread: they read S from TMEM, keep the online softmax (reference
// maximum and running sum, fp32, exp2) in registers and write P as packed bf16 back over the S columns,
// from where the second product takes it as its A operand.  O accumulates in TMEM across tiles; it is
// rescaled only when a row's maximum has grown by more than 2^8 since the reference maximum was taken
// (probabilities stay below 256, the normalisation by the running sum cancels the stale reference), so
// the softmax of tile j+1 overlaps P V of tile j, and Q K^T runs one tile ahead (two S buffers).  Two CTAs
// share an SM.  V is consumed as it lies in memory ([key][dh], an MN-major B operand).  Every wait is
// bounded; on a timeout the CTA records the error, drains and frees its TMEM.
#include "kernels.h"

namespace vl {

namespace {

constexpr int TC_BM = 128;
constexpr int TC_BN = 64;
constexpr int TC_THREADS = 160;
constexpr int TC_KSTAGES = 3;  // key tiles in flight (a key tile is free as soon as its Q K^T is done); value tiles: 2
constexpr int TC_TMEM_COLS = 256;  // S0/P0 [0,64), S1/P1 [64,128), O [128, 128 + dh)
constexpr float TC_RESCALE_LOG2 = 8.f;  // rescale O when a row maximum exceeds its reference by this (log2)

template <int DH>
struct TcSmem {
    static constexpr uint32_t Q_BYTES = TC_BM * DH * 2;
    static constexpr uint32_t KV_BYTES = TC_BN * DH * 2;
    static constexpr uint32_t K_OFF = Q_BYTES;
    static constexpr uint32_t V_OFF = K_OFF + TC_KSTAGES * KV_BYTES;
    static constexpr uint32_t BAR_OFF = V_OFF + 2 * KV_BYTES;
    static constexpr uint32_t TOTAL = BAR_OFF + 256;
};

// K-major operand whose rows are 128 bytes (64 bf16) with the 128-byte swizzle: see umma_desc_k_sw128.
// MN-major operand (V as stored: [key][dh]): 64 dh-columns contiguous per key row of 128 bytes, 8 key rows
// per 1024-byte swizzle atom; `lbo_bytes` separates the 64-column blocks of a wider head.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t tile_smem, uint32_t lbo_bytes) {
    const uint64_t lo = static_cast<uint64_t>((tile_smem & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16);
    const uint64_t hi = static_cast<uint64_t>(1024u >> 4) | (1ull << 14) | (2ull << 29);
    return lo | (hi << 32);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int DH>
__global__ void __launch_bounds__(TC_THREADS, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
               const int* __restrict__ cu_seqlens, int batch, int n_qblocks, int n_heads, int n_kv_heads,
               __nv_bfloat16* __restrict__ out, int* status) {
    using L = TcSmem<DH>;
    constexpr int QB = DH / 64;  // 64-column blocks per head
    extern __shared__ __align__(1024) uint8_t tc_smem[];

    // Work order: all (sequence, head) pairs of the last query tile first, then the tile before it, ...: the
    // CTAs with the most key tiles start first (longest-processing-time order), heads of a KV group adjacent.
    const int pairs = n_heads * batch;
    const int qb = n_qblocks - 1 - static_cast<int>(blockIdx.x) / pairs;
    const int rem = static_cast<int>(blockIdx.x) % pairs;
    const int seq = rem / n_heads, head = rem % n_heads;
    const int seq_start = cu_seqlens[seq];
    const int len = cu_seqlens[seq + 1] - seq_start;
    const int q0 = qb * TC_BM;
    if (q0 >= len) return;
    const uint32_t sbase = smem_u32(tc_smem);
    if ((sbase & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, VERILLM_DEV_WAIT_TIMEOUT);
        return;
    }
    const int kvh = head * n_kv_heads / n_heads;
    const int dq = n_heads * DH, dkv = n_kv_heads * DH;
    const int last_row = min(q0 + TC_BM, len) - 1;
    const int nb = last_row / TC_BN + 1;  // causal: key tiles up to the last valid row

    const uint32_t q_s = sbase;
    auto k_s = [&](int b) { return sbase + L::K_OFF + b * L::KV_BYTES; };
    auto v_s = [&](int b) { return sbase + L::V_OFF + b * L::KV_BYTES; };
    const uint32_t bar = sbase + L::BAR_OFF;
    const uint32_t q_full = bar, o_done = bar + 8;
    auto p_ready = [&](int b) { return bar + 16 + 8 * b; };
    auto s_full = [&](int b) { return bar + 32 + 8 * b; };
    auto k_full = [&](int b) { return bar + 48 + 8 * b; };
    auto k_empty = [&](int b) { return bar + 72 + 8 * b; };
    auto v_full = [&](int b) { return bar + 96 + 8 * b; };
    auto v_empty = [&](int b) { return bar + 112 + 8 * b; };
    const uint32_t tmem_slot = bar + 128;
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(tc_smem + L::BAR_OFF + 128);
    volatile int* failed = reinterpret_cast<volatile int*>(tc_smem + L::BAR_OFF + 132);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        *failed = 0;
        mbar_init(q_full, 1);
        mbar_init(o_done, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(p_ready(b), 4);  // one arrival per softmax warp
            mbar_init(s_full(b), 1);
            mbar_init(v_full(b), 1);
            mbar_init(v_empty(b), 1);
        }
        for (int b = 0; b < TC_KSTAGES; ++b) {
            mbar_init(k_full(b), 1);
            mbar_init(k_empty(b), 1);
        }
        fence_mbar_init();
    }
    if (warp == 4) {
        tmem_alloc(tmem_slot, TC_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 4) {
        // ------------------------------------------------------------ TMA + MMA driver (one thread)
        if (lane == 0) {
            bool ok = true;
            auto load_k = [&](int j) {
                const int kb = j % TC_KSTAGES;
                mbar_arrive_expect_tx(k_full(kb), L::KV_BYTES);
#pragma unroll
                for (int c = 0; c < QB; ++c)
                    tma_load_2d(k_s(kb) + c * (TC_BN * 128), &tmap_kv, dq + kvh * DH + c * 64, seq_start + j * TC_BN, k_full(kb));
            };
            auto load_v = [&](int j) {
                const int b = j & 1;
                mbar_arrive_expect_tx(v_full(b), L::KV_BYTES);
#pragma unroll
                for (int c = 0; c < QB; ++c)
                    tma_load_2d(v_s(b) + c * (TC_BN * 128), &tmap_kv, dq + dkv + kvh * DH + c * 64, seq_start + j * TC_BN, v_full(b));
            };
            auto issue_qk = [&](int j) {  // S[j & 1] = Q K_j^T : M 128, N 64, K = DH
                const int b = j & 1, kb = j % TC_KSTAGES;
                constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, TC_BN);
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint64_t a = umma_desc_k_sw128(q_s + (kk / 4) * (TC_BM * 128)) + 2u * (kk % 4);
                    const uint64_t bd = umma_desc_k_sw128(k_s(kb) + (kk / 4) * (TC_BN * 128)) + 2u * (kk % 4);
                    umma_bf16(tmem_base + static_cast<uint32_t>(b * TC_BN), a, bd, idesc, kk != 0 ? 1u : 0u);
                }
                umma_commit(s_full(b));
                umma_commit(k_empty(kb));  // the key tile can be replaced once this product is done
            };
            mbar_arrive_expect_tx(q_full, L::Q_BYTES);
#pragma unroll
            for (int c = 0; c < QB; ++c) tma_load_2d(q_s + c * (TC_BM * 128), &tmap_q, head * DH + c * 64, seq_start + q0, q_full);
            for (int j = 0; j < TC_KSTAGES && j < nb; ++j) load_k(j);
            for (int j = 0; j < 2 && j < nb; ++j) load_v(j);
            ok = mbar_wait(q_full, 0, status) && mbar_wait(k_full(0), 0, status);
            if (ok) {
                tc_fence_after();
                issue_qk(0);
            }
            for (int j = 0; j < nb && ok; ++j) {
                const int b = j & 1;
                if (j + 1 < nb) {  // Q K^T runs one tile ahead of the softmax
                    if (!mbar_wait(k_full((j + 1) % TC_KSTAGES), ((j + 1) / TC_KSTAGES) & 1, status)) { ok = false; break; }
                    tc_fence_after();
                    issue_qk(j + 1);
                }
                if (j + TC_KSTAGES < nb) {  // key tile j is consumed (its product was issued an iteration ago): refill
                    if (!mbar_wait(k_empty(j % TC_KSTAGES), (j / TC_KSTAGES) & 1, status)) { ok = false; break; }
                    load_k(j + TC_KSTAGES);
                }
                if (!mbar_wait(v_full(b), (j >> 1) & 1, status)) { ok = false; break; }
                if (!mbar_wait(p_ready(b), (j >> 1) & 1, status)) { ok = false; break; }
                tc_fence_after();
                {   // O (+)= P V_j : M 128, N = DH, K = 64 keys; P from TMEM (8 packed columns per 16 keys),
                    // V is the MN-major B operand
                    constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, DH) | (1u << 16);
#pragma unroll
                    for (int kk = 0; kk < TC_BN / 16; ++kk) {
                        const uint64_t bd = umma_desc_mn_sw128(v_s(b) + kk * 2048, TC_BN * 128);
                        umma_bf16_ts(tmem_base + 128u, tmem_base + static_cast<uint32_t>(b * TC_BN + kk * 8), bd, idesc,
                                     (j | kk) != 0 ? 1u : 0u);
                    }
                }
                umma_commit(o_done);
                umma_commit(v_empty(b));
                if (j >= 1 && j + 1 < nb) {  // value tile j-1 was consumed an iteration ago: fetch tile j+1 into its place
                    if (!mbar_wait(v_empty(b ^ 1), ((j - 1) >> 1) & 1, status)) { ok = false; break; }
                    load_v(j + 1);
                }
            }
            if (!ok) *failed = 1;
        }
    } else {
        // ------------------------------------------------------------ softmax / output warps: one row per thread
        const int r = warp * 32 + lane;
        const int row = q0 + r;  // position inside the sequence
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        const uint32_t o_addr = lane_base + 128u;
        const float scale_log2 = rsqrtf(static_cast<float>(DH)) * 1.4426950408889634f;
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < nb; ++j) {
            const int b = j & 1;
            if (!mbar_wait(s_full(b), (j >> 1) & 1, status)) { ok = false; break; }
            tc_fence_after();
            const int key0 = j * TC_BN;
            const bool need_mask = key0 + TC_BN - 1 > q0;  // uniform over the CTA
            const uint32_t s_addr = lane_base + static_cast<uint32_t>(b * TC_BN);
            uint32_t v0[32], v1[32];
            tmem_ld32(s_addr, v0);
            tmem_ld32(s_addr + 32, v1);
            tmem_ld_wait();
            // raw scores: mask the future on the diagonal tiles only, then one maximum per row
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (key0 + i > row) v0[i] = 0xFF800000u;       // -inf
                    if (key0 + 32 + i > row) v1[i] = 0xFF800000u;
                }
            }
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fmaxf(__uint_as_float(v0[i]), __uint_as_float(v1[i])));
            mx *= scale_log2;  // the scale is positive: max commutes with it
            if (j == 0) {
                m_ref = mx;  // tile 0 holds key 0 <= row: finite
            } else {
                const bool grow = mx > m_ref + TC_RESCALE_LOG2;
                if (__any_sync(0xFFFFFFFFu, grow)) {
                    // O holds tiles 0..j-1 relative to the old reference: wait for P V_{j-1}, then rescale
                    const float corr = grow ? ex2(m_ref - mx) : 1.f;
                    if (!mbar_wait(o_done, (j - 1) & 1, status)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < DH / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(o_addr + c * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
                        tmem_st32(o_addr + c * 32, o);
                    }
                    tmem_st_wait();
                    l_run *= corr;
                    if (grow) m_ref = mx;
                }
            }
            // probabilities relative to the reference maximum, packed bf16 over the first 32 S columns
            float rs = 0.f;
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float a0 = ex2(fmaf(__uint_as_float(v0[2 * i]), scale_log2, -m_ref));
                const float a1 = ex2(fmaf(__uint_as_float(v0[2 * i + 1]), scale_log2, -m_ref));
                const float b0 = ex2(fmaf(__uint_as_float(v1[2 * i]), scale_log2, -m_ref));
                const float b1 = ex2(fmaf(__uint_as_float(v1[2 * i + 1]), scale_log2, -m_ref));
                rs += (a0 + a1) + (b0 + b1);
                pk[i] = pack_bf16(a0, a1);
                pk[16 + i] = pack_bf16(b0, b1);
            }
            l_run += rs;
            tmem_st32(s_addr, pk);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready(b));  // 32 arrivals on one barrier word would serialise
        }
        // The last P V must have landed before O is read.  A parity wait can only tell apart the current
        // phase and the one before it, and so far only P V_{nb-3} is known to be complete (Q K^T of the last
        // tile was issued ahead of P V_{nb-2}): wait for the phases one at a time.
        if (ok && nb >= 2 && !mbar_wait(o_done, (nb - 2) & 1, status)) ok = false;
        if (ok && !mbar_wait(o_done, (nb - 1) & 1, status)) ok = false;
        if (!ok) *failed = 1;
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l_run;
            __nv_bfloat16* dst = out + static_cast<size_t>(seq_start + (row < len ? row : 0)) * dq + head * DH;
#pragma unroll 1
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(o_addr + c * 32, o);
                tmem_ld_wait();
                if (row < len) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 u;
                        u.x = pack_bf16(__uint_as_float(o[8 * q + 0]) * inv, __uint_as_float(o[8 * q + 1]) * inv);
                        u.y = pack_bf16(__uint_as_float(o[8 * q + 2]) * inv, __uint_as_float(o[8 * q + 3]) * inv);
                        u.z = pack_bf16(__uint_as_float(o[8 * q + 4]) * inv, __uint_as_float(o[8 * q + 5]) * inv);
                        u.w = pack_bf16(__uint_as_float(o[8 * q + 6]) * inv, __uint_as_float(o[8 * q + 7]) * inv);
                        reinterpret_cast<uint4*>(dst + c * 32)[q] = u;
                    }
                }
                __syncwarp();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*failed) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {
        }
        __syncthreads();
    }
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TC_TMEM_COLS);
    }
}

}  // namespace

cudaError_t attention_tc_init() {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(TcSmem<64>::TOTAL));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(TcSmem<128>::TOTAL));
}

cudaError_t launch_attention_tc(const CUtensorMap& tmap_q, const CUtensorMap& tmap_kv, const int* cu_seqlens_dev,
                                int batch, int max_seqlen, int n_heads, int n_kv_heads, int head_dim, void* out,
                                int* status, cudaStream_t stream) {
    if (batch <= 0 || max_seqlen <= 0) return cudaSuccess;
    const int n_qblocks = (max_seqlen + TC_BM - 1) / TC_BM;
    const dim3 grid(static_cast<unsigned>(n_qblocks) * n_heads * batch);
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out);
    if (head_dim == 64)
        attn_tc_kernel<64><<<grid, TC_THREADS, TcSmem<64>::TOTAL, stream>>>(tmap_q, tmap_kv, cu_seqlens_dev, batch,
                                                                           n_qblocks, n_heads, n_kv_heads, o, status);
    else if (head_dim == 128)
        attn_tc_kernel<128><<<grid, TC_THREADS, TcSmem<128>::TOTAL, stream>>>(tmap_q, tmap_kv, cu_seqlens_dev, batch,
                                                                             n_qblocks, n_heads, n_kv_heads, o, status);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace vl
