// Causal grouped-query attention over packed sequences on the fifth-generation tensor cores:
// softmax(q k^T / sqrt(dh) + causal mask) v, flash style ("a single forward pass under the causal mask").
//
// One CTA owns 128 query rows of one (sequence, query head) and walks the key/value tiles of 64 positions
// up to the diagonal.  Three single-thread roles drive the asynchronous work: warp 5 issues the TMA loads
// of Q and of separate key (3 tiles) and value (2 tiles) rings (128-byte swizzle); warp 4 issues
// S = Q K^T and warp 6 issues O += P V (tcgen05.mma).  The products have a thread each because issuing
// one tcgen05 instruction costs its thread several tens of cycles whatever its size.
// Warps 0-3 own one query row per thread: they read S from TMEM, keep the online softmax (reference
// maximum and running sum, fp32, exp2, packed fp32 arithmetic) in registers and write P as packed bf16
// back over the S columns, from where the second product takes it as its A operand; the registers that
// held S receive the next tile's S while P is still being finished.  O accumulates in TMEM across tiles;
// it is rescaled only when a row's maximum has grown by more than 2^8 since the reference maximum was
// taken (probabilities stay below 256, the normalisation by the running sum cancels the stale reference).
// S_{t} is started as soon as P V_{t-2} has read P_{t-2} out of its buffer (two S/P buffers).  Two CTAs
// share an SM.  V is consumed as it lies in memory ([key][dh], an MN-major B operand).  Every wait is
// bounded; on a timeout the CTA records the error, drains and frees its TMEM.
#include "kernels.h"

namespace vl {

namespace {

constexpr int TC_BM = 128;
constexpr int TC_BN = 64;
constexpr int TC_THREADS = 224;
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

// max of three values in one instruction
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// packed fp32 pairs: d = a * b + c and d = a + b on both halves at once
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return reinterpret_cast<float2&>(d);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return reinterpret_cast<float2&>(d);
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
    const uint32_t q_full = bar;
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

    if (warp == 5) {
        // ------------------------------------------------------------ TMA producer (one thread)
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
            mbar_arrive_expect_tx(q_full, L::Q_BYTES);
#pragma unroll
            for (int c = 0; c < QB; ++c) tma_load_2d(q_s + c * (TC_BM * 128), &tmap_q, head * DH + c * 64, seq_start + q0, q_full);
            for (int j = 0; j < TC_KSTAGES && j < nb; ++j) load_k(j);
            for (int j = 0; j < 2 && j < nb; ++j) load_v(j);
            for (int j = 0; j < nb && ok; ++j) {
                if (j + TC_KSTAGES < nb) {  // key tile j is free once its Q K^T is done
                    if (!mbar_wait(k_empty(j % TC_KSTAGES), (j / TC_KSTAGES) & 1, status)) { ok = false; break; }
                    load_k(j + TC_KSTAGES);
                }
                if (j + 2 < nb) {  // value tile j is free once its P V is done
                    if (!mbar_wait(v_empty(j & 1), (j >> 1) & 1, status)) { ok = false; break; }
                    load_v(j + 2);
                }
            }
            if (!ok) *failed = 1;
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ Q K^T issuer (one thread)
        // Issuing one tcgen05 instruction costs this thread several tens of cycles whatever its size, so the
        // two products have an issuing thread each: S_{t} is started as soon as its buffer is free (P V_{t-2}
        // complete) without queueing behind the P V issue of the tile in between.
        if (lane == 0) {
            bool ok = true;
            // operand descriptors: a step of 16 elements along K inside a swizzled 128-byte row adds 2
            // (16-byte units), the next 64-column block adds a whole tile
            const uint64_t q_desc = umma_desc_k_sw128(q_s);
            const uint64_t k_desc0 = umma_desc_k_sw128(k_s(0));
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, TC_BN);
            ok = mbar_wait(q_full, 0, status);
            for (int t = 0; t < nb && ok; ++t) {  // S[t & 1] = Q K_t^T : M 128, N 64, K = DH
                const int b = t & 1, kb = t % TC_KSTAGES;
                // keys first (they arrive early); the buffer is free once P V_{t-2} has read P_{t-2} out of it
                if (!mbar_wait(k_full(kb), (t / TC_KSTAGES) & 1, status)) { ok = false; break; }
                if (t >= 2 && !mbar_wait(v_empty(b), ((t - 2) >> 1) & 1, status)) { ok = false; break; }
                tc_fence_after();
                const uint64_t kd = k_desc0 + static_cast<uint64_t>(kb * (L::KV_BYTES >> 4));
#pragma unroll
                for (int kk = 0; kk < DH / 16; ++kk) {
                    const uint64_t a = q_desc + static_cast<uint64_t>((kk / 4) * ((TC_BM * 128) >> 4) + 2 * (kk % 4));
                    const uint64_t bd = kd + static_cast<uint64_t>((kk / 4) * ((TC_BN * 128) >> 4) + 2 * (kk % 4));
                    umma_bf16(tmem_base + static_cast<uint32_t>(b * TC_BN), a, bd, idesc, kk != 0 ? 1u : 0u);
                }
                umma_commit(s_full(b));
                umma_commit(k_empty(kb));  // the key tile can be replaced once this product is done
            }
            if (!ok) *failed = 1;
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------ P V issuer (one thread)
        if (lane == 0) {
            bool ok = true;
            const uint64_t v_desc0 = umma_desc_mn_sw128(v_s(0), TC_BN * 128);
            // O (+)= P V_j : M 128, N = DH, K = 64 keys; P from TMEM (8 packed columns per 16 keys), V is the
            // MN-major B operand (16 keys = two 8-row swizzle atoms = 2048 bytes)
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, DH) | (1u << 16);
            for (int j = 0; j < nb && ok; ++j) {
                const int b = j & 1;
                if (!mbar_wait(v_full(b), (j >> 1) & 1, status)) { ok = false; break; }
                if (!mbar_wait(p_ready(b), (j >> 1) & 1, status)) { ok = false; break; }
                tc_fence_after();
                const uint64_t vd = v_desc0 + static_cast<uint64_t>(b * (L::KV_BYTES >> 4));
#pragma unroll
                for (int kk = 0; kk < TC_BN / 16; ++kk)
                    umma_bf16_ts(tmem_base + 128u, tmem_base + static_cast<uint32_t>(b * TC_BN + kk * 8),
                                 vd + static_cast<uint64_t>(kk * (2048 >> 4)), idesc, (j | kk) != 0 ? 1u : 0u);
                umma_commit(v_empty(b));  // P V_j complete: frees the value tile and the S/P buffer, O is current
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
        // S of tile j sits in registers when iteration j starts: each half is fetched (asynchronously) as soon
        // as the previous tile's exponentials have consumed the registers it lands in, so the TMEM read
        // latency overlaps the arithmetic.  Q K^T runs one tile ahead, so S_{j+1} is normally complete by then.
        uint32_t v0[32], v1[32];
        if (!mbar_wait(s_full(0), 0, status)) ok = false;
        if (ok) {
            tc_fence_after();
            tmem_ld32(lane_base, v0);
            tmem_ld32(lane_base + 32, v1);
            tmem_ld_wait_regs(v0);
            tmem_ld_wait_regs(v1);
        }
        for (int j = 0; j < nb && ok; ++j) {
            const int b = j & 1;
            const int key0 = j * TC_BN;
            const bool need_mask = key0 + TC_BN - 1 > q0;  // uniform over the CTA
            const uint32_t s_addr = lane_base + static_cast<uint32_t>(b * TC_BN);
            const uint32_t s_next = lane_base + static_cast<uint32_t>((b ^ 1) * TC_BN);
            // raw scores: mask the future on the diagonal tiles only, then one maximum per row
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (key0 + i > row) v0[i] = 0xFF800000u;       // -inf
                    if (key0 + 32 + i > row) v1[i] = 0xFF800000u;
                }
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four independent chains
#pragma unroll
            for (int i = 0; i < 32; ++i) mx4[i & 3] = max3(mx4[i & 3], __uint_as_float(v0[i]), __uint_as_float(v1[i]));
            float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            mx *= scale_log2;  // the scale is positive: max commutes with it
            if (j == 0) {
                m_ref = mx;  // tile 0 holds key 0 <= row: finite
            } else {
                const bool grow = mx > m_ref + TC_RESCALE_LOG2;
                if (__any_sync(0xFFFFFFFFu, grow)) {
                    // O holds tiles 0..j-1 relative to the old reference: wait for P V_{j-1}, then rescale
                    const float corr = grow ? ex2(m_ref - mx) : 1.f;
                    // (tile j-1 is phase (j-1)/2 of its value barrier; the next phase of that barrier needs
                    // P_{j+1}, so the parity cannot be ambiguous here)
                    if (!mbar_wait(v_empty(b ^ 1), ((j - 1) >> 1) & 1, status)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < DH / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(o_addr + c * 32, o);
                        tmem_ld_wait_regs(o);
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
                        tmem_st32(o_addr + c * 32, o);
                    }
                    tmem_st_wait();
                    l_run *= corr;
                    if (grow) m_ref = mx;
                }
            }
            // probabilities relative to the reference maximum, packed bf16 over the first 32 S columns; each
            // half is written back as soon as it is complete, and the same registers then receive S_{j+1}
            const bool more = j + 1 < nb;
            // two elements per instruction for the scaling and the row sum (packed fp32 arithmetic)
            const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(-m_ref, -m_ref);
            float2 rs2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            uint32_t pk0[16], pk1[16];  // separate registers: the first store may still be reading its sources
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float2 t = ffma2(make_float2(__uint_as_float(v0[2 * i]), __uint_as_float(v0[2 * i + 1])), sc2, nm2);
                const float2 e = make_float2(ex2(t.x), ex2(t.y));
                rs2[i & 1] = fadd2(rs2[i & 1], e);
                pk0[i] = pack_bf16(e.x, e.y);
            }
            tmem_st16(s_addr, pk0);
            // S_{j+1}: fetched here if it is already complete (it then lands while the second half is
            // computed), otherwise after the second half, so that P_j is never held back by the wait
            bool early = false;
            if (more) {
                early = __all_sync(0xFFFFFFFFu, mbar_test_wait(s_full(b ^ 1), ((j + 1) >> 1) & 1));
                if (early) {
                    tc_fence_after();
                    tmem_ld32(s_next, v0);
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float2 t = ffma2(make_float2(__uint_as_float(v1[2 * i]), __uint_as_float(v1[2 * i + 1])), sc2, nm2);
                const float2 e = make_float2(ex2(t.x), ex2(t.y));
                rs2[i & 1] = fadd2(rs2[i & 1], e);
                pk1[i] = pack_bf16(e.x, e.y);
            }
            tmem_st16(s_addr + 16, pk1);
            if (early) tmem_ld32(s_next + 32, v1);
            l_run += (rs2[0].x + rs2[0].y) + (rs2[1].x + rs2[1].y);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_ready(b));  // 32 arrivals on one barrier word would serialise
            if (more) {
                if (!early) {
                    if (!mbar_wait(s_full(b ^ 1), ((j + 1) >> 1) & 1, status)) { ok = false; break; }
                    tc_fence_after();
                    tmem_ld32(s_next, v0);
                    tmem_ld32(s_next + 32, v1);
                }
                tmem_ld_wait_regs(v0);
                tmem_ld_wait_regs(v1);
            }
        }
        // The last P V must have landed before O is read (the products complete in issue order).  Its value
        // barrier completes no further phase afterwards, so this wait holds however late it is reached.
        if (ok && !mbar_wait(v_empty((nb - 1) & 1), ((nb - 1) >> 1) & 1, status)) ok = false;
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
