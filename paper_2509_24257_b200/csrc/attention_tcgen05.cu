// Causal grouped-query attention over packed sequences on the fifth-generation tensor cores:
// softmax(q k^T / sqrt(dh) + causal mask) v, flash style (the one causal pass of Full-Sequence Prefill, Eq. 1).
//
// A unit of work is 128 query rows of one (sequence, query head), walking the key/value tiles of 64
// positions up to the diagonal.  CTAs are persistent, two per SM: each takes its share of the units
// (longest first, dealt in rounds of alternating direction) and treats their tiles as one stream, so that
// the loads and the first Q K^T of the next unit run under the softmax tail and the output pass of the
// current one.  Three single-thread roles drive the asynchronous work: warp 5 issues the TMA loads of the
// key (3 tiles) and value (2 tiles) rings (128-byte swizzle); warp 4 fetches Q and issues S = Q K^T; warp 6
// issues O += P V (tcgen05.mma).  The products have a thread each because issuing one tcgen05 instruction
// costs its thread several tens of cycles whatever its size.
// Warps 0-3 own one query row per thread: they read S from TMEM, keep the online softmax (reference
// maximum and running sum, fp32, exp2, packed fp32 arithmetic) in registers and write P as packed bf16
// back over the S columns, from where the second product takes it as its A operand; the registers that
// held S receive the next tile's S while P is still being finished.  O accumulates in TMEM across tiles;
// it is rescaled only when a row's maximum has grown by more than 2^8 since the reference maximum was
// taken (probabilities stay below 256, the normalisation by the running sum cancels the stale reference).
// S of a tile is started as soon as the P V two tiles back has read P out of its buffer (two S/P
// buffers).  V is consumed as it lies in memory ([key][dh], an MN-major B operand).  Every wait is
// bounded; on a timeout the CTA records the error, drains and frees its TMEM.
#include "kernels.h"

namespace vl {

namespace {

constexpr int TC_BM = 128;
constexpr int TC_BN = 64;
constexpr int TC_THREADS = 224;
constexpr int TC_KSTAGES = 3;  // key tiles in flight (a key tile is free as soon as its Q K^T is done); value tiles: 2
constexpr int TC_TMEM_COLS = 256;  // S0/P0 [0,64), S1/P1 [64,128), O [128, 128 + dh)
constexpr int TC_TABLE = 48;  // work units per CTA kept in shared memory (two CTAs of head_dim 128 then just fit an SM)
constexpr float TC_RESCALE_LOG2 = 8.f;  // rescale O when a row maximum exceeds its reference by this (log2)

template <int DH>
struct TcSmem {
    static constexpr uint32_t Q_BYTES = TC_BM * DH * 2;
    static constexpr uint32_t KV_BYTES = TC_BN * DH * 2;
    static constexpr uint32_t K_OFF = Q_BYTES;
    static constexpr uint32_t V_OFF = K_OFF + TC_KSTAGES * KV_BYTES;
    static constexpr uint32_t BAR_OFF = V_OFF + 2 * KV_BYTES;
    static constexpr uint32_t TABLE_OFF = BAR_OFF + 256;  // the CTA's first TC_TABLE work units, 16 bytes each
    static constexpr uint32_t TOTAL = TABLE_OFF + TC_TABLE * 16;
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

// 32-byte store (the address must be 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&r)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
                 "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
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

// One unit of work: 128 query rows of one (sequence, query head).
struct AttnItem {
    int seq_start, len, q0, head, kvh, nb;
};

// The CTA's k-th unit of work.  Units are ordered by decreasing number of key tiles (last query tile of
// every (sequence, head) first, heads of a KV group adjacent) and dealt to the CTAs in rounds whose
// direction alternates, so that every CTA receives a similar total.  Returns false past the end; a unit
// that lies beyond its sequence's length has nb = 0.
__device__ __forceinline__ bool attn_item(int k, const int* __restrict__ cu_seqlens, int batch, int n_qblocks,
                                          int n_heads, int n_kv_heads, AttnItem& w) {
    const int G = static_cast<int>(gridDim.x), x = static_cast<int>(blockIdx.x);
    const int pairs = n_heads * batch;
    const int idx = k * G + ((k & 1) ? G - 1 - x : x);
    if (idx >= n_qblocks * pairs) return false;
    const int qb = n_qblocks - 1 - idx / pairs;
    const int rem = idx % pairs;
    const int seq = rem / n_heads;
    w.head = rem % n_heads;
    w.kvh = w.head * n_kv_heads / n_heads;
    w.seq_start = __ldg(cu_seqlens + seq);
    w.len = __ldg(cu_seqlens + seq + 1) - w.seq_start;
    w.q0 = qb * TC_BM;
    w.nb = w.q0 < w.len ? (min(w.q0 + TC_BM, w.len) - 1) / TC_BN + 1 : 0;  // causal: tiles up to the last valid row
    return true;
}

template <int DH>
__global__ void __launch_bounds__(TC_THREADS, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
               const int* __restrict__ cu_seqlens, int batch, int n_qblocks, int n_heads, int n_kv_heads,
               __nv_bfloat16* __restrict__ out, int* status) {
    using L = TcSmem<DH>;
    constexpr int QB = DH / 64;  // 64-column blocks per head
    extern __shared__ __align__(1024) uint8_t tc_smem[];

    const uint32_t sbase = smem_u32(tc_smem);
    if ((sbase & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, VERILLM_DEV_WAIT_TIMEOUT);
        return;
    }
    const int dq = n_heads * DH, dkv = n_kv_heads * DH;

    const uint32_t q_s = sbase;
    auto k_s = [&](int b) { return sbase + L::K_OFF + b * L::KV_BYTES; };
    auto v_s = [&](int b) { return sbase + L::V_OFF + b * L::KV_BYTES; };
    const uint32_t bar = sbase + L::BAR_OFF;
    const uint32_t q_full = bar, q_empty = bar + 8;
    auto p_ready = [&](int b) { return bar + 16 + 8 * b; };
    auto s_full = [&](int b) { return bar + 32 + 8 * b; };
    auto k_full = [&](int b) { return bar + 48 + 8 * b; };
    auto k_empty = [&](int b) { return bar + 72 + 8 * b; };
    auto v_full = [&](int b) { return bar + 96 + 8 * b; };
    auto v_empty = [&](int b) { return bar + 112 + 8 * b; };
    const uint32_t tmem_slot = bar + 128;
    volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(tc_smem + L::BAR_OFF + 128);
    volatile int* failed = reinterpret_cast<volatile int*>(tc_smem + L::BAR_OFF + 132);

    // Work units are looked up once, by many threads at a time, and kept in shared memory (head, kv head and
    // tile count packed into one word, bit 31 = past the end); only a CTA with more than TC_TABLE units
    // computes the later ones on the spot.
    int4* table = reinterpret_cast<int4*>(tc_smem + L::TABLE_OFF);
    for (int k = threadIdx.x; k < TC_TABLE; k += TC_THREADS) {
        AttnItem w;
        const bool valid = attn_item(k, cu_seqlens, batch, n_qblocks, n_heads, n_kv_heads, w);
        table[k] = valid ? make_int4(w.seq_start, w.len, w.q0, w.head | (w.kvh << 10) | (w.nb << 20))
                         : make_int4(0, 0, 0, static_cast<int>(0x80000000u));
    }
    auto item = [&](int k, AttnItem& w) {
        if (k >= TC_TABLE) return attn_item(k, cu_seqlens, batch, n_qblocks, n_heads, n_kv_heads, w);
        const int4 t = table[k];
        if (t.w < 0) return false;
        w.seq_start = t.x;
        w.len = t.y;
        w.q0 = t.z;
        w.head = t.w & 1023;
        w.kvh = (t.w >> 10) & 1023;
        w.nb = t.w >> 20;
        return true;
    };

    // The CTA's key/value tiles form one stream over all its units: tile g of the stream uses key slot
    // g % 3 (phase g / 3), value slot and S/P buffer g & 1 (phase g / 2); the unit's Q is phase `unit`.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        *failed = 0;
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
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
    // up to here only the CTA's own resources and the sequence boundaries (written before the chain of layer
    // kernels started) were touched: all of it may run under the tail of the projection that produces q, k, v
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 5) {
        // ------------------------------------------------------------ TMA producer of keys and values (one thread)
        // Two cursors walk the CTA's tile stream: keys run three tiles ahead of the tile whose Q K^T has
        // completed, values two tiles ahead of the tile whose P V has completed.
        if (lane == 0) {
            struct Cursor {
                int k, j;  // unit number, tile inside the unit
                AttnItem w;
                bool valid;
            };
            auto seek = [&](Cursor& c) {  // first unit from c.k on that has tiles
                c.j = 0;
                while ((c.valid = item(c.k, c.w)) && c.w.nb == 0) ++c.k;
            };
            auto step = [&](Cursor& c) {
                if (++c.j == c.w.nb) {
                    ++c.k;
                    seek(c);
                }
            };
            Cursor kc, vc;
            kc.k = 0;
            seek(kc);
            vc = kc;
            int gk = 0, gv = 0;  // stream index of the next key / value tile to fetch
            auto load_k = [&]() {
                const int kb = gk % TC_KSTAGES;
                mbar_arrive_expect_tx(k_full(kb), L::KV_BYTES);
#pragma unroll
                for (int c = 0; c < QB; ++c)
                    tma_load_2d(k_s(kb) + c * (TC_BN * 128), &tmap_kv, dq + kc.w.kvh * DH + c * 64,
                                kc.w.seq_start + kc.j * TC_BN, k_full(kb));
                step(kc);
                ++gk;
            };
            auto load_v = [&]() {
                const int b = gv & 1;
                mbar_arrive_expect_tx(v_full(b), L::KV_BYTES);
#pragma unroll
                for (int c = 0; c < QB; ++c)
                    tma_load_2d(v_s(b) + c * (TC_BN * 128), &tmap_kv, dq + dkv + vc.w.kvh * DH + c * 64,
                                vc.w.seq_start + vc.j * TC_BN, v_full(b));
                step(vc);
                ++gv;
            };
            for (int n = 0; n < TC_KSTAGES && kc.valid; ++n) load_k();
            for (int n = 0; n < 2 && vc.valid; ++n) load_v();
            bool ok = true;
            for (int g = 0; (kc.valid || vc.valid) && ok; ++g) {
                if (kc.valid) {  // key tile g is free once its Q K^T is done
                    if (!mbar_wait(k_empty(g % TC_KSTAGES), (g / TC_KSTAGES) & 1, status)) { ok = false; break; }
                    load_k();
                }
                if (vc.valid) {  // value tile g is free once its P V is done
                    if (!mbar_wait(v_empty(g & 1), (g >> 1) & 1, status)) { ok = false; break; }
                    load_v();
                }
            }
            if (!ok) *failed = 1;
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ Q K^T issuer (one thread); also fetches Q
        // Issuing one tcgen05 instruction costs this thread several tens of cycles whatever its size, so the
        // two products have an issuing thread each: S of a tile is started as soon as its buffer is free (the
        // P V two tiles back complete) without queueing behind the P V issue of the tile in between.
        if (lane == 0) {
            bool ok = true;
            // operand descriptors: a step of 16 elements along K inside a swizzled 128-byte row adds 2
            // (16-byte units), the next 64-column block adds a whole tile
            const uint64_t q_desc = umma_desc_k_sw128(q_s);
            const uint64_t k_desc0 = umma_desc_k_sw128(k_s(0));
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, TC_BN);
            AttnItem w;
            int g = 0, unit = 0;
            for (int k = 0; ok && item(k, w); ++k) {
                if (w.nb == 0) continue;
                // the single Q buffer is free once every Q K^T of the previous unit has completed; the softmax
                // of that unit's last tiles and its output pass hide this fetch
                if (unit > 0 && !mbar_wait(q_empty, (unit - 1) & 1, status)) { ok = false; break; }
                mbar_arrive_expect_tx(q_full, L::Q_BYTES);
#pragma unroll
                for (int c = 0; c < QB; ++c)
                    tma_load_2d(q_s + c * (TC_BM * 128), &tmap_q, w.head * DH + c * 64, w.seq_start + w.q0, q_full);
                if (!mbar_wait(q_full, unit & 1, status)) { ok = false; break; }
                for (int t = 0; t < w.nb; ++t, ++g) {  // S[g & 1] = Q K_t^T : M 128, N 64, K = DH
                    const int b = g & 1, kb = g % TC_KSTAGES;
                    // keys first (they arrive early); the buffer is free once P V of stream tile g-2 has read P out of it
                    if (!mbar_wait(k_full(kb), (g / TC_KSTAGES) & 1, status)) { ok = false; break; }
                    if (g >= 2 && !mbar_wait(v_empty(b), ((g - 2) >> 1) & 1, status)) { ok = false; break; }
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
                umma_commit(q_empty);
                ++unit;
            }
            if (!ok) *failed = 1;
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------ P V issuer (one thread)
        if (lane == 0) {
            bool ok = true;
            const uint64_t v_desc0 = umma_desc_mn_sw128(v_s(0), TC_BN * 128);
            // O (+)= P V_j : M 128, N = DH, K = 64 keys; P from TMEM (8 packed columns per 16 keys), V is the
            // MN-major B operand (16 keys = two 8-row swizzle atoms = 2048 bytes).  The first tile of a unit
            // overwrites O: its P arrives only after every softmax warp has read the previous unit's O.
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, DH) | (1u << 16);
            AttnItem w;
            int g = 0;
            for (int k = 0; ok && item(k, w); ++k) {
                for (int j = 0; j < w.nb; ++j, ++g) {
                    const int b = g & 1;
                    if (!mbar_wait(v_full(b), (g >> 1) & 1, status)) { ok = false; break; }
                    if (!mbar_wait(p_ready(b), (g >> 1) & 1, status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t vd = v_desc0 + static_cast<uint64_t>(b * (L::KV_BYTES >> 4));
#pragma unroll
                    for (int kk = 0; kk < TC_BN / 16; ++kk)
                        umma_bf16_ts(tmem_base + 128u, tmem_base + static_cast<uint32_t>(b * TC_BN + kk * 8),
                                     vd + static_cast<uint64_t>(kk * (2048 >> 4)), idesc, (j | kk) != 0 ? 1u : 0u);
                    umma_commit(v_empty(b));  // P V complete: frees the value tile and the S/P buffer, O is current
                }
            }
            if (!ok) *failed = 1;
        }
    } else {
        // ------------------------------------------------------------ softmax / output warps: one row per thread
        const int r = warp * 32 + lane;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        const uint32_t o_addr = lane_base + 128u;
        const float scale_log2 = rsqrtf(static_cast<float>(DH)) * 1.4426950408889634f;
        bool ok = true;
        AttnItem w;
        int g0 = 0;  // stream index of the unit's first tile
        for (int unit_k = 0; ok && item(unit_k, w); ++unit_k) {
        if (w.nb == 0) continue;
        const int nb = w.nb, q0 = w.q0, len = w.len;
        const int row = q0 + r;  // position inside the sequence
        float m_ref = -INFINITY, l_run = 0.f;
        // S of tile j sits in registers when iteration j starts: each half is fetched (asynchronously) as soon
        // as the previous tile's exponentials have consumed the registers it lands in, so the TMEM read
        // latency overlaps the arithmetic.
        uint32_t v0[32], v1[32];
        if (!mbar_wait(s_full(g0 & 1), (g0 >> 1) & 1, status)) { ok = false; break; }
        tc_fence_after();
        tmem_ld32(lane_base + static_cast<uint32_t>((g0 & 1) * TC_BN), v0);
        tmem_ld32(lane_base + static_cast<uint32_t>((g0 & 1) * TC_BN) + 32, v1);
        tmem_ld_wait_regs(v0);
        tmem_ld_wait_regs(v1);
        for (int j = 0; j < nb && ok; ++j) {
            const int g = g0 + j;  // stream index: buffer g & 1, phase g / 2
            const int b = g & 1;
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
                    // (the previous tile is phase (g-1)/2 of its value barrier; the next phase of that barrier
                    // needs the P after this one, so the parity cannot be ambiguous here)
                    if (!mbar_wait(v_empty(b ^ 1), ((g - 1) >> 1) & 1, status)) { ok = false; break; }
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
                early = __all_sync(0xFFFFFFFFu, mbar_test_wait(s_full(b ^ 1), ((g + 1) >> 1) & 1));
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
                    if (!mbar_wait(s_full(b ^ 1), ((g + 1) >> 1) & 1, status)) { ok = false; break; }
                    tc_fence_after();
                    tmem_ld32(s_next, v0);
                    tmem_ld32(s_next + 32, v1);
                }
                tmem_ld_wait_regs(v0);
                tmem_ld_wait_regs(v1);
            }
        }
        if (!ok) break;
        // The unit's last P V must have landed before O is read (the products complete in issue order).  Its
        // value barrier completes no further phase until this warp has delivered another P, so the wait holds
        // however late it is reached.
        const int g_last = g0 + nb - 1;
        if (!mbar_wait(v_empty(g_last & 1), (g_last >> 1) & 1, status)) { ok = false; break; }
        tc_fence_after();
        {
            const float inv = 1.f / l_run;
            __nv_bfloat16* dst = out + static_cast<size_t>(w.seq_start + (row < len ? row : 0)) * dq + w.head * DH;
#pragma unroll 1
            for (int c = 0; c < DH / 64; ++c) {  // two 32-column blocks in flight
                uint32_t o0[32], o1[32];
                tmem_ld32(o_addr + c * 64, o0);
                tmem_ld32(o_addr + c * 64 + 32, o1);
                tmem_ld_wait_regs(o0);
                tmem_ld_wait_regs(o1);
                if (row < len) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {  // 32-byte stores: one full sector per row and instruction
                        uint32_t u[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            u[i] = pack_bf16(__uint_as_float(o0[16 * q + 2 * i]) * inv, __uint_as_float(o0[16 * q + 2 * i + 1]) * inv);
                        st_global_v8(dst + c * 64 + 16 * q, u);
                    }
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        uint32_t u[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            u[i] = pack_bf16(__uint_as_float(o1[16 * q + 2 * i]) * inv, __uint_as_float(o1[16 * q + 2 * i + 1]) * inv);
                        st_global_v8(dst + c * 64 + 32 + 16 * q, u);
                    }
                }
                __syncwarp();
            }
        }
        // the reads of O above are ordered before the next unit's first P V by the fence that precedes the
        // arrival on its P barrier
        g0 += nb;
        }  // units
        if (!ok) *failed = 1;
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
                                int* status, int num_sms, int overlap_prologue, cudaStream_t stream) {
    if (batch <= 0 || max_seqlen <= 0) return cudaSuccess;
    const int n_qblocks = (max_seqlen + TC_BM - 1) / TC_BM;
    if (n_heads > 1024 || n_qblocks * (TC_BM / TC_BN) > 2047) return cudaErrorInvalidValue;  // packed work-unit fields
    // persistent CTAs, two per SM (each holds half of the SM's tensor memory)
    const long long units = static_cast<long long>(n_qblocks) * n_heads * batch;
    const dim3 grid(static_cast<unsigned>(units < 2LL * num_sms ? units : 2LL * num_sms));
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(TC_THREADS);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prologue ? 1 : 0;
    if (head_dim == 64) {
        cfg.dynamicSmemBytes = TcSmem<64>::TOTAL;
        return cudaLaunchKernelEx(&cfg, attn_tc_kernel<64>, tmap_q, tmap_kv, cu_seqlens_dev, batch, n_qblocks, n_heads,
                                  n_kv_heads, o, status);
    }
    if (head_dim == 128) {
        cfg.dynamicSmemBytes = TcSmem<128>::TOTAL;
        return cudaLaunchKernelEx(&cfg, attn_tc_kernel<128>, tmap_q, tmap_kv, cu_seqlens_dev, batch, n_qblocks, n_heads,
                                  n_kv_heads, o, status);
    }
    return cudaErrorInvalidValue;
}

}  // namespace vl
