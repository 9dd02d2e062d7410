// Causal grouped-query attention over packed sequences, flash style: softmax(q k^T / sqrt(dh) + causal
// mask) v with an online softmax kept per warp in fp32 ("a single forward pass under the causal mask").
//
// One CTA owns 128 consecutive query rows of one (sequence, query head): 8 warps x 16 rows.  Key/value
// tiles of 64 positions stream through a double-buffered cp.async ring; q k^T and p v run on
// mma.sync m16n8k16 (bf16 in, fp32 out) with fragments fetched by ldmatrix from XOR-swizzled shared
// memory.  The four query heads of a KV group are neighbours in the grid, so their key/value tiles are
// shared through L2.
#include "kernels.h"

namespace vl {

namespace {

constexpr int ATT_BM = 128;
constexpr int ATT_BN = 64;
constexpr int ATT_THREADS = 256;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory tiles are [rows][DH] bf16; the 16-byte chunk c of row r lives at chunk c ^ (r & 7).
template <int DH>
__device__ __forceinline__ uint32_t tile_addr(uint32_t base, int row, int chunk) {
    return base + static_cast<uint32_t>(row * (DH * 2) + ((chunk ^ (row & 7)) << 4));
}

// Copies `rows` rows of DH bf16 (global row stride ld elements) into a swizzled tile; row indices at or
// beyond `valid_rows` re-read the last valid row (finite data that the causal mask discards).
template <int DH>
__device__ __forceinline__ void load_tile(uint32_t smem_base, const __nv_bfloat16* g, int ld, int rows, int first_row,
                                          int valid_rows) {
    constexpr int CH = DH / 8;
    for (int i = threadIdx.x; i < rows * CH; i += ATT_THREADS) {
        const int r = i / CH, c = i - r * CH;
        int gr = first_row + r;
        gr = gr < valid_rows ? gr : valid_rows - 1;
        cp_async16(tile_addr<DH>(smem_base, r, c), g + static_cast<size_t>(gr) * ld + c * 8);
    }
}

template <int DH>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attn_causal_gqa_kernel(const __nv_bfloat16* __restrict__ qkv, const int* __restrict__ cu_seqlens, int n_heads,
                       int n_kv_heads, __nv_bfloat16* __restrict__ out) {
    extern __shared__ __align__(128) uint8_t att_smem[];
    const int seq = blockIdx.z, head = blockIdx.y;
    const int seq_start = cu_seqlens[seq];
    const int len = cu_seqlens[seq + 1] - seq_start;
    const int qb = static_cast<int>(gridDim.x) - 1 - static_cast<int>(blockIdx.x);  // longest rows first
    const int q0 = qb * ATT_BM;
    if (q0 >= len) return;

    const int kvh = head * n_kv_heads / n_heads;
    const int dq = n_heads * DH, dkv = n_kv_heads * DH;
    const int ld = dq + 2 * dkv;
    const __nv_bfloat16* qg = qkv + static_cast<size_t>(seq_start) * ld + head * DH;
    const __nv_bfloat16* kg = qkv + static_cast<size_t>(seq_start) * ld + dq + kvh * DH;
    const __nv_bfloat16* vg = kg + dkv;

    const uint32_t sbase = smem_u32(att_smem);
    const uint32_t q_s = sbase;
    constexpr uint32_t Q_BYTES = ATT_BM * DH * 2, KV_BYTES = ATT_BN * DH * 2;
    auto k_s = [&](int b) { return sbase + Q_BYTES + b * KV_BYTES; };
    auto v_s = [&](int b) { return sbase + Q_BYTES + 2 * KV_BYTES + b * KV_BYTES; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int r0 = q0 + warp * 16;                        // first query row of this warp
    const int last_row = min(q0 + ATT_BM, len) - 1;       // last valid query row of the CTA
    const int n_kv_blocks = last_row / ATT_BN + 1;        // causal: keys up to the last row
    const float scale_log2 = rsqrtf(static_cast<float>(DH)) * 1.4426950408889634f;

    load_tile<DH>(q_s, qg, ld, ATT_BM, q0, len);
    load_tile<DH>(k_s(0), kg, ld, ATT_BN, 0, len);
    load_tile<DH>(v_s(0), vg, ld, ATT_BN, 0, len);
    cp_async_commit();

    float o[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    for (int kb = 0; kb < n_kv_blocks; ++kb) {
        const int buf = kb & 1;
        if (kb + 1 < n_kv_blocks) {
            load_tile<DH>(k_s(buf ^ 1), kg, ld, ATT_BN, (kb + 1) * ATT_BN, len);
            load_tile<DH>(v_s(buf ^ 1), vg, ld, ATT_BN, (kb + 1) * ATT_BN, len);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();

        const int key0 = kb * ATT_BN;
        if (key0 <= r0 + 15) {  // otherwise every key of the block is in the future of all 16 rows
            // ---- S = Q K^T (16 x 64 per warp)
            float s[ATT_BN / 8][4];
#pragma unroll
            for (int n = 0; n < ATT_BN / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < DH / 16; ++kk) {
                uint32_t a0, a1, a2, a3;
                ldsm_x4(tile_addr<DH>(q_s, warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, kk * 2 + (lane >> 4)), a0, a1,
                        a2, a3);
#pragma unroll
                for (int np = 0; np < ATT_BN / 16; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(tile_addr<DH>(k_s(buf), np * 16 + (lane & 7) + (lane >> 4) * 8, kk * 2 + ((lane >> 3) & 1)),
                            b0, b1, b2, b3);
                    mma_bf16_16816(s[2 * np], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(s[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
            }
            // ---- scale, causal mask, online softmax (rows g and g + 8 of the warp's 16)
            const bool need_mask = key0 + ATT_BN - 1 > r0;
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int n = 0; n < ATT_BN / 8; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = s[n][e] * scale_log2;
                    if (need_mask) {
                        const int key = key0 + n * 8 + 2 * t + (e & 1);
                        const int row = r0 + g + (e >> 1) * 8;
                        if (key > row) v = -INFINITY;
                    }
                    s[n][e] = v;
                    mx[e >> 1] = fmaxf(mx[e >> 1], v);
                }
            }
            float corr[2], m_new[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xFFFFFFFFu, mx[h], 1));
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xFFFFFFFFu, mx[h], 2));
                m_new[h] = fmaxf(m_run[h], mx[h]);
                // block 0 always holds key 0 <= row, so m_new is finite from the first block on
                corr[h] = fast_exp2(m_run[h] - m_new[h]);
                m_run[h] = m_new[h];
            }
            float rs[2] = {0.f, 0.f};
#pragma unroll
            for (int n = 0; n < ATT_BN / 8; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float pv = fast_exp2(s[n][e] - m_new[e >> 1]);
                    s[n][e] = pv;
                    rs[e >> 1] += pv;
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                rs[h] += __shfl_xor_sync(0xFFFFFFFFu, rs[h], 1);
                rs[h] += __shfl_xor_sync(0xFFFFFFFFu, rs[h], 2);
                l_run[h] = l_run[h] * corr[h] + rs[h];
            }
#pragma unroll
            for (int n = 0; n < DH / 8; ++n) {
                o[n][0] *= corr[0];
                o[n][1] *= corr[0];
                o[n][2] *= corr[1];
                o[n][3] *= corr[1];
            }
            // ---- O += P V
#pragma unroll
            for (int kc = 0; kc < ATT_BN / 16; ++kc) {
                const uint32_t a0 = pack_bf16(s[2 * kc][0], s[2 * kc][1]);
                const uint32_t a1 = pack_bf16(s[2 * kc][2], s[2 * kc][3]);
                const uint32_t a2 = pack_bf16(s[2 * kc + 1][0], s[2 * kc + 1][1]);
                const uint32_t a3 = pack_bf16(s[2 * kc + 1][2], s[2 * kc + 1][3]);
#pragma unroll
                for (int np = 0; np < DH / 16; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_trans(tile_addr<DH>(v_s(buf), kc * 16 + (lane & 7) + ((lane >> 3) & 1) * 8,
                                                np * 2 + (lane >> 4)),
                                  b0, b1, b2, b3);
                    mma_bf16_16816(o[2 * np], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(o[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        }
        __syncthreads();  // the buffer just read is refilled at the top of the next iteration
    }

    // ---- normalise and store
    const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
    const int row_a = r0 + g, row_b = r0 + g + 8;
    __nv_bfloat16* og = out + static_cast<size_t>(seq_start) * dq + head * DH;
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) {
        const int col = n * 8 + 2 * t;
        if (row_a < len)
            *reinterpret_cast<uint32_t*>(og + static_cast<size_t>(row_a) * dq + col) = pack_bf16(o[n][0] * inv0, o[n][1] * inv0);
        if (row_b < len)
            *reinterpret_cast<uint32_t*>(og + static_cast<size_t>(row_b) * dq + col) = pack_bf16(o[n][2] * inv1, o[n][3] * inv1);
    }
}

template <int DH>
constexpr int att_smem_bytes() {
    return ATT_BM * DH * 2 + 4 * ATT_BN * DH * 2;
}

}  // namespace

cudaError_t attention_init() {
    cudaError_t e = cudaFuncSetAttribute(attn_causal_gqa_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         att_smem_bytes<64>());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attn_causal_gqa_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                att_smem_bytes<128>());
}

cudaError_t launch_attention(const void* qkv, const int* cu_seqlens_dev, int batch, int max_seqlen, int n_heads,
                             int n_kv_heads, int head_dim, void* out, cudaStream_t stream) {
    if (batch <= 0 || max_seqlen <= 0) return cudaSuccess;
    const dim3 grid((max_seqlen + ATT_BM - 1) / ATT_BM, n_heads, batch);
    const __nv_bfloat16* in = reinterpret_cast<const __nv_bfloat16*>(qkv);
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out);
    if (head_dim == 64)
        attn_causal_gqa_kernel<64><<<grid, ATT_THREADS, att_smem_bytes<64>(), stream>>>(in, cu_seqlens_dev, n_heads,
                                                                                       n_kv_heads, o);
    else if (head_dim == 128)
        attn_causal_gqa_kernel<128><<<grid, ATT_THREADS, att_smem_bytes<128>(), stream>>>(in, cu_seqlens_dev, n_heads,
                                                                                         n_kv_heads, o);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace vl
