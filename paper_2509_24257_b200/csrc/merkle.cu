// Merkle commitment of hidden-state vectors (Inference Scheme, commitment step: a tree over all scalar entries,
// its root submitted; canonical float32 serialisation, SHA-256): one root per vector.
//
// Tree: leaf j = SHA-256 of the 4 bytes of entry j as a little-endian IEEE-754 float32; inner node =
// SHA-256(left || right) over the two 32-byte children; a level with an odd number of nodes pairs its last
// node with itself; a single leaf is its own root.  One CTA per vector: every thread hashes subtrees of four
// leaves straight from global memory, the upper levels are folded in shared memory.
// SHA-256 follows FIPS 180-4; its round constants are derived on the host from their definition (fractional
// parts of the cube / square roots of the first primes) rather than typed in.
#include "kernels.h"

namespace vl {

namespace {

__constant__ uint32_t c_k[64];
__constant__ uint32_t c_h0[8];
// K[t] + W[t] of the block that pads a 64-byte message (0x80, zeros, length 512): the same for every inner
// node, so its message schedule is expanded once on the host.
__constant__ uint32_t c_kw_pad[64];

__device__ __forceinline__ uint32_t rotr(uint32_t x, int n) { return __funnelshift_r(x, x, n); }

#define VL_SHA_ROUND(kw)                                                      \
    {                                                                         \
        const uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25);           \
        const uint32_t ch = (e & f) ^ (~e & g);                               \
        const uint32_t t1 = h + S1 + ch + (kw);                               \
        const uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22);           \
        const uint32_t mj = (a & b) ^ (a & c) ^ (b & c);                      \
        h = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + S0 + mj; \
    }

// One compression: state += F(state, block), block given as 16 big-endian words.
__device__ __forceinline__ void sha256_compress(uint32_t (&st)[8], uint32_t (&w)[16]) {
    uint32_t a = st[0], b = st[1], c = st[2], d = st[3], e = st[4], f = st[5], g = st[6], h = st[7];
#pragma unroll
    for (int t = 0; t < 64; ++t) {
        if (t >= 16) {
            const uint32_t w15 = w[(t - 15) & 15], w2 = w[(t - 2) & 15];
            const uint32_t s0 = rotr(w15, 7) ^ rotr(w15, 18) ^ (w15 >> 3);
            const uint32_t s1 = rotr(w2, 17) ^ rotr(w2, 19) ^ (w2 >> 10);
            w[t & 15] = w[t & 15] + s0 + w[(t - 7) & 15] + s1;
        }
        VL_SHA_ROUND(c_k[t] + w[t & 15])
    }
    st[0] += a; st[1] += b; st[2] += c; st[3] += d; st[4] += e; st[5] += f; st[6] += g; st[7] += h;
}

// The compression of the constant padding block of a 64-byte message: no schedule to compute.
__device__ __forceinline__ void sha256_compress_pad64(uint32_t (&st)[8]) {
    uint32_t a = st[0], b = st[1], c = st[2], d = st[3], e = st[4], f = st[5], g = st[6], h = st[7];
#pragma unroll
    for (int t = 0; t < 64; ++t) VL_SHA_ROUND(c_kw_pad[t])
    st[0] += a; st[1] += b; st[2] += c; st[3] += d; st[4] += e; st[5] += f; st[6] += g; st[7] += h;
}
#undef VL_SHA_ROUND

// Digests live in shared memory, word k of a digest at p[k * stride].  The two hash routines are not inlined:
// the kernel then holds one copy of each (about 3600 instructions together) instead of one per call site, which
// keeps it inside the instruction cache, and each copy gets its own register allocation.

// SHA-256 of the 4-byte little-endian serialisation of one float32.  All words of the block but the first are
// compile-time constants, so most of the schedule folds away when the rounds are unrolled.
__device__ __noinline__ void hash_leaf(float x, uint32_t* out, int os) {
    uint32_t w[16], st[8];
    w[0] = __byte_perm(__float_as_uint(x), 0, 0x0123);  // message bytes b0 b1 b2 b3 = LSB first
    w[1] = 0x80000000u;
#pragma unroll
    for (int i = 2; i < 15; ++i) w[i] = 0u;
    w[15] = 32u;  // message length in bits
#pragma unroll
    for (int i = 0; i < 8; ++i) st[i] = c_h0[i];
    sha256_compress(st, w);
#pragma unroll
    for (int i = 0; i < 8; ++i) out[i * os] = st[i];
}

// SHA-256 of the 64-byte concatenation of two digests.  Both inputs are read before the output is written, so
// `out` may be one of them.
__device__ __noinline__ void hash_pair(const uint32_t* l, int ls, const uint32_t* r, int rs, uint32_t* out, int os) {
    uint32_t w[16], st[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w[i] = l[i * ls];
        w[8 + i] = r[i * rs];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) st[i] = c_h0[i];
    sha256_compress(st, w);
    sha256_compress_pad64(st);
#pragma unroll
    for (int i = 0; i < 8; ++i) out[i * os] = st[i];
}

constexpr int kMerkleThreads = 512;
constexpr int kMerkleCtasPerSm = 3;  // 48 warps per SM: a serial chain of rounds needs many warps to fill the issue slots
constexpr int kMerkleScratchWords = 2 * 8 * kMerkleThreads;  // two digests per thread, word-major

__global__ void __launch_bounds__(kMerkleThreads, kMerkleCtasPerSm)
merkle_root_kernel(const float* __restrict__ states, int d, uint8_t* __restrict__ roots) {
    // scratch [2][8][threads] (a thread's two leaf digests), then nodes [ceil(ceil(d/2)/2)][8]: the current level
    extern __shared__ uint32_t merkle_smem[];
    uint32_t* s0 = merkle_smem + threadIdx.x;
    uint32_t* s1 = s0 + 8 * kMerkleThreads;
    uint32_t* nodes = merkle_smem + kMerkleScratchWords;
    const float* x = states + static_cast<size_t>(blockIdx.x) * d;
    const int n1 = (d + 1) / 2;  // nodes on level 1
    // level-1 node j (the hash of leaves 2j and 2j+1; the last leaf pairs with itself) -> out
    auto level1 = [&](int j, uint32_t* out, int os) {
        hash_leaf(x[2 * j], s0, kMerkleThreads);
        if (2 * j + 1 < d) {
            hash_leaf(x[2 * j + 1], s1, kMerkleThreads);
            hash_pair(s0, kMerkleThreads, s1, kMerkleThreads, out, os);
        } else {
            hash_pair(s0, kMerkleThreads, s0, kMerkleThreads, out, os);
        }
    };
    if (n1 == 1) {  // one or two entries: the root is the leaf or the only level-1 node
        if (threadIdx.x == 0) {
            if (d == 1) hash_leaf(x[0], nodes, 1);
            else level1(0, nodes, 1);
        }
    } else {
        // every thread hashes subtrees of four leaves straight from global memory: only level 2 reaches the node array
        const int n2 = (n1 + 1) / 2;
#pragma unroll 1
        for (int i = threadIdx.x; i < n2; i += kMerkleThreads) {
            uint32_t* mine = nodes + i * 8;
            level1(2 * i, mine, 1);
            if (2 * i + 1 < n1) {
                level1(2 * i + 1, s0, kMerkleThreads);
                hash_pair(mine, 1, s0, kMerkleThreads, mine, 1);
            } else {
                hash_pair(mine, 1, mine, 1, mine, 1);
            }
        }
        __syncthreads();
#pragma unroll 1
        for (int cnt = n2; cnt > 1; cnt = (cnt + 1) / 2) {
            const int next = (cnt + 1) / 2;
            // rounds of kMerkleThreads outputs: a round reads [2 r T, 2 r T + 2 T) and writes [r T, r T + T);
            // only inside a round can a write land on another thread's input: the result waits in the thread's
            // scratch until every thread of the round has read its inputs
#pragma unroll 1
            for (int base = 0; base < next; base += kMerkleThreads) {
                const int i = base + threadIdx.x;
                const bool active = i < next;
                if (active) {
                    const int ri = 2 * i + 1 < cnt ? 2 * i + 1 : 2 * i;
                    hash_pair(nodes + 2 * i * 8, 1, nodes + ri * 8, 1, s0, kMerkleThreads);
                }
                __syncthreads();
                if (active)
                    for (int k = 0; k < 8; ++k) nodes[i * 8 + k] = s0[k * kMerkleThreads];
                __syncthreads();
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {  // digest bytes are the state words in big-endian order
        const uint32_t wv = nodes[threadIdx.x >> 2];
        roots[static_cast<size_t>(blockIdx.x) * 32 + threadIdx.x] = static_cast<uint8_t>(wv >> (24 - 8 * (threadIdx.x & 3)));
    }
}

// floor(2^frac_bits * root) of n^(1/k) for k = 2 or 3, by binary search on integers (no floating point).
uint32_t frac_root_bits(uint32_t n, int k) {
    // find the largest r with r^k <= n * 2^(32 k); the answer's low 32 bits are the fractional part
    unsigned __int128 target = static_cast<unsigned __int128>(n) << (32 * k);
    uint64_t lo = 0, hi = static_cast<uint64_t>(1) << 40;
    while (hi - lo > 1) {
        const uint64_t mid = lo + (hi - lo) / 2;
        unsigned __int128 p = mid;
        for (int i = 1; i < k; ++i) p *= mid;  // mid < 2^40: mid^3 < 2^120 fits
        if (p <= target) lo = mid; else hi = mid;
    }
    return static_cast<uint32_t>(lo & 0xFFFFFFFFu);
}

}  // namespace

cudaError_t merkle_init() {
    uint32_t k[64], h0[8];
    int found = 0;
    for (uint32_t n = 2; found < 64; ++n) {
        bool prime = true;
        for (uint32_t q = 2; q * q <= n; ++q)
            if (n % q == 0) { prime = false; break; }
        if (!prime) continue;
        if (found < 8) h0[found] = frac_root_bits(n, 2);
        k[found] = frac_root_bits(n, 3);
        ++found;
    }
    // message schedule of the block that pads a 64-byte message, added to the round constants
    uint32_t w[64], kw[64];
    auto rot = [](uint32_t v, int n) { return (v >> n) | (v << (32 - n)); };
    for (int t = 0; t < 16; ++t) w[t] = 0u;
    w[0] = 0x80000000u;
    w[15] = 512u;
    for (int t = 16; t < 64; ++t) {
        const uint32_t s0 = rot(w[t - 15], 7) ^ rot(w[t - 15], 18) ^ (w[t - 15] >> 3);
        const uint32_t s1 = rot(w[t - 2], 17) ^ rot(w[t - 2], 19) ^ (w[t - 2] >> 10);
        w[t] = w[t - 16] + s0 + w[t - 7] + s1;
    }
    for (int t = 0; t < 64; ++t) kw[t] = k[t] + w[t];
    cudaError_t e = cudaMemcpyToSymbol(c_k, k, sizeof(k));
    if (e != cudaSuccess) return e;
    e = cudaMemcpyToSymbol(c_kw_pad, kw, sizeof(kw));
    if (e != cudaSuccess) return e;
    return cudaMemcpyToSymbol(c_h0, h0, sizeof(h0));
}

cudaError_t launch_merkle_roots(const float* states, int n_vec, int d, uint8_t* roots, cudaStream_t stream) {
    if (n_vec <= 0) return cudaSuccess;
    const size_t smem = sizeof(uint32_t) * kMerkleScratchWords + static_cast<size_t>(((d + 1) / 2 + 1) / 2) * 32;  // scratch + one digest per four entries
    // the attribute belongs to the (function, device) pair: remember what each device was given
    static size_t configured[64] = {0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (smem > 48 * 1024 && smem > configured[dev]) {
        e = cudaFuncSetAttribute(merkle_root_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        configured[dev] = smem;
    }
    merkle_root_kernel<<<n_vec, kMerkleThreads, smem, stream>>>(states, d, roots);
    return cudaGetLastError();
}

}  // namespace vl
