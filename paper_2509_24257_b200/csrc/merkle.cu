// Merkle commitment of hidden-state vectors ("constructs a Merkle tree over all scalar entries ... and submits
// the Merkle root"; canonical float32 serialisation, SHA-256): one root per vector.
//
// Tree: leaf j = SHA-256 of the 4 bytes of entry j as a little-endian IEEE-754 float32; inner node =
// SHA-256(left || right) over the two 32-byte children; a level with an odd number of nodes pairs its last
// node with itself; a single leaf is its own root.  One CTA per vector: every thread hashes two leaves and
// their parent straight from global memory, the upper levels are folded in shared memory.
// SHA-256 follows FIPS 180-4; its round constants are derived on the host from their definition (fractional
// parts of the cube / square roots of the first primes) rather than typed in.
#include "kernels.h"

namespace vl {

namespace {

__constant__ uint32_t c_k[64];
__constant__ uint32_t c_h0[8];

__device__ __forceinline__ uint32_t rotr(uint32_t x, int n) { return __funnelshift_r(x, x, n); }

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
        const uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25);
        const uint32_t ch = (e & f) ^ (~e & g);
        const uint32_t t1 = h + S1 + ch + c_k[t] + w[t & 15];
        const uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22);
        const uint32_t mj = (a & b) ^ (a & c) ^ (b & c);
        const uint32_t t2 = S0 + mj;
        h = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + t2;
    }
    st[0] += a; st[1] += b; st[2] += c; st[3] += d; st[4] += e; st[5] += f; st[6] += g; st[7] += h;
}

__device__ __forceinline__ void sha256_init(uint32_t (&st)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) st[i] = c_h0[i];
}

// SHA-256 of the 4-byte little-endian serialisation of one float32.
__device__ __forceinline__ void hash_leaf(float x, uint32_t (&out)[8]) {
    uint32_t w[16];
    w[0] = __byte_perm(__float_as_uint(x), 0, 0x0123);  // message bytes b0 b1 b2 b3 = LSB first
    w[1] = 0x80000000u;
#pragma unroll
    for (int i = 2; i < 15; ++i) w[i] = 0u;
    w[15] = 32u;  // message length in bits
    sha256_init(out);
    sha256_compress(out, w);
}

// SHA-256 of the 64-byte concatenation of two digests (given as their 8 state words each).
__device__ __forceinline__ void hash_pair(const uint32_t (&l)[8], const uint32_t (&r)[8], uint32_t (&out)[8]) {
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        w[i] = l[i];
        w[8 + i] = r[i];
    }
    sha256_init(out);
    sha256_compress(out, w);
    w[0] = 0x80000000u;
#pragma unroll
    for (int i = 1; i < 15; ++i) w[i] = 0u;
    w[15] = 512u;
    sha256_compress(out, w);
}

constexpr int kMerkleThreads = 256;

__global__ void __launch_bounds__(kMerkleThreads)
merkle_root_kernel(const float* __restrict__ states, int d, uint8_t* __restrict__ roots) {
    extern __shared__ uint32_t nodes[];  // [ceil(d/2)][8] digests of the current level
    const float* x = states + static_cast<size_t>(blockIdx.x) * d;
    uint32_t dg[8];
    if (d == 1) {
        if (threadIdx.x == 0) {
            hash_leaf(x[0], dg);
            for (int i = 0; i < 8; ++i) nodes[i] = dg[i];
        }
    } else {
        const int half = (d + 1) / 2;
        for (int i = threadIdx.x; i < half; i += kMerkleThreads) {
            uint32_t a[8], b[8];
            hash_leaf(x[2 * i], a);
            if (2 * i + 1 < d) hash_leaf(x[2 * i + 1], b);
            else
                for (int k = 0; k < 8; ++k) b[k] = a[k];
            hash_pair(a, b, dg);
            for (int k = 0; k < 8; ++k) nodes[i * 8 + k] = dg[k];
        }
        __syncthreads();
        for (int cnt = half; cnt > 1; cnt = (cnt + 1) / 2) {
            const int next = (cnt + 1) / 2;
            // rounds of kMerkleThreads outputs: a round reads [2 r T, 2 r T + 2 T) and writes [r T, r T + T);
            // only inside a round can a write land on another thread's input, hence read - sync - write - sync
            for (int base = 0; base < next; base += kMerkleThreads) {
                const int i = base + threadIdx.x;
                uint32_t l[8], r[8];
                const bool active = i < next;
                if (active) {
                    const int ri = 2 * i + 1 < cnt ? 2 * i + 1 : 2 * i;
                    for (int k = 0; k < 8; ++k) {
                        l[k] = nodes[2 * i * 8 + k];
                        r[k] = nodes[ri * 8 + k];
                    }
                }
                __syncthreads();
                if (active) {
                    hash_pair(l, r, dg);
                    for (int k = 0; k < 8; ++k) nodes[i * 8 + k] = dg[k];
                }
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
    cudaError_t e = cudaMemcpyToSymbol(c_k, k, sizeof(k));
    if (e != cudaSuccess) return e;
    return cudaMemcpyToSymbol(c_h0, h0, sizeof(h0));
}

cudaError_t launch_merkle_roots(const float* states, int n_vec, int d, uint8_t* roots, cudaStream_t stream) {
    if (n_vec <= 0) return cudaSuccess;
    const size_t smem = static_cast<size_t>((d + 1) / 2) * 32;
    static size_t configured = 48 * 1024;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(merkle_root_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    merkle_root_kernel<<<n_vec, kMerkleThreads, smem < 32 ? 32 : smem, stream>>>(states, d, roots);
    return cudaGetLastError();
}

}  // namespace vl
