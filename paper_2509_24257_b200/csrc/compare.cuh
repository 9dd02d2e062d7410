// Element-wise deviation statistics of a recomputed hidden state against the committed one
// (Delta = S_hat - S; offline battery T_off; bit-aware exponent/mantissa comparison).
// Used by the fused gather-and-compare epilogue of the down projection and by the standalone
// comparison kernel; the partial sums it produces are reduced by the verdict kernels.
#pragma once

#include "common.cuh"

namespace vl {

// Number of 32-bit words one partial record holds (floats first, then counters).
constexpr int kNPart = 12;

struct CmpParams {
    int commit_dtype;  // VERILLM_BF16 / VERILLM_F32
    float tau_large;   // Z_large threshold
    // Both thresholds of the bit-aware test are integers in the units of a float32 bit pattern (a bf16
    // mantissa field sits in bits 16..22 of the widened value, the implicit one at bit 23):
    int thr_dev;  // largest significand distance counted as small, -1 if none qualifies
    int thr_em;   // mantissa-field distance above which an exponent mismatch is large
};

// Host-side conversion of (e_w, e_m) to those units.  `dev <= e_w * 2^mantissa_bits` on an integer
// distance is `dev <= floor(e_w * 2^mantissa_bits)`; distances never exceed 2^(mantissa_bits + 2).
inline CmpParams make_cmp_params(int commit_dtype, float tau_large, float e_w, int e_m) {
    const int mbits = commit_dtype == VERILLM_BF16 ? 7 : 23;
    const int mshift = 23 - mbits;
    const float thr_w = e_w * static_cast<float>(1 << mbits);
    const int max_dev = 1 << (mbits + 2);
    int k = -1;
    if (thr_w >= static_cast<float>(max_dev)) k = max_dev;
    else if (thr_w >= 0.f) k = static_cast<int>(thr_w);  // floor of a non-negative value
    int em = e_m;
    if (em < -1) em = -1;
    if (em > (1 << mbits)) em = 1 << mbits;
    CmpParams c;
    c.commit_dtype = commit_dtype;
    c.tau_large = tau_large;
    c.thr_dev = k < 0 ? -1 : k * (1 << mshift);
    c.thr_em = em * (1 << mshift);
    return c;
}

// packed fp32 pairs: d = a * b + c and d = a + b on both halves in one instruction
__device__ __forceinline__ float2 cmp_ffma2(float2 a, float2 b, float2 c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return reinterpret_cast<float2&>(d);
}
__device__ __forceinline__ float2 cmp_fadd2(float2 a, float2 b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return reinterpret_cast<float2&>(d);
}

struct CmpAcc {
    float ss, rr, sa, sg, mx;
    uint32_t n_mis, n_large_m, n_small_w, n_exact, n_qsmall, n_zlarge, n_nonfinite;

    __device__ __forceinline__ void clear() {
        ss = rr = sa = sg = mx = 0.f;
        n_mis = n_large_m = n_small_w = n_exact = n_qsmall = n_zlarge = n_nonfinite = 0u;
    }
    // Adds what a CmpPairAcc gathered (sums of the even and odd elements, in that order).
    __device__ __forceinline__ void fold(const float2 ss2, const float2 rr2, const float2 sg2, const float2 sa2) {
        ss += ss2.x + ss2.y;
        rr += rr2.x + rr2.y;
        sg += sg2.x + sg2.y;
        sa += sa2.x + sa2.y;
    }

    // h: recomputed value (fp32); hb: h rounded to the commit dtype, as a float32 bit pattern; cb: the
    // committed value as a float32 bit pattern (a bf16 value widened by 16 zero bits, or the float32).
    // kChecked = false leaves out the test for non-finite operands: the caller then inspects `sa` after
    // the pass (any non-finite operand makes |h - c|, and with it the sum, non-finite) and repeats the
    // pass with kChecked = true from cleared accumulators.
    template <bool kChecked>
    __device__ __forceinline__ void add_bits(float h, uint32_t hb, uint32_t cb, const CmpParams& p) {
        const float c = __uint_as_float(cb);
        const float d = h - c;
        const float ad = fabsf(d);
        if constexpr (kChecked) {
            if (!(ad < INFINITY)) {
                // a non-finite operand is counted and left out of every sum; a finite pair whose
                // difference overflowed is kept
                if ((__float_as_uint(h) & 0x7F800000u) == 0x7F800000u || (cb & 0x7F800000u) == 0x7F800000u) {
                    n_nonfinite++;
                    return;
                }
            }
        }
        ss = fmaf(d, d, ss);
        rr = fmaf(c, c, rr);
        sa += ad;
        sg += d;
        mx = fmaxf(mx, ad);
        n_qsmall += (ad <= 1e-5f) ? 1u : 0u;
        n_zlarge += (ad > p.tau_large) ? 1u : 0u;

        // sign / exponent field / mantissa field of both values in the commit dtype
        const uint32_t x = hb ^ cb;
        const bool same_exp = (x & 0x7F800000u) == 0u;
        const uint32_t mh = hb & 0x7FFFFFu, mc = cb & 0x7FFFFFu;
        int dev = static_cast<int>(__usad(mh, mc, 0u));  // mantissa-field distance; also the significand
                                                          // distance when exponent and sign agree
        n_mis += same_exp ? 0u : 1u;
        n_large_m += (!same_exp && dev > p.thr_em) ? 1u : 0u;
        if (same_exp && static_cast<int>(x) < 0) {
            // rare: equal exponent fields, opposite signs: the signed significands (implicit one unless the
            // exponent field is zero) lie on both sides of zero
            const uint32_t one = (hb & 0x7F800000u) != 0u ? 0x800000u : 0u;
            dev = static_cast<int>(mh + mc + 2u * one);
        }
        n_small_w += (same_exp && dev <= p.thr_dev) ? 1u : 0u;
        n_exact += (x == 0u) ? 1u : 0u;
    }

    // Two neighbouring elements against a packed pair of committed bf16 values (low half first).
    template <bool kChecked = true>
    __device__ __forceinline__ void add_bf16x2(float h_lo, float h_hi, uint32_t c_pair, const CmpParams& p) {
        const uint32_t h_pair = pack_bf16(h_lo, h_hi);
        add_bits<kChecked>(h_lo, h_pair << 16, c_pair << 16, p);
        add_bits<kChecked>(h_hi, h_pair & 0xFFFF0000u, c_pair & 0xFFFF0000u, p);
    }
    // The same two elements without the test for non-finite operands, on the packed words: the float sums run on
    // packed fp32 pairs (the caller owns the four pair accumulators and folds them in at the end), the field tests
    // on the two 16-bit halves in place.  Counts are identical to add_bits'; the sums differ only in their order.
    __device__ __forceinline__ void add_bf16x2_packed(float h_lo, float h_hi, uint32_t c_pair, const CmpParams& p,
                                                      float2& ss2, float2& rr2, float2& sg2, float2& sa2) {
        const uint32_t h_pair = pack_bf16(h_lo, h_hi);
        const float2 c2 = make_float2(__uint_as_float(c_pair << 16), __uint_as_float(c_pair & 0xFFFF0000u));
        const float2 d2 = cmp_ffma2(c2, make_float2(-1.f, -1.f), make_float2(h_lo, h_hi));  // h - c, exactly
        ss2 = cmp_ffma2(d2, d2, ss2);
        rr2 = cmp_ffma2(c2, c2, rr2);
        sg2 = cmp_fadd2(sg2, d2);
        const float a0 = fabsf(d2.x), a1 = fabsf(d2.y);
        sa2.x += a0;
        sa2.y += a1;
        mx = fmaxf(mx, fmaxf(a0, a1));
        n_qsmall += (a0 <= 1e-5f) ? 1u : 0u;
        n_qsmall += (a1 <= 1e-5f) ? 1u : 0u;
        n_zlarge += (a0 > p.tau_large) ? 1u : 0u;
        n_zlarge += (a1 > p.tau_large) ? 1u : 0u;

        const uint32_t x = h_pair ^ c_pair;
        // low half: fields at bits 15 / 14..7 / 6..0, distances in units of 1 (thresholds scaled down by 2^16)
        {
            const bool same_exp = (x & 0x7F80u) == 0u;
            const uint32_t mh = h_pair & 0x7Fu, mc = c_pair & 0x7Fu;
            int dev = static_cast<int>(__usad(mh, mc, 0u));
            n_mis += same_exp ? 0u : 1u;
            n_large_m += (!same_exp && dev > (p.thr_em >> 16)) ? 1u : 0u;
            if (same_exp && (x & 0x8000u) != 0u) {
                const uint32_t one = (h_pair & 0x7F80u) != 0u ? 0x80u : 0u;
                dev = static_cast<int>(mh + mc + 2u * one);
            }
            n_small_w += (same_exp && dev <= (p.thr_dev >> 16)) ? 1u : 0u;
            n_exact += ((x & 0xFFFFu) == 0u) ? 1u : 0u;
        }
        // high half: the same fields 16 bits up, distances in the units of the float32 bit pattern
        {
            const bool same_exp = (x & 0x7F800000u) == 0u;
            const uint32_t mh = h_pair & 0x7F0000u, mc = c_pair & 0x7F0000u;
            int dev = static_cast<int>(__usad(mh, mc, 0u));
            n_mis += same_exp ? 0u : 1u;
            n_large_m += (!same_exp && dev > p.thr_em) ? 1u : 0u;
            if (same_exp && static_cast<int>(x) < 0) {
                const uint32_t one = (h_pair & 0x7F800000u) != 0u ? 0x800000u : 0u;
                dev = static_cast<int>(mh + mc + 2u * one);
            }
            n_small_w += (same_exp && dev <= p.thr_dev) ? 1u : 0u;
            n_exact += ((x & 0xFFFF0000u) == 0u) ? 1u : 0u;
        }
    }
    template <bool kChecked = true>
    __device__ __forceinline__ void add_f32(float h, uint32_t c_bits, const CmpParams& p) {
        add_bits<kChecked>(h, __float_as_uint(h), c_bits, p);
    }

    __device__ __forceinline__ void store(float* dst) const {
        float4* d4 = reinterpret_cast<float4*>(dst);
        d4[0] = make_float4(ss, rr, sa, sg);
        d4[1] = make_float4(mx, __uint_as_float(n_mis), __uint_as_float(n_large_m), __uint_as_float(n_small_w));
        d4[2] = make_float4(__uint_as_float(n_exact), __uint_as_float(n_qsmall), __uint_as_float(n_zlarge),
                            __uint_as_float(n_nonfinite));
    }
};

}  // namespace vl
