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
    float thr_w;       // e_w * 2^mantissa_bits: largest significand distance counted as small
    int e_m;           // mantissa-field distance above which a mismatch is large
};

struct CmpAcc {
    float ss, rr, sa, sg, mx;
    uint32_t n_mis, n_large_m, n_small_w, n_exact, n_qsmall, n_zlarge, n_nonfinite;

    __device__ __forceinline__ void clear() {
        ss = rr = sa = sg = mx = 0.f;
        n_mis = n_large_m = n_small_w = n_exact = n_qsmall = n_zlarge = n_nonfinite = 0u;
    }

    // h: recomputed value (fp32); c_bits: committed value as a float32 bit pattern (a bf16 value widened
    // by 16 zero bits, or the float32 itself).  kBf16 selects the commit dtype at compile time.
    template <bool kBf16>
    __device__ __forceinline__ void add(float h, uint32_t c_bits, const CmpParams& p) {
        const float c = __uint_as_float(c_bits);
        const uint32_t h_bits = __float_as_uint(h);
        // finite <=> exponent field below 255
        if ((h_bits & 0x7F800000u) == 0x7F800000u || (c_bits & 0x7F800000u) == 0x7F800000u) {
            n_nonfinite++;
            return;
        }
        const float d = h - c;
        const float ad = fabsf(d);
        ss = fmaf(d, d, ss);
        rr = fmaf(c, c, rr);
        sa += ad;
        sg += d;
        mx = fmaxf(mx, ad);
        n_qsmall += (ad <= 1e-5f) ? 1u : 0u;
        n_zlarge += (ad > p.tau_large) ? 1u : 0u;

        // both values in the commit dtype, then sign / exponent field / mantissa field
        constexpr int mshift = kBf16 ? 16 : 0;
        constexpr int mbits = kBf16 ? 7 : 23;
        uint32_t hb;
        if constexpr (kBf16) {
            const __nv_bfloat16 hr = __float2bfloat16_rn(h);
            hb = static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(&hr)) << 16;
        } else {
            hb = h_bits;
        }
        const uint32_t cb = c_bits;
        const uint32_t eh = hb & 0x7F800000u, ec = cb & 0x7F800000u;  // exponent fields, in place
        const uint32_t mh = (hb & 0x7FFFFFu) >> mshift, mc = (cb & 0x7FFFFFu) >> mshift;
        if (eh != ec) {
            n_mis++;
            n_large_m += (__usad(mh, mc, 0u) > static_cast<uint32_t>(p.e_m)) ? 1u : 0u;
        } else {
            // signed significands (implicit one unless the exponent field is zero), distance in steps
            const uint32_t one = eh != 0u ? (1u << mbits) : 0u;
            const uint32_t sh = one + mh, sc = one + mc;
            const uint32_t dev = ((hb ^ cb) >> 31) ? sh + sc : __usad(sh, sc, 0u);
            n_small_w += (static_cast<float>(dev) <= p.thr_w) ? 1u : 0u;
            n_exact += (hb == cb) ? 1u : 0u;
        }
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
