// The per-group arithmetic of the token-group quantizer's fast path (g = 32, one thread per group):
// Algorithm S1 steps 2-7 on a group held in registers.  Shared by the stand-alone quantizer
// kernels and by the linear layer's fused producer.
#pragma once
#include <cmath>

#include "tdq_common.cuh"

namespace tdq {
namespace {

// True when the binary32 moments prove that 7 tau sigma exceeds cmin by a safe margin, i.e.
// the C1 bound cannot be the minimum.  s1 = sum x, s2 = sum x^2 over the 32 elements.
// The estimate var = s2/32 - mean^2 has relative error below 1e-4 once var >= s2/512, and
// the test keeps a 1 % margin on the squared radius, so a true result is always right; a
// false one only means the deviation is recomputed exactly.
__device__ __forceinline__ bool c1_cannot_bind(float s1, float s2, float seven_tau, float cmin) {
    const float mean = s1 * (1.0f / 32.0f);
    const float ex2 = s2 * (1.0f / 32.0f);
    const float var = fmaf(-mean, mean, ex2);
    const float lhs = seven_tau * seven_tau * var * 0.99f;
    const float rhs = cmin * cmin;
    return (var >= ex2 * (1.0f / 16.0f)) && (lhs > rhs) && (rhs >= 1e-30f) && (s2 < 1e37f) && (lhs < 1e37f);
}

// sigma = Std(x_k) + 1e-12 in binary64, sequentially over the group, rounded to binary32.
template <typename GetF>
__device__ __forceinline__ float sigma_exact32(GetF get) {
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < 32; ++i) s = __dadd_rn(s, (double)get(i));
    const double mu = s / 32.0;
    double ss = 0.0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        double d = __dsub_rn((double)get(i), mu);
        ss = __dadd_rn(ss, __dmul_rn(d, d));
    }
    return __fadd_rn(__double2float_rn(sqrt(ss / 32.0)), kStdEps);
}

// Nibble of one element: exact quotient, round half to even via the magic add.  The clip to
// [-c, c] bounds |x / Delta| by 7 (1 + 2^-23), so the rounded code is always inside [-7, 7]
// and the 4-bit clamp of the definition never acts for finite input.
__device__ __forceinline__ uint32_t nibble_fast(float x, float c, float delta, float rcp) {
    const float xt = fminf(fmaxf(x, -c), c);
    const float q0 = __fmul_rn(xt, rcp);
    const float e = __fmaf_rn(-q0, delta, xt);
    const float q1 = __fmaf_rn(e, rcp, q0);
    return __float_as_uint(__fadd_rn(q1, kRoundMagic)) & 0xFu;
}

// The same test on moments accumulated in bf16 pairs (2^-9 unit roundoff, 16 sequential adds per
// half): s2 is within 4 % and the mean within 0.032 rms, so the variance estimate is off by at
// most 0.105 E[x^2].  Requiring var >= E[x^2] / 2 turns that into var_true >= 0.78 var, and the
// factor 0.7 then leaves 7 tau sigma_true >= 1.05 cmin.  Anything else goes to the exact path.
__device__ __forceinline__ bool c1_cannot_bind_rough(float s1, float s2, float seven_tau, float cmin) {
    const float mean = s1 * (1.0f / 32.0f);
    const float ex2 = s2 * (1.0f / 32.0f);
    const float var = fmaf(-mean, mean, ex2);
    const float lhs = seven_tau * seven_tau * var * 0.7f;
    const float rhs = cmin * cmin;
    return (var >= ex2 * 0.5f) && (lhs > rhs) && (rhs >= 1e-30f) && (s2 < 1e37f) && (lhs < 1e37f);
}

// two binary32 lanes in one 64-bit register; each lane rounds exactly like the scalar .rn instruction
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t p, uint32_t& lo, uint32_t& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p));
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Two elements at once: the sequence of nibble_fast on both lanes, with 8 added to the rounding
// constant so that the low nibble of each result is q + 8 in 1..15 and nothing borrows from the
// bits above it.  The results are pushed into `acc` with integer multiply-adds (acc = 16 acc + t),
// last element first; pack_word() removes what the upper bits of the eight t's add up to.
constexpr float kRoundMagic8 = kRoundMagic + 8.0f;
constexpr uint32_t kMagicBits = 0x4B400000u;   // bit pattern of kRoundMagic
constexpr uint32_t kMagicSum = kMagicBits + (kMagicBits << 4) + (kMagicBits << 8);   // higher terms vanish mod 2^32
__device__ __forceinline__ void nibbles_fast2(uint64_t xt, uint64_t neg_delta2, uint64_t rcp2, uint64_t magic2,
                                              uint32_t& acc) {
    const uint64_t q0 = f2_mul(xt, rcp2);
    const uint64_t e = f2_fma(q0, neg_delta2, xt);     // xt - q0 * Delta, exact
    const uint64_t q1 = f2_fma(e, rcp2, q0);
    uint32_t t0, t1;
    f2_unpack(f2_add(q1, magic2), t0, t1);
    acc = acc * 16u + t1;
    acc = acc * 16u + t0;
}
// eight nibbles q + 8 plus the constant part -> eight two's complement nibbles
__device__ __forceinline__ uint32_t pack_word(uint32_t acc) { return (acc - kMagicSum) ^ 0x88888888u; }

__device__ __forceinline__ uint32_t nibble_ieee(float x, float c, float delta) {
    return (uint32_t)quantize_ieee(x, c, delta) & 0xFu;
}

// K-th smallest of 32 magnitudes given as two sorted halves (even and odd channels of a bf16 group in
// the low and high 16 bits of s[0..15]; s[0..15] and s[16..31] of an fp32 group): the maximum over
// i + j = K - 1 of min(E[i], O[j]), an index past the end counting as +inf.
template <int K>
__device__ __forceinline__ uint32_t kth_of_sorted_halves_u16(const uint32_t (&s)[16]) {
    constexpr int lo_i = (K > 16) ? K - 16 : 0;
    constexpr int hi_i = (K - 1 < 15) ? K - 1 : 15;
    constexpr int mid_i = (lo_i + hi_i) / 2;
    uint32_t r = (K > 16) ? s[(K > 16) ? K - 17 : 0] : 0u;
#pragma unroll
    for (int i = lo_i; i <= mid_i && i <= hi_i; ++i)
        r = __vmaxu2(r, __vminu2(s[i], __byte_perm(s[K - 1 - i], 0u, 0x1032u)));
    return max(r & 0xffffu, r >> 16);
}
template <int K>
__device__ __forceinline__ float kth_of_sorted_halves_f32(const float (&s)[32]) {
    constexpr int lo_i = (K > 16) ? K - 16 : 0;
    constexpr int hi_i = (K - 1 < 15) ? K - 1 : 15;
    float r = (K > 16) ? fmaxf(s[(K > 16) ? K - 17 : 0], s[(K > 16) ? K - 1 : 16]) : 0.0f;
#pragma unroll
    for (int i = lo_i; i <= hi_i; ++i) r = fmaxf(r, fminf(s[i], s[16 + K - 1 - i]));
    return r;
}

// The same with the rank known only at run time: a switch over the 32 compile-time instances, so that the sorted
// halves are only ever indexed with constants and stay in registers.
#define TDQ_RANK_CASES \
    TDQ_RC(1) TDQ_RC(2) TDQ_RC(3) TDQ_RC(4) TDQ_RC(5) TDQ_RC(6) TDQ_RC(7) TDQ_RC(8) TDQ_RC(9) TDQ_RC(10) TDQ_RC(11) \
    TDQ_RC(12) TDQ_RC(13) TDQ_RC(14) TDQ_RC(15) TDQ_RC(16) TDQ_RC(17) TDQ_RC(18) TDQ_RC(19) TDQ_RC(20) TDQ_RC(21) \
    TDQ_RC(22) TDQ_RC(23) TDQ_RC(24) TDQ_RC(25) TDQ_RC(26) TDQ_RC(27) TDQ_RC(28) TDQ_RC(29) TDQ_RC(30) TDQ_RC(31) TDQ_RC(32)
__device__ __forceinline__ uint32_t kth_of_sorted_halves_u16_rt(const uint32_t (&s)[16], int k) {
    switch (k) {
#define TDQ_RC(K_) case K_: return kth_of_sorted_halves_u16<K_>(s);
        TDQ_RANK_CASES
#undef TDQ_RC
    }
    return 0u;
}
__device__ __forceinline__ float kth_of_sorted_halves_f32_rt(const float (&s)[32], int k) {
    switch (k) {
#define TDQ_RC(K_) case K_: return kth_of_sorted_halves_f32<K_>(s);
        TDQ_RANK_CASES
#undef TDQ_RC
    }
    return 0.0f;
}

// One group held in registers (w: 16 packed bf16 pairs or 32 floats, in channel order): statistics,
// projection, quantization.  out: the group's 32 two's complement nibbles, channel 8 w + n in
// nibble n of word w; delta: its step.  KB: rank of the base radius among the magnitudes (32: the maximum,
// Eq. 5; less: the percentile option of Supp. S4.8, which takes the group's KB-th smallest magnitude).
// KB == 0: both ranks are run-time values (rt_kzr, rt_kb in 1..32), for the settings that have no instance of their own.
template <bool BF16, int KZR, int KB = 32>
__device__ __forceinline__ void quantize_group32(const uint32_t (&w)[BF16 ? 16 : 32], float seven_tau, uint32_t flags,
                                                 uint32_t (&out)[4], float& delta, int rt_kzr = 0, int rt_kb = 0) {
    auto get = [&](int i) -> float {
        if (BF16) return (i & 1) ? __uint_as_float(w[i >> 1] & 0xffff0000u) : __uint_as_float(w[i >> 1] << 16);
        return __uint_as_float(w[i]);
    };

    // base radius, rank-KZR magnitude, moments
    float c_base, thr = 0.0f;
    if (KB < 32) {
        // percentile base radius: both ranks come from the same two sorted halves
        if (BF16) {
            uint32_t s[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) s[i] = w[i] & 0x7fff7fffu;
#define TDQ_CE(i, j) { uint32_t lo_ = __vminu2(s[i], s[j]); s[j] = __vmaxu2(s[i], s[j]); s[i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
            if (KB == 0) {
                c_base = __uint_as_float(kth_of_sorted_halves_u16_rt(s, rt_kb) << 16);
                if (flags & TDQ_ENABLE_C2) thr = __uint_as_float(kth_of_sorted_halves_u16_rt(s, rt_kzr) << 16);
            } else {
                c_base = __uint_as_float(kth_of_sorted_halves_u16<(KB ? KB : 1)>(s) << 16);
                if (flags & TDQ_ENABLE_C2) thr = __uint_as_float(kth_of_sorted_halves_u16<(KZR ? KZR : 1)>(s) << 16);
            }
        } else {
            float s[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) s[i] = fabsf(__uint_as_float(w[i]));
#define TDQ_CE(i, j) { float lo_ = fminf(s[i], s[j]); s[j] = fmaxf(s[i], s[j]); s[i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
#define TDQ_CE(i, j) { float lo_ = fminf(s[16 + i], s[16 + j]); s[16 + j] = fmaxf(s[16 + i], s[16 + j]); s[16 + i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
            if (KB == 0) {
                c_base = kth_of_sorted_halves_f32_rt(s, rt_kb);
                if (flags & TDQ_ENABLE_C2) thr = kth_of_sorted_halves_f32_rt(s, rt_kzr);
            } else {
                c_base = kth_of_sorted_halves_f32<(KB ? KB : 1)>(s);
                if (flags & TDQ_ENABLE_C2) thr = kth_of_sorted_halves_f32<(KZR ? KZR : 1)>(s);
            }
        }
    } else if (BF16) {
        // |x| of a bf16 is a 15-bit key whose unsigned order is the numeric order, so the network
        // runs on packed 16-bit integer min/max (two channels per instruction, integer pipe)
        uint32_t s[16];
        uint32_t mx = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            s[i] = w[i] & 0x7fff7fffu;
            mx = __vmaxu2(mx, s[i]);
        }
        c_base = __uint_as_float(max(mx & 0xffffu, mx >> 16) << 16);
        if (flags & TDQ_ENABLE_C2) {
#define TDQ_CE(i, j) { uint32_t lo_ = __vminu2(s[i], s[j]); s[j] = __vmaxu2(s[i], s[j]); s[i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
            // low halves: sorted even channels E, high halves: sorted odd channels O.  The KZR-th
            // smallest of the union is max over i + j = KZR - 1 of min(E[i], O[j]), where an
            // index past the end counts as +inf (so for KZR > 16 the terms E[KZR-17] and
            // O[KZR-17] stand alone).  One packed min with the partner's halves swapped covers
            // index i and its mirror at once.
            constexpr int lo_i = (KZR > 16) ? KZR - 16 : 0;
            constexpr int hi_i = (KZR - 1 < 15) ? KZR - 1 : 15;
            constexpr int mid_i = (lo_i + hi_i) / 2;
            uint32_t r = (KZR > 16) ? s[(KZR > 16) ? KZR - 17 : 0] : 0u;
#pragma unroll
            for (int i = lo_i; i <= mid_i && i <= hi_i; ++i)
                r = __vmaxu2(r, __vminu2(s[i], __byte_perm(s[KZR - 1 - i], 0u, 0x1032u)));
            thr = __uint_as_float(max(r & 0xffffu, r >> 16) << 16);
        }
    } else {
        float s[32];
        float mx = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            s[i] = fabsf(__uint_as_float(w[i]));
            mx = fmaxf(mx, s[i]);
        }
        c_base = mx;
        if (flags & TDQ_ENABLE_C2) {
#define TDQ_CE(i, j) { float lo_ = fminf(s[i], s[j]); s[j] = fmaxf(s[i], s[j]); s[i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
#define TDQ_CE(i, j) { float lo_ = fminf(s[16 + i], s[16 + j]); s[16 + j] = fmaxf(s[16 + i], s[16 + j]); s[16 + i] = lo_; }
#include "sort16_network.inc"
#undef TDQ_CE
            constexpr int lo_i = (KZR > 16) ? KZR - 16 : 0;
            constexpr int hi_i = (KZR - 1 < 15) ? KZR - 1 : 15;
            float r = (KZR > 16) ? fmaxf(s[(KZR > 16) ? KZR - 17 : 0], s[(KZR > 16) ? KZR - 1 : 16]) : 0.0f;
#pragma unroll
            for (int i = lo_i; i <= hi_i; ++i) r = fmaxf(r, fminf(s[i], s[16 + KZR - 1 - i]));
            thr = r;
        }
    }

    float sigma = INFINITY;   // an idle C1 bound
    if (flags & TDQ_ENABLE_C1) {
        float cmin = c_base;
        if (flags & TDQ_ENABLE_C2) cmin = fminf(cmin, __fmul_rn(14.0f, thr));
        bool idle;
        if (BF16) {   // rough moments, two channels per instruction
            __nv_bfloat162 s1b = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
            __nv_bfloat162 s2b = __hmul2(s1b, s1b);
#pragma unroll
            for (int i = 1; i < 16; ++i) {
                const __nv_bfloat162 xi = *reinterpret_cast<const __nv_bfloat162*>(&w[i]);
                s1b = __hadd2(s1b, xi);
                s2b = __hfma2(xi, xi, s2b);
            }
            idle = c1_cannot_bind_rough(__low2float(s1b) + __high2float(s1b), __low2float(s2b) + __high2float(s2b),
                                        seven_tau, cmin);
        } else {
            float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                float v = get(i);
                s1 += v;
                s2 = fmaf(v, v, s2);
            }
            idle = c1_cannot_bind(s1, s2, seven_tau, cmin);
        }
        if (!idle) sigma = sigma_exact32(get);
    }

    float c;
    dcrp_project(c_base, sigma, thr, seven_tau, flags, c, delta);

    if (delta <= 1e30f) {
        const float rcp = __frcp_rn(delta);
        const uint64_t rcp2 = f2_pack(rcp, rcp), neg_delta2 = f2_pack(-delta, -delta);
        const uint64_t magic2 = f2_pack(kRoundMagic8, kRoundMagic8);
        // bf16 input is clipped two channels at a time against c rounded up to a bf16: a value
        // between c and that bound still divides to less than 7.5 (or 1.5 under the step floor),
        // so it rounds to the same code as c itself
        const uint32_t cup = (__float_as_uint(c) + 0xffffu) >> 16;
        const uint32_t cpos = cup | (cup << 16), cneg = cpos | 0x80008000u;
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
            uint32_t acc = 0;
#pragma unroll
            for (int n = 6; n >= 0; n -= 2) {
                uint64_t xt;
                if (BF16) {
                    const __nv_bfloat162 lim_hi = *reinterpret_cast<const __nv_bfloat162*>(&cpos);
                    const __nv_bfloat162 lim_lo = *reinterpret_cast<const __nv_bfloat162*>(&cneg);
                    const __nv_bfloat162 xp = __hmin2(__hmax2(*reinterpret_cast<const __nv_bfloat162*>(&w[wd * 4 + n / 2]), lim_lo), lim_hi);
                    const uint32_t u = *reinterpret_cast<const uint32_t*>(&xp);
                    xt = f2_pack(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
                } else {
                    xt = f2_pack(fminf(fmaxf(get(wd * 8 + n), -c), c), fminf(fmaxf(get(wd * 8 + n + 1), -c), c));
                }
                nibbles_fast2(xt, neg_delta2, rcp2, magic2, acc);
            }
            out[wd] = pack_word(acc);
        }
    } else {   // 1 / Delta would be subnormal: take the IEEE division
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
            uint32_t acc = 0;
#pragma unroll
            for (int n = 0; n < 8; ++n) acc |= nibble_ieee(get(wd * 8 + n), c, delta) << (4 * n);
            out[wd] = acc;
        }
    }
}


// The same result as quantize_group32<., 7> with a small register footprint, for callers that have
// few registers to spare: the group (64 or 128 bytes at src, 16-byte aligned) is read twice instead
// of being held in registers, and the seven smallest magnitudes are kept by insertion.  Every
// quantity that reaches the output is computed by the same operations in the same precision; only
// the screen that decides whether the exact deviation is needed differs, and both screens are safe.
template <bool BF16>
__device__ __forceinline__ void quantize_group32_lean(const uint4* src, float seven_tau, uint32_t flags,
                                                      uint32_t (&out)[4], float& delta) {
    constexpr int kChunks = BF16 ? 4 : 8;           // 16-byte chunks of the group
    constexpr int kPer = 32 / kChunks;              // elements per chunk
    auto elem = [](const uint4& t, int e) -> float {
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
        if (BF16) return (e & 1) ? __uint_as_float(w[e >> 1] & 0xffff0000u) : __uint_as_float(w[e >> 1] << 16);
        return __uint_as_float(w[e]);
    };
    uint32_t small[7];                              // the seven smallest |x| so far (binary32 bit patterns), ascending
#pragma unroll
    for (int j = 0; j < 7; ++j) small[j] = 0x7f800000u;
    uint32_t kmax = 0u;
    float s1 = 0.0f, s2 = 0.0f;
#pragma unroll 1
    for (int q = 0; q < kChunks; ++q) {
        const uint4 t = __ldg(src + q);
#pragma unroll
        for (int e = 0; e < kPer; ++e) {
            const float x = elem(t, e);
            uint32_t key = __float_as_uint(x) & 0x7fffffffu;
            kmax = max(kmax, key);
            s1 += x;
            s2 = fmaf(x, x, s2);
#pragma unroll
            for (int j = 0; j < 7; ++j) {
                const uint32_t lo = min(small[j], key);
                key = max(small[j], key);
                small[j] = lo;
            }
        }
    }
    const float c_base = __uint_as_float(kmax);
    const float thr = (flags & TDQ_ENABLE_C2) ? __uint_as_float(small[6]) : 0.0f;
    float sigma = INFINITY;                         // an idle C1 bound
    if (flags & TDQ_ENABLE_C1) {
        float cmin = c_base;
        if (flags & TDQ_ENABLE_C2) cmin = fminf(cmin, __fmul_rn(14.0f, thr));
        if (!c1_cannot_bind(s1, s2, seven_tau, cmin)) {
            auto get = [&](int i) -> float {
                if (BF16) return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(src) + i) << 16);
                return __ldg(reinterpret_cast<const float*>(src) + i);
            };
            sigma = sigma_exact32(get);
        }
    }
    float c;
    dcrp_project(c_base, sigma, thr, seven_tau, flags, c, delta);
    const bool fast = delta <= 1e30f;               // otherwise 1 / Delta would be subnormal: take the IEEE division
    const float rcp = fast ? __frcp_rn(delta) : 0.0f;
#pragma unroll
    for (int wd = 0; wd < 4; ++wd) {
        uint32_t acc = 0u;
#pragma unroll
        for (int h = 0; h < 8 / kPer; ++h) {
            const uint4 t = __ldg(src + wd * (8 / kPer) + h);
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                const float x = elem(t, e);
                const uint32_t nib = fast ? nibble_fast(x, c, delta, rcp) : nibble_ieee(x, c, delta);
                acc |= nib << (4 * (h * kPer + e));
            }
        }
        out[wd] = acc;
    }
}

}  // namespace
}  // namespace tdq
