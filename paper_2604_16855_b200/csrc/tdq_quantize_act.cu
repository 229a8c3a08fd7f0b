// tdq_quantize_act: token-group dual-constraint activation quantizer (Algorithm S1 steps 1-7).
//
// Two kernels:
//   * act_g32_kernel   g = 32, C % 32 == 0, 16-byte aligned rows.  A CTA stages a tile of
//     consecutive token-groups in shared memory with coalesced 128-bit loads (XOR-swizzled
//     so the read-back is conflict free); then every thread owns one whole group in
//     registers: max, sums, a pruned sorting network for the rank-k magnitude, the DCRP
//     projection, an exact quotient, round-half-even, and one 128-bit store of 32 nibbles.
//     One pass over HBM: 2 (bf16) or 4 (fp32) bytes in, 0.5 + 0.125 bytes out per element.
//   * act_generic_kernel   any even g <= 4096, any C, any alignment: one warp per group,
//     rank selection by bisection on the bit patterns of |x|, IEEE division.
//
// Exactness.  Codes must equal clip(rint(fl(fl(clip(x)) / Delta))) in binary32.  The fast
// kernel replaces the division by y = RN(1/Delta), q0 = RN(x y), e = x - q0 Delta (one FMA,
// exact), q1 = RN(q0 + e y).  q0 + e y differs from x / Delta by less than 2^-23 ulp, so q1
// is the correctly rounded quotient unless x / Delta lies within that distance of a midpoint
// between two floats; a quotient that is exactly a multiple of 0.5 is reproduced exactly.
// The group standard deviation only matters when the C1 bound can be the minimum; a cheap
// binary32 test with a 0.5 % margin proves it cannot for almost every zero-mean group, and
// the other groups recompute it in binary64 in the sequential order of the definition.
#include <cmath>

#include "tdq_common.cuh"

namespace tdq {

std::atomic<uint64_t> g_launch_count{0};

namespace {

struct ActArgs {
    const void* x;
    int64_t M, C, row_stride;  // elements
    int64_t total_groups;      // M * K
    int32_t g, K;              // group size, groups per token
    int32_t k_zr, k_base;      // 1-indexed ranks
    float seven_tau;
    uint32_t flags;
    uint8_t* codes;
    float* scale;
    float* offset;
};

// ------------------------------------------------------------------------------------------
// generic kernel: one warp per group

constexpr int kGenericWarps = 4;

template <bool BF16>
__device__ __forceinline__ float load_elem(const void* x, int64_t idx) {
    if (BF16) return bf16_bits_to_float(reinterpret_cast<const uint16_t*>(x)[idx]);
    return reinterpret_cast<const float*>(x)[idx];
}

// k-th smallest (1-indexed) key of the warp's group by bisection over the key space:
// the smallest v with #{key <= v} >= k.  Keys are bit patterns of non-negative floats.
__device__ __forceinline__ uint32_t warp_kth_key(const float* sm, int g, int lane, int k, uint32_t key_max) {
    uint32_t lo = 0, hi = key_max;
    while (lo < hi) {   // at most 32 rounds: hi - lo halves each time
        uint32_t mid = lo + ((hi - lo) >> 1);
        int cnt = 0;
        for (int i = lane; i < g; i += 32) cnt += (__float_as_uint(fabsf(sm[i])) <= mid) ? 1 : 0;
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (cnt >= k) hi = mid; else lo = mid + 1;
    }
    return lo;
}

template <bool BF16>
__global__ void __launch_bounds__(kGenericWarps * 32) act_generic_kernel(ActArgs a) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* sm = smem + (size_t)warp * a.g;
    const int g = a.g;
    const int64_t C_pad = (int64_t)a.K * g;
    for (int64_t gi = (int64_t)blockIdx.x * kGenericWarps + warp; gi < a.total_groups;
         gi += (int64_t)gridDim.x * kGenericWarps) {
        const int64_t m = gi / a.K;
        const int k = (int)(gi - m * a.K);
        uint32_t kmax = 0;
        double s = 0.0;
        for (int i = lane; i < g; i += 32) {
            int64_t ch = (int64_t)k * g + i;
            float v = (ch < a.C) ? load_elem<BF16>(a.x, m * a.row_stride + ch) : 0.0f;
            sm[i] = v;
            kmax = max(kmax, __float_as_uint(fabsf(v)));
            s += (double)v;
        }
        __syncwarp();
        kmax = __reduce_max_sync(0xffffffffu, kmax);
        float c_base = __uint_as_float(kmax);
        if (a.k_base < g) c_base = __uint_as_float(warp_kth_key(sm, g, lane, a.k_base, kmax));
        float thr = 0.0f, sigma = 0.0f;
        if (a.flags & TDQ_ENABLE_C2) thr = __uint_as_float(warp_kth_key(sm, g, lane, a.k_zr, kmax));
        if (a.flags & TDQ_ENABLE_C1) {
            for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const double mu = s / (double)g;
            double ss = 0.0;
            for (int i = lane; i < g; i += 32) {
                double d = (double)sm[i] - mu;
                ss = __dadd_rn(ss, __dmul_rn(d, d));
            }
            for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            sigma = __fadd_rn(__double2float_rn(sqrt(ss / (double)g)), kStdEps);
        }
        float c, delta;
        dcrp_project(c_base, sigma, thr, a.seven_tau, a.flags, c, delta);
        uint8_t* row_codes = a.codes + (m * C_pad + (int64_t)k * g) / 2;
        for (int j = lane; j < g / 2; j += 32) {
            int q0 = quantize_ieee(sm[2 * j], c, delta);
            int q1 = quantize_ieee(sm[2 * j + 1], c, delta);
            row_codes[j] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
        }
        if (lane == 0) {
            a.scale[gi] = delta;
            if (a.offset) a.offset[gi] = 0.0f;
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------
// fast kernel: g = 32, one thread per group

constexpr int kFastThreads = 256;   // groups per CTA tile

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

// One group held in registers (w: 16 packed bf16 pairs or 32 floats, in channel order): statistics,
// projection, quantization; writes the group's 16 code bytes and its scale.
template <bool BF16, int KZR>
__device__ __forceinline__ void process_group(const uint32_t (&w)[BF16 ? 16 : 32], const ActArgs& a, int64_t gi) {
    auto get = [&](int i) -> float {
        if (BF16) return (i & 1) ? __uint_as_float(w[i >> 1] & 0xffff0000u) : __uint_as_float(w[i >> 1] << 16);
        return __uint_as_float(w[i]);
    };

    // base radius, rank-KZR magnitude, moments
    float c_base, thr = 0.0f;
    if (BF16) {
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
        if (a.flags & TDQ_ENABLE_C2) {
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
        if (a.flags & TDQ_ENABLE_C2) {
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
    if (a.flags & TDQ_ENABLE_C1) {
        float cmin = c_base;
        if (a.flags & TDQ_ENABLE_C2) cmin = fminf(cmin, __fmul_rn(14.0f, thr));
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
                                        a.seven_tau, cmin);
        } else {
            float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                float v = get(i);
                s1 += v;
                s2 = fmaf(v, v, s2);
            }
            idle = c1_cannot_bind(s1, s2, a.seven_tau, cmin);
        }
        if (!idle) sigma = sigma_exact32(get);
    }

    float c, delta;
    dcrp_project(c_base, sigma, thr, a.seven_tau, a.flags, c, delta);

    uint32_t out[4];
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
    reinterpret_cast<uint4*>(a.codes)[gi] = make_uint4(out[0], out[1], out[2], out[3]);
    a.scale[gi] = delta;
    if (a.offset) a.offset[gi] = 0.0f;
}

template <bool BF16, int KZR>
__global__ void __launch_bounds__(kFastThreads) act_g32_kernel(ActArgs a) {
    constexpr int kGroupBytes = BF16 ? 64 : 128;
    constexpr int kChunks = kGroupBytes / 16;          // 16-byte chunks per group
    constexpr int kSwzMask = kChunks - 1;
    __shared__ __align__(16) uint4 tile[kFastThreads * kChunks];

    const int t = threadIdx.x;
    const int64_t g0 = (int64_t)blockIdx.x * kFastThreads;
    const char* xb = reinterpret_cast<const char*>(a.x);
    const int64_t esize = BF16 ? 2 : 4;
    const bool flat = (a.row_stride == a.C);

    // stage: coalesced 16-byte loads; chunk p of local group l lands at l*kChunks + (p ^ swz(l))
#pragma unroll
    for (int j = 0; j < kChunks; ++j) {
        const int ch = t + j * kFastThreads;
        const int l = ch / kChunks, p = ch % kChunks;
        const int64_t gi = g0 + l;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (gi < a.total_groups) {
            int64_t off;
            if (flat) {
                off = gi * kGroupBytes + p * 16;
            } else {
                const int64_t m = gi / a.K;
                const int64_t k = gi - m * a.K;
                off = (m * a.row_stride + k * 32) * esize + p * 16;
            }
            v = __ldg(reinterpret_cast<const uint4*>(xb + off));
        }
        const int swz = BF16 ? ((l >> 1) & kSwzMask) : (l & kSwzMask);
        tile[l * kChunks + (p ^ swz)] = v;
    }
    __syncthreads();

    const int64_t gi = g0 + t;
    if (gi >= a.total_groups) return;

    // this thread's group: words w[], 16 packed bf16 pairs or 32 floats
    uint32_t w[kChunks * 4];
    {
        const int swz = BF16 ? ((t >> 1) & kSwzMask) : (t & kSwzMask);
#pragma unroll
        for (int p = 0; p < kChunks; ++p) {
            uint4 v = tile[t * kChunks + (p ^ swz)];
            w[4 * p + 0] = v.x; w[4 * p + 1] = v.y; w[4 * p + 2] = v.z; w[4 * p + 3] = v.w;
        }
    }
    process_group<BF16, KZR>(w, a, gi);
}

// ------------------------------------------------------------------------------------------
// fast kernel for dense rows (row stride == C): persistent CTAs, bulk-copy ring
//
// Consecutive groups are consecutive in memory, so a tile of 256 groups is one contiguous
// piece (16 KB of bf16, 32 KB of fp32).  A producer lane streams tiles into a ring of
// shared-memory stages with cp.async.bulk; the 256 consumer threads take one group each out of
// a stage, hand the stage back, and then spend their time on the selection network while the
// next tiles are already landing.  Waits are bounded (see kRingTimeout).

constexpr int kRingStagesBf16 = 4, kRingStagesF32 = 3;
constexpr int kRingThreads = kFastThreads + 32;
constexpr long long kRingTimeout = 2000000000LL;

__device__ __forceinline__ uint32_t ring_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool ring_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(ring_smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// false when the phase did not complete in about a second (the caller then stops working)
__device__ __forceinline__ bool ring_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (ring_test(bar, parity)) return true;
    long long t0 = 0;
    uint32_t polls = 0;
#pragma unroll 1
    while (!ring_test(bar, parity)) {
        if ((++polls & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > kRingTimeout) { *abort_flag = 1; return false; }
        }
    }
    return true;
}

template <bool BF16, int KZR>
__global__ void __launch_bounds__(kRingThreads) act_g32_ring_kernel(ActArgs a, int64_t n_tiles) {
    constexpr int kGroupBytes = BF16 ? 64 : 128;
    constexpr int kChunks = kGroupBytes / 16;
    constexpr int kStages = BF16 ? kRingStagesBf16 : kRingStagesF32;
    constexpr int kStageBytes = kFastThreads * kGroupBytes;
    extern __shared__ __align__(128) uint8_t ring_smem[];
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ volatile int abort_flag;
    const int t = threadIdx.x;
    if (t == 0) {
        for (int i = 0; i < kStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ring_smem_u32(&full[i])), "r"(1) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ring_smem_u32(&empty[i])), "r"(kFastThreads / 32) : "memory");
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const char* xb = reinterpret_cast<const char*>(a.x);
    if (t >= kFastThreads) {
        if (t == kFastThreads) {   // producer lane
            uint32_t s = 0, ph = 0;
            for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
                if (!ring_wait(&empty[s], ph ^ 1, &abort_flag)) break;
                const int64_t g0 = tile * kFastThreads;
                const int64_t ng = min((int64_t)kFastThreads, a.total_groups - g0);
                const uint32_t bytes = (uint32_t)(ng * kGroupBytes);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ring_smem_u32(&full[s])), "r"(bytes) : "memory");
                asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(ring_smem_u32(ring_smem + (size_t)s * kStageBytes)), "l"(xb + g0 * kGroupBytes), "r"(bytes),
                               "r"(ring_smem_u32(&full[s]))
                             : "memory");
                if (++s == kStages) { s = 0; ph ^= 1; }
            }
        }
        return;
    }
    uint32_t s = 0, ph = 0;
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        if (!__all_sync(0xffffffffu, ring_wait(&full[s], ph, &abort_flag))) break;
        const int64_t gi = tile * kFastThreads + t;
        uint32_t w[kChunks * 4];
        // volatile loads: the stage is handed back right below, so these must be the only reads of it
        const uint32_t src = ring_smem_u32(ring_smem + (size_t)s * kStageBytes + (size_t)t * kGroupBytes);
#pragma unroll
        for (int p = 0; p < kChunks; ++p)
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[4 * p + 0]), "=r"(w[4 * p + 1]), "=r"(w[4 * p + 2]), "=r"(w[4 * p + 3])
                         : "r"(src + p * 16)
                         : "memory");
        // The producer refills the stage through the async proxy as soon as the eighth warp has
        // arrived.  Reads made through the generic proxy are only ordered before such writes by a
        // proxy fence; without it the refill was observed to overtake these loads.
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if ((t & 31) == 0)
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ring_smem_u32(&empty[s])) : "memory");
        if (++s == kStages) { s = 0; ph ^= 1; }
        if (gi < a.total_groups) process_group<BF16, KZR>(w, a, gi);
    }
}

template <bool BF16, int KZR>
cudaError_t launch_ring(const ActArgs& a, cudaStream_t st) {
    constexpr int kStages = BF16 ? kRingStagesBf16 : kRingStagesF32;
    constexpr int smem = kStages * kFastThreads * (BF16 ? 64 : 128);
    static int n_sm = 0;
    static bool attr_done = false;
    if (n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorUnknown;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorUnknown;
    }
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(act_g32_ring_kernel<BF16, KZR>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int64_t n_tiles = (a.total_groups + kFastThreads - 1) / kFastThreads;
    const int64_t grid = n_tiles < 2 * n_sm ? n_tiles : 2 * n_sm;
    act_g32_ring_kernel<BF16, KZR><<<(unsigned)grid, kRingThreads, smem, st>>>(a, n_tiles);
    return cudaGetLastError();
}

template <bool BF16>
cudaError_t launch_fast(const ActArgs& a, cudaStream_t st) {
    const int64_t blocks = (a.total_groups + kFastThreads - 1) / kFastThreads;
    dim3 grid((unsigned)blocks), block(kFastThreads);
    if (a.row_stride == a.C) {   // dense rows: the persistent ring kernel
        switch (a.k_zr) {
#define TDQ_CASE(KZ) case KZ: return launch_ring<BF16, KZ>(a, st);
            TDQ_CASE(4) TDQ_CASE(7) TDQ_CASE(10) TDQ_CASE(13) TDQ_CASE(16) TDQ_CASE(32)
#undef TDQ_CASE
            default: return cudaErrorInvalidValue;
        }
    }
    switch (a.k_zr) {
#define TDQ_CASE(KZ) case KZ: act_g32_kernel<BF16, KZ><<<grid, block, 0, st>>>(a); break;
        TDQ_CASE(4) TDQ_CASE(7) TDQ_CASE(10) TDQ_CASE(13) TDQ_CASE(16) TDQ_CASE(32)
#undef TDQ_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

bool fast_rank(int k) { return k == 4 || k == 7 || k == 10 || k == 13 || k == 16 || k == 32; }

}  // namespace

// Argument checks shared with the fused entry point.
tdq_status check_act_args(const void* x, tdq_dtype dt, int64_t B, int64_t N, int64_t C, int64_t stride,
                          const tdq_act_params* p) {
    if (!x || !p) return TDQ_ERR_INVALID_ARG;
    if (dt != TDQ_F32 && dt != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || C <= 0 || stride < C) return TDQ_ERR_INVALID_ARG;
    if (p->group_size < 2 || p->group_size > 4096 || (p->group_size & 1)) return TDQ_ERR_INVALID_ARG;
    if (!(p->tau > 0.0f) || !(p->zr > 0.0f && p->zr <= 1.0f)) return TDQ_ERR_INVALID_ARG;
    if (!(p->base_percentile > 0.0f && p->base_percentile <= 1.0f)) return TDQ_ERR_INVALID_ARG;
    if (p->flags & ~(TDQ_ENABLE_C1 | TDQ_ENABLE_C2)) return TDQ_ERR_INVALID_ARG;
    return TDQ_OK;
}

bool act_fast_path_ok(const void* x, tdq_dtype dt, int64_t C, int64_t stride, const tdq_act_params* p) {
    const int32_t g = p->group_size;
    const int64_t esize = dt == TDQ_BF16 ? 2 : 4;
    return g == 32 && C % 32 == 0 && (reinterpret_cast<uintptr_t>(x) % 16 == 0) &&
           (stride * esize) % 16 == 0 && rank_of(p->base_percentile, g) == g &&
           (!(p->flags & TDQ_ENABLE_C2) || fast_rank(rank_of(p->zr, g)));
}

}  // namespace tdq

using namespace tdq;

extern "C" void tdq_default_act_params(tdq_act_params* p) {
    if (!p) return;
    p->group_size = 32;
    p->tau = 1.0f;
    p->zr = 0.2f;
    p->base_percentile = 1.0f;
    p->flags = TDQ_ENABLE_C1 | TDQ_ENABLE_C2;
}

extern "C" tdq_status tdq_quantize_act(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                       int64_t row_stride_elems, const tdq_act_params* p, uint8_t* codes,
                                       float* scale, float* offset, void* cuda_stream) {
    tdq_status st = check_act_args(x, x_dtype, B, N, C, row_stride_elems, p);
    if (st != TDQ_OK) return st;
    if (!codes || !scale) return TDQ_ERR_INVALID_ARG;
    const int64_t M = B * N;
    if (M == 0) return TDQ_OK;
    const int32_t g = p->group_size;
    ActArgs a;
    a.x = x;
    a.M = M;
    a.C = C;
    a.row_stride = row_stride_elems;
    a.g = g;
    const int64_t K = (C + g - 1) / g;
    if (K > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    a.K = (int32_t)K;
    a.total_groups = M * K;
    a.k_zr = rank_of(p->zr, g);
    a.k_base = rank_of(p->base_percentile, g);
    a.seven_tau = 7.0f * p->tau;
    a.flags = p->flags;
    a.codes = codes;
    a.scale = scale;
    a.offset = offset;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    const bool out_aligned = reinterpret_cast<uintptr_t>(codes) % 16 == 0;
    if (out_aligned && act_fast_path_ok(x, x_dtype, C, row_stride_elems, p) &&
        a.total_groups / kFastThreads < INT32_MAX) {
        if (!(a.flags & TDQ_ENABLE_C2)) a.k_zr = 7;   // rank unused; pick an instantiated kernel
        e = (x_dtype == TDQ_BF16) ? launch_fast<true>(a, stream) : launch_fast<false>(a, stream);
    } else {
        const size_t smem = (size_t)kGenericWarps * g * sizeof(float);
        int64_t blocks = (a.total_groups + kGenericWarps - 1) / kGenericWarps;
        if (blocks > 148 * 64) blocks = 148 * 64;
        if (smem > 48 * 1024) {
            cudaFuncSetAttribute(act_generic_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            cudaFuncSetAttribute(act_generic_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        }
        if (x_dtype == TDQ_BF16)
            act_generic_kernel<true><<<(unsigned)blocks, kGenericWarps * 32, smem, stream>>>(a);
        else
            act_generic_kernel<false><<<(unsigned)blocks, kGenericWarps * 32, smem, stream>>>(a);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}
