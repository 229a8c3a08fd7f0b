// tdq_quantize_act: token-group dual-constraint activation quantizer (Algorithm S1 steps 1-7).
//
// Five kernels:
//   * act_g32_ring_kernel   the fast path on dense rows (row stride == C): persistent, two CTAs per
//     SM; one producer lane streams 16 KB tiles of 256 groups into a shared-memory ring with 1-D
//     bulk copies and mbarrier transaction counts, eight consumer warps take one group per thread
//     (the per-group arithmetic is in tdq_act_group.cuh).
//   * act_g32_kernel   the same per-group code for strided rows: g = 32, C % 32 == 0, 16-byte
//     aligned rows.  A CTA stages a tile of
//     consecutive token-groups in shared memory with coalesced 128-bit loads (XOR-swizzled
//     so the read-back is conflict free); then every thread owns one whole group in
//     registers: max, sums, a pruned sorting network for the rank-k magnitude, the DCRP
//     projection, an exact quotient, round-half-even, and one 128-bit store of 32 nibbles.
//     One pass over HBM: 2 (bf16) or 4 (fp32) bytes in, 0.5 + 0.125 bytes out per element.
//   * act_g32_nchw_kernel   channel-major input [B, C, H*W]: a tile of 32 channel rows is staged in
//     shared memory and each thread gathers one position's 32 channels (tdq_quantize_act_nchw).
//   * act_fixed_kernel   the fixed-radius control: no reductions, 8 channels per thread
//     (tdq_quantize_act_fixed).
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

#include "tdq_act_group.cuh"
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

// One group: quantize it in registers, write its 16 code bytes and its scale.
template <bool BF16, int KZR, int KB = 32>
__device__ __forceinline__ void process_group(const uint32_t (&w)[BF16 ? 16 : 32], const ActArgs& a, int64_t gi) {
    uint32_t out[4];
    float delta;
    quantize_group32<BF16, KZR, KB>(w, a.seven_tau, a.flags, out, delta, a.k_zr, a.k_base);
    reinterpret_cast<uint4*>(a.codes)[gi] = make_uint4(out[0], out[1], out[2], out[3]);
    a.scale[gi] = delta;
    if (a.offset) a.offset[gi] = 0.0f;
}

template <bool BF16, int KZR, int KB = 32>
__global__ void __launch_bounds__(kFastThreads) act_g32_kernel(ActArgs a) {
    constexpr int kGroupBytes = BF16 ? 64 : 128;
    constexpr int kChunks = kGroupBytes / 16;          // 16-byte chunks per group
    constexpr int kSwzMask = kChunks - 1;
    __shared__ __align__(16) uint4 tile[kFastThreads * kChunks];

    pdl_wait();
    pdl_trigger();
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
    process_group<BF16, KZR, KB>(w, a, gi);
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
// A ring wait that ran out leaves its code here (first writer wins): bits 0-7 name the wait (12 producer, 13 consumer,
// 14 the self-test), bits 8-31 the CTA.  One word per device, read and cleared by tdq_quantize_status().
__device__ uint32_t g_act_wait_status = 0u;

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
__device__ __forceinline__ bool ring_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t code,
                                          long long limit = kRingTimeout) {
    if (ring_test(bar, parity)) return true;
    long long t0 = 0;
    uint32_t polls = 0;
#pragma unroll 1
    while (!ring_test(bar, parity)) {
        if ((++polls & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit) {
                atomicCAS(&g_act_wait_status, 0u, code | ((uint32_t)blockIdx.x << 8));
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}

template <bool BF16, int KZR, int KB = 32>
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
    pdl_wait();          // everything above overlaps the tail of the kernel before this one
    pdl_trigger();
    const char* xb = reinterpret_cast<const char*>(a.x);
    if (t >= kFastThreads) {
        if (t == kFastThreads) {   // producer lane
            uint32_t s = 0, ph = 0;
            for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
                if (!ring_wait(&empty[s], ph ^ 1, &abort_flag, 12u)) break;
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
        if (!__all_sync(0xffffffffu, ring_wait(&full[s], ph, &abort_flag, 13u))) break;
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
        if (gi < a.total_groups) process_group<BF16, KZR, KB>(w, a, gi);
    }
}

template <bool BF16, int KZR, int KB = 32>
cudaError_t launch_ring(const ActArgs& a, cudaStream_t st) {
    constexpr int kStages = BF16 ? kRingStagesBf16 : kRingStagesF32;
    constexpr int smem = kStages * kFastThreads * (BF16 ? 64 : 128);
    static std::atomic<uint64_t> attr_done{0};      // per template instance, one bit per device
    int dev = 0;
    const int n_sm = current_device_sm_count(&dev);
    if (n_sm <= 0) return cudaErrorUnknown;
    if (!device_marked(attr_done, dev)) {
        cudaError_t e = cudaFuncSetAttribute(act_g32_ring_kernel<BF16, KZR, KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        mark_device(attr_done, dev);
    }
    const int64_t n_tiles = (a.total_groups + kFastThreads - 1) / kFastThreads;
    const int64_t grid = n_tiles < 2 * n_sm ? n_tiles : 2 * n_sm;
    return launch_pdl(act_g32_ring_kernel<BF16, KZR, KB>, dim3((unsigned)grid), dim3(kRingThreads), smem, st, a, n_tiles);
}

// every zero-bin rank of a group of 32 has its instance of the two row-major kernels
#define TDQ_ALL_RANKS \
    TDQ_CASE(1) TDQ_CASE(2) TDQ_CASE(3) TDQ_CASE(4) TDQ_CASE(5) TDQ_CASE(6) TDQ_CASE(7) TDQ_CASE(8) \
    TDQ_CASE(9) TDQ_CASE(10) TDQ_CASE(11) TDQ_CASE(12) TDQ_CASE(13) TDQ_CASE(14) TDQ_CASE(15) TDQ_CASE(16) \
    TDQ_CASE(17) TDQ_CASE(18) TDQ_CASE(19) TDQ_CASE(20) TDQ_CASE(21) TDQ_CASE(22) TDQ_CASE(23) TDQ_CASE(24) \
    TDQ_CASE(25) TDQ_CASE(26) TDQ_CASE(27) TDQ_CASE(28) TDQ_CASE(29) TDQ_CASE(30) TDQ_CASE(31) TDQ_CASE(32)
template <bool BF16>
cudaError_t launch_fast(const ActArgs& a, cudaStream_t st) {
    const int64_t blocks = (a.total_groups + kFastThreads - 1) / kFastThreads;
    dim3 grid((unsigned)blocks), block(kFastThreads);
    if (a.k_base != 32 && (a.k_base < 29 || a.k_zr != 7)) {
        // any other pair of ranks: the instance that takes both at run time
        if (a.row_stride == a.C) return launch_ring<BF16, 0, 0>(a, st);
        return launch_pdl(act_g32_kernel<BF16, 0, 0>, grid, block, 0, st, a);
    }
    if (a.k_base != 32) {        // percentile base radius: ranks 29..31 beside the default zero-bin rank
        switch (a.k_base) {
#define TDQ_CASE(KB_)                                                                  \
            case KB_:                                                                  \
                if (a.row_stride == a.C) return launch_ring<BF16, 7, KB_>(a, st);      \
                return launch_pdl(act_g32_kernel<BF16, 7, KB_>, grid, block, 0, st, a);
            TDQ_CASE(29) TDQ_CASE(30) TDQ_CASE(31)
#undef TDQ_CASE
            default: return cudaErrorInvalidValue;
        }
    }
    if (a.row_stride == a.C) {   // dense rows: the persistent ring kernel
        switch (a.k_zr) {
#define TDQ_CASE(KZ) case KZ: return launch_ring<BF16, KZ>(a, st);
            TDQ_ALL_RANKS
#undef TDQ_CASE
            default: return cudaErrorInvalidValue;
        }
    }
    switch (a.k_zr) {
#define TDQ_CASE(KZ) case KZ: return launch_pdl(act_g32_kernel<BF16, KZ>, grid, block, 0, st, a);
        TDQ_ALL_RANKS
#undef TDQ_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// channel-major input: x is [B][C][H*W] (a convolutional feature map) and is quantized along C
// without a permuted copy.  A CTA takes one group of 32 channels and 256 consecutive positions of
// one image: the 32 channel rows are read with coalesced loads into a shared-memory tile, then
// thread t gathers position t's 32 channels down the tile's columns and quantizes them like any
// other group.  Codes and scales come out token-major, [B*H*W, C/2] and [B*H*W, C/32].

struct NchwArgs {
    ActArgs a;          // x, K, k_zr, seven_tau, flags, codes, scale, offset
    int64_t HW;         // positions per image
    int32_t vec_ok;     // channel rows can be read with 16-byte loads
};

template <bool BF16, int KZR>
__global__ void __launch_bounds__(kFastThreads) act_g32_nchw_kernel(NchwArgs n) {
    constexpr int esz = BF16 ? 2 : 4;
    constexpr int kRowBytes = kFastThreads * esz + 16;        // 16 bytes of padding per channel row
    constexpr int kVecPerRow = kFastThreads * esz / 16;       // 16-byte pieces of a channel row
    __shared__ __align__(16) uint8_t tile[32 * kRowBytes];
    const ActArgs& a = n.a;
    const int t = threadIdx.x;
    const int64_t s0 = (int64_t)blockIdx.x * kFastThreads;    // first position of the tile
    const int k = blockIdx.y;                                  // channel group
    const int64_t b = blockIdx.z;
    const uint8_t* img = reinterpret_cast<const uint8_t*>(a.x) + ((b * a.C + (int64_t)k * 32) * n.HW + s0) * esz;
    const int64_t left = n.HW - s0;                            // positions from s0 to the end of the image
    if (n.vec_ok) {
#pragma unroll
        for (int j = 0; j < 32 * kVecPerRow / kFastThreads; ++j) {
            const int idx = t + j * kFastThreads;
            const int c = idx / kVecPerRow, piece = idx % kVecPerRow;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if ((int64_t)(piece + 1) * (16 / esz) <= left)     // HW is a multiple of 16 bytes here: pieces are whole
                v = __ldg(reinterpret_cast<const uint4*>(img + (int64_t)c * n.HW * esz) + piece);
            *reinterpret_cast<uint4*>(tile + c * kRowBytes + piece * 16) = v;
        }
    } else {
#pragma unroll 4
        for (int c = 0; c < 32; ++c) {
            const uint8_t* src = img + ((int64_t)c * n.HW + t) * esz;
            if (BF16)
                *reinterpret_cast<uint16_t*>(tile + c * kRowBytes + t * 2) =
                    t < left ? __ldg(reinterpret_cast<const uint16_t*>(src)) : (uint16_t)0;
            else
                *reinterpret_cast<uint32_t*>(tile + c * kRowBytes + t * 4) =
                    t < left ? __ldg(reinterpret_cast<const uint32_t*>(src)) : 0u;
        }
    }
    __syncthreads();
    if (t >= left) return;
    uint32_t w[BF16 ? 16 : 32];
    if (BF16) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t lo = *reinterpret_cast<const uint16_t*>(tile + (2 * i) * kRowBytes + t * 2);
            const uint32_t hi = *reinterpret_cast<const uint16_t*>(tile + (2 * i + 1) * kRowBytes + t * 2);
            w[i] = lo | (hi << 16);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) w[i] = *reinterpret_cast<const uint32_t*>(tile + i * kRowBytes + t * 4);
    }
    process_group<BF16, KZR>(w, a, ((b * n.HW + s0 + t) * a.K) + k);
}

template <bool BF16>
cudaError_t launch_nchw(const NchwArgs& n, int64_t B, cudaStream_t st) {
    dim3 grid((unsigned)((n.HW + kFastThreads - 1) / kFastThreads), (unsigned)n.a.K, (unsigned)B);
    switch (n.a.k_zr) {
#define TDQ_CASE(KZ) case KZ: act_g32_nchw_kernel<BF16, KZ><<<grid, kFastThreads, 0, st>>>(n); break;
        TDQ_CASE(4) TDQ_CASE(7) TDQ_CASE(10) TDQ_CASE(13) TDQ_CASE(16) TDQ_CASE(32)
#undef TDQ_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// fixed-radius control: no reductions at all.  A thread takes 8 consecutive channels of a row:
// one or two 16-byte loads, eight exact quotients, one 4-byte store of codes.

struct FixedArgs {
    const void* x;
    int64_t M, C, row_stride;   // elements
    int64_t chunks_per_row;     // C / 8
    int32_t g, K;
    float c, delta;
    uint8_t* codes;
    float* scale;
    float* offset;
};

template <bool BF16>
__global__ void __launch_bounds__(256) act_fixed_kernel(FixedArgs f) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= f.M * f.chunks_per_row) return;
    int64_t m, ch8;
    if (f.M * f.chunks_per_row <= 0xffffffffll) {   // the usual case: 32-bit division
        const uint32_t q32 = (uint32_t)idx / (uint32_t)f.chunks_per_row;
        m = q32;
        ch8 = (uint32_t)idx - q32 * (uint32_t)f.chunks_per_row;
    } else {
        m = idx / f.chunks_per_row;
        ch8 = idx - m * f.chunks_per_row;
    }
    float v[8];
    if (BF16) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(f.x) + m * f.row_stride + ch8 * 8));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else {
        const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(f.x) + m * f.row_stride + ch8 * 8);
        const uint4 t0 = __ldg(src), t1 = __ldg(src + 1);
        v[0] = __uint_as_float(t0.x); v[1] = __uint_as_float(t0.y); v[2] = __uint_as_float(t0.z); v[3] = __uint_as_float(t0.w);
        v[4] = __uint_as_float(t1.x); v[5] = __uint_as_float(t1.y); v[6] = __uint_as_float(t1.z); v[7] = __uint_as_float(t1.w);
    }
    uint32_t word = 0u;
    if (f.delta <= 1e30f) {   // two channels at a time, as in the token-group kernels
        const float rcp = __frcp_rn(f.delta);
        const uint64_t rcp2 = f2_pack(rcp, rcp), neg_delta2 = f2_pack(-f.delta, -f.delta);
        const uint64_t magic2 = f2_pack(kRoundMagic8, kRoundMagic8);
        uint32_t acc = 0u;
#pragma unroll
        for (int n = 6; n >= 0; n -= 2)
            nibbles_fast2(f2_pack(fminf(fmaxf(v[n], -f.c), f.c), fminf(fmaxf(v[n + 1], -f.c), f.c)), neg_delta2, rcp2, magic2, acc);
        word = pack_word(acc);
    } else {                  // 1 / Delta would be subnormal: take the IEEE division
#pragma unroll
        for (int n = 0; n < 8; ++n) word |= nibble_ieee(v[n], f.c, f.delta) << (4 * n);
    }
    reinterpret_cast<uint32_t*>(f.codes)[idx] = word;
    const int64_t ch = ch8 * 8;
    if (ch % f.g == 0) {
        const int64_t gi = m * f.K + ch / f.g;
        f.scale[gi] = f.delta;
        if (f.offset) f.offset[gi] = 0.0f;
    }
}

// the zero-bin ranks the channel-major kernel is instantiated for (those of the paper's sweep over zr)
bool fast_rank(int k) { return k == 4 || k == 7 || k == 10 || k == 13 || k == 16 || k == 32; }
// base radius: any rank (the maximum and ranks 29-31 with the default zero-bin rank have instances of their own, the
// other pairs share the instance that takes its ranks at run time)
bool fast_base_rank(const tdq_act_params*) { return true; }

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
    if (p->flags & ~(TDQ_ENABLE_C1 | TDQ_ENABLE_C2 | TDQ_POW2_STEP)) return TDQ_ERR_INVALID_ARG;
    return TDQ_OK;
}

bool act_fast_path_ok(const void* x, tdq_dtype dt, int64_t C, int64_t stride, const tdq_act_params* p) {
    const int32_t g = p->group_size;
    const int64_t esize = dt == TDQ_BF16 ? 2 : 4;
    return g == 32 && C % 32 == 0 && (reinterpret_cast<uintptr_t>(x) % 16 == 0) &&
           (stride * esize) % 16 == 0 && fast_base_rank(p);   // every zero-bin rank has its instance
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

extern "C" tdq_status tdq_quantize_act_nchw(const void* x, tdq_dtype x_dtype, int64_t B, int64_t C, int64_t H, int64_t W,
                                            const tdq_act_params* p, uint8_t* codes, float* scale, float* offset,
                                            void* cuda_stream) {
    if (H < 0 || W < 0) return TDQ_ERR_INVALID_ARG;
    const int64_t HW = H * W;
    if (B >= 0 && C > 0 && p && B * HW == 0) return TDQ_OK;   // an empty map: nothing to read, x may be null
    tdq_status st = check_act_args(x, x_dtype, B, HW, C, C, p);
    if (st != TDQ_OK) return st;
    if (!codes || !scale) return TDQ_ERR_INVALID_ARG;
    if (B * HW == 0) return TDQ_OK;
    const int32_t g = p->group_size;
    // the channel-major kernel is the fast path only: 32-channel groups, max-abs base radius, a rank it has
    if (g != 32 || C % 32 != 0 || rank_of(p->base_percentile, g) != g || reinterpret_cast<uintptr_t>(codes) % 16 ||
        ((p->flags & TDQ_ENABLE_C2) && !fast_rank(rank_of(p->zr, g))))
        return TDQ_ERR_UNSUPPORTED;
    if (C / 32 > 65535 || B > 65535 || (HW + kFastThreads - 1) / kFastThreads > INT32_MAX) return TDQ_ERR_UNSUPPORTED;
    NchwArgs n;
    n.a.x = x;
    n.a.M = B * HW;
    n.a.C = C;
    n.a.row_stride = C;
    n.a.g = g;
    n.a.K = (int32_t)(C / 32);
    n.a.total_groups = n.a.M * n.a.K;
    n.a.k_zr = (p->flags & TDQ_ENABLE_C2) ? rank_of(p->zr, g) : 7;   // rank unused without C2; pick an instantiated kernel
    n.a.k_base = g;
    n.a.seven_tau = 7.0f * p->tau;
    n.a.flags = p->flags;
    n.a.codes = codes;
    n.a.scale = scale;
    n.a.offset = offset;
    n.HW = HW;
    const int64_t esz = x_dtype == TDQ_BF16 ? 2 : 4;
    n.vec_ok = (reinterpret_cast<uintptr_t>(x) % 16 == 0 && (HW * esz) % 16 == 0) ? 1 : 0;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const cudaError_t e = (x_dtype == TDQ_BF16) ? launch_nchw<true>(n, B, stream) : launch_nchw<false>(n, B, stream);
    if (e != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

extern "C" tdq_status tdq_quantize_act_fixed(const void* x, tdq_dtype x_dtype, int64_t B, int64_t N, int64_t C,
                                             int64_t row_stride_elems, int32_t group_size, float radius, uint8_t* codes,
                                             float* scale, float* offset, void* cuda_stream) {
    if (!x || !codes || !scale) return TDQ_ERR_INVALID_ARG;
    if (x_dtype != TDQ_F32 && x_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (B < 0 || N < 0 || C <= 0 || row_stride_elems < C) return TDQ_ERR_INVALID_ARG;
    if (group_size < 2 || group_size > 4096 || (group_size & 1) || !(radius > 0.0f)) return TDQ_ERR_INVALID_ARG;
    const int64_t M = B * N;
    if (M == 0) return TDQ_OK;
    const int64_t esz = x_dtype == TDQ_BF16 ? 2 : 4;
    if (group_size % 8 || C % group_size || reinterpret_cast<uintptr_t>(x) % 16 || (row_stride_elems * esz) % 16 ||
        reinterpret_cast<uintptr_t>(codes) % 4)
        return TDQ_ERR_UNSUPPORTED;
    FixedArgs f;
    f.x = x; f.M = M; f.C = C; f.row_stride = row_stride_elems; f.chunks_per_row = C / 8;
    f.g = group_size; f.K = (int32_t)(C / group_size);
    f.c = fmaxf(radius, kClipFloor);
    f.delta = fmaxf(f.c / kQmax, kStepFloor);      // binary32 division on the host: the same IEEE operation
    f.codes = codes; f.scale = scale; f.offset = offset;
    const int64_t blocks = (M * f.chunks_per_row + 255) / 256;
    if (blocks > INT32_MAX) return TDQ_ERR_UNSUPPORTED;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (x_dtype == TDQ_BF16)
        act_fixed_kernel<true><<<(unsigned)blocks, 256, 0, stream>>>(f);
    else
        act_fixed_kernel<false><<<(unsigned)blocks, 256, 0, stream>>>(f);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

// ------------------------------------------------------------------------------------------
// bounded waits of the quantizer: the status word and the self-test

namespace tdq {
namespace {
// One warp: a fresh barrier with one expected arrival that never comes, waited on with the ring kernel's own
// routine and a short limit.  Nothing is in flight when the warp leaves.
__global__ void __launch_bounds__(32) act_wait_selftest_kernel(long long limit) {
    __shared__ uint64_t bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(ring_smem_u32(&bar)) : "memory");
        abort_flag = 0;
    }
    __syncwarp();
    ring_wait(&bar, 0u, &abort_flag, 14u, limit);
}
}  // namespace

tdq_status act_wait_selftest(long long limit_cycles, cudaStream_t stream) {
    act_wait_selftest_kernel<<<1, 32, 0, stream>>>(limit_cycles);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}
}  // namespace tdq

extern "C" tdq_status tdq_quantize_status(void* cuda_stream, uint32_t* detail) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    const uint32_t zero = 0;
    if (cudaMemcpyFromSymbolAsync(&word, g_act_wait_status, sizeof word, 0, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return TDQ_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (word != 0 &&
        (cudaMemcpyToSymbolAsync(g_act_wait_status, &zero, sizeof zero, 0, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
         cudaStreamSynchronize(stream) != cudaSuccess))
        return TDQ_ERR_CUDA;
    if (detail) *detail = word;
    return word == 0 ? TDQ_OK : TDQ_ERR_DEVICE_TIMEOUT;
}
