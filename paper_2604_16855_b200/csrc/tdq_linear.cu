// tdq_w4a4_linear: W4A4 linear layer on the 5th-generation tensor cores (Algorithm S1 step 10).
//
//   acc[m,o,k] = sum_{i in group k} q_x[m,i] q_w[o,i]      tcgen05.mma kind::i8, int32 in TMEM
//   y[m,o]     = s_o * sum_k Delta[m,k] * acc[m,o,k] + b_o  fp32 in registers
//
// The activation scale changes every g codes along the contraction axis, so an int32
// accumulator may only span one token-group.  Each group gets its own TMEM slot (a fresh
// accumulation; groups wider than 32 codes chain g/32 instructions into the same slot), is
// read back with tcgen05.ld, converted, multiplied by its Delta and added to a float
// accumulator that stays in registers for the whole contraction ("promotion").
//
// One persistent CTA per SM walks over 128 x 128 output tiles.  Warp roles:
//   warps 0-7   promotion + epilogue: warp w owns TMEM lanes 32 (w % 4) .. +31 (its rows) and
//               columns 64 (w / 4) .. +63; a thread keeps 64 float accumulators of one row.
//   warp  8     one lane issues the MMAs and the commits that release buffers.
//   warps 9-11  operand producers: 128-bit loads of packed codes, unpack to int8, store in
//               the tensor core's shared-memory layout, publish with an mbarrier.
// Two rings decouple the roles: kStages operand stages (one K-step of 32 codes each) and
// kSlots TMEM accumulator slots, each with a full and an empty mbarrier.
//
// Operands.  A nibble is moved to the HIGH half of its byte, which is the two's complement
// byte 16 q: no sign extension is needed, the integer result is 256 acc (exactly;
// |256 acc| < 2^31 for g <= 4096) and the factor 1/256 is folded into Delta, an exact
// power-of-two scaling.  Even channels fill the first 16 bytes of a row and odd channels the
// second 16; both operands use the same order, so the sum is unchanged.
//
// Shared-memory operand layout: K-major, no swizzle.  A 32-byte row splits into two 16-byte
// chunks; 8 rows x 16 bytes form one contiguous 128-byte core matrix; the two K-chunks of an
// 8-row band are 128 bytes apart (leading byte offset), bands are 256 bytes apart (stride
// byte offset).
//
// Every wait on an mbarrier is bounded: after about a second the thread records a code in
// the workspace status word and raises a CTA-wide flag; every role then leaves its loops,
// the CTA releases its TMEM and returns.
#include "tdq_common.cuh"

namespace tdq {
namespace {

constexpr int kBM = 128;              // rows per tile = TMEM lanes
constexpr int kBN = 128;              // columns per tile = one TMEM slot
constexpr int kStages = 8;            // operand ring, one K-step (32 codes) per stage
constexpr int kSlots = 4;             // TMEM accumulator ring (4 x 128 = 512 columns)
constexpr int kPromoWarps = 8;
constexpr int kMmaWarp = 8;
constexpr int kProdWarp0 = 9;
constexpr int kProdWarps = 3;
constexpr int kThreads = (kPromoWarps + 1 + kProdWarps) * 32;   // 384: 12 warps leave 168 registers per thread
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kJobs = (kBM + kBN + kProdThreads - 1) / kProdThreads;   // operand rows per producer thread
constexpr int kABytes = kBM * 32, kBBytes = kBN * 32;
static_assert(kABytes == kBBytes, "the producers address both operand rings with one stage stride");
constexpr uint32_t kTmemCols = kSlots * kBN;
constexpr long long kTimeoutCycles = 2000000000LL;
// S32 accumulator, signed 8-bit A and B, both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                            ((uint32_t)(kBM >> 4) << 24);

struct LinArgs {
    const uint8_t* xcodes;
    const float* xscale;
    const uint8_t* wcodes;
    const float* wscale;
    const float* bias;
    int64_t M, O;
    int32_t row_bytes;      // I_pad / 2
    int32_t n_steps;        // I_pad / 32
    int32_t steps_per_grp;  // g / 32
    int32_t Kg;             // groups per token
    int32_t tiles_m, tiles_n;
    void* y;
    int64_t y_stride;
    int32_t* acc_debug;
    uint32_t* status;
    int32_t vec_ok;         // y, wscale, bias 16-byte aligned and y_stride % 4 == 0: float4 epilogue
};

struct __align__(128) Smem {
    uint8_t a[kStages][kABytes];
    uint8_t b[kStages][kBBytes];
    uint64_t full[kStages], empty[kStages];
    uint64_t tfull[kSlots], tempty[kSlots];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: false when the phase did not complete within the time limit or another
// role of this CTA already gave up.  `code` names the wait in the status word.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Smem* sm, uint32_t* status, uint32_t code) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_test(bar, parity)) return true;
        if (sm->abort_flag) return false;
        if (clock64() - t0 > kTimeoutCycles) {
            atomicCAS(status, 0u, code | ((uint32_t)blockIdx.x << 8));
            sm->abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ uint64_t smem_desc_kmajor_noswizzle(uint32_t saddr) {
    // start address, leading byte offset 128, stride byte offset 256 (all >> 4), version 1
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 16) | ((uint64_t)(256 >> 4) << 32) |
           (1ull << 46);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 16 packed bytes (32 codes) -> two 16-byte chunks of bytes 16*q: even channels, odd channels.
__device__ __forceinline__ void unpack16(const uint4 p, uint4& even, uint4& odd) {
    even = make_uint4((p.x << 4) & 0xF0F0F0F0u, (p.y << 4) & 0xF0F0F0F0u, (p.z << 4) & 0xF0F0F0F0u,
                      (p.w << 4) & 0xF0F0F0F0u);
    odd = make_uint4(p.x & 0xF0F0F0F0u, p.y & 0xF0F0F0F0u, p.z & 0xF0F0F0F0u, p.w & 0xF0F0F0F0u);
}

// byte offset of row r, K-chunk 0 inside one K-step's operand block (see the layout note above)
__device__ __forceinline__ uint32_t row_off(int r) { return (uint32_t)((r >> 3) * 256 + (r & 7) * 16); }

template <bool YBF16>
__global__ void __launch_bounds__(kThreads, 1) w4a4_linear_kernel(LinArgs a) {
    extern __shared__ uint8_t smem_raw[];
    Smem* sm = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;

    if (t == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&sm->full[i], kProdWarps); mbar_init(&sm->empty[i], 1); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(&sm->tfull[i], 1); mbar_init(&sm->tempty[i], kPromoWarps); }
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    const int64_t n_tiles = (int64_t)a.tiles_m * a.tiles_n;
    const int grp_per_tile = a.n_steps / a.steps_per_grp;

    if (warp < kPromoWarps) {
        // ------------------------------------------------------------ promotion + epilogue
        const int row = (warp & 3) * 32 + lane;
        const int col0 = (warp >> 2) * (kBN / 2);
        uint32_t gc = 0;   // groups consumed so far (across tiles): slot = gc % kSlots
        for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            const int64_t m = (tile / a.tiles_n) * kBM + row;
            const int64_t n0 = (tile % a.tiles_n) * kBN + col0;
            const bool row_ok = m < a.M;
            const float* srow = a.xscale + (row_ok ? m : 0) * a.Kg;
            float yacc[kBN / 2];
#pragma unroll
            for (int j = 0; j < kBN / 2; ++j) yacc[j] = 0.0f;
            float d_next = row_ok ? __ldg(srow) * (1.0f / 256.0f) : 0.0f;
            bool ok = true;
            for (int grp = 0; grp < grp_per_tile && ok; ++grp, ++gc) {
                const float d256 = d_next;
                if (grp + 1 < grp_per_tile) d_next = row_ok ? __ldg(srow + grp + 1) * (1.0f / 256.0f) : 0.0f;
                const uint32_t slot = gc % kSlots;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm->tfull[slot], (gc / kSlots) & 1, sm, a.status, 2u));
                if (!ok) break;   // warp-uniform: the TMEM loads below are warp-collective
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + slot * kBN + col0;
                uint32_t v0[32], v1[32];
                tmem_ld32(taddr, v0);
                tmem_ld32(taddr + 32, v1);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->tempty[slot]);   // slot may be overwritten from here on
#pragma unroll
                for (int j = 0; j < 32; ++j) yacc[j] = fmaf(d256, (float)(int32_t)v0[j], yacc[j]);
#pragma unroll
                for (int j = 0; j < 32; ++j) yacc[32 + j] = fmaf(d256, (float)(int32_t)v1[j], yacc[32 + j]);
                if (a.acc_debug && row_ok) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (n0 + j < a.O) a.acc_debug[(m * a.O + n0 + j) * a.Kg + grp] = ((int32_t)v0[j]) >> 8;
                        if (n0 + 32 + j < a.O) a.acc_debug[(m * a.O + n0 + 32 + j) * a.Kg + grp] = ((int32_t)v1[j]) >> 8;
                    }
                }
            }
            if (!ok) break;
            // epilogue: y = s_o * sum + bias
            if (row_ok) {
                if (!YBF16 && a.vec_ok && n0 + kBN / 2 <= a.O) {
                    float* yrow = reinterpret_cast<float*>(a.y) + m * a.y_stride + n0;
#pragma unroll
                    for (int j = 0; j < kBN / 2; j += 4) {
                        const float4 s4 = __ldg(reinterpret_cast<const float4*>(a.wscale + n0 + j));
                        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (a.bias) b4 = __ldg(reinterpret_cast<const float4*>(a.bias + n0 + j));
                        float4 o;
                        o.x = __fmaf_rn(s4.x, yacc[j], b4.x);
                        o.y = __fmaf_rn(s4.y, yacc[j + 1], b4.y);
                        o.z = __fmaf_rn(s4.z, yacc[j + 2], b4.z);
                        o.w = __fmaf_rn(s4.w, yacc[j + 3], b4.w);
                        __stcs(reinterpret_cast<float4*>(yrow + j), o);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < kBN / 2; ++j) {
                        const int64_t n = n0 + j;
                        if (n < a.O) {
                            const float b = a.bias ? __ldg(a.bias + n) : 0.0f;
                            const float v = __fmaf_rn(__ldg(a.wscale + n), yacc[j], b);
                            if (YBF16)
                                reinterpret_cast<__nv_bfloat16*>(a.y)[m * a.y_stride + n] = __float2bfloat16_rn(v);
                            else
                                reinterpret_cast<float*>(a.y)[m * a.y_stride + n] = v;
                        }
                    }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issue (one lane)
        if (lane == 0) {
            uint32_t it = 0, gc = 0;
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                for (int step = 0; step < a.n_steps && ok; ++step, ++it) {
                    const uint32_t s = it % kStages;
                    const int sub = step % a.steps_per_grp;
                    const uint32_t slot = gc % kSlots;
                    if (sub == 0) ok = mbar_wait(&sm->tempty[slot], ((gc / kSlots) & 1) ^ 1, sm, a.status, 3u);
                    if (ok) ok = mbar_wait(&sm->full[s], (it / kStages) & 1, sm, a.status, 4u);
                    if (!ok) break;
                    tc_fence_after();
                    mma_i8(tmem_base + slot * kBN, smem_desc_kmajor_noswizzle(smem_u32(sm->a[s])),
                           smem_desc_kmajor_noswizzle(smem_u32(sm->b[s])), kIdesc, sub == 0 ? 0u : 1u);
                    mma_commit(&sm->empty[s]);
                    if (sub == a.steps_per_grp - 1) {
                        mma_commit(&sm->tfull[slot]);
                        ++gc;
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ operand producers
        // row job j: j < kBM is row j of the A tile, otherwise row j - kBM of the B tile
        const int pt = (warp - kProdWarp0) * 32 + lane;
        uint32_t it = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const int64_t m0 = (tile / a.tiles_n) * kBM, n0 = (tile % a.tiles_n) * kBN;
            const uint8_t* src[kJobs];
            uint32_t dst[kJobs];
#pragma unroll
            for (int q = 0; q < kJobs; ++q) {
                const int j = pt + q * kProdThreads;
                src[q] = nullptr;
                dst[q] = 0xffffffffu;
                if (j < kBM) {
                    if (m0 + j < a.M) src[q] = a.xcodes + (m0 + j) * a.row_bytes;
                    dst[q] = row_off(j);
                } else if (j < kBM + kBN) {
                    if (n0 + (j - kBM) < a.O) src[q] = a.wcodes + (n0 + (j - kBM)) * a.row_bytes;
                    dst[q] = (uint32_t)(kStages * kABytes) + row_off(j - kBM);   // b[] follows a[] in Smem
                }
            }
            for (int s0 = 0; s0 < a.n_steps && ok; s0 += 4) {
                uint4 pk[kJobs][4];
#pragma unroll
                for (int q = 0; q < kJobs; ++q)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        pk[q][b] = make_uint4(0, 0, 0, 0);
                        if (src[q] && s0 + b < a.n_steps)
                            pk[q][b] = __ldg(reinterpret_cast<const uint4*>(src[q] + (size_t)(s0 + b) * 16));
                    }
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    if (s0 + b >= a.n_steps) break;
                    const uint32_t s = it % kStages;
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm->empty[s], ((it / kStages) & 1) ^ 1, sm, a.status, 5u));
                    if (!ok) break;   // warp-uniform: the warp synchronises below
#pragma unroll
                    for (int q = 0; q < kJobs; ++q) {
                        if (dst[q] == 0xffffffffu) continue;
                        uint4 ev, od;
                        unpack16(pk[q][b], ev, od);
                        // a[s] and b[s] blocks: stage stride is kABytes for A rows and kBBytes for B rows (equal)
                        uint8_t* d = sm->a[0] + dst[q] + s * kABytes;
                        *reinterpret_cast<uint4*>(d) = ev;
                        *reinterpret_cast<uint4*>(d + 128) = od;
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->full[s]);
                    ++it;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        // all MMAs this CTA issued have completed unless a wait gave up; in that case give the
        // tensor core a moment before the columns are handed back
        if (sm->abort_flag) __nanosleep(1000000);
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace
}  // namespace tdq

using namespace tdq;

extern "C" size_t tdq_linear_workspace_bytes(int64_t, int64_t, int64_t, int32_t) { return 256; }

extern "C" tdq_status tdq_w4a4_linear(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                      const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                      int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                      int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream) {
    if (!xcodes || !xscale || !wcodes || !wscale || !y) return TDQ_ERR_INVALID_ARG;
    if (M < 0 || O <= 0 || I_pad <= 0 || y_row_stride < O) return TDQ_ERR_INVALID_ARG;
    if (y_dtype != TDQ_F32 && y_dtype != TDQ_BF16) return TDQ_ERR_INVALID_ARG;
    if (group_size <= 0 || I_pad % group_size) return TDQ_ERR_INVALID_ARG;
    if (group_size % 32 || group_size > 4096) return TDQ_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < tdq_linear_workspace_bytes(M, I_pad, O, group_size)) return TDQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(xcodes) % 16 || reinterpret_cast<uintptr_t>(wcodes) % 16 ||
        reinterpret_cast<uintptr_t>(workspace) % 16)
        return TDQ_ERR_ALIGNMENT;
    if (I_pad / 2 > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    if (M == 0) return TDQ_OK;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);

    LinArgs a;
    a.xcodes = xcodes; a.xscale = xscale; a.wcodes = wcodes; a.wscale = wscale; a.bias = bias;
    a.M = M; a.O = O;
    a.row_bytes = (int32_t)(I_pad / 2);
    a.n_steps = (int32_t)(I_pad / 32);
    a.steps_per_grp = group_size / 32;
    a.Kg = (int32_t)(I_pad / group_size);
    const int64_t tm = (M + kBM - 1) / kBM, tn = (O + kBN - 1) / kBN;
    if (tm > INT32_MAX || tn > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    a.tiles_m = (int32_t)tm;
    a.tiles_n = (int32_t)tn;
    a.y = y; a.y_stride = y_row_stride; a.acc_debug = acc_debug;
    a.status = reinterpret_cast<uint32_t*>(workspace);
    a.vec_ok = (reinterpret_cast<uintptr_t>(y) % 16 == 0 && reinterpret_cast<uintptr_t>(wscale) % 16 == 0 &&
                (!bias || reinterpret_cast<uintptr_t>(bias) % 16 == 0) && y_row_stride % 4 == 0)
                   ? 1
                   : 0;

    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return TDQ_ERR_CUDA;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TDQ_ERR_CUDA;
    }
    const size_t smem = sizeof(Smem) + 128;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(w4a4_linear_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess ||
            cudaFuncSetAttribute(w4a4_linear_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess)
            return TDQ_ERR_CUDA;
        attr_set = true;
    }
    if (cudaMemsetAsync(workspace, 0, 16, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    const int64_t tiles = tm * tn;
    const unsigned grid = (unsigned)(tiles < n_sm ? tiles : n_sm);
    if (y_dtype == TDQ_BF16)
        w4a4_linear_kernel<true><<<grid, kThreads, smem, stream>>>(a);
    else
        w4a4_linear_kernel<false><<<grid, kThreads, smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

extern "C" tdq_status tdq_workspace_status(const void* workspace, void* cuda_stream, uint32_t* detail) {
    if (!workspace) return TDQ_ERR_INVALID_ARG;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TDQ_ERR_CUDA;
    if (detail) *detail = word;
    return word == 0 ? TDQ_OK : TDQ_ERR_DEVICE_TIMEOUT;
}
