// Shared pieces of the W4A4 linear layer's kernels: tile constants, the argument block, mbarrier /
// bulk-copy / tcgen05 wrappers (inline PTX), the nibble-to-operand-byte expansion, the tensor map
// of y and the shared-memory plan.  Included by tdq_linear.cu (all group widths, the fused and the
// power-of-two variants) and tdq_linear_g32.cu (the g = 32 kernel).
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cstring>
#include <type_traits>

#include "tdq_common.cuh"

namespace tdq {

constexpr int kBM = 128;                 // rows per tile = TMEM lanes
constexpr int kBN = 128;                 // columns per tile = one TMEM slot
constexpr int kSlots = 4;                // TMEM accumulator ring (4 x 128 = 512 columns)
constexpr int kChunk = 4;                // K-steps (of 32 codes) per ring stage
constexpr int kBlock = 128 * 32;         // operand bytes of one 128-row block and one K-step
constexpr int kScaleBlock = 128 * 4;     // the scales of one 128-row block and one group
constexpr int kMaxStages = 8;
constexpr int kProdWarps = 2;
constexpr int kMmaWarp = 2;
constexpr int kPromoWarp0 = 4;
constexpr int kPromoWarps = 16;
constexpr int kCols = kBN / (kPromoWarps / 4);   // 32 columns of one row per promotion thread
constexpr int kThreads = (kPromoWarp0 + kPromoWarps) * 32;   // 640
constexpr int kStripBytes = kCols * 4;   // one thread's 32 raw fp32 sums
constexpr int kStagingBytes = kPromoWarps * 32 * kStripBytes;
constexpr int kWsbBytes = kPromoWarps * 256;   // per warp: 32 output-channel scales and 32 biases
constexpr int kCtrlBytes = 384;
constexpr int kMaxItemBufs = 4;          // copies of a work item's scales and resident A block in flight
constexpr int kSmemLimit = 232448;       // 227 KB per CTA
constexpr uint32_t kTmemCols = kSlots * kBN;
constexpr long long kTimeoutCycles = 2000000000LL;
constexpr uint32_t kSuspendHintNs = 20000;   // longest sleep of one try_wait
constexpr int kExpandThreads = 512;
constexpr int kRegsControl = 40, kRegsPromo = 104;   // 128 * 40 + 512 * 104 <= 640 * 96

// instruction descriptors: M = 128, N = 128, both operands K-major
constexpr uint32_t kIdescShape = ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
constexpr uint32_t kIdescI8 = (2u << 4) | (1u << 7) | (1u << 10) | kIdescShape;   // S32 += S8 * S8
constexpr uint32_t kIdescF8 = (1u << 4) | (0u << 7) | (0u << 10) | kIdescShape;   // F32 += E4M3 * E4M3

struct LinArgs {
    const uint8_t* a_blocks;   // [tiles_m][n_steps] operand blocks
    const uint8_t* b_blocks;   // [tiles_n][n_steps] operand blocks
    const uint8_t* s_blocks;   // [tiles_m][Kg] scale blocks
    const float* wscale;
    const float* bias;
    int64_t M, O;
    int32_t n_steps;           // I_pad / 32
    int32_t steps_per_grp;     // g / 32
    int32_t Kg;                // groups per token
    int32_t tiles_m, tiles_n, n_parts;
    int32_t a_resident;        // the item's whole A block stays in shared memory
    int32_t n_stages;
    uint32_t ring_off, stage_bytes, staging_off;   // shared-memory carve-up
    uint32_t staging_bytes;    // all sixteen strips: 64 KB, 32 KB when a strip holds 32 rows of 64 bytes, 16 KB with rows of 32 bytes
    int32_t half_strips;       // 1: fp32 output written in two passes of 16 columns through 64-byte strip rows; 2: any output in
                               // passes through 32-byte strip rows
    uint32_t ibuf_bytes;       // one item buffer: the item's scales, then its A blocks if resident
    int32_t n_ibuf;            // item buffers (1..kMaxItemBufs): the producer runs that many items ahead
    void* y;
    int64_t y_stride;
    int32_t* acc_debug;
    uint32_t* status;
    int32_t tma_ok;            // y can be written with bulk tensor stores (16-byte aligned base and row pitch)
    float out_scale;           // 2^18 (E4M3 route) or 2^-8 (int8 route)
    int32_t y_f16;             // 16-bit output is fp16 (else bf16); the kernels' 16-bit instances serve both
    // resident A without the fused producer: the promotion warps unpack the item's codes themselves
    const uint8_t* xcodes;
    const float* xscale;
    int32_t row_bytes;         // I_pad / 2
    int32_t unpack_a;
    int32_t pair_groups;       // groups of a multiple of four steps: 1 = two or more per tile, the two MMA warps take them in turn;
                               // 2 = one per tile, the warps take its chunks in turn into two accumulators
    // fused producer only: the activations themselves and the quantizer's parameters
    const void* x;
    int64_t x_stride;          // elements between rows of x
    float seven_tau;
    uint32_t act_flags;
};

struct Ctrl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t tfull[kSlots], tempty[kSlots];
    uint64_t a_full[kMaxItemBufs], a_empty[kMaxItemBufs];
    uint64_t sfull, sfree;     // g = 32 kernel: the staged output tile is complete / has been read by the copy engine
    uint32_t tmem_base;
    volatile int abort_flag;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block outgrew its reservation");

struct Plan {
    int64_t tiles_m, tiles_n;
    int32_t n_steps, n_chunks, Kg, n_parts, a_resident, n_stages;
    uint32_t ring_off, stage_bytes, staging_off, smem_bytes, ibuf_bytes;
    int32_t n_ibuf;
    size_t a_bytes, b_bytes, s_bytes;   // operand and scale blocks in the workspace
};

// The g = 32 kernel (tdq_linear_g32.cu); the caller has run the operand expansion and built the plan and the map.
tdq_status launch_linear_g32(const LinArgs& a, const CUtensorMap& ymap, uint32_t smem_bytes, unsigned grid, bool ybf,
                             bool dbg, cudaStream_t stream);

namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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

__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;   // the thread is suspended until the phase completes or the time hint (in ns) has passed: no busy polling
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}

// Slow path of a bounded wait: sleeps on the barrier until the phase completes, another role of
// this CTA has given up, or about a second has passed; then it records which wait gave up
// (first writer wins) and raises the CTA-wide flag.
__device__ __forceinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, Ctrl* c, uint32_t* status, uint32_t code,
                                               long long limit = kTimeoutCycles) {
    long long t0 = 0;
#pragma unroll 1
    for (;;) {
        // a burst of sleeping waits between two looks at the abort flag and the clock: waiting warps
        // share their scheduler with working ones, so the waiting loop is kept to a few instructions
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try(bar, parity)) return true;
        if (c->abort_flag) return false;
        const long long now = clock64();
        if (t0 == 0) t0 = now;
        if (now - t0 > limit) {
            atomicCAS(status, 0u, code | ((uint32_t)blockIdx.x << 8));
            c->abort_flag = 1;
            return false;
        }
    }
}

// Bounded wait by a converged warp; the answer is the same in every lane.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, Ctrl* c, uint32_t* status, uint32_t code,
                                               long long limit = kTimeoutCycles) {
    if (__all_sync(0xffffffffu, mbar_test(bar, parity))) return true;
    return __all_sync(0xffffffffu, mbar_wait_slow(bar, parity, c, status, code, limit));
}

// The same primitives on 32-bit shared-window addresses, for the hot loops (no pointer conversion).
__device__ __forceinline__ bool mbar_test_s(uint32_t bar_s, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_s), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void mbar_arrive_lane0_s(uint32_t bar_s, int lane) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.s32 p, %1, 0;\n\t"
        "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
        ::"r"(bar_s), "r"(lane)
        : "memory");
}

// lane 0 of a converged warp arrives; predicated, so the warp does not diverge
__device__ __forceinline__ void mbar_arrive_lane0(uint64_t* bar, int lane) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.s32 p, %1, 0;\n\t"
        "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
        ::"r"(smem_u32(bar)), "r"(lane)
        : "memory");
}

// global -> shared bulk copy that reports its bytes to an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// K-major, no swizzle: 8 rows x 16 bytes are one contiguous 128-byte core matrix; the two
// K-halves of an 8-row band are 128 bytes apart (leading byte offset) and bands are 256 bytes
// apart (stride byte offset).  Offsets are stored >> 4; bit 46 is the descriptor version.
// The start address sits in the low 14 bits, so adding (bytes >> 4) moves the descriptor.
// MMA issue and commit for a converged warp: every lane executes them and the predicate lets
// one through (`on` is non-zero in lane 0 only, and only if the step is to be issued), so there
// is no branch.  Descriptors are passed as their low words; the high word is constant.
constexpr uint32_t kDescHi = (256u >> 4) | (1u << 14);   // stride byte offset 256, descriptor version 1
template <bool I8>
__device__ __forceinline__ void mma_issue_if(uint32_t on, uint32_t d_tmem, uint32_t adesc_lo, uint32_t bdesc_lo,
                                             uint32_t accumulate) {
    if (I8)
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
            "mov.b64 da, {%1, %6};\n\tmov.b64 db, {%2, %6};\n\t"
            "@q tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(kIdescI8), "r"(accumulate), "r"(on), "r"(kDescHi)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\t"
            "mov.b64 da, {%1, %6};\n\tmov.b64 db, {%2, %6};\n\t"
            "@q tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(kIdescF8), "r"(accumulate), "r"(on), "r"(kDescHi)
            : "memory");
}
// Four instructions on consecutive K-steps of the same accumulator (operand blocks 4096 bytes apart): the
// predicates and the descriptors are built once, the descriptors move by an add.
template <bool I8>
__device__ __forceinline__ void mma_issue4_if(uint32_t on, uint32_t d_tmem, uint32_t adesc_lo, uint32_t bdesc_lo,
                                              uint32_t accumulate_first) {
#define TDQ_MMA4(KIND, IDESC)                                                                       \
    asm volatile(                                                                                   \
        "{\n\t.reg .pred p, q, t;\n\t.reg .b64 da, db;\n\t"                                        \
        "setp.ne.b32 p, %4, 0;\n\tsetp.ne.b32 q, %5, 0;\n\tsetp.eq.b32 t, 0, 0;\n\t"                 \
        "mov.b64 da, {%1, %6};\n\tmov.b64 db, {%2, %6};\n\t"                                        \
        "@q tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, p;\n\t"                        \
        "add.s64 da, da, 256;\n\tadd.s64 db, db, 256;\n\t"                                          \
        "@q tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, t;\n\t"                        \
        "add.s64 da, da, 256;\n\tadd.s64 db, db, 256;\n\t"                                          \
        "@q tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, t;\n\t"                        \
        "add.s64 da, da, 256;\n\tadd.s64 db, db, 256;\n\t"                                          \
        "@q tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, t;\n\t}"                       \
        ::"r"(d_tmem), "r"(adesc_lo), "r"(bdesc_lo), "r"(IDESC), "r"(accumulate_first), "r"(on), "r"(kDescHi) \
        : "memory")
    if (I8) TDQ_MMA4("i8", kIdescI8);
    else TDQ_MMA4("f8f6f4", kIdescF8);
#undef TDQ_MMA4
}
__device__ __forceinline__ void mma_commit_if(uint32_t on, uint32_t bar_s) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar_s), "r"(on)
        : "memory");
}
// low word of the operand descriptor of a block at shared address saddr (leading byte offset 128)
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | ((128u >> 4) << 16); }

// 32 consecutive columns of this warp's 32 TMEM lanes: lane i receives row i, v[j] = column j.
// The operands are declared read-write so that a landing buffer keeps its registers for the
// whole kernel (pure outputs would be renamed at every load and copied at every loop edge).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
          "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
          "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
          "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
        : "r"(taddr)
        : "memory");
}

// the same for 16 columns
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
          "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
// acc = v * d + acc on two packed floats
__device__ __forceinline__ void fma2(uint64_t& acc, uint64_t v, uint64_t d) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(v), "l"(d));
}

// two floats -> one word of two bf16 or two fp16 (round to nearest even), low half first
__device__ __forceinline__ uint32_t pack16(float lo, float hi, int f16) {
    if (f16) {
        __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&h);
    }
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&b);
}

// shared memory by 32-bit shared-window address
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// shared -> global bulk tensor store of one box (coordinates: column, row), tracked by bulk groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src_smem, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src_smem), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
    return v;
}

template <int N>
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// ------------------------------------------------------------------------------------------
// kernel 1: nibbles -> operand bytes in core-matrix order, scales regrouped by row block

// four two's complement bytes 16 q -> four sign-magnitude bytes (q < 0) << 7 | |q|
__device__ __forceinline__ uint32_t to_sign_magnitude(uint32_t b16) {
    uint32_t neg;   // 0xFF where the byte is negative: prmt with the selector's replicate-sign bit set
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(neg) : "r"(b16), "r"(0u), "r"(0xBA98u));
    const uint32_t abs16 = (b16 ^ neg) + (neg & 0x01010101u);             // 16 |q| per byte, no carry leaves a byte
    return (abs16 >> 4) | (neg & 0x80808080u);
}

// 8 packed codes (even channel in the low nibble) -> 8 operand bytes in channel order
template <bool I8>
__device__ __forceinline__ void expand8(uint32_t p, uint32_t& lo, uint32_t& hi) {
    uint32_t ev = (p << 4) & 0xF0F0F0F0u;   // channels 0,2,4,6 as bytes 16 q
    uint32_t od = p & 0xF0F0F0F0u;          // channels 1,3,5,7
    if (!I8) {
        ev = to_sign_magnitude(ev);
        od = to_sign_magnitude(od);
    }
    lo = __byte_perm(ev, od, 0x5140u);
    hi = __byte_perm(ev, od, 0x7362u);
}

// Test-only dump of 32 integer group sums of one output row (the debug instantiation of the kernel).
template <bool I8>
__device__ __noinline__ void debug_store(const LinArgs& a, const uint32_t* v, int64_t m, int64_t n0, int grp) {
#pragma unroll 1
    for (int q = 0; q < 32; ++q)
        if (n0 + q < a.O)
            a.acc_debug[(m * a.O + n0 + q) * a.Kg + grp] =
                I8 ? ((int32_t)v[q] >> 8) : __float2int_rn(__uint_as_float(v[q]) * 262144.0f);
}

// Descriptor of y for the epilogue's bulk tensor stores: a [M][O] matrix with a row pitch, written in
// boxes of 32 (or box_rows) rows x 32 columns whose 16-byte chunks are swizzled in shared memory the way the
// kernel lays them out (128-byte rows: chunk ^ (row & 7); 64-byte rows: chunk ^ ((row >> 1) & 3)).
// The driver's encoder is looked up once; false when it is not there or refuses the shape.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool encode_y_map(CUtensorMap* map, void* y, bool bf16, int64_t M, int64_t O, int64_t y_row_stride, int box_cols,
                  int box_rows = 32, bool f16 = false) {
    static const TensorMapEncodeFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<TensorMapEncodeFn>(fn);
    }();
    if (!encode) return false;
    const cuuint64_t esz = bf16 ? 2 : 4;
    const cuuint64_t dims[2] = {(cuuint64_t)O, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)y_row_stride * esz};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const size_t row_bytes = (size_t)box_cols * esz;    // strip rows of 128, 64 or 32 bytes, swizzled alike
    const cuuint32_t elem_strides[2] = {1u, 1u};
    return encode(map, bf16 ? (f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, y, dims, strides, box,
                  elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


constexpr size_t kWorkspaceHeader = 256;   // status word, then the blocks

// false: sizes out of range, or the problem's scales plus two ring stages do not fit in shared memory
bool make_plan(int64_t M, int64_t I_pad, int64_t O, int32_t g, int n_sm, Plan& p, int64_t staging_bytes = kStagingBytes) {
    p.tiles_m = (M + kBM - 1) / kBM;
    p.tiles_n = (O + kBN - 1) / kBN;
    if (p.tiles_m > INT32_MAX / 4096 || p.tiles_n > INT32_MAX / 4096 || I_pad / 32 > INT32_MAX / 8) return false;
    p.n_steps = (int32_t)(I_pad / 32);
    p.n_chunks = (p.n_steps + kChunk - 1) / kChunk;
    p.Kg = (int32_t)(I_pad / g);
    p.a_bytes = (size_t)p.tiles_m * p.n_steps * kBlock;
    p.b_bytes = (size_t)p.tiles_n * p.n_steps * kBlock;
    p.s_bytes = (size_t)p.tiles_m * p.Kg * kScaleBlock;
    // shared memory: control, the item's scales, [resident A], ring, output strips, channel scales
    const int64_t scales = (int64_t)p.Kg * kScaleBlock;
    const int64_t fixed = 1024 + kCtrlBytes + scales + staging_bytes + kWsbBytes;   // 1024: the strips start on a 1 KB boundary
    const int64_t a_res = (int64_t)p.n_steps * kBlock;
    const int64_t stage_b = (int64_t)kChunk * kBlock, stage_ab = 2 * stage_b;
    const int64_t stages_res = (kSmemLimit - fixed - a_res) / stage_b;
    if (stages_res >= 3) {
        p.a_resident = 1;
        p.ibuf_bytes = (uint32_t)(scales + a_res);
        // further item buffers while enough stages remain for two tiles' worth of B (at most six, at least three):
        // with short contractions the hand-over between work items, not the ring, is what the tensor core waits for
        const int64_t want_stages = 2 * p.n_chunks < 3 ? 3 : (2 * p.n_chunks > 6 ? 6 : 2 * p.n_chunks);
        p.n_ibuf = 1;
        while (p.n_ibuf < kMaxItemBufs && (kSmemLimit - fixed - a_res - (int64_t)p.n_ibuf * p.ibuf_bytes) / stage_b >= want_stages) ++p.n_ibuf;
        const int64_t st = (kSmemLimit - fixed - a_res - (int64_t)(p.n_ibuf - 1) * p.ibuf_bytes) / stage_b;
        p.n_stages = (int32_t)(st > kMaxStages ? kMaxStages : st);
        p.stage_bytes = (uint32_t)stage_b;
    } else {
        const int64_t st = (kSmemLimit - fixed) / stage_ab;
        if (st < 2) return false;
        p.a_resident = 0;
        p.ibuf_bytes = (uint32_t)scales;
        p.n_ibuf = 1;
        p.n_stages = (int32_t)(st > kMaxStages ? kMaxStages : st);
        p.stage_bytes = (uint32_t)stage_ab;
    }
    p.ring_off = (uint32_t)kCtrlBytes + (uint32_t)p.n_ibuf * p.ibuf_bytes;
    p.staging_off = p.ring_off + (uint32_t)p.n_stages * p.stage_bytes;
    p.smem_bytes = p.staging_off + 1024 + (uint32_t)staging_bytes + kWsbBytes;
    // split the column tiles of a row block into parts so that the items fill the SMs evenly
    int best = 1;
    int64_t best_cost = INT64_MAX;
    for (int parts = 1; parts <= p.tiles_n; ++parts) {
        const int64_t items = p.tiles_m * parts;
        const int64_t waves = (items + n_sm - 1) / n_sm;
        const int64_t per_item = (p.tiles_n + parts - 1) / parts;
        const int64_t cost = waves * (per_item * 16 + 1);   // +1: an item reloads its A block
        if (cost < best_cost) { best_cost = cost; best = parts; }
    }
    p.n_parts = best;
    return true;
}

}  // namespace
}  // namespace tdq
