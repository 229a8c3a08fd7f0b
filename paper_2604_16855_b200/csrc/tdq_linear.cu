// tdq_w4a4_linear: W4A4 linear layer on the 5th-generation tensor cores (Algorithm S1 step 10).
//
//   acc[m,o,k] = sum_{i in group k} q_x[m,i] q_w[o,i]      tcgen05.mma, exact, accumulator in TMEM
//   y[m,o]     = s_o * sum_k Delta[m,k] * acc[m,o,k] + b_o  fp32 in registers
//
// The activation scale changes every g codes along the contraction axis, so one tensor-core
// accumulator may only span one token-group.  Each group gets a fresh TMEM slot (groups wider
// than 32 codes chain g/32 instructions into it), is read back with tcgen05.ld, multiplied by
// its Delta and added to a float accumulator that stays in registers for the whole
// contraction ("promotion").  At g = 32 the promotion, not the tensor pipe, sets the pace: one
// 128 x 128 x 32 instruction takes 64 clocks, while 16384 fp32 FMAs take 128 clocks of the SM's
// FMA pipes.  The operand encoding is chosen so that nothing else is added to that:
//
//   * g <= 128: kind::f8f6f4, E4M3 operands, fp32 accumulator.  A code q in [-8, 8] is stored as
//     the byte sign(q) << 7 | |q|, which E4M3 reads as q * 2^-9 (the values are subnormal, or
//     2^-6 for |q| = 8).  g / 32 instructions contract one group into a fresh slot; the products
//     (|p| <= 64) and their sum (<= 8192) are exact in the fp32 accumulator, so TMEM holds
//     acc * 2^-18 exactly and the promotion needs no integer-to-float conversion: one packed fp32
//     FMA per two values.  (Measured with adversarial codes: the accumulator stays exact up to the
//     largest sum 4096 codes can produce, 2^18; the limit of 128 is caution, not need.)
//   * g > 128: kind::i8, int32 accumulator (many instructions chain into one slot, so the
//     sum stays in integers; promotion is rarer).  A code is stored as the two's complement
//     byte 16 q; TMEM holds 256 acc.
//   The power of two is folded into the output-channel scale in the epilogue; both routes
//   give bit-identical integer sums and the same float sequence.
//
// Two kernels per call:
//   1. expand_kernel   rewrites the packed nibbles of both operands as operand bytes, in 128-row
//      x 32-code blocks laid out in the tensor core's K-major core-matrix order (8 rows x 16
//      bytes contiguous), and regroups the activation scales as [row block][group][128 rows].
//      The blocks live in the caller's workspace; a block is one contiguous piece, so the GEMM
//      moves operands with plain 1-D bulk copies (cp.async.bulk + mbarrier) and no tensor maps.
//   2. w4a4_gemm_kernel   persistent, one CTA per SM, 128 x 128 output tiles.  Warp roles:
//        warps 0-1   producers: one lane each issues the bulk copies of alternate ring stages
//        warps 2-3   MMA issue and the commits that release buffers.  Group k of a tile uses TMEM slot
//                    k & 3.  The issue loop is straight-line, predicated code (a lone warp runs
//                    dependent scalar code slowly, and branches cost most): at g = 32 the two warps take
//                    the even and the odd slots, at g = 64 the first and the second group of a stage.
//                    At g a multiple of 128 a ring stage belongs to one group: with two or more groups per
//                    tile the two warps take the groups in turn, with one group per tile (g = C) they take
//                    its stages in turn, each into an accumulator of its own that the promotion warps add
//                    (integer sums); either way each warp has its own half of the ring, fed by the
//                    producer warp of its parity.  Otherwise warp 2 issues alone.
//        warps 4-19  promotion + epilogue: warp w owns TMEM lanes 32 (w % 4).. (its rows) and 32
//                    columns; a thread keeps 32 float accumulators of one output row and one
//                    32-value landing buffer.  Sixteen warps, four per scheduler: a warp executes
//                    dependent instructions only every few clocks, so the TMEM load and the
//                    barrier traffic of one warp hide behind the FMAs of the other three.  The loop
//                    is unrolled over the four slots, so slot, barrier and TMEM addresses are constants.
//      A work item is one 128-row block of A with a range of column tiles.  The item's scales,
//      and its A block when the whole K extent fits, are loaded once per item; B (and A
//      otherwise) streams through a ring of stages of 4 K-steps.  TMEM holds four 128-column
//      accumulator slots, each with a full/empty mbarrier pair.
//      In the epilogue a warp needs no other warp: every thread scales its 32 sums and parks them in
//      the warp's own 4 KB strip of shared memory, laid out (and swizzled) as the source box of a
//      bulk tensor store; lane 0 starts one 32 x 32 store per tile, a few groups into the next
//      tile, and the copy engine clips it at the edges of y.  Unaligned y is written element by
//      element from the same strip.
//      Where the ring needs the shared memory more (wide groups), the strips have rows of 64 or 32 bytes
//      and a tile is written in two or four passes.
//   The fused instantiation (tdq_quant_linear_fused) replaces the load of an item's A block and
//   scales: the promotion warps quantize the item's 128 activation rows into the same shared-memory
//   regions before they start on its tiles.
//
// Every wait on an mbarrier is bounded: after about a second the thread records a code in the
// workspace status word and raises a CTA-wide flag; every role then leaves its loops, the CTA
// releases its TMEM and returns.
#include <cuda_fp8.h>

#include <mutex>

#include "tdq_act_group.cuh"
#include "tdq_tc.cuh"

namespace tdq {
namespace {

struct ExpandArgs {
    const uint8_t* xcodes;
    const float* xscale;
    const uint8_t* wcodes;
    uint8_t* a_blocks;
    uint8_t* b_blocks;
    uint8_t* s_blocks;
    int64_t M, O;
    int32_t row_bytes;       // I_pad / 2
    int32_t n_steps, n_chunks, steps_per_grp, Kg;
    int32_t tiles_m, tiles_n;
    uint32_t* status;        // the workspace's status words, cleared here for the GEMM that follows
};

// Waits for this thread's outstanding TMEM loads; the 16 landing registers pass through as operands, so that no
// use of them can be scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait_on16(uint32_t* v) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :
                 : "memory");
}

// One CTA rewrites one (128-row block, 4 K-steps) piece: thread t takes row t / 4 and K-step t % 4.
template <bool I8>
__global__ void __launch_bounds__(kExpandThreads) expand_kernel(ExpandArgs a) {
    pdl_trigger();                                         // the GEMM may set itself up meanwhile
    const int piece = blockIdx.x;
    if (piece == 0 && threadIdx.x < 4) a.status[threadIdx.x] = 0u;   // saves a separate memset in front of every call
    const int blk = piece / a.n_chunks, kc = piece % a.n_chunks;
    const int r = threadIdx.x >> 2;
    const int ks = kc * kChunk + (threadIdx.x & 3);
    if (ks >= a.n_steps) return;
    const bool is_a = blk < a.tiles_m;
    const int tile = is_a ? blk : blk - a.tiles_m;
    const int64_t row = (int64_t)tile * 128 + r;
    const int64_t rows = is_a ? a.M : a.O;
    const uint8_t* src = is_a ? a.xcodes : a.wcodes;
    uint4 p = make_uint4(0, 0, 0, 0);
    if (row < rows) p = __ldg(reinterpret_cast<const uint4*>(src + row * a.row_bytes + (int64_t)ks * 16));
    uint4 c0, c1;
    expand8<I8>(p.x, c0.x, c0.y);
    expand8<I8>(p.y, c0.z, c0.w);
    expand8<I8>(p.z, c1.x, c1.y);
    expand8<I8>(p.w, c1.z, c1.w);
    uint8_t* dst = (is_a ? a.a_blocks : a.b_blocks) + ((int64_t)tile * a.n_steps + ks) * kBlock;
    const int off = (r >> 3) * 256 + (r & 7) * 16;
    *reinterpret_cast<uint4*>(dst + off) = c0;
    *reinterpret_cast<uint4*>(dst + off + 128) = c1;
    if (is_a && ks % a.steps_per_grp == 0) {
        const int grp = ks / a.steps_per_grp;
        float s = 0.0f;
        if (row < rows) s = __ldg(a.xscale + row * a.Kg + grp);
        reinterpret_cast<float*>(a.s_blocks + ((int64_t)tile * a.Kg + grp) * kScaleBlock)[r] = s;
    }
}

// Power-of-two steps (tdq_w4a4_linear_pow2): the group scale goes into the operand.  With every step of a
// row a power of two, Delta[m,k] = 2^(e_m + s), a code is stored as the E4M3 value q * 2^(s - 9), where
// e_m is the row's largest step exponent minus 14, so s runs over 0..14: |q| <= 8 has at most three
// significant bits and E4M3 four, and q * 2^(s-9) lies between 2^-9 (the smallest subnormal) and 256, so
// the byte is exact.  Steps more than 2^14 below the row's largest have s < 0 and lose their low bits
// (truncated).  The whole contraction then accumulates in one fp32 accumulator and the row needs one
// scale, 2^e_m, in the epilogue.
// Four codes (the nibbles of h, lowest first) as four such bytes.  shr = max(-s, 0) low bits of |q| are dropped first;
// mul = 2^(max(s, 0) - 9).  q * mul is exact in binary32 and in E4M3, so the hardware conversion is exact too.
__device__ __forceinline__ uint32_t pow2_bytes4(uint32_t h, int shr, float mul) {
    int q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        q[i] = ((int)(h << (28 - 4 * i))) >> 28;           // sign-extended nibble
        if (shr) q[i] = q[i] >= 0 ? (q[i] >> shr) : -((-q[i]) >> shr);   // toward zero
    }
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2((float)q[0] * mul, (float)q[1] * mul), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2((float)q[2] * mul, (float)q[3] * mul), __NV_SATFINITE, __NV_E4M3);
    return lo | (hi << 16);
}

// Eight codes (the nibbles of p, lowest first) through a 16-entry byte table held in four registers (entry n
// is the byte of the code whose two's-complement nibble is n): one byte permute per four codes and table half,
// and a select on the nibble's top bit.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void table_bytes8(uint32_t p, const uint4& tab, uint32_t& lo, uint32_t& hi) {
    const uint32_t sel = p & 0x77777777u;                  // selectors 0..7; only the low 16 bits of a selector count
    const uint32_t ev = (p << 4) & 0x80808080u;            // top bits of nibbles 0, 2, 4, 6 as byte signs
    const uint32_t od = p & 0x80808080u;                   // of nibbles 1, 3, 5, 7
    const uint32_t m_lo = prmt(ev, od, 0xd9c8u);           // sign-replicating selectors: 0xff where the nibble is >= 8
    const uint32_t m_hi = prmt(ev, od, 0xfbeau);
    const uint32_t a_lo = prmt(tab.x, tab.y, sel), b_lo = prmt(tab.z, tab.w, sel);
    const uint32_t a_hi = prmt(tab.x, tab.y, sel >> 16), b_hi = prmt(tab.z, tab.w, sel >> 16);
    lo = (a_lo & ~m_lo) | (b_lo & m_lo);
    hi = (a_hi & ~m_hi) | (b_hi & m_hi);
}

constexpr int kPow2MinShift = -4;                          // |q| <= 8: four or more dropped bits leave nothing
constexpr int kPow2Tables = 14 - kPow2MinShift + 1;        // one table per s in -4..14
constexpr int kPow2Chunks = 2;                             // chunks of K-steps per CTA of the expansion

// A step that is not a positive power of two is reported as the status word 11 | epoch << 8, stored by
// whichever thread meets one.  The epoch is the workspace's third status word: the GEMM kernel of every call
// adds one to it, after this kernel has finished, so it is fixed while this kernel runs and differs from the
// epoch of the call before (also when the calls are replays of one captured graph).  The CTA that clears the
// status word for this call leaves exactly the value 11 | epoch << 8 alone, so the order of the clear and the
// reports does not matter, and a report left by an earlier call is cleared like any other stale word.
__global__ void __launch_bounds__(kExpandThreads) expand_pow2_kernel(ExpandArgs a, int32_t act_steps_per_grp, int32_t act_Kg) {
    __shared__ __align__(16) uint8_t s_tab[kPow2Tables][16];
    static_assert(kPow2Tables * 16 <= kExpandThreads, "one thread per table byte");
    if (threadIdx.x < kPow2Tables * 16) {
        const int s = (int)(threadIdx.x >> 4) + kPow2MinShift;
        const float mul = __uint_as_float((uint32_t)((s > 0 ? s : 0) - 9 + 127) << 23);
        s_tab[threadIdx.x >> 4][threadIdx.x & 15] = (uint8_t)pow2_bytes4(threadIdx.x & 15u, s < 0 ? -s : 0, mul);
    }
    __syncthreads();
    pdl_trigger();                                         // the GEMM may set itself up meanwhile
    if (blockIdx.x == 0 && threadIdx.x < 4) {
        if (threadIdx.x == 0) {
            const uint32_t keep = 11u | (*reinterpret_cast<volatile uint32_t*>(a.status + 2) << 8);
            const uint32_t old = *reinterpret_cast<volatile uint32_t*>(a.status);
            if (old != keep) atomicCAS(a.status, old, 0u);   // fails only if a report of this call came in between
        } else if (threadIdx.x != 2) {
            a.status[threadIdx.x] = 0u;
        }
    }
    // one CTA takes a 128-row block and kPow2Chunks chunks of K-steps: thread t takes row t / 4 and, in every
    // chunk, K-step t % 4, with all its loads issued before the first use
    const int piece = blockIdx.x;
    const int n_cp = (a.n_chunks + kPow2Chunks - 1) / kPow2Chunks;
    const int blk = piece / n_cp, kc0 = (piece % n_cp) * kPow2Chunks;
    const int r = threadIdx.x >> 2;
    const bool is_a = blk < a.tiles_m;
    const int tile = is_a ? blk : blk - a.tiles_m;
    const int64_t row = (int64_t)tile * 128 + r;
    const int64_t rows = is_a ? a.M : a.O;
    const uint8_t* src = is_a ? a.xcodes : a.wcodes;
    int ks[kPow2Chunks];
    uint4 p[kPow2Chunks];
#pragma unroll
    for (int j = 0; j < kPow2Chunks; ++j) {
        ks[j] = (kc0 + j) * kChunk + (threadIdx.x & 3);
        p[j] = make_uint4(0, 0, 0, 0);
        if (row < rows && ks[j] < a.n_steps) p[j] = __ldg(reinterpret_cast<const uint4*>(src + row * a.row_bytes + (int64_t)ks[j] * 16));
    }
    int e_m = 0;
    const float* sc = a.xscale + row * act_Kg;
    if (is_a && row < rows) {
        uint32_t emax = 0u, bad = 0u;
        int k = 0;
        if ((act_Kg & 3) == 0 && (reinterpret_cast<uintptr_t>(sc) & 15) == 0) {   // four steps per load
#pragma unroll 2
            for (; k < act_Kg; k += 4) {
                const uint4 b4 = __ldg(reinterpret_cast<const uint4*>(sc + k));
                emax = max(max(emax, b4.x >> 23), max(max(b4.y >> 23, b4.z >> 23), b4.w >> 23));
                bad |= (b4.x | b4.y | b4.z | b4.w) & 0x807fffffu;
            }
        }
        for (; k < act_Kg; ++k) {
            const uint32_t bits = __float_as_uint(__ldg(sc + k));
            emax = max(emax, bits >> 23);
            bad |= bits & 0x807fffffu;                     // a mantissa or a sign: not a power of two
        }
        if (bad) atomicExch(a.status, 11u | (*reinterpret_cast<volatile uint32_t*>(a.status + 2) << 8));   // see above
        e_m = (int)emax - 14;
    }
#pragma unroll
    for (int j = 0; j < kPow2Chunks; ++j) {
        if (ks[j] >= a.n_steps) break;
        uint4 c0, c1;
        if (!is_a) {
            expand8<false>(p[j].x, c0.x, c0.y);
            expand8<false>(p[j].y, c0.z, c0.w);
            expand8<false>(p[j].z, c1.x, c1.y);
            expand8<false>(p[j].w, c1.z, c1.w);
        } else {
            int s = 0;
            if (row < rows) s = (int)(__float_as_uint(__ldg(sc + ks[j] / act_steps_per_grp)) >> 23) - e_m;
            // s <= 14 by the choice of e_m (a step with its sign bit set is reported above; its bytes are not used)
            const int ti = min(max(s, kPow2MinShift), 14) - kPow2MinShift;
            const uint4 tab = *reinterpret_cast<const uint4*>(s_tab[ti]);
            table_bytes8(p[j].x, tab, c0.x, c0.y);
            table_bytes8(p[j].y, tab, c0.z, c0.w);
            table_bytes8(p[j].z, tab, c1.x, c1.y);
            table_bytes8(p[j].w, tab, c1.z, c1.w);
            if (ks[j] == 0)                                // bits of 2^e_m, the row's one scale
                reinterpret_cast<uint32_t*>(a.s_blocks + (int64_t)tile * kScaleBlock)[r] = row < rows && e_m > 0 ? (uint32_t)e_m << 23 : 0u;
        }
        uint8_t* dst = (is_a ? a.a_blocks : a.b_blocks) + ((int64_t)tile * a.n_steps + ks[j]) * kBlock;
        const int off = (r >> 3) * 256 + (r & 7) * 16;
        *reinterpret_cast<uint4*>(dst + off) = c0;
        *reinterpret_cast<uint4*>(dst + off + 128) = c1;
    }
}

// ------------------------------------------------------------------------------------------
// kernel 2: the GEMM


// FUSED: 0 the A operand comes as blocks from the workspace; 1 / 2: the promotion warps quantize the
// work item's 128 rows of bf16 / fp32 activations themselves and write operand bytes and scales
// straight into shared memory (A must be resident), so codes and scales never reach global memory.
template <bool I8, bool YBF16, bool DBG, int FUSED = 0>
__global__ void __launch_bounds__(kThreads, 1) w4a4_gemm_kernel(const LinArgs a, const __grid_constant__ CUtensorMap ymap) {
    extern __shared__ __align__(128) uint8_t smem_raw[];   // no static shared memory: the window starts aligned
    Ctrl* c = reinterpret_cast<Ctrl*>(smem_raw);
    const uint32_t sm_s = smem_u32(smem_raw);
    // item buffer b: [Kg][128] floats of the item's scales, then its [n_steps] operand blocks if resident.
    // Item number ic of this CTA uses buffer ic % n_ibuf; (ib, iu) below are that index and the parity of
    // ic / n_ibuf, which is the phase of the buffer's two barriers.
    const uint32_t ibuf_s = sm_s + kCtrlBytes;
    const uint32_t a_in_ibuf = (uint32_t)a.Kg * kScaleBlock;
    const uint32_t ring_s = sm_s + a.ring_off;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const bool resident = a.a_resident != 0;

    if (t == 0) {
        // MMA-issuing warps: two that share every ring stage (groups of one or two steps), two that take whole
        // groups in turn (a.pair_groups), else one
        const uint32_t n_issuers = (a.steps_per_grp <= 2 || a.pair_groups) ? 2u : 1u;
        const uint32_t per_stage = a.steps_per_grp <= 2 ? 2u : 1u;   // of them, how many read one stage
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&c->full[i], 1); mbar_init(&c->empty[i], per_stage); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(&c->tfull[i], 1); mbar_init(&c->tempty[i], kPromoWarps); }
        for (int i = 0; i < kMaxItemBufs; ++i) {
            mbar_init(&c->a_full[i], (FUSED || a.unpack_a) ? kPromoWarps : 1);
            mbar_init(&c->a_empty[i], n_issuers + kPromoWarps);
        }
        c->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();          // barrier set-up and the TMEM allocation overlap the tail of the kernel before this one
    pdl_trigger();
    if (blockIdx.x == 0 && t == 0) atomicAdd(a.status + 2, 1u);   // the call's epoch (see expand_pow2_kernel)
    const uint32_t tmem_base = c->tmem_base;

    const int n_items = a.tiles_m * a.n_parts;
    const int n_chunks = (a.n_steps + kChunk - 1) / kChunk;
    const int spg = a.steps_per_grp;
    auto part_begin = [&](int part) { return (int)(((int64_t)part * a.tiles_n) / a.n_parts); };

    if (warp < kPromoWarp0) {
        setmaxnreg_dec<kRegsControl>();
        // The control roles run with the whole warp converged and let lane 0 issue: a lone lane whose
        // warp-mates sit at the final barrier was measured to execute several times slower.
        if (warp < kProdWarps) {
            // ------------------------------------------------------------ producers (lane 0 issues)
            uint32_t sc = 0, s = 0, ph = 0;   // stage counter, its ring slot and phase
            uint32_t ps = 0, pph = 0;         // paired groups: position and phase in this warp's half of the ring
            const uint32_t n_mine = ((uint32_t)a.n_stages + 1 - (uint32_t)warp) / 2;
            uint32_t ib = 0, iu = 0;          // item buffer and its phase
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int mt = item / a.n_parts, part = item % a.n_parts;
                const uint8_t* a_src = a.a_blocks + (int64_t)mt * a.n_steps * kBlock;
                if (warp == 0 && !FUSED && !a.unpack_a) {
                    ok = mbar_wait_warp(&c->a_empty[ib], iu ^ 1, c, a.status, 1u);
                    if (!ok) break;
                    if (lane == 0) {
                    const uint32_t sbytes = (uint32_t)a.Kg * kScaleBlock;
                    const uint32_t scales_s = ibuf_s + ib * a.ibuf_bytes, ares_s = scales_s + a_in_ibuf;
                    mbar_expect_tx(&c->a_full[ib], sbytes + (resident ? (uint32_t)a.n_steps * kBlock : 0u));
                    const uint8_t* s_src = a.s_blocks + (int64_t)mt * a.Kg * kScaleBlock;
                    for (uint32_t off = 0; off < sbytes; off += 16384u)
                        bulk_load(scales_s + off, s_src + off, min(16384u, sbytes - off), &c->a_full[ib]);
                    if (resident)
                        for (int kc = 0; kc < n_chunks; ++kc) {
                            const int nk = min(kChunk, a.n_steps - kc * kChunk);
                            bulk_load(ares_s + kc * kChunk * kBlock, a_src + (int64_t)kc * kChunk * kBlock,
                                      (uint32_t)nk * kBlock, &c->a_full[ib]);
                        }
                    }
                    __syncwarp();
                }
                if (++ib == (uint32_t)a.n_ibuf) { ib = 0; iu ^= 1; }
                for (int nt = part_begin(part); nt < part_begin(part + 1) && ok; ++nt) {
                    const uint8_t* b_src = a.b_blocks + (int64_t)nt * a.n_steps * kBlock;
                    if (!FUSED && a.pair_groups) {   // (not compiled into the fused kernels, which never take these modes)
                        // two rings: this warp feeds the MMA warp of its parity through the stages of its parity, with
                        // the chunks of that warp's groups (group = steps_per_grp / 4 consecutive chunks of a tile)
                        // (pair_groups == 2: one group per tile, its chunks go to the two warps in turn)
                        const int cpg = a.pair_groups == 2 ? 1 : a.steps_per_grp / kChunk;
                        for (int kc0 = warp * cpg; kc0 < n_chunks && ok; kc0 += 2 * cpg) {
                            for (int kc = kc0; kc < kc0 + cpg; ++kc) {
                                const uint32_t st = 2 * ps + (uint32_t)warp;
                                ok = mbar_wait_warp(&c->empty[st], pph ^ 1, c, a.status, 5u);
                                if (!ok) break;
                                if (lane == 0) {
                                    const uint32_t stage = ring_s + st * a.stage_bytes;
                                    mbar_expect_tx(&c->full[st], (uint32_t)kChunk * kBlock * (resident ? 1u : 2u));
                                    bulk_load(stage, b_src + (int64_t)kc * kChunk * kBlock, (uint32_t)kChunk * kBlock, &c->full[st]);
                                    if (!resident)
                                        bulk_load(stage + kChunk * kBlock, a_src + (int64_t)kc * kChunk * kBlock,
                                                  (uint32_t)kChunk * kBlock, &c->full[st]);
                                }
                                __syncwarp();
                                if (++ps == n_mine) { ps = 0; pph ^= 1; }
                            }
                        }
                        continue;
                    }
                    for (int kc = 0; kc < n_chunks; ++kc, ++sc) {
                        if ((int)(sc & 1u) == warp) {
                            ok = mbar_wait_warp(&c->empty[s], ph ^ 1, c, a.status, 5u);
                            if (!ok) break;
                            if (lane == 0) {
                            const int nk = min(kChunk, a.n_steps - kc * kChunk);
                            const uint32_t stage = ring_s + s * a.stage_bytes;
                            mbar_expect_tx(&c->full[s], (uint32_t)nk * kBlock * (resident ? 1u : 2u));
                            bulk_load(stage, b_src + (int64_t)kc * kChunk * kBlock, (uint32_t)nk * kBlock, &c->full[s]);
                            if (!resident)
                                bulk_load(stage + kChunk * kBlock, a_src + (int64_t)kc * kChunk * kBlock,
                                          (uint32_t)nk * kBlock, &c->full[s]);
                            }
                            __syncwarp();
                        }
                        if (++s == (uint32_t)a.n_stages) { s = 0; ph ^= 1; }
                    }
                }
            }
        } else if (warp == kMmaWarp || spg <= 2 || (!FUSED && a.pair_groups)) {
            // ------------------------------------------------------------ MMA issue (lane 0 issues)
            // A warp runs dependent scalar code at one instruction every few clocks, so this loop is
            // what paces the tensor pipe: everything that can be is hoisted, and the two cases are
            // compiled separately.  With one instruction per group (g = 32) the groups are
            // independent and two warps take them in turn (even and odd slots), so that each has two
            // groups' time for its bookkeeping; wider groups chain into one slot and stay with one warp.
            const uint32_t me = (uint32_t)(warp - kMmaWarp);
            const uint32_t lane0 = lane == 0 ? 1u : 0u;
            const uint32_t ring_lo = desc_lo(ring_s);
            const uint32_t stage_step = a.stage_bytes >> 4, n_stages = (uint32_t)a.n_stages;
            const uint32_t a_in_stage = resident ? 0u : (uint32_t)(kChunk * (kBlock >> 4));
            const uint32_t empty_s = smem_u32(&c->empty[0]), tfull_s = smem_u32(&c->tfull[0]);
            const uint32_t tempty_s = smem_u32(&c->tempty[0]);
            const int n_steps = a.n_steps;
            // Group k of a tile uses TMEM slot k & 3, so a chunk of four steps always starts at slot 0.
            // 5: one group per tile whose chunks the two warps take in turn, each into an accumulator of its own, which
            // the promotion warps add (integer sums, so the split changes nothing): slots 0 and 1 for even tiles of this
            // CTA, 2 and 3 for odd ones (SPLITQ);
            // mode 0: one instruction per group, two warps that take the even and the odd slots (DUAL); 3: two
            // instructions per group, two warps that take the first and the second group of a chunk (DUAL2);
            // 1: groups of a multiple of four steps, so that a chunk belongs to one group and is issued as
            // straight-line code (QUAD), by one warp when a tile has a single group; 4: the same with two or more
            // groups per tile, which two warps take in turn, each on its own half of the ring (PAIRQ); 2: any
            // other group width, one step at a time
            auto role = [&](auto mode_tag) {
                constexpr int MODE = decltype(mode_tag)::value;
                constexpr bool DUAL = MODE == 0, QUAD = MODE == 1, DUAL2 = MODE == 3, PAIRQ = MODE == 4, SPLITQ = MODE == 5;
                uint32_t s = 0, ph = 0, ib = 0, iu = 0;
                bool ok = true;
                // DUAL: this warp's two slots (me and me + 2), everything about them precomputed
                const uint32_t tm_a = tmem_base + me * kBN, tm_b = tm_a + 2 * kBN;
                const uint32_t off_a = me * (kBlock >> 4), off_b = off_a + 2 * (kBlock >> 4);
                const uint32_t tfull_a = tfull_s + me * 8, tfull_b = tfull_a + 16;
                const uint32_t tempty_a = tempty_s + me * 8, tempty_b = tempty_a + 16;
                uint32_t q_a = 1, q_b = 1;     // parity to wait for on tempty of each slot; a fresh barrier passes parity 1
                // otherwise: one slot at a time
                uint32_t qm = 0xFu;            // the same parities as a mask, bit = slot
                uint32_t ps = 0, pph = 0;      // PAIRQ, SPLITQ: position and phase in this warp's half of the ring (stages me, me + 2, ...)
                uint32_t tpar = 0;             // SPLITQ: parity of the tile among this CTA's tiles
                const uint32_t n_mine = (n_stages + 1 - me) / 2;
                for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                    const int part = item % a.n_parts;
                    const int n_tiles = part_begin(part + 1) - part_begin(part);
                    ok = mbar_wait_warp(&c->a_full[ib], iu, c, a.status, 6u);
                    const uint32_t ares_lo = desc_lo(ibuf_s + ib * a.ibuf_bytes + a_in_ibuf);
                    for (int tl = 0; tl < n_tiles && ok; ++tl) {
                        int sub = 0;
                        uint32_t slot = 0;
                        bool slot_ready = false;   // the early answer about the next slot, if it was yes
                        uint32_t a_lo = ares_lo;   // resident: walks through the item's A blocks
                        if (PAIRQ) {
                            // this warp's groups only (me, me + 2, ...): a group is spg / 4 consecutive chunks into slot
                            // group & 3.  The warp has every second ring stage to itself (fed by the producer warp of the
                            // same parity): two independent rings, so neither warp ever looks at a barrier of the other's.
                            const int cpg = spg / kChunk;
                            const uint32_t full_s = smem_u32(&c->full[0]);
                            for (uint32_t g2 = me; g2 < (uint32_t)a.Kg && ok; g2 += 2) {
                                const uint32_t gslot = g2 & (kSlots - 1), d_tmem = tmem_base + gslot * kBN;
                                uint32_t a_g = ares_lo + g2 * (uint32_t)spg * (uint32_t)(kBlock >> 4);
                                for (int cc = 0; cc < cpg; ++cc) {
                                    const uint32_t st = 2 * ps + me;
                                    if (!mbar_test_s(full_s + st * 8, pph)) {
                                        ok = mbar_wait_warp(&c->full[st], pph, c, a.status, 4u);
                                        if (!ok) break;
                                    }
                                    if (cc == 0 && !mbar_test_s(tempty_s + gslot * 8, (qm >> gslot) & 1u)) {
                                        ok = mbar_wait_warp(&c->tempty[gslot], (qm >> gslot) & 1u, c, a.status, 3u);
                                        if (!ok) break;
                                    }
                                    tc_fence_after();
                                    const uint32_t b_st = ring_lo + st * stage_step;
                                    mma_issue4_if<I8>(lane0, d_tmem, resident ? a_g : b_st + a_in_stage, b_st, cc == 0 ? 0u : 1u);
                                    if (cc == cpg - 1) {
                                        mma_commit_if(lane0, tfull_s + gslot * 8);
                                        qm ^= 1u << gslot;
                                    }
                                    mma_commit_if(lane0, empty_s + st * 8);
                                    a_g += kChunk * (kBlock >> 4);
                                    if (++ps == n_mine) { ps = 0; pph ^= 1; }
                                }
                            }
                            continue;
                        }
                        if (SPLITQ) {
                            // this warp's chunks only (me, me + 2, ...), with as little scalar work around the four
                            // instructions as possible: a lone warp pays several clocks for every dependent instruction
                            const int n_own = (n_chunks - (int)me + 1) / 2;
                            const uint32_t gslot = 2u * tpar + me, d_tmem = tmem_base + gslot * kBN;
                            const uint32_t full_s = smem_u32(&c->full[0]);
                            uint32_t a_own = ares_lo + me * (uint32_t)(kChunk * (kBlock >> 4));
                            for (int i = 0; i < n_own; ++i) {
                                const uint32_t st = 2 * ps + me;
                                if (!mbar_test_s(full_s + st * 8, pph)) {
                                    ok = mbar_wait_warp(&c->full[st], pph, c, a.status, 4u);
                                    if (!ok) break;
                                }
                                if (i == 0 && !mbar_test_s(tempty_s + gslot * 8, (qm >> gslot) & 1u)) {
                                    ok = mbar_wait_warp(&c->tempty[gslot], (qm >> gslot) & 1u, c, a.status, 3u);
                                    if (!ok) break;
                                }
                                tc_fence_after();
                                const uint32_t b_st = ring_lo + st * stage_step;
                                mma_issue4_if<I8>(lane0, d_tmem, resident ? a_own : b_st + a_in_stage, b_st, i == 0 ? 0u : 1u);
                                if (i == n_own - 1) {
                                    mma_commit_if(lane0, tfull_s + gslot * 8);
                                    qm ^= 1u << gslot;
                                }
                                mma_commit_if(lane0, empty_s + st * 8);
                                a_own += 2 * kChunk * (kBlock >> 4);
                                if (++ps == n_mine) { ps = 0; pph ^= 1; }
                            }
                            tpar ^= 1u;
                            continue;
                        }
                        for (int k0 = 0; k0 < n_steps && ok; k0 += kChunk) {
                            ok = mbar_wait_warp(&c->full[s], ph, c, a.status, 4u);
                            if (!ok) break;
                            const uint32_t b_lo = ring_lo + s * stage_step;
                            if (!resident) a_lo = b_lo + a_in_stage;
                            const int nk = min(kChunk, n_steps - k0);
                            if (DUAL) {
                                // straight-line: both of this warp's steps, predicated off past the end of K
                                const uint32_t act_a = me < (uint32_t)nk ? 1u : 0u, act_b = me + 2 < (uint32_t)nk ? 1u : 0u;
                                const bool rdy_a = mbar_test_s(tempty_a, q_a) || !act_a;
                                const bool rdy_b = mbar_test_s(tempty_b, q_b) || !act_b;
                                if (!__all_sync(0xffffffffu, rdy_a)) {
                                    ok = mbar_wait_warp(&c->tempty[me], q_a, c, a.status, 3u);
                                    if (!ok) break;
                                }
                                tc_fence_after();
                                mma_issue_if<I8>(lane0 & act_a, tm_a, a_lo + off_a, b_lo + off_a, 0u);
                                mma_commit_if(lane0 & act_a, tfull_a);
                                q_a ^= act_a;
                                if (!__all_sync(0xffffffffu, rdy_b)) {
                                    ok = mbar_wait_warp(&c->tempty[me + 2], q_b, c, a.status, 3u);
                                    if (!ok) break;
                                    tc_fence_after();
                                }
                                mma_issue_if<I8>(lane0 & act_b, tm_b, a_lo + off_b, b_lo + off_b, 0u);
                                mma_commit_if(lane0 & act_b, tfull_b);
                                q_b ^= act_b;
                            } else if (DUAL2) {
                                // group h of chunk c sits in slot 2 (c & 1) + h: this warp (h = me) alternates between its two slots
                                const bool odd = (k0 & kChunk) != 0;
                                const uint32_t act = 2 * me < (uint32_t)nk ? 1u : 0u;
                                const uint32_t q = odd ? q_b : q_a;
                                const bool rdy = mbar_test_s(odd ? tempty_b : tempty_a, q) || !act;
                                if (!__all_sync(0xffffffffu, rdy)) {
                                    ok = mbar_wait_warp(&c->tempty[me + (odd ? 2u : 0u)], q, c, a.status, 3u);
                                    if (!ok) break;
                                }
                                tc_fence_after();
                                const uint32_t d_tmem = odd ? tm_b : tm_a;
                                mma_issue_if<I8>(lane0 & act, d_tmem, a_lo + 2 * off_a, b_lo + 2 * off_a, 0u);
                                mma_issue_if<I8>(lane0 & act, d_tmem, a_lo + 2 * off_a + (kBlock >> 4), b_lo + 2 * off_a + (kBlock >> 4), 1u);
                                mma_commit_if(lane0 & act, odd ? tfull_b : tfull_a);
                                if (odd) q_b ^= act; else q_a ^= act;
                            } else if (QUAD) {
                                // all four steps of the chunk go to the same slot; n_steps is a multiple of four
                                if (sub == 0 && !slot_ready) {
                                    ok = mbar_wait_warp(&c->tempty[slot], (qm >> slot) & 1u, c, a.status, 3u);
                                    if (!ok) break;
                                }
                                tc_fence_after();
                                const uint32_t d_tmem = tmem_base + slot * kBN;
                                static_assert((kBlock >> 4) == 256, "mma_issue4_if moves the descriptors by 256");
                                mma_issue4_if<I8>(lane0, d_tmem, a_lo, b_lo, sub == 0 ? 0u : 1u);
                                sub += kChunk;
                                if (sub == spg) {
                                    sub = 0;
                                    mma_commit_if(lane0, tfull_s + slot * 8);
                                    qm ^= 1u << slot;
                                    slot = (slot + 1) & (kSlots - 1);
                                    slot_ready = __all_sync(0xffffffffu, mbar_test_s(tempty_s + slot * 8, (qm >> slot) & 1u));
                                }
                            } else {
                                uint32_t a_j = a_lo, b_j = b_lo;
#pragma unroll 1
                                for (int j = 0; j < nk; ++j, a_j += kBlock >> 4, b_j += kBlock >> 4) {
                                    if (sub == 0 && !slot_ready) {
                                        ok = mbar_wait_warp(&c->tempty[slot], (qm >> slot) & 1u, c, a.status, 3u);
                                        if (!ok) break;
                                    }
                                    tc_fence_after();
                                    mma_issue_if<I8>(lane0, tmem_base + slot * kBN, a_j, b_j, sub == 0 ? 0u : 1u);
                                    if (++sub == spg) {
                                        sub = 0;
                                        mma_commit_if(lane0, tfull_s + slot * 8);
                                        qm ^= 1u << slot;
                                        slot = (slot + 1) & (kSlots - 1);
                                        slot_ready = __all_sync(0xffffffffu, mbar_test_s(tempty_s + slot * 8, (qm >> slot) & 1u));
                                    }
                                }
                                if (!ok) break;
                            }
                            if (resident) a_lo += kChunk * (kBlock >> 4);
                            mma_commit_if(lane0, empty_s + s * 8);
                            if (++s == n_stages) { s = 0; ph ^= 1; }
                        }
                    }
                    if (ok) mma_commit_if(lane0, smem_u32(&c->a_empty[ib]));
                    if (++ib == (uint32_t)a.n_ibuf) { ib = 0; iu ^= 1; }
                }
            };
            if (spg == 1) role(std::integral_constant<int, 0>{});
            else if (spg == 2) role(std::integral_constant<int, 3>{});
            else if (!FUSED && a.pair_groups == 2) role(std::integral_constant<int, 5>{});
            else if (!FUSED && a.pair_groups) role(std::integral_constant<int, 4>{});
            else if (spg % kChunk == 0) role(std::integral_constant<int, 1>{});
            else role(std::integral_constant<int, 2>{});
        }
    } else {
        setmaxnreg_inc<kRegsPromo>();
        // ------------------------------------------------------------ promotion + epilogue
        const int pw = warp - kPromoWarp0;
        const int quarter = warp & 3;                 // TMEM lanes 32 * quarter .. + 31
        const int row = quarter * 32 + lane;
        const int col0 = (pw >> 2) * kCols;
        const uint32_t tmem_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + col0;
        // Epilogue geometry.  A warp owns one 32 x 32 block of every tile (the rows of its TMEM lanes,
        // its 32 columns) and needs no other warp to write it out: it scales the sums, parks them in
        // 4 KB of shared memory of its own in the layout of a bulk tensor store (rows of 128 or 64
        // bytes, 16-byte chunks swizzled by the row so that the writes are conflict-free), and lane 0
        // starts the store.  The copy engine clips the box at the edges of y and runs while the warp
        // promotes the next tile; the strip is reused only after the engine has read it.
        constexpr int esz = YBF16 ? 2 : 4;
        constexpr uint32_t kRowBytes = kCols * esz;   // one row of the strip
        const uint32_t strips_s = (sm_s + a.staging_off + 1023u) & ~1023u;   // the swizzle pattern repeats every 1024 bytes
        const bool narrow = YBF16 || a.half_strips;   // 64-byte strip rows (32-byte rows when a.half_strips == 2)
        const uint32_t strip_w = strips_s + (uint32_t)pw * (a.staging_bytes / kPromoWarps);
        const uint32_t strip_row = strip_w + (uint32_t)lane * (a.half_strips == 2 ? 32u : narrow ? 64u : 128u);
        const uint32_t swz = narrow ? (((uint32_t)lane >> 1) & 3u) : ((uint32_t)lane & 7u);   // chunk c sits at c ^ swz
        const uint32_t wsb_s = strips_s + a.staging_bytes + (uint32_t)pw * 256;
        uint32_t ib = 0, iu = 0;                      // item buffer and its phase
        uint32_t my_scale_s = ibuf_s + (uint32_t)row * 4;   // this row's scales in the current item buffer

        uint64_t yacc[kCols / 2];      // 32 floats of one output row, packed in pairs
        // landing buffer: this thread's 32 columns of a slot; 16 at a time in the fused kernel, whose
        // quantizer code leaves the promotion loop fewer registers
        constexpr int kLand = FUSED ? kCols / 2 : kCols;
        uint32_t v[kLand];
#pragma unroll
        for (int q = 0; q < kLand; ++q) v[q] = 0u;
        uint32_t ic = 0;                 // items so far
        uint32_t p_full[kSlots] = {0u, 0u, 0u, 0u};   // parity of the completion of tfull[s] to wait for next
        int item = blockIdx.x, mt = 0, nt = 0, nt_end = 0;
        int64_t n0 = 0;
        float w0 = 0.f, b0 = 0.f;        // channel scale and bias of column n0 + lane
        bool ok = true;

        auto begin_item = [&]() {
            mt = item / a.n_parts;
            const int part = item % a.n_parts;
            nt = part_begin(part);
            nt_end = part_begin(part + 1);
            const uint32_t scales_s = ibuf_s + ib * a.ibuf_bytes, ares_s = scales_s + a_in_ibuf;
            my_scale_s = scales_s + (uint32_t)row * 4;
            if (FUSED) {
                // The previous item's A and scales are free once every MMA that read them has completed and
                // every promotion warp has left the item (a_empty counts both).  Then thread = (row, group
                // mod 4) quantizes its groups: Algorithm S1 steps 2-7 in registers, codes expanded to operand
                // bytes in the block's core-matrix order, the step to the scale block.
                ok = mbar_wait_warp(&c->a_empty[ib], iu ^ 1, c, a.status, 1u);
                if (ok) {
                    constexpr bool XBF = FUSED == 1;
                    const int pt = pw * 32 + lane, r = pt & (kBM - 1);
                    const int64_t mr = (int64_t)mt * kBM + r;
                    const uint32_t off = (uint32_t)((r >> 3) * 256 + (r & 7) * 16);
                    for (int k = pt >> 7; k < a.Kg; k += kPromoWarps * 32 / kBM) {
                        uint32_t out[4] = {0u, 0u, 0u, 0u};
                        float delta = 0.0f;
                        if (mr < a.M)
                            quantize_group32_lean<XBF>(
                                reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(a.x) +
                                                               ((size_t)mr * a.x_stride + (size_t)k * 32) * (XBF ? 2 : 4)),
                                a.seven_tau, a.act_flags, out, delta);
                        uint4 c0, c1;
                        expand8<I8>(out[0], c0.x, c0.y);
                        expand8<I8>(out[1], c0.z, c0.w);
                        expand8<I8>(out[2], c1.x, c1.y);
                        expand8<I8>(out[3], c1.z, c1.w);
                        const uint32_t dst = ares_s + (uint32_t)k * kBlock + off;
                        sts128(dst, c0.x, c0.y, c0.z, c0.w);
                        sts128(dst + 128, c1.x, c1.y, c1.z, c1.w);
                        sts32(scales_s + (uint32_t)k * kScaleBlock + (uint32_t)r * 4, __float_as_uint(delta));
                    }
                    // written through the generic proxy, read by the tensor core through the async proxy
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    mbar_arrive_lane0(&c->a_full[ib], lane);
                }
            }
            if (!FUSED && a.unpack_a) {
                // Packed codes -> operand bytes, straight into the item buffer (no pass through global
                // memory): thread pt takes row pt / 4 and every fourth K-step from pt % 4, so that a warp
                // reads 64 contiguous bytes of each of 8 rows.
                ok = mbar_wait_warp(&c->a_empty[ib], iu ^ 1, c, a.status, 1u);
                if (ok) {
                    const int pt = pw * 32 + lane, r = pt >> 2;
                    const int64_t mr = (int64_t)mt * kBM + r;
                    const uint32_t off = (uint32_t)((r >> 3) * 256 + (r & 7) * 16);
                    const uint8_t* src = a.xcodes + mr * a.row_bytes;
#pragma unroll 1
                    for (int ks = pt & 3; ks < a.n_steps; ks += 4) {
                        uint4 p4 = make_uint4(0u, 0u, 0u, 0u);
                        if (mr < a.M) p4 = __ldg(reinterpret_cast<const uint4*>(src + ks * 16));
                        uint4 c0, c1;
                        expand8<I8>(p4.x, c0.x, c0.y);
                        expand8<I8>(p4.y, c0.z, c0.w);
                        expand8<I8>(p4.z, c1.x, c1.y);
                        expand8<I8>(p4.w, c1.z, c1.w);
                        const uint32_t dst = ares_s + (uint32_t)ks * kBlock + off;
                        sts128(dst, c0.x, c0.y, c0.z, c0.w);
                        sts128(dst + 128, c1.x, c1.y, c1.z, c1.w);
                    }
                    // scales: [group][128 rows]; thread pt takes row pt % 128 and every fourth group
                    const int rs = pt & (kBM - 1);
                    const int64_t ms = (int64_t)mt * kBM + rs;
#pragma unroll 1
                    for (int k = pt >> 7; k < a.Kg; k += kPromoWarps * 32 / kBM)
                        sts32(scales_s + (uint32_t)k * kScaleBlock + (uint32_t)rs * 4,
                              ms < a.M ? __float_as_uint(__ldg(a.xscale + ms * a.Kg + k)) : 0u);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    mbar_arrive_lane0(&c->a_full[ib], lane);
                }
            }
            if (ok) ok = mbar_wait_warp(&c->a_full[ib], iu, c, a.status, 7u);
        };
        auto begin_tile = [&]() {
            n0 = (int64_t)nt * kBN + col0;
#pragma unroll
            for (int j = 0; j < kCols / 2; ++j) yacc[j] = 0ull;
            // loaded now, used at the end of the tile: the latency is not waited for
            const int64_t ca = n0 + lane;
            w0 = ca < a.O ? __ldg(a.wscale + ca) : 0.f;
            b0 = (a.bias && ca < a.O) ? __ldg(a.bias + ca) : 0.f;
        };
        bool store_pending = false;      // a staged tile whose bulk tensor store has not been started
        int32_t store_x = 0, store_y = 0;
        const int store_turn = (pw >> 2) * 4;   // group of the next tile at which this warp starts its store
        auto issue_store = [&]() {
            if (lane == 0) {
                tma_store_2d(&ymap, strip_w, store_x, store_y);
                bulk_commit_group();
            }
            store_pending = false;
        };
        // y = (s_o * 2^e) * sum + bias for the tile that just finished, then on to the next tile
        // The same epilogue in two passes of 16 columns (fp32 output of wide groups, where the promotion warps
        // have time to spare): a strip is 32 rows of 64 bytes, half the shared memory, and the ring gets the
        // other half as two more stages.  The second pass waits until the engine has read the first.
        auto finish_tile_half = [&]() {
            float* wsb = reinterpret_cast<float*>(smem_raw + (wsb_s - sm_s));
            wsb[lane] = __fmul_rn(w0, a.out_scale);
            wsb[32 + lane] = b0;
            uint8_t* strip = smem_raw + (strip_row - sm_s);
            const int64_t m0 = (int64_t)mt * kBM + quarter * 32;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (lane == 0) bulk_wait_group_read0();      // the previous pass's store has read the strip
                __syncwarp();
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * h + jj;
                    float o0, o1, o2, o3;
                    unpack2(yacc[2 * j], o0, o1);
                    unpack2(yacc[2 * j + 1], o2, o3);
                    const float4 s4 = reinterpret_cast<const float4*>(wsb)[j], b4 = reinterpret_cast<const float4*>(wsb + 32)[j];
                    *reinterpret_cast<float4*>(strip + (((uint32_t)jj ^ swz) << 4)) =
                        make_float4(__fmaf_rn(s4.x, o0, b4.x), __fmaf_rn(s4.y, o1, b4.y), __fmaf_rn(s4.z, o2, b4.z),
                                    __fmaf_rn(s4.w, o3, b4.w));
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && m0 < a.M && n0 + 16 * h < a.O) {
                    tma_store_2d(&ymap, strip_w, (int32_t)n0 + 16 * h, (int32_t)m0);
                    bulk_commit_group();
                }
            }
        };
        // The same with strip rows of 32 bytes (a.half_strips == 2: one group per tile with streamed operands, where a
        // tile takes tens of thousands of clocks and the ring can use the shared memory): four passes of 8 columns for
        // fp32 output, two of 16 for 16-bit output; 16 KB of strips in all.  The two 16-byte chunks of a row swap
        // places in rows 4-7 of every eight (the 32-byte swizzle of the tensor map), which keeps the writes
        // conflict-free.
        auto finish_tile_quarter = [&]() {
            float* wsb = reinterpret_cast<float*>(smem_raw + (wsb_s - sm_s));
            wsb[lane] = __fmul_rn(w0, a.out_scale);
            wsb[32 + lane] = b0;
            uint8_t* strip = smem_raw + (strip_row - sm_s);
            const uint32_t sw32 = ((uint32_t)lane >> 2) & 1u;
            const int64_t m0 = (int64_t)mt * kBM + quarter * 32;
            constexpr int kPasses = YBF16 ? 2 : 4, kColsPass = kCols / kPasses;
#pragma unroll
            for (int h = 0; h < kPasses; ++h) {
                if (lane == 0) bulk_wait_group_read0();      // the previous pass's store has read the strip
                __syncwarp();
#pragma unroll
                for (int jj = 0; jj < 2; ++jj) {             // the row's two 16-byte chunks
                    if (YBF16) {                             // eight columns per chunk
                        const int j = 4 * h + 2 * jj;        // yacc pairs j .. j + 3 = columns 2 j .. 2 j + 7 ... in units of four columns below
                        float o[8];
                        unpack2(yacc[2 * j], o[0], o[1]);
                        unpack2(yacc[2 * j + 1], o[2], o[3]);
                        unpack2(yacc[2 * j + 2], o[4], o[5]);
                        unpack2(yacc[2 * j + 3], o[6], o[7]);
                        const float4 sa = reinterpret_cast<const float4*>(wsb)[j], sb = reinterpret_cast<const float4*>(wsb)[j + 1];
                        const float4 ba = reinterpret_cast<const float4*>(wsb + 32)[j], bb = reinterpret_cast<const float4*>(wsb + 32)[j + 1];
                        *reinterpret_cast<uint4*>(strip + (((uint32_t)jj ^ sw32) << 4)) =
                            make_uint4(pack16(__fmaf_rn(sa.x, o[0], ba.x), __fmaf_rn(sa.y, o[1], ba.y), a.y_f16),
                                       pack16(__fmaf_rn(sa.z, o[2], ba.z), __fmaf_rn(sa.w, o[3], ba.w), a.y_f16),
                                       pack16(__fmaf_rn(sb.x, o[4], bb.x), __fmaf_rn(sb.y, o[5], bb.y), a.y_f16),
                                       pack16(__fmaf_rn(sb.z, o[6], bb.z), __fmaf_rn(sb.w, o[7], bb.w), a.y_f16));
                    } else {                                 // four columns per chunk
                        const int j = 2 * h + jj;
                        float o0, o1, o2, o3;
                        unpack2(yacc[2 * j], o0, o1);
                        unpack2(yacc[2 * j + 1], o2, o3);
                        const float4 s4 = reinterpret_cast<const float4*>(wsb)[j], b4 = reinterpret_cast<const float4*>(wsb + 32)[j];
                        *reinterpret_cast<float4*>(strip + (((uint32_t)jj ^ sw32) << 4)) =
                            make_float4(__fmaf_rn(s4.x, o0, b4.x), __fmaf_rn(s4.y, o1, b4.y), __fmaf_rn(s4.z, o2, b4.z),
                                        __fmaf_rn(s4.w, o3, b4.w));
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && m0 < a.M && n0 + kColsPass * h < a.O) {
                    tma_store_2d(&ymap, strip_w, (int32_t)n0 + kColsPass * h, (int32_t)m0);
                    bulk_commit_group();
                }
            }
        };
        auto finish_tile = [&]() {
            if (a.half_strips == 2) {
                finish_tile_quarter();
            } else if (!YBF16 && a.half_strips) {
                finish_tile_half();
            } else {
            if (store_pending) issue_store();            // a short tile: the previous store is still waiting for its turn
            if (lane == 0) bulk_wait_group_read0();      // the previous tile's store has read the strip
            float* wsb = reinterpret_cast<float*>(smem_raw + (wsb_s - sm_s));
            wsb[lane] = __fmul_rn(w0, a.out_scale);
            wsb[32 + lane] = b0;
            __syncwarp();
            uint8_t* strip = smem_raw + (strip_row - sm_s);
#pragma unroll
            for (int j = 0; j < kCols / 4; ++j) {
                float o0, o1, o2, o3;
                unpack2(yacc[2 * j], o0, o1);
                unpack2(yacc[2 * j + 1], o2, o3);
                const float4 s4 = reinterpret_cast<const float4*>(wsb)[j], b4 = reinterpret_cast<const float4*>(wsb + 32)[j];
                o0 = __fmaf_rn(s4.x, o0, b4.x);
                o1 = __fmaf_rn(s4.y, o1, b4.y);
                o2 = __fmaf_rn(s4.z, o2, b4.z);
                o3 = __fmaf_rn(s4.w, o3, b4.w);
                if (YBF16) {       // columns 4 j .. 4 j + 3: half of chunk j / 2
                    *reinterpret_cast<uint2*>(strip + ((((uint32_t)j >> 1) ^ swz) << 4) + ((uint32_t)j & 1u) * 8) =
                        make_uint2(pack16(o0, o1, a.y_f16), pack16(o2, o3, a.y_f16));
                } else {
                    *reinterpret_cast<float4*>(strip + (((uint32_t)j ^ swz) << 4)) = make_float4(o0, o1, o2, o3);
                }
            }
            const int64_t m0 = (int64_t)mt * kBM + quarter * 32;   // first row of this warp's block
            if (a.tma_ok) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes before the engine's reads
                __syncwarp();
                // The store is started a few groups into the next tile, each block of columns at its own
                // time: sixteen warps that hand 4 KB to the copy engine at the same moment queue up behind
                // one another, and starting a store blocks the warp until the engine has taken it.
                store_pending = m0 < a.M && n0 < a.O;
                store_x = (int32_t)n0;
                store_y = (int32_t)m0;
            } else {          // any alignment: a row at a time, lane = column
                __syncwarp();
                const int rows = (int)min((int64_t)32, a.M - m0);
                if (n0 + lane < a.O) {
#pragma unroll 1
                    for (int r = 0; r < rows; ++r) {
                        const size_t at = (size_t)(m0 + r) * a.y_stride + (size_t)(n0 + lane);
                        if (YBF16) {
                            const uint32_t rs = ((uint32_t)r >> 1) & 3u;
                            reinterpret_cast<uint16_t*>(a.y)[at] = (uint16_t)lds16(
                                strip_w + (uint32_t)r * kRowBytes + ((((uint32_t)lane >> 3) ^ rs) << 4) + ((uint32_t)lane & 7u) * 2);
                        } else {
                            const uint32_t rs = (uint32_t)r & 7u;
                            reinterpret_cast<uint32_t*>(a.y)[at] = lds32(
                                strip_w + (uint32_t)r * kRowBytes + ((((uint32_t)lane >> 2) ^ rs) << 4) + ((uint32_t)lane & 3u) * 4);
                        }
                    }
                }
                __syncwarp();     // the strip may be overwritten by the next tile
            }
            }
            // next tile, next item
            if (++nt == nt_end) {
                // the item's scales were read through the generic proxy; the next item's bulk copies
                // overwrite them through the async proxy, which only a proxy fence orders after the reads
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                mbar_arrive_lane0(&c->a_empty[ib], lane);
                if (++ib == (uint32_t)a.n_ibuf) { ib = 0; iu ^= 1; }
                item += gridDim.x;
                if (item < n_items) begin_item();
            }
            if (ok && item < n_items) begin_tile();
        };
        // Group k of a tile lives in TMEM slot k & 3, so the slot is a compile-time constant in a loop
        // unrolled by four.  request<U>: wait until slot U is full, start loading this thread's 32
        // columns into v.  consume<U>: wait for them, hand the slot back at once, fold them in; it also
        // asks whether the next slot is full already, an answer that is only needed after the FMAs.
        // With four promotion warps per scheduler the load of one warp hides behind the FMAs of the others.
        uint32_t tfull_s = smem_u32(&c->tfull[0]), tempty_s = smem_u32(&c->tempty[0]), tmem_row_r = tmem_row;
        // opaque to the compiler: kept in registers instead of being recomputed from the thread index at every use
        asm volatile("" : "+r"(tfull_s), "+r"(tempty_s), "+r"(tmem_row_r));
        auto request = [&](auto u_tag, bool ready) {
            constexpr uint32_t U = decltype(u_tag)::value;
            if (!__all_sync(0xffffffffu, ready)) ok = mbar_wait_warp(&c->tfull[U], p_full[U], c, a.status, 2u);
            p_full[U] ^= 1u;
            tc_fence_after();
            if (FUSED) tmem_ld16(tmem_row_r + U * kBN, v);
            else tmem_ld32(tmem_row_r + U * kBN, v);
        };
        auto consume = [&](auto u_tag, uint32_t scale_q, int k) -> bool {
            constexpr uint32_t U = decltype(u_tag)::value, N = (U + 1) & (kSlots - 1);
            const uint32_t dbits = lds32(scale_q + U * kScaleBlock);
            const uint64_t d2 = pack2(dbits, dbits);
            const bool next_ready = mbar_test_s(tfull_s + N * 8, p_full[N]);
            tmem_ld_wait();                               // v has landed
            if (FUSED) {                                  // first half folded in, then the second half takes its place
#pragma unroll
                for (int q = 0; q < kLand / 2; ++q) fma2(yacc[q], pack2(v[2 * q], v[2 * q + 1]), d2);
                tmem_ld16(tmem_row_r + U * kBN + kLand, v);
                tmem_ld_wait();
            }
            tc_fence_before();                            // the slot is drained
            __syncwarp();
            mbar_arrive_lane0_s(tempty_s + U * 8, lane);
            if (DBG) {
                const int64_t m = (int64_t)mt * kBM + row;
                if (a.acc_debug && m < a.M) debug_store<I8>(a, v, m, n0, k + (int)U);
            }
            if (I8) {
#pragma unroll
                for (int q = 0; q < kLand; ++q) v[q] = __float_as_uint((float)(int32_t)v[q]);
            }
#pragma unroll
            for (int q = 0; q < kLand / 2; ++q) fma2(yacc[(FUSED ? kLand / 2 : 0) + q], pack2(v[2 * q], v[2 * q + 1]), d2);
            return next_ready;
        };
        // One group per tile in two accumulators (a.pair_groups == 2): slots UA and UA + 1 hold the sums over the even
        // and the odd chunks of K.  Integer sums: their sum is the group's sum whatever the split.  (The power-of-two
        // variant accumulates scaled values in fp32; there the split adds one rounding to the K the variant already has.)
        auto consume_split = [&](auto u_tag) {
            constexpr uint32_t UA = decltype(u_tag)::value, UB = UA + 1;
            ok = mbar_wait_warp(&c->tfull[UA], p_full[UA], c, a.status, 2u);
            if (ok) ok = mbar_wait_warp(&c->tfull[UB], p_full[UB], c, a.status, 2u);
            p_full[UA] ^= 1u;
            p_full[UB] ^= 1u;
            if (!ok) return;
            const uint32_t dbits = lds32(my_scale_s);
            const uint64_t d2 = pack2(dbits, dbits);
            tc_fence_after();
            if (!FUSED) {
                tmem_ld32(tmem_row_r + UA * kBN, v);
                tmem_ld_wait();
                uint32_t v2[kCols / 2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int q = 0; q < kCols / 2; ++q) v2[q] = 0u;
                    tmem_ld16(tmem_row_r + UB * kBN + h * (kCols / 2), v2);
                    tmem_ld_wait_on16(v2);
#pragma unroll
                    for (int q = 0; q < kCols / 2; ++q) {
                        uint32_t& d = v[h * (kCols / 2) + q];
                        if (I8) d += v2[q];
                        else d = __float_as_uint(__fadd_rn(__uint_as_float(d), __uint_as_float(v2[q])));   // power-of-two variant
                    }
                }
            }
            tc_fence_before();                            // both slots are drained
            __syncwarp();
            mbar_arrive_lane0_s(tempty_s + UA * 8, lane);
            mbar_arrive_lane0_s(tempty_s + UB * 8, lane);
            if (DBG) {
                const int64_t m = (int64_t)mt * kBM + row;
                if (a.acc_debug && m < a.M) debug_store<I8>(a, v, m, n0, 0);
            }
            if (!FUSED) {
#pragma unroll
                for (int q = 0; q < kCols; ++q)
                    if (I8) v[q] = __float_as_uint((float)(int32_t)v[q]);
#pragma unroll
                for (int q = 0; q < kCols / 2; ++q) fma2(yacc[q], pack2(v[2 * q], v[2 * q + 1]), d2);
            }
        };
        const std::integral_constant<uint32_t, 0> u0{};
        const std::integral_constant<uint32_t, 1> u1{};
        const std::integral_constant<uint32_t, 2> u2{};
        const std::integral_constant<uint32_t, 3> u3{};

        if (!FUSED && a.pair_groups == 2) {
            if (item < n_items) {
                begin_item();
                if (ok) begin_tile();
                uint32_t tpar = 0;
#pragma unroll 1
                while (ok && item < n_items) {
                    if (tpar) consume_split(u2); else consume_split(u0);
                    tpar ^= 1u;
                    if (!ok) break;
                    finish_tile();
                }
            }
        } else if (item < n_items) {
            begin_item();
            if (ok) {
                begin_tile();
                request(u0, false);
            }
#pragma unroll 1
            while (ok && item < n_items) {
                // one tile; the load of its first group is in flight
                const int Kg = a.Kg;
                uint32_t scale_q = my_scale_s;
                int k = 0;
#pragma unroll 1
                for (; k + 4 < Kg && ok; k += 4, scale_q += 4 * kScaleBlock) {   // four groups, and more behind them
                    if (store_pending && k >= store_turn) issue_store();
                    request(u1, consume(u0, scale_q, k));
                    request(u2, consume(u1, scale_q, k));
                    request(u3, consume(u2, scale_q, k));
                    request(u0, consume(u3, scale_q, k));
                }
                if (!ok) break;
                const int rem = Kg - k;                   // the last one to four groups
                bool r = consume(u0, scale_q, k);
                if (rem > 1) {
                    request(u1, r);
                    r = consume(u1, scale_q, k);
                    if (rem > 2) {
                        request(u2, r);
                        r = consume(u2, scale_q, k);
                        if (rem > 3) {
                            request(u3, r);
                            consume(u3, scale_q, k);
                        }
                    }
                }
                if (!ok) break;
                // The epilogue comes before the wait for the next tile's first group: that group may belong
                // to the next work item, which cannot start before this warp has handed the item's buffers back.
                finish_tile();
                if (ok && item < n_items) request(u0, false);
            }
        }
        tmem_ld_wait();            // nothing may still be landing when TMEM is released
        if (store_pending) issue_store();
        if (lane == 0) bulk_wait_group0();   // nor may a store still be reading this CTA's shared memory
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        // all MMAs this CTA issued have completed unless a wait gave up; in that case give the
        // tensor core a moment before the columns are handed back
        if (c->abort_flag) __nanosleep(1000000);
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------
// host side


}  // namespace
}  // namespace tdq

using namespace tdq;

static int sm_count() { return current_device_sm_count(); }

extern "C" size_t tdq_linear_workspace_bytes(int64_t M, int64_t I_pad, int64_t O, int32_t group_size) {
    if (M < 0 || I_pad <= 0 || O <= 0 || group_size <= 0 || group_size % 32 || I_pad % group_size)
        return kWorkspaceHeader;
    Plan p;
    if (!make_plan(M, I_pad, O, group_size, 148, p)) return kWorkspaceHeader;
    return kWorkspaceHeader + p.a_bytes + p.b_bytes + p.s_bytes;
}

namespace tdq {

tdq_status linear_check_shape(int64_t M, int64_t I_pad, int64_t O, int32_t group_size, size_t workspace_bytes) {
    if (M < 0 || O <= 0 || I_pad <= 0) return TDQ_ERR_INVALID_ARG;
    if (group_size <= 0 || I_pad % group_size) return TDQ_ERR_INVALID_ARG;
    if (group_size % 32 || group_size > 4096) return TDQ_ERR_UNSUPPORTED;
    if (I_pad / 2 > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    Plan p;
    if (!make_plan(M, I_pad, O, group_size, 148, p)) return TDQ_ERR_UNSUPPORTED;
    if (workspace_bytes < kWorkspaceHeader + p.a_bytes + p.b_bytes + p.s_bytes) return TDQ_ERR_WORKSPACE;
    return TDQ_OK;
}

tdq_status linear_impl(const FusedSrc* fx, const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                       const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O, int32_t group_size,
                       void* y, tdq_dtype y_dtype, int64_t y_row_stride, int32_t* acc_debug, void* workspace,
                       size_t workspace_bytes, void* cuda_stream, int pow2_steps) {
    if (!fx && (!xcodes || !xscale)) return TDQ_ERR_INVALID_ARG;
    if (pow2_steps && (fx || acc_debug)) return TDQ_ERR_UNSUPPORTED;
    if (fx && (!fx->x || group_size != 32 || acc_debug)) return TDQ_ERR_UNSUPPORTED;
    if (!wcodes || !wscale || !y) return TDQ_ERR_INVALID_ARG;
    if (M < 0 || O <= 0 || I_pad <= 0 || y_row_stride < O) return TDQ_ERR_INVALID_ARG;
    if (y_dtype != TDQ_F32 && y_dtype != TDQ_BF16 && y_dtype != TDQ_F16) return TDQ_ERR_INVALID_ARG;
    const bool y_f16 = y_dtype == TDQ_F16;
    if (y_f16) y_dtype = TDQ_BF16;      // the 16-bit kernels serve both types; a flag picks the conversion
    if (group_size <= 0 || I_pad % group_size) return TDQ_ERR_INVALID_ARG;
    if (group_size % 32 || group_size > 4096) return TDQ_ERR_UNSUPPORTED;
    if (I_pad / 2 > INT32_MAX) return TDQ_ERR_INVALID_ARG;
    // power-of-two steps: the activation groups only matter to the operand encoding; the kernel sees one
    // group that spans the whole contraction
    const int32_t act_group = group_size;
    if (pow2_steps) {
        if (I_pad > INT32_MAX) return TDQ_ERR_UNSUPPORTED;
        group_size = (int32_t)I_pad;
    }
    Plan p;
    if (!make_plan(M, I_pad, O, group_size, 148, p)) return TDQ_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < kWorkspaceHeader + p.a_bytes + p.b_bytes + p.s_bytes) return TDQ_ERR_WORKSPACE;
    if ((!fx && reinterpret_cast<uintptr_t>(xcodes) % 16) || reinterpret_cast<uintptr_t>(wcodes) % 16 ||
        reinterpret_cast<uintptr_t>(workspace) % 16)
        return TDQ_ERR_ALIGNMENT;
    if (M == 0) return TDQ_OK;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    const int n_sm = sm_count();
    if (n_sm <= 0) return TDQ_ERR_CUDA;
    // Output strips: 64-byte rows (32 KB in all) for bf16 output, and for fp32 output of wide groups, which is
    // then written in two passes of 16 columns; the ring gets the other 32 KB.  Both need the bulk tensor store.
    const int64_t y_esz = y_dtype == TDQ_BF16 ? 2 : 4;
    const bool y_tma = reinterpret_cast<uintptr_t>(y) % 16 == 0 && (y_row_stride * y_esz) % 16 == 0 && O <= INT32_MAX &&
                       M <= INT32_MAX;
    const bool half_strips = y_tma && y_dtype == TDQ_F32 && !fx && !acc_debug && group_size >= 128;
    const bool narrow_strips = y_tma && (y_dtype == TDQ_BF16 || half_strips);
    // several instructions chain into one slot: keep the integer accumulator (the power-of-two variant
    // accumulates scaled values, which only the fp32 accumulator can hold)
    const bool wide = group_size > 64 && !pow2_steps;   // a ring stage belongs to one group: the two-warp modes
    // Up to 128 codes per group the E4M3 route is taken (at most four chained instructions per accumulator; the sums, below
    // 2^13 in units of 2^-18, are exact in the fp32 accumulator, and the promotion needs no integer-to-float conversion);
    // wider groups keep the integer accumulator.
    const bool i8 = group_size > 128 && !pow2_steps;
    int64_t staging_bytes = narrow_strips ? kStagingBytes / 2 : kStagingBytes;
    if (!make_plan(M, I_pad, O, group_size, n_sm, p, staging_bytes)) return TDQ_ERR_UNSUPPORTED;
    // Wide groups run with two MMA-issuing warps, each with half of the ring, and the ring is what bounds them: strips
    // with 32-byte rows (16 KB in all, written in passes) leave room for more stages.  Taken when that gives the smaller
    // half of the ring another stage without changing whether A stays resident; with several groups per tile only where
    // the operands stream (a long contraction), since the passes cost a short tile more than the stage gives.
    bool quarter_strips = y_tma && !fx && !acc_debug && (wide || pow2_steps) && p.n_chunks >= 2 &&
                          ((p.Kg == 1 && p.n_steps % kChunk == 0) ||
                           (wide && (group_size / 32) % kChunk == 0 && p.Kg >= 2 && !p.a_resident));
    if (quarter_strips) {
        Plan q;
        if (make_plan(M, I_pad, O, group_size, n_sm, q, kStagingBytes / 4) && q.a_resident == p.a_resident &&
            q.n_stages / 2 > p.n_stages / 2) {
            p = q;
            staging_bytes = kStagingBytes / 4;
        } else {
            quarter_strips = false;
        }
    }
    if (fx && !p.a_resident) return TDQ_ERR_UNSUPPORTED;   // the fused producer writes a whole row block's A into shared memory

    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);

    ExpandArgs e;
    e.xcodes = xcodes; e.xscale = xscale; e.wcodes = wcodes;
    e.a_blocks = ws + kWorkspaceHeader;
    e.b_blocks = e.a_blocks + p.a_bytes;
    e.s_blocks = e.b_blocks + p.b_bytes;
    e.M = M; e.O = O;
    e.row_bytes = (int32_t)(I_pad / 2);
    e.n_steps = p.n_steps; e.n_chunks = p.n_chunks;
    e.steps_per_grp = group_size / 32;
    e.Kg = p.Kg;
    // The kernel can unpack a resident A block itself, which saves the pass that writes A blocks to the
    // workspace; its promotion warps do that at the start of an item, though, with the tensor core idle,
    // so it only pays when an item carries much more work than its own unpacking.
    const int64_t steps_per_item = (p.tiles_n + p.n_parts - 1) / p.n_parts * (int64_t)p.n_steps;
    const bool unpack_a = !fx && !pow2_steps && p.a_resident && steps_per_item >= 256;
    e.tiles_m = (fx || unpack_a) ? 0 : (int32_t)p.tiles_m;   // then only the weights are expanded here
    e.tiles_n = (int32_t)p.tiles_n;
    e.status = reinterpret_cast<uint32_t*>(workspace);

    LinArgs a;
    a.a_blocks = e.a_blocks; a.b_blocks = e.b_blocks; a.s_blocks = e.s_blocks;
    a.wscale = wscale; a.bias = bias;
    a.M = M; a.O = O;
    a.n_steps = p.n_steps; a.steps_per_grp = e.steps_per_grp; a.Kg = p.Kg;
    a.tiles_m = (int32_t)p.tiles_m; a.tiles_n = e.tiles_n; a.n_parts = p.n_parts;
    a.a_resident = p.a_resident; a.n_stages = p.n_stages;
    a.ring_off = p.ring_off; a.stage_bytes = p.stage_bytes;
    a.ibuf_bytes = p.ibuf_bytes; a.n_ibuf = p.n_ibuf;
    a.staging_off = p.staging_off;
    a.y = y; a.y_stride = y_row_stride; a.acc_debug = acc_debug;
    a.status = reinterpret_cast<uint32_t*>(workspace);
    const int64_t esz = y_dtype == TDQ_BF16 ? 2 : 4;
    // bulk tensor stores want a 16-byte aligned base and row pitch; anything else goes element by element
    CUtensorMap ymap;
    memset(&ymap, 0, sizeof(ymap));
    a.tma_ok = 0;
    // g = 32 with y that tensor stores can write goes to the kernel built for it (tdq_linear_g32.cu)
    const bool use_g32 = group_size == 32 && !pow2_steps && !fx && y_tma;
    if (y_tma && encode_y_map(&ymap, y, y_dtype == TDQ_BF16, M, O, y_row_stride,
                              quarter_strips ? (y_dtype == TDQ_BF16 ? kCols / 2 : kCols / 4) : half_strips ? kCols / 2 : kCols,
                              use_g32 ? kBM : 32, y_f16))
        a.tma_ok = 1;
    else if (narrow_strips || quarter_strips)
        return TDQ_ERR_CUDA;   // the plan counted on the tensor store
    a.staging_bytes = (uint32_t)staging_bytes;
    a.half_strips = quarter_strips ? 2 : half_strips ? 1 : 0;
    a.out_scale = i8 ? 0.00390625f : 262144.0f;
    a.y_f16 = y_f16 ? 1 : 0;
    a.xcodes = xcodes; a.xscale = xscale; a.row_bytes = e.row_bytes; a.unpack_a = unpack_a ? 1 : 0;
    a.pair_groups = (wide && a.steps_per_grp % kChunk == 0 && a.Kg >= 2) ? 1 : 0;
    // one group per tile: the group's chunks go to the two MMA warps in turn, each with an accumulator of its own
    if ((wide || pow2_steps) && !fx && a.Kg == 1 && a.steps_per_grp % kChunk == 0 && p.n_chunks >= 2) a.pair_groups = 2;
    a.x = fx ? fx->x : nullptr;
    a.x_stride = fx ? fx->row_stride : 0;
    a.seven_tau = fx ? fx->seven_tau : 0.0f;
    a.act_flags = fx ? fx->flags : 0u;

    const bool ybf = y_dtype == TDQ_BF16, dbg = acc_debug != nullptr;
    void (*kernel)(LinArgs, CUtensorMap) = nullptr;
#define TDQ_PICK(I8_, YB_, DBG_) if (i8 == I8_ && ybf == YB_ && dbg == DBG_) kernel = w4a4_gemm_kernel<I8_, YB_, DBG_>;
    TDQ_PICK(false, false, false) TDQ_PICK(false, true, false) TDQ_PICK(true, false, false) TDQ_PICK(true, true, false)
    TDQ_PICK(false, false, true) TDQ_PICK(false, true, true) TDQ_PICK(true, false, true) TDQ_PICK(true, true, true)
#undef TDQ_PICK
    if (fx) {
        if (fx->bf16) kernel = ybf ? w4a4_gemm_kernel<false, true, false, 1> : w4a4_gemm_kernel<false, false, false, 1>;
        else kernel = ybf ? w4a4_gemm_kernel<false, true, false, 2> : w4a4_gemm_kernel<false, false, false, 2>;
    }
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess)
        return TDQ_ERR_CUDA;

    const unsigned pieces = (unsigned)((e.tiles_m + e.tiles_n) * p.n_chunks);
    if (pow2_steps) {
        const unsigned pieces2 = (unsigned)((e.tiles_m + e.tiles_n) * ((p.n_chunks + kPow2Chunks - 1) / kPow2Chunks));
        expand_pow2_kernel<<<pieces2, kExpandThreads, 0, stream>>>(e, (int32_t)(act_group / 32), (int32_t)(I_pad / act_group));
    }
    else if (i8) expand_kernel<true><<<pieces, kExpandThreads, 0, stream>>>(e);
    else expand_kernel<false><<<pieces, kExpandThreads, 0, stream>>>(e);
    // (Ordinary launches: as programmatic dependents of the kernel before them the expansions were measured 1 to 4 us
    // per call slower; their CTAs need next to no shared memory, so they can become resident beside a running GEMM
    // and wait there.  The GEMM that follows is a programmatic dependent of the expansion: its set-up overlaps it.)
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);

    const int64_t items = p.tiles_m * p.n_parts;
    const unsigned grid = (unsigned)(items < n_sm ? items : n_sm);
    if (use_g32 && a.tma_ok) return launch_linear_g32(a, ymap, p.smem_bytes, grid, ybf, dbg, stream);
    if (launch_pdl(kernel, dim3(grid), dim3(kThreads), p.smem_bytes, stream, a, ymap) != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

}  // namespace tdq

extern "C" tdq_status tdq_w4a4_linear(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                      const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                      int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                      int32_t* acc_debug, void* workspace, size_t workspace_bytes,
                                      void* cuda_stream) {
    return linear_impl(nullptr, xcodes, xscale, wcodes, wscale, bias, M, I_pad, O, group_size, y, y_dtype, y_row_stride,
                       acc_debug, workspace, workspace_bytes, cuda_stream, 0);
}

extern "C" tdq_status tdq_w4a4_linear_pow2(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                           const float* wscale, const float* bias, int64_t M, int64_t I_pad, int64_t O,
                                           int32_t group_size, void* y, tdq_dtype y_dtype, int64_t y_row_stride,
                                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return linear_impl(nullptr, xcodes, xscale, wcodes, wscale, bias, M, I_pad, O, group_size, y, y_dtype, y_row_stride,
                       nullptr, workspace, workspace_bytes, cuda_stream, 1);
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

// ------------------------------------------------------------------------------------------
// tdq_selftest_wait_timeout: makes a bounded wait run out, the way a lost arrival would

namespace tdq {
namespace {
// One warp: a fresh barrier with one expected arrival that never comes, waited on with the GEMM kernels' own
// routine and a short limit; the code lands in the workspace's status word.  Nothing is in flight when the
// warp leaves.
__global__ void __launch_bounds__(32) linear_wait_selftest_kernel(uint32_t* status, long long limit) {
    __shared__ Ctrl c;
    if (threadIdx.x == 0) {
        mbar_init(&c.full[0], 1);
        c.abort_flag = 0;
    }
    __syncwarp();
    mbar_wait_warp(&c.full[0], 0u, &c, status, 15u, limit);
}
}  // namespace
}  // namespace tdq

extern "C" tdq_status tdq_selftest_wait_timeout(int32_t which, int64_t limit_cycles, void* workspace, void* cuda_stream) {
    if (which != 0 && which != 1) return TDQ_ERR_INVALID_ARG;
    if (limit_cycles < 1000 || limit_cycles > 2000000000LL) return TDQ_ERR_INVALID_ARG;   // at most about a second
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (which == 1) return act_wait_selftest(limit_cycles, stream);
    if (!workspace) return TDQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return TDQ_ERR_ALIGNMENT;
    if (cudaMemsetAsync(workspace, 0, 16, stream) != cudaSuccess) return TDQ_ERR_CUDA;
    linear_wait_selftest_kernel<<<1, 32, 0, stream>>>(reinterpret_cast<uint32_t*>(workspace), limit_cycles);
    if (cudaGetLastError() != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

// ------------------------------------------------------------------------------------------
// tdq_w4a4_linear_static: the same two kernels, with the operand blocks in a fixed device array

namespace {
constexpr size_t kStaticScratchBytes = TDQ_LINEAR_STATIC_BYTES;
// Lives in every CUDA context that loads this library, from load to exit.  Host code may only
// use the name to look its device address up; the kernels get that address as a plain pointer.
static __device__ __align__(256) uint8_t g_static_scratch[kStaticScratchBytes];

std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};
}  // namespace

extern "C" tdq_status tdq_w4a4_linear_static(const uint8_t* xcodes, const float* xscale, const uint8_t* wcodes,
                                             const float* wscale, const float* bias, int64_t M, int64_t I_pad,
                                             int64_t O, int32_t group_size, void* y, tdq_dtype y_dtype,
                                             int64_t y_row_stride, int32_t wait, void* cuda_stream) {
    // the argument checks that do not depend on the scratch come first, as in tdq_w4a4_linear
    if (!wcodes || !wscale || !y) return TDQ_ERR_INVALID_ARG;
    if (M < 0 || O <= 0 || I_pad <= 0 || y_row_stride < O) return TDQ_ERR_INVALID_ARG;
    if (group_size <= 0 || I_pad % group_size) return TDQ_ERR_INVALID_ARG;
    if (group_size % 32 || group_size > 4096) return TDQ_ERR_UNSUPPORTED;
    const size_t need = tdq_linear_workspace_bytes(M, I_pad, O, group_size);
    if (need > kStaticScratchBytes) return TDQ_ERR_WORKSPACE;   // the problem is too large for the fixed array

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TDQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return TDQ_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {   // first call on this device: ask the runtime where the array lives here
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return TDQ_ERR_CUDA;
            g_static_ptr[dev] = p;
        }
        scratch = g_static_ptr[dev];
    }
    tdq_status st = tdq_w4a4_linear(xcodes, xscale, wcodes, wscale, bias, M, I_pad, O, group_size, y, y_dtype,
                                    y_row_stride, nullptr, scratch, kStaticScratchBytes, cuda_stream);
    if (st != TDQ_OK || !wait || M == 0) return st;
    return tdq_workspace_status(scratch, cuda_stream, nullptr);
}
