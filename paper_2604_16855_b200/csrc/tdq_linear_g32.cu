// The W4A4 linear layer at the paper's group size g = 32 (Algorithm S1 step 10 with Eq. 9 and Eq. 4
// substituted), with y that bulk tensor stores can write (16-byte aligned base and row pitch):
//
//   acc[m,o,k] = sum_{i in group k} q_x[m,i] q_w[o,i]      one tcgen05.mma (E4M3 operands, exact) per group
//   y[m,o]     = s_o * sum_k Delta[m,k] * acc[m,o,k] + b_o  fp32 in registers ("promotion")
//
// At g = 32 every K-step of the tensor core ends an accumulator, so the per-group pass over the
// 128 x 128 accumulators (16384 fp32 multiply-adds, 128 clocks of the SM's FMA pipes, against 64
// clocks of tensor time) bounds the kernel.  This kernel is built around keeping those pipes fed:
//
//   * eight promotion warps, each owning 32 TMEM lanes (rows) and 64 columns: 64 float sums and two
//     32-register landing buffers per thread.  The tcgen05.ld of the next half group is always in
//     flight while the multiply-adds of the current half run, so a warp never waits for a load it
//     has only just issued, and a TMEM slot is handed back as soon as its second half has landed
//     (before its arithmetic), which lets the tensor core refill it a group-time earlier.
//   * the first load of the next tile is started before the epilogue of the current one.
//   * the epilogue only scales (s_o, b_o) and parks the tile in shared memory, laid out as four
//     32-column boxes of a bulk tensor store; a control warp of its own issues the four stores and
//     hands the staging area back when the copy engine has read it, so the promotion warps never
//     block on the engine.
//   * a lone warp runs dependent scalar code at one instruction every several clocks, so the per-group
//     bookkeeping of the tensor-core side is spread over four MMA-issuing warps, one per TMEM slot, and
//     every wait in a hot loop is one barrier test with the bounded, sleeping wait out of line.
//   Warps 0-1 stream the weight blocks (and A when it does not stay resident), warps 2-5 issue the
//   MMAs (warp 2 + j owns TMEM slot j), warp 6 issues the stores; warp 7 only keeps the register
//   partitions of the four schedulers even.  Operand blocks, the ring, the item buffers and the bounded
//   waits are those of the general kernel (tdq_linear.cu).
#include "tdq_tc.cuh"

namespace tdq {
namespace {

constexpr int kCtlWarps = 8;
constexpr int kMmaWarps = kSlots;                          // warps 2..5, one per TMEM slot
constexpr int kStoreWarp = kMmaWarp + kMmaWarps;           // 6
constexpr int kPWarp0 = kCtlWarps;
constexpr int kPWarps = 8;
constexpr int kPCols = kBN / (kPWarps / 4);                 // 64 columns of one row per promotion thread
constexpr int kThreadsG32 = (kCtlWarps + kPWarps) * 32;     // 512
constexpr int kRegsCtl = 40, kRegsP = 208;                  // 256 * 40 + 256 * 208 <= 65536
#ifndef TDQ_ACC_SWAP
#define TDQ_ACC_SWAP 0
#endif
// Which accumulator pair takes which column pair of a landing buffer (pair q goes to accumulator q ^ kAccSwap):
// a packed multiply-add whose accumulator and multiplicand pairs sit in the same register banks issues at half rate.
constexpr int kAccSwap = TDQ_ACC_SWAP;
constexpr uint32_t kBoxF32 = 128 * 128, kBoxBF16 = 128 * 64;   // one 32-column box of 128 rows in the staging area
static_assert(2 * kBN * 4 <= kWsbBytes, "the tile's channel scales and biases outgrew their reservation");
static_assert(4 * kBoxF32 <= kStagingBytes, "the staged tile outgrew its reservation");

// Waits for this thread's outstanding TMEM loads.  The landing registers are passed through as operands so
// that no use of them can be scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait_on(uint32_t* v) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                   "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :
                 : "memory");
}

// Waits in the hot loops: one test of the barrier; if the phase is not complete yet, the bounded sleeping
// wait, out of line.  Every lane asks about the same barrier in the same instruction, so the lanes agree
// without a vote.  A wait that gives up raises the CTA's abort flag (and records its code); the loops look
// at that flag once per tile, and every later wait returns at once.
__device__ __forceinline__ void wait_cold(uint32_t bar_s, uint32_t parity, Ctrl* c, uint32_t* status, uint32_t code) {
    uint64_t* bar = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(c) + (bar_s - smem_u32(c)));
    mbar_wait_slow(bar, parity, c, status, code);
}
__device__ __forceinline__ void wait_hot(uint32_t bar_s, uint32_t parity, Ctrl* c, uint32_t* status, uint32_t code) {
    if (!mbar_test_s(bar_s, parity)) wait_cold(bar_s, parity, c, status, code);
}

template <bool YBF16, bool DBG>
__global__ void __launch_bounds__(kThreadsG32, 1) w4a4_g32_kernel(const LinArgs a, const __grid_constant__ CUtensorMap ymap) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    Ctrl* c = reinterpret_cast<Ctrl*>(smem_raw);
    const uint32_t sm_s = smem_u32(smem_raw);
    // item buffer b: [Kg][128] floats of the item's scales, then its [n_steps] operand blocks if resident
    const uint32_t ibuf_s = sm_s + kCtrlBytes;
    const uint32_t a_in_ibuf = (uint32_t)a.Kg * kScaleBlock;
    const uint32_t ring_s = sm_s + a.ring_off;
    const uint32_t stage_s = (sm_s + a.staging_off + 1023u) & ~1023u;   // the swizzle patterns repeat every 1024 bytes
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const bool resident = a.a_resident != 0;

    if (t == 0) {
        for (int i = 0; i < kMaxStages; ++i) { mbar_init(&c->full[i], 1); mbar_init(&c->empty[i], kMmaWarps); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(&c->tfull[i], 1); mbar_init(&c->tempty[i], kPWarps); }
        for (int i = 0; i < kMaxItemBufs; ++i) {
            mbar_init(&c->a_full[i], a.unpack_a ? kPWarps : 1);
            mbar_init(&c->a_empty[i], kMmaWarps + kPWarps);
        }
        mbar_init(&c->sfull, kPWarps);
        mbar_init(&c->sfree, 1);
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
    const uint32_t tmem_base = c->tmem_base;

    const int n_items = a.tiles_m * a.n_parts;
    const int n_chunks = (a.n_steps + kChunk - 1) / kChunk;
    auto part_begin = [&](int part) { return (int)(((int64_t)part * a.tiles_n) / a.n_parts); };

    if (warp < kCtlWarps) {
        setmaxnreg_dec<kRegsCtl>();
        // The control roles run with the whole warp converged and let lane 0 issue.
        if (warp < kProdWarps) {
            // ------------------------------------------------------------ producers: alternate ring stages
            uint32_t sc = 0, s = 0, ph = 0;   // stage counter, its ring slot and phase
            uint32_t ib = 0, iu = 0;          // item buffer and its phase
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int mt = item / a.n_parts, part = item % a.n_parts;
                const uint8_t* a_src = a.a_blocks + (int64_t)mt * a.n_steps * kBlock;
                if (warp == 0 && !a.unpack_a) {
                    wait_hot(smem_u32(&c->a_empty[ib]), iu ^ 1, c, a.status, 1u);
                    if (c->abort_flag) break;
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
                    for (int kc = 0; kc < n_chunks; ++kc, ++sc) {
                        if ((int)(sc & 1u) == warp) {
                            wait_hot(smem_u32(&c->empty[s]), ph ^ 1, c, a.status, 5u);
                            if (c->abort_flag) { ok = false; break; }
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
        } else if (warp < kMmaWarp + kMmaWarps) {
            // ------------------------------------------------------------ MMA issue (lane 0 issues)
            // One instruction per group; group k of a tile goes to TMEM slot k & 3, and this warp owns slot
            // `me`: per ring stage (four K-steps) it issues step `me`, if the contraction reaches that far.
            const uint32_t me = (uint32_t)(warp - kMmaWarp);
            const uint32_t lane0 = lane == 0 ? 1u : 0u;
            const uint32_t ring_lo = desc_lo(ring_s);
            const uint32_t stage_step = a.stage_bytes >> 4, n_stages = (uint32_t)a.n_stages;
            const uint32_t a_in_stage = resident ? 0u : (uint32_t)(kChunk * (kBlock >> 4));
            const uint32_t full_s = smem_u32(&c->full[0]), empty_s = smem_u32(&c->empty[0]);
            const uint32_t tfull_me = smem_u32(&c->tfull[me]), tempty_me = smem_u32(&c->tempty[me]);
            const uint32_t tm_me = tmem_base + me * kBN, off_me = me * (kBlock >> 4);
            const int n_steps = a.n_steps;
            uint32_t s = 0, ph = 0, ib = 0, iu = 0;
            uint32_t q_me = 1;             // parity to wait for on tempty; a fresh barrier passes parity 1
            for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
                const int part = item % a.n_parts;
                const int n_tiles = part_begin(part + 1) - part_begin(part);
                wait_hot(smem_u32(&c->a_full[ib]), iu, c, a.status, 6u);
                if (c->abort_flag) break;
                const uint32_t ares_lo = desc_lo(ibuf_s + ib * a.ibuf_bytes + a_in_ibuf);
                for (int tl = 0; tl < n_tiles; ++tl) {
                    uint32_t a_lo = ares_lo + off_me;   // resident: walks through the item's A blocks
#pragma unroll 1
                    for (int k0 = 0; k0 < n_steps; k0 += kChunk) {
                        const uint32_t act = (k0 + (int)me < n_steps) ? lane0 : 0u;
                        wait_hot(full_s + s * 8, ph, c, a.status, 4u);
                        const uint32_t b_lo = ring_lo + s * stage_step + off_me;
                        if (k0 + (int)me < n_steps) {
                            wait_hot(tempty_me, q_me, c, a.status, 3u);
                            q_me ^= 1u;
                        }
                        tc_fence_after();
                        mma_issue_if<false>(act, tm_me, resident ? a_lo : b_lo + a_in_stage, b_lo, 0u);
                        mma_commit_if(act, tfull_me);
                        mma_commit_if(lane0, empty_s + s * 8);
                        a_lo += kChunk * (kBlock >> 4);
                        if (++s == n_stages) { s = 0; ph ^= 1; }
                    }
                    if (c->abort_flag) break;
                }
                if (c->abort_flag) break;
                mma_commit_if(lane0, smem_u32(&c->a_empty[ib]));
                if (++ib == (uint32_t)a.n_ibuf) { ib = 0; iu ^= 1; }
            }
        } else if (warp == kStoreWarp) {
            // ------------------------------------------------------------ output stores, channel scales
            // A staged tile is four boxes of 32 columns x 128 rows; the copy engine clips them at the edges of
            // y.  The staging area goes back to the promotion warps when the engine has read it.  The same
            // hand-over carries the next tile's 128 channel scales (times the accumulator's power of two) and
            // biases, which this warp fetches into shared memory while the stores run: phase n of `sfree`
            // says that tile n of this CTA may be staged and that its scales are in place.
            constexpr uint32_t box_bytes = YBF16 ? kBoxBF16 : kBoxF32;
            float* wsb = reinterpret_cast<float*>(smem_raw + (stage_s + a.staging_bytes - sm_s));   // [128] scales, [128] biases
            auto fetch_scales = [&](int nt) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int64_t col = (int64_t)nt * kBN + 32 * i + lane;
                    wsb[32 * i + lane] = col < a.O ? __fmul_rn(__ldg(a.wscale + col), a.out_scale) : 0.f;
                    wsb[128 + 32 * i + lane] = (a.bias && col < a.O) ? __ldg(a.bias + col) : 0.f;
                }
                __syncwarp();
            };
            uint32_t sph = 0;
            bool ok = true;
            if ((int)blockIdx.x < n_items) {
                fetch_scales(part_begin((int)blockIdx.x % a.n_parts));
                mbar_arrive_lane0(&c->sfree, lane);
            }
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int mt = item / a.n_parts, part = item % a.n_parts;
                for (int nt = part_begin(part); nt < part_begin(part + 1) && ok; ++nt) {
                    wait_hot(smem_u32(&c->sfull), sph, c, a.status, 8u);
                    if (c->abort_flag) { ok = false; break; }
                    sph ^= 1u;
                    if (lane == 0) {
                        const int64_t n0 = (int64_t)nt * kBN;
#pragma unroll
                        for (int cb = 0; cb < 4; ++cb)
                            if (n0 + 32 * cb < a.O)
                                tma_store_2d(&ymap, stage_s + (uint32_t)cb * box_bytes, (int32_t)n0 + 32 * cb, mt * kBM);
                        bulk_commit_group();
                    }
                    // the next tile of this CTA, if there is one: its scales go in while the stores run
                    int nnt = nt + 1;
                    bool more = true;
                    if (nnt == part_begin(part + 1)) {
                        const int nitem = item + (int)gridDim.x;
                        more = nitem < n_items;
                        nnt = more ? part_begin(nitem % a.n_parts) : 0;
                    }
                    if (more) fetch_scales(nnt);
                    if (lane == 0) bulk_wait_group_read0();
                    __syncwarp();
                    mbar_arrive_lane0(&c->sfree, lane);
                }
            }
            if (lane == 0) bulk_wait_group0();   // no store may still be reading this CTA's shared memory at exit
        }
    } else {
        setmaxnreg_inc<kRegsP>();
        // ------------------------------------------------------------ promotion + epilogue
        const int pw = warp - kPWarp0;
        const int quarter = warp & 3;                 // TMEM lanes 32 * quarter .. + 31
        const int half = pw >> 2;                     // columns 64 * half .. + 63 of the tile
        const int row = quarter * 32 + lane;
        const int col0 = half * kPCols;
        const uint32_t wsb_s = stage_s + a.staging_bytes;   // [128] channel scales, [128] biases of the current tile
        uint32_t ib = 0, iu = 0;                      // item buffer and its phase
        uint32_t my_scale_s = ibuf_s + (uint32_t)row * 4;   // this row's scales in the current item buffer

        uint64_t yacc[kPCols / 2];     // 64 floats of one output row, packed in pairs
        uint32_t va[32], vb[32];       // landing buffers: columns 0-31 and 32-63 of this thread's share of a slot
#pragma unroll
        for (int q = 0; q < 32; ++q) { va[q] = 0u; vb[q] = 0u; }
        uint32_t p_full[kSlots] = {0u, 0u, 0u, 0u};   // parity of the completion of tfull[s] to wait for next
        uint32_t sf_par = 0u;            // parity to wait for on sfree
        int item = blockIdx.x, mt = 0, nt = 0, nt_end = 0;
        int64_t n0 = 0;
        const uint32_t sfree_s = smem_u32(&c->sfree);

        auto begin_item = [&]() {
            mt = item / a.n_parts;
            const int part = item % a.n_parts;
            nt = part_begin(part);
            nt_end = part_begin(part + 1);
            const uint32_t scales_s = ibuf_s + ib * a.ibuf_bytes, ares_s = scales_s + a_in_ibuf;
            my_scale_s = scales_s + (uint32_t)row * 4;
            if (a.unpack_a) {
                // Packed codes -> operand bytes, straight into the item buffer: thread pt takes row pt / 2 and
                // every second K-step from pt % 2 (a warp reads 32 contiguous bytes of each of 16 rows).
                wait_hot(smem_u32(&c->a_empty[ib]), iu ^ 1, c, a.status, 1u);
                {
                    const int pt = pw * 32 + lane, r = pt >> 1;
                    const int64_t mr = (int64_t)mt * kBM + r;
                    const uint32_t off = (uint32_t)((r >> 3) * 256 + (r & 7) * 16);
                    const uint8_t* src = a.xcodes + mr * a.row_bytes;
#pragma unroll 2
                    for (int ks = pt & 1; ks < a.n_steps; ks += 2) {
                        uint4 p4 = make_uint4(0u, 0u, 0u, 0u);
                        if (mr < a.M) p4 = __ldg(reinterpret_cast<const uint4*>(src + ks * 16));
                        uint4 c0, c1;
                        expand8<false>(p4.x, c0.x, c0.y);
                        expand8<false>(p4.y, c0.z, c0.w);
                        expand8<false>(p4.z, c1.x, c1.y);
                        expand8<false>(p4.w, c1.z, c1.w);
                        const uint32_t dst = ares_s + (uint32_t)ks * kBlock + off;
                        sts128(dst, c0.x, c0.y, c0.z, c0.w);
                        sts128(dst + 128, c1.x, c1.y, c1.z, c1.w);
                    }
                    // scales: [group][128 rows]; thread pt takes row pt % 128 and every second group
                    const int rs = pt & (kBM - 1);
                    const int64_t ms = (int64_t)mt * kBM + rs;
#pragma unroll 1
                    for (int k = pt >> 7; k < a.Kg; k += kPWarps * 32 / kBM)
                        sts32(scales_s + (uint32_t)k * kScaleBlock + (uint32_t)rs * 4,
                              ms < a.M ? __float_as_uint(__ldg(a.xscale + ms * a.Kg + k)) : 0u);
                    // written through the generic proxy, read by the tensor core through the async proxy
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    mbar_arrive_lane0(&c->a_full[ib], lane);
                }
            }
            wait_hot(smem_u32(&c->a_full[ib]), iu, c, a.status, 7u);
        };
        auto begin_tile = [&]() {
            n0 = (int64_t)nt * kBN + col0;
#pragma unroll
            for (int j = 0; j < kPCols / 2; ++j) yacc[j] = 0ull;
        };
        // y = (s_o * 2^18) * sum + bias for the tile that just finished, parked as the source of the bulk
        // tensor stores: box cb = columns 32 cb .. + 31 of all 128 rows, rows of 128 bytes whose 16-byte chunk j
        // sits at j ^ (row & 7) (fp32), or rows of 64 bytes with chunk j at j ^ ((row >> 1) & 3) (bf16).  Then on
        // to the next tile.
        auto finish_tile = [&]() {
            wait_hot(sfree_s, sf_par, c, a.status, 9u);   // the previous tile's stores have read the area
            sf_par ^= 1u;
            {
                // scales of columns 4 i .. 4 i + 3 of the tile at wsb4[i], biases at wsb4[32 + i]
                const float4* wsb4 = reinterpret_cast<const float4*>(smem_raw + (wsb_s - sm_s)) + 16 * half;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {          // one box of 32 columns at a time: all loads first
                    float4 s4[8], b4[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) { s4[j] = wsb4[8 * hh + j]; b4[j] = wsb4[32 + 8 * hh + j]; }
                    if (!YBF16) {
                        const uint32_t row_s = stage_s + (uint32_t)(2 * half + hh) * kBoxF32 + (uint32_t)row * 128u;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float o0, o1, o2, o3;
                            unpack2(yacc[16 * hh + ((2 * j) ^ kAccSwap)], o0, o1);
                            unpack2(yacc[16 * hh + ((2 * j + 1) ^ kAccSwap)], o2, o3);
                            o0 = __fmaf_rn(s4[j].x, o0, b4[j].x);
                            o1 = __fmaf_rn(s4[j].y, o1, b4[j].y);
                            o2 = __fmaf_rn(s4[j].z, o2, b4[j].z);
                            o3 = __fmaf_rn(s4[j].w, o3, b4[j].w);
                            sts128(row_s + (((uint32_t)j ^ ((uint32_t)lane & 7u)) << 4), __float_as_uint(o0), __float_as_uint(o1),
                                   __float_as_uint(o2), __float_as_uint(o3));
                        }
                    } else {
                        const uint32_t row_s = stage_s + (uint32_t)(2 * half + hh) * kBoxBF16 + (uint32_t)row * 64u;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {       // eight columns = one 16-byte chunk of bf16
                            float o[8];
                            unpack2(yacc[16 * hh + ((4 * j) ^ kAccSwap)], o[0], o[1]);
                            unpack2(yacc[16 * hh + ((4 * j + 1) ^ kAccSwap)], o[2], o[3]);
                            unpack2(yacc[16 * hh + ((4 * j + 2) ^ kAccSwap)], o[4], o[5]);
                            unpack2(yacc[16 * hh + ((4 * j + 3) ^ kAccSwap)], o[6], o[7]);
                            const float4 sa = s4[2 * j], sb = s4[2 * j + 1], ba = b4[2 * j], bb = b4[2 * j + 1];
                            sts128(row_s + (((uint32_t)j ^ (((uint32_t)lane >> 1) & 3u)) << 4),
                                   pack16(__fmaf_rn(sa.x, o[0], ba.x), __fmaf_rn(sa.y, o[1], ba.y), a.y_f16),
                                   pack16(__fmaf_rn(sa.z, o[2], ba.z), __fmaf_rn(sa.w, o[3], ba.w), a.y_f16),
                                   pack16(__fmaf_rn(sb.x, o[4], bb.x), __fmaf_rn(sb.y, o[5], bb.y), a.y_f16),
                                   pack16(__fmaf_rn(sb.z, o[6], bb.z), __fmaf_rn(sb.w, o[7], bb.w), a.y_f16));
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes before the engine's reads
                __syncwarp();
                mbar_arrive_lane0(&c->sfull, lane);
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
            if (item < n_items) begin_tile();
        };

        uint32_t tfull_s = smem_u32(&c->tfull[0]), tempty_s = smem_u32(&c->tempty[0]);
        uint32_t tmem_row_r = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)col0;
        // opaque to the compiler: kept in registers instead of being recomputed from the thread index at every use
        asm volatile("" : "+r"(tfull_s), "+r"(tempty_s), "+r"(tmem_row_r));

        // Starts the load of the first half of a tile's first group (slot 0) into va.
        auto first_load = [&]() {
            wait_hot(tfull_s, p_full[0], c, a.status, 2u);
            p_full[0] ^= 1u;
            tc_fence_after();
            tmem_ld32(tmem_row_r, va);
        };
        // One group (slot U) whose first half is on its way into va: start the second half, fold the first in,
        // hand the slot back once the second has landed, start the next group's first half, fold the second in.
        // A barrier test answers only about a hundred clocks after it is issued, and a shared-memory load after
        // about thirty, so both are issued well before their results are needed: the test of the next group's
        // barrier at the top of a group (its answer is looked at after the first half's arithmetic), and the
        // next group's step while the current group's second half is folded in.
        uint32_t dnext = 0u;
        auto group = [&](auto u_tag, uint32_t scale_q, int k, bool prefetch) {
            constexpr uint32_t U = decltype(u_tag)::value, N = (U + 1) & (kSlots - 1);
            const bool next_ready = prefetch ? mbar_test_s(tfull_s + N * 8, p_full[N]) : true;
            const uint64_t d2 = pack2(dnext, dnext);
            tmem_ld_wait_on(va);
            tmem_ld32(tmem_row_r + U * kBN + 32, vb);
            if (DBG) {
                const int64_t m = (int64_t)mt * kBM + row;
                if (a.acc_debug && m < a.M) debug_store<false>(a, va, m, n0, k + (int)U);
            }
#pragma unroll
            for (int q = 0; q < 16; ++q) fma2(yacc[q ^ kAccSwap], pack2(va[2 * q], va[2 * q + 1]), d2);
            tmem_ld_wait_on(vb);
            tc_fence_before();                            // the slot is drained
            __syncwarp();
            mbar_arrive_lane0_s(tempty_s + U * 8, lane);
            if (prefetch) {
                if (!next_ready) wait_cold(tfull_s + N * 8, p_full[N], c, a.status, 2u);
                p_full[N] ^= 1u;
                tc_fence_after();
                tmem_ld32(tmem_row_r + N * kBN, va);
            }
            // the step of the group after this one (past the tile's last group this reads the start of the
            // next region of shared memory; the value is then replaced before it is used)
            dnext = lds32(scale_q + (U + 1) * kScaleBlock);
            if (DBG) {
                const int64_t m = (int64_t)mt * kBM + row;
                if (a.acc_debug && m < a.M) debug_store<false>(a, vb, m, n0 + 32, k + (int)U);
            }
#pragma unroll
            for (int q = 0; q < 16; ++q) fma2(yacc[16 + (q ^ kAccSwap)], pack2(vb[2 * q], vb[2 * q + 1]), d2);
        };
        const std::integral_constant<uint32_t, 0> u0{};
        const std::integral_constant<uint32_t, 1> u1{};
        const std::integral_constant<uint32_t, 2> u2{};
        const std::integral_constant<uint32_t, 3> u3{};

        if (item < n_items) {
            begin_item();
            begin_tile();
            first_load();
#pragma unroll 1
            while (item < n_items && !c->abort_flag) {
                // one tile; the first half of its first group is in flight
                const int Kg = a.Kg;
                uint32_t scale_q = my_scale_s;
                int k = 0;
                dnext = lds32(scale_q);
#pragma unroll 1
                for (; k + 4 < Kg; k += 4, scale_q += 4 * kScaleBlock) {   // four groups, and more behind them
                    group(u0, scale_q, k, true);
                    group(u1, scale_q, k, true);
                    group(u2, scale_q, k, true);
                    group(u3, scale_q, k, true);
                }
                const int rem = Kg - k;                   // the last one to four groups
                group(u0, scale_q, k, rem > 1);
                if (rem > 1) {
                    group(u1, scale_q, k, rem > 2);
                    if (rem > 2) {
                        group(u2, scale_q, k, rem > 3);
                        if (rem > 3) group(u3, scale_q, k, false);
                    }
                }
                // The next tile's first load runs under the epilogue when it belongs to the same work item; the
                // first group of another item cannot start before this warp has handed the item's buffers back.
                const bool same_item = nt + 1 < nt_end;
                if (same_item) first_load();
                finish_tile();
                if (!same_item && item < n_items) first_load();
            }
        }
        tmem_ld_wait_on(va);       // nothing may still be landing when TMEM is released
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

}  // namespace

tdq_status launch_linear_g32(const LinArgs& a, const CUtensorMap& ymap, uint32_t smem_bytes, unsigned grid, bool ybf,
                             bool dbg, cudaStream_t stream) {
    void (*kernel)(LinArgs, CUtensorMap) = nullptr;
    if (!ybf && !dbg) kernel = w4a4_g32_kernel<false, false>;
    if (ybf && !dbg) kernel = w4a4_g32_kernel<true, false>;
    if (!ybf && dbg) kernel = w4a4_g32_kernel<false, true>;
    if (ybf && dbg) kernel = w4a4_g32_kernel<true, true>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess)
        return TDQ_ERR_CUDA;
    if (launch_pdl(kernel, dim3(grid), dim3(kThreadsG32), smem_bytes, stream, a, ymap) != cudaSuccess) return TDQ_ERR_CUDA;
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return TDQ_OK;
}

}  // namespace tdq
