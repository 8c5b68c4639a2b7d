// K2 for head_dim 128: the software-pipelined backward (see peagle_bwd.cu for the formulation and
// for the head_dim-64 kernel this one mirrors).  What differs at 128 elements per head:
//   - Tensor memory is full with S^T | dP^T | dK | dV (128 columns each), so K and V stay in shared
//     memory as the A operands of S^T and dP^T, and dQ = dS K is accumulated over the dP^T columns
//     once the compute warps hold dP^T in registers; dP^T of the next step follows when the drain
//     warps have read dQ out.
//   - Shared memory is full with K, V (one stage), the dS^T tile, two stages of Q, ONE stage of dO
//     (its last reader of a step, dV, runs early in the step and its first reader of the next
//     step, dP^T, late, so the reload fits between them) and a 32 KB fp32 tile through which dQ
//     leaves in two halves by tiled reduce-adds (8-byte reductions from registers cost 0.6 of
//     1.65 ms).  -LSE*log2e and -Delta of a step's rows (1 KB) come in with its Q tile; that
//     they fit at all takes the 1 KB usually kept as slack for aligning the tiles, so the kernel
//     requires a 1024-byte aligned base and reports an error otherwise.  Read from global memory
//     (broadcast loads, other rows every step) they cost 16 % of the kernel.  The packed metadata
//     of the rows, needed by the steps that are not FULL, is still read from global memory.
// Roles (512 threads): warps 0-7 compute (a thread owns one key lane and 64 of the 128 query
// columns), warp 8 lane 0 issues the MMAs one step ahead (dV(i), S^T(i+1) while the compute warps
// form dS^T(i); dK(i), dQ(i), then dP^T(i+1) while they form P^T(i+1)), warp 9 produces (TMA),
// warps 12-15 drain dQ per step and dK / dV per work item.
#include <math_constants.h>

#include "peagle_bwd_common.cuh"

namespace peagle {
using namespace sm100;

// Registers per thread after the roles re-split the CTA's allocation (512 threads x 128): two
// warpgroups of compute warps, the warpgroup of the issuing / producing warps, the drain warpgroup.
// The thread that issues the products wants its descriptors resident: with 56 (head_dim 128: 40)
// registers for its warpgroup the compiler spilled them and re-formed them per product, and the
// kernel was 9 (7) per cent slower than with 88.
#ifndef BWD128_COMPUTE_REGS
#define BWD128_COMPUTE_REGS 144
#define BWD128_ISSUE_REGS 88
#define BWD128_DRAIN_REGS 136
#endif
namespace {
constexpr int COMPUTE_REGS = BWD128_COMPUTE_REGS, ISSUE_REGS = BWD128_ISSUE_REGS, DRAIN_REGS = BWD128_DRAIN_REGS;
static_assert(256 * COMPUTE_REGS + 128 * ISSUE_REGS + 128 * DRAIN_REGS <= 512 * 128,
              "the re-split must fit the launch allocation, or setmaxnreg.inc waits for ever");
} // namespace

struct Bwd128Cfg {
    static constexpr int D = 128;
    static constexpr int NSQ = 2;
    static constexpr int PANEL_BYTES = 128 * 128;        // 128 rows x 64 bf16
    static constexpr int TILE_BYTES = 2 * PANEL_BYTES;   // 128 rows x 128 bf16, two panels
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = TILE_BYTES;
    static constexpr int OFF_DS = 2 * TILE_BYTES;                // [key][q 0..63], [key][q 64..127]
    static constexpr int OFF_Q = OFF_DS + TILE_BYTES;            // two stages of Q
    static constexpr int OFF_DO = OFF_Q + NSQ * TILE_BYTES;      // one stage of dO
    static constexpr int OFF_DQ = OFF_DO + TILE_BYTES;           // fp32 dQ half tile on its way out: 2 panels of 32 columns
    static constexpr int OFF_BAR = OFF_DQ + TILE_BYTES;
    static constexpr int N_BAR = 2 * NSQ + 13 + 4;               // the last four: work-queue slots
    static constexpr int OFF_MISC = OFF_BAR + N_BAR * 8;         // tensor-memory base, abort flag, queue
    // per stage of Q: -LSE*log2e and -Delta of the step's 128 query rows (2 x 512 bytes)
    static constexpr int OFF_ROW = (OFF_MISC + 32 + 15) / 16 * 16;
    static constexpr int ROW_BYTES = 1024;
    // No slack for alignment is left: the kernel declares its shared memory 1024-byte aligned and
    // leaves with an error if the base is not.
    static constexpr int SMEM_BYTES = OFF_ROW + NSQ * ROW_BYTES;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
    static constexpr int TM_S = 0, TM_DP = 128, TM_DQ = 128, TM_DK = 256, TM_DV = 384;
};

__global__ void __launch_bounds__(512, 1)
bwd128_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmdO,
              const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ CUtensorMap tmDQ, const BwdParams P)
{
    using C = Bwd128Cfg;
    constexpr int D = 128, NSQ = C::NSQ, TB = C::TILE_BYTES, PB = C::PANEL_BYTES;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t sb = smem_u32(smem_raw);
    uint8_t *sp = smem_raw;
    if (sb & 1023u) { // the swizzled tiles need this alignment; nothing has been set up yet
        if (threadIdx.x == 0)
            atomicCAS(P.status, 0, PEAGLE_ERR_ALIGN);
        return;
    }
    const uint32_t bar0 = sb + C::OFF_BAR;
    auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    constexpr int B_QFULL = 0, B_QEMPTY = NSQ, B_KVFULL = 2 * NSQ, B_KVEMPTY = B_KVFULL + 1,
                  B_SFULL = B_KVFULL + 2, B_DPFULL = B_KVFULL + 3, B_PFULL = B_KVFULL + 4,
                  B_DSFULL = B_KVFULL + 5, B_DQFULL = B_KVFULL + 6, B_DQEMPTY = B_KVFULL + 7,
                  B_ACCFREE = B_KVFULL + 8, B_DOFULL = B_KVFULL + 9, B_DOEMPTY = B_KVFULL + 10,
                  B_WQ = 2 * NSQ + 13;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(sp + C::OFF_MISC);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 4);
    volatile int *wq = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 16);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < NSQ; ++s) {
            mbar_init(BAR(B_QFULL + s), 1);
            mbar_init(BAR(B_QEMPTY + s), 1);
        }
        for (int s = 0; s < 4; ++s)
            mbar_init(BAR(B_WQ + s), 1);
        mbar_init(BAR(B_KVFULL), 1);
        mbar_init(BAR(B_KVEMPTY), 1);
        mbar_init(BAR(B_SFULL), 1);
        mbar_init(BAR(B_DPFULL), 1);
        mbar_init(BAR(B_PFULL), 8);   // one arrival per compute warp
        mbar_init(BAR(B_DSFULL), 8);
        mbar_init(BAR(B_DQFULL), 1);
        mbar_init(BAR(B_DQEMPTY), 4); // one arrival per drain warp
        mbar_init(BAR(B_ACCFREE), 4);
        mbar_init(BAR(B_DOFULL), 1);
        mbar_init(BAR(B_DOEMPTY), 1);
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc(sb + C::OFF_MISC, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp >= 12) {
        // ------------------------------------------------------------ drain (warps 12-15)
        reg_set<DRAIN_REGS, 128>();
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int sub = lane >> 2, cq = 2 * (lane & 3); // row inside a 16-lane load, first column
        BwdWalk wk;
        wk.init(P, wq, BAR(B_WQ), abort_flag, false, lane);
        int2 ktile = make_int2(0, 0);
        bool ok = true;
        // Adds a [32 lanes x 64 columns] block of tensor memory, scaled, to fp32 rows in global
        // memory; row_ptr(lane) gives the destination row or null.  A quad of threads holds 32
        // contiguous bytes of a row, so a reduction instruction covers whole 32-byte sectors.
        auto drain_block = [&](uint32_t tcol, float f, auto row_ptr, int coff, int barrier) {
            uint32_t o[2][32];
            tmem_ld_16x256b_x8(tmem + lane_base + tcol, o[0]);
            tmem_ld_16x256b_x8(tmem + lane_base + (16u << 16) + tcol, o[1]);
            tmem_wait_ld();
            if (barrier >= 0) {
                tc_fence_before();
                warp_arrive(BAR(barrier));
            }
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float *ra = row_ptr((warp & 3) * 32 + hf * 16 + sub);
                float *rb = row_ptr((warp & 3) * 32 + hf * 16 + sub + 8);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (ra)
                        red_add_v2(ra + coff + 8 * i + cq, __uint_as_float(o[hf][4 * i]) * f,
                                   __uint_as_float(o[hf][4 * i + 1]) * f);
                    if (rb)
                        red_add_v2(rb + coff + 8 * i + cq, __uint_as_float(o[hf][4 * i + 2]) * f,
                                   __uint_as_float(o[hf][4 * i + 3]) * f);
                }
            }
        };
        for (int it = 0; ok && wk.valid; ++it) {
            if (wk.first())
                ktile = P.ktile[wk.kt];
            const int row0 = wk.qt() * BM; // row of the partition
            const int h = wk.head();
            const bool last = wk.last();
            const int q_len = P.q_end - P.q_begin;
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_DQFULL), it & 1, abort_flag));
            if (!ok)
                break;
            tc_fence_after();
            // dQ(it), one 64-column half at a time: tensor memory -> registers -> swizzled fp32
            // tile in shared memory -> one tiled reduce-add per 32-column panel (rows past the
            // partition's end are clipped by the tensor map).  The columns are released as soon
            // as the second half is in registers.
            (void)q_len;
            uint32_t o[4][32];
#pragma unroll
            for (int pn = 0; pn < 4; ++pn)
                tmem_ld32(tmem + lane_base + C::TM_DQ + pn * 32, o[pn]);
            tmem_wait_ld();
            tc_fence_before();
            warp_arrive(BAR(B_DQEMPTY));
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                if (!ok)
                    break;
                const int rw = (warp & 3) * 32 + lane; // row of the tile = tensor-memory lane
                if (threadIdx.x == 384)
                    bulk_wait_group_read<0>(); // the previous half has left shared memory
                ok = bar_and(3, 128, ok);      // the four warps go on, or leave, together
                if (!ok)
                    break;
#pragma unroll
                for (int pn = 0; pn < 2; ++pn) {
                    uint8_t *dst = sp + C::OFF_DQ + pn * PB + rw * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 v;
                        v.x = __uint_as_float(o[2 * half + pn][4 * c]) * P.scale;
                        v.y = __uint_as_float(o[2 * half + pn][4 * c + 1]) * P.scale;
                        v.z = __uint_as_float(o[2 * half + pn][4 * c + 2]) * P.scale;
                        v.w = __uint_as_float(o[2 * half + pn][4 * c + 3]) * P.scale;
                        *reinterpret_cast<float4 *>(dst + ((c ^ (rw & 7)) << 4)) = v;
                    }
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 3, 128;" ::: "memory");
                if (threadIdx.x == 384) {
                    tma_reduce_add_3d(&tmDQ, sb + C::OFF_DQ, half * 64, h, row0);
                    tma_reduce_add_3d(&tmDQ, sb + C::OFF_DQ + PB, half * 64 + 32, h, row0);
                    bulk_commit_group();
                }
            }
            if (!ok)
                break;
            if (last) {
                // every MMA of the work item is complete (the barrier above covers them all)
                const int g = wk.g;
                auto k_row = [&](int i) -> float * {
                    return i < ktile.y ? P.dK_acc + ((size_t)(ktile.x + i) * P.Hkv + g) * D : nullptr;
                };
                auto v_row = [&](int i) -> float * {
                    return i < ktile.y ? P.dV_acc + ((size_t)(ktile.x + i) * P.Hkv + g) * D : nullptr;
                };
                drain_block(C::TM_DK, P.scale, k_row, 0, -1);
                drain_block(C::TM_DK + 64, P.scale, k_row, 64, -1);
                drain_block(C::TM_DV, 1.f, v_row, 0, -1);
                drain_block(C::TM_DV + 64, 1.f, v_row, 64, B_ACCFREE);
            }
            wk.next();
        }
        if (threadIdx.x == 384)
            bulk_wait_group<0>();
    } else if (warp >= 8) {
        reg_set<ISSUE_REGS, 128>();
        if (warp == 9) {
            // -------------------------------------------------------- producer
            if (lane == 0) {
                tma_prefetch_desc(&tmQ);
                tma_prefetch_desc(&tmdO);
                tma_prefetch_desc(&tmK);
                tma_prefetch_desc(&tmV);
            }
            BwdWalk wk;
            wk.init(P, wq, BAR(B_WQ), abort_flag, true, lane);
            // K / V have one stage: the next item's tiles are requested once the last product of
            // the current item has read them
            auto load_kv = [&](int w, int kt, int g) -> bool {
                bool ok = true;
                if (lane == 0) {
                    ok = mbar_wait(BAR(B_KVEMPTY), (w & 1) ^ 1, abort_flag);
                    if (ok) {
                        const int start = P.ktile[kt].x;
                        mbar_arrive_expect_tx(BAR(B_KVFULL), 2 * TB);
                        for (int pn = 0; pn < 2; ++pn) {
                            tma_load_3d(sb + C::OFF_K + pn * PB, &tmK, BAR(B_KVFULL), pn * 64, g, start);
                            tma_load_3d(sb + C::OFF_V + pn * PB, &tmV, BAR(B_KVFULL), pn * 64, g, start);
                        }
                    }
                }
                return __all_sync(0xffffffffu, ok);
            };
            bool ok = true;
            if (wk.valid)
                ok = load_kv(0, wk.kt, wk.g);
            for (int it = 0; ok && wk.valid; ++it) {
                const int st = it % NSQ, ph = (it / NSQ) & 1;
                const int row0 = P.q_begin + wk.qt() * BM;
                const int h = wk.head();
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QEMPTY + st), ph ^ 1, abort_flag));
                if (!ok)
                    break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(BAR(B_QFULL + st), TB + C::ROW_BYTES);
                    const uint32_t qa = sb + C::OFF_Q + st * TB;
                    for (int pn = 0; pn < 2; ++pn)
                        tma_load_3d(qa + pn * PB, &tmQ, BAR(B_QFULL + st), pn * 64, h, row0);
                    const uint32_t ra = sb + C::OFF_ROW + st * C::ROW_BYTES;
                    const size_t ri = (size_t)h * P.q_pad + (size_t)wk.qt() * BM;
                    bulk_load(ra, P.nl2 + ri, 512, BAR(B_QFULL + st));
                    bulk_load(ra + 512, P.nd + ri, 512, BAR(B_QFULL + st));
                }
                // dO has one stage: free once dV of the previous step has run
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_DOEMPTY), (it & 1) ^ 1, abort_flag));
                if (!ok)
                    break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(BAR(B_DOFULL), TB);
                    for (int pn = 0; pn < 2; ++pn)
                        tma_load_3d(sb + C::OFF_DO + pn * PB, &tmdO, BAR(B_DOFULL), pn * 64, h, row0);
                }
                const bool was_last = wk.last();
                wk.next();
                if (was_last && wk.valid)
                    ok = load_kv(wk.w, wk.kt, wk.g);
            }
        } else if (warp == 8) {
            // -------------------------------------------------------- MMA issue: the whole warp
            // walks the steps and waits, its elected lane issues (see elect_one)
            const uint32_t lead = elect_one();
            constexpr uint32_t IDESC_S = idesc_bf16_f32(128, 128, 0, 0);
            constexpr uint32_t IDESC_KV = idesc_bf16_f32(128, D, 0, 1);
            constexpr uint32_t IDESC_DQ = idesc_bf16_f32(128, D, 1, 1);
            // Lower descriptor words (16-byte units).  "k" = K-major operand, "m" = MN-major
            // (its second 64-wide panel one PANEL_BYTES further on).
            const uint32_t k_k = desc_lo_sw128(sb + C::OFF_K, 16), k_m = desc_lo_sw128(sb + C::OFF_K, PB);
            const uint32_t v_k = desc_lo_sw128(sb + C::OFF_V, 16);
            const uint32_t ds_k = desc_lo_sw128(sb + C::OFF_DS, 16), ds_m = desc_lo_sw128(sb + C::OFF_DS, PB);
            const uint32_t q_k = desc_lo_sw128(sb + C::OFF_Q, 16), q_m = desc_lo_sw128(sb + C::OFF_Q, PB);
            const uint32_t do_k = desc_lo_sw128(sb + C::OFF_DO, 16), do_m = desc_lo_sw128(sb + C::OFF_DO, PB);
            constexpr uint32_t TBU = TB >> 4, PBU = PB >> 4;
            // slice k of a K-major operand: panel k / 4, 32 bytes per slice inside the 128-byte rows
            auto koff = [](int k) { return (uint32_t)((k / 4) * PBU + (k % 4) * 2); };
            auto issue_s = [&](uint32_t q) { // S^T = K Q^T
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    if (lead) mma_ss_lo(tmem + C::TM_S, k_k + koff(k), q_k + q + koff(k), IDESC_S, k > 0);
            };
            auto issue_dp = [&]() { // dP^T = V dO^T
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    if (lead) mma_ss_lo(tmem + C::TM_DP, v_k + koff(k), do_k + koff(k), IDESC_S, k > 0);
            };
            const int G = P.Hq / P.Hkv;
            bool ok = true;
            int it = 0, w = 0;
            for (;; ++w) {
                if (!mbar_wait(BAR(B_WQ + (w & 3)), (w >> 2) & 1, abort_flag))
                    break;
                const int idx = wq[w & 3];
                if (idx < 0)
                    break;
                const int n_cur = P.bitems[idx / P.Hkv].w * G;
                ok = mbar_wait(BAR(B_KVFULL), w & 1, abort_flag) &&
                     mbar_wait(BAR(B_QFULL + (it & 1)), (it >> 1) & 1, abort_flag) &&
                     mbar_wait(BAR(B_DOFULL), it & 1, abort_flag);
                // dQ of the previous item's last step must have left the dP^T columns
                if (ok && it > 0)
                    ok = mbar_wait(BAR(B_DQEMPTY), (it - 1) & 1, abort_flag);
                if (!ok)
                    break;
                tc_fence_after();
                issue_s((it & 1) * TBU);
                if (lead) tc_commit(BAR(B_SFULL));
                issue_dp();
                if (lead) tc_commit(BAR(B_DPFULL));
                for (int i = 0; ok && i < n_cur; ++i, ++it) {
                    const int st = it & 1, nst = st ^ 1;
                    static_assert(NSQ == 2, "stage = step parity");
                    const uint32_t qo = st * TBU, nqo = nst * TBU;
                    const bool first = i == 0, last = i == n_cur - 1;
                    // ---- dV(it) once P^T(it) is in tensor memory, then S^T(it+1)
                    ok = mbar_wait(BAR(B_PFULL), it & 1, abort_flag);
                    if (ok && first)
                        ok = mbar_wait(BAR(B_ACCFREE), (w & 1) ^ 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k) // query rows 16k..16k+15 of P^T (bf16 over S^T)
                        if (lead) mma_ts_lo(tmem + C::TM_DV, tmem + C::TM_S + (k / 4) * 64 + (k % 4) * 8,
                                  do_m + k * 128, IDESC_KV, !first || k > 0);
                    if (lead) tc_commit(BAR(B_DOEMPTY)); // dV is the step's last product with dO
                    if (!last) {
                        ok = mbar_wait(BAR(B_QFULL + nst), ((it + 1) >> 1) & 1, abort_flag);
                        if (!ok)
                            break;
                        tc_fence_after();
                        issue_s(nqo);
                        if (lead) tc_commit(BAR(B_SFULL));
                    }
                    // ---- dK(it), dQ(it) once dS^T(it) is in shared memory (the compute warps then
                    // hold dP^T(it) in registers: dQ goes over its columns)
                    ok = mbar_wait(BAR(B_DSFULL), it & 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lead) mma_ss_lo(tmem + C::TM_DK, ds_k + koff(k), q_m + qo + k * 128, IDESC_KV,
                                  !first || k > 0);
                    if (lead) tc_commit(BAR(B_QEMPTY + st)); // dQ reads neither Q nor dO
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lead) mma_ss_lo(tmem + C::TM_DQ, ds_m + k * 128, k_m + k * 128, IDESC_DQ, k > 0);
                    if (lead) tc_commit(BAR(B_DQFULL));
                    if (last) {
                        if (lead) tc_commit(BAR(B_KVEMPTY));
                    } else {
                        // ---- dP^T(it+1) over the columns dQ(it) has just left
                        ok = mbar_wait(BAR(B_DQEMPTY), it & 1, abort_flag) &&
                             mbar_wait(BAR(B_DOFULL), (it + 1) & 1, abort_flag);
                        if (!ok)
                            break;
                        tc_fence_after();
                        issue_dp();
                        if (lead) tc_commit(BAR(B_DPFULL));
                    }
                }
                if (!ok)
                    break;
            }
        }
    } else {
        reg_set<COMPUTE_REGS, 128>();
        // ------------------------------------------------------------ compute (warps 0-7)
        const int wg = warp >> 2;        // half of the query columns
        const int r = threadIdx.x & 127; // key lane
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_sel + C::TM_S + wg * 64;
        const uint32_t tDP = tmem + lane_sel + C::TM_DP + wg * 64;
        uint8_t *dsrow = sp + C::OFF_DS + wg * PB + r * 128;
        BwdWalk wk;
        wk.init(P, wq, BAR(B_WQ), abort_flag, false, lane);
        bool ok = true;
        int32_t mk = META_NONE_K;
        for (int it = 0; ok && wk.valid; ++it) {
            if (wk.first()) {
                const int2 ktile = P.ktile[wk.kt];
                mk = (r < ktile.y) ? P.meta[ktile.x + r] : META_NONE_K;
            }
            const bool full = wk.full();
            // per-row values of this step's 64 query columns
            const size_t rb = (size_t)wk.qt() * BM + wg * 64;
            const uint8_t *rowv = sp + C::OFF_ROW + (it % NSQ) * C::ROW_BYTES + wg * 256;
            const float4 *nl4 = reinterpret_cast<const float4 *>(rowv);
            const float4 *nd4 = reinterpret_cast<const float4 *>(rowv + 512);
            const int4 *mq4 = reinterpret_cast<const int4 *>(P.mqp + rb);
            // The metadata of the next query tile is sent towards L1 now (read by the steps that are
            // not FULL; every thread of a column group reads the same 64 values, broadcast loads)
            {
                int qn, hn;
                if (lane < 2 && wk.peek(qn, hn) && qn != wk.qt())
                    asm volatile("prefetch.global.L1 [%0];" ::"l"(P.mqp + (size_t)qn * BM + wg * 64 + lane * 32));
            }
            // ---- P^T (the row values arrive with the step's Q tile)
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_SFULL), it & 1, abort_flag) &&
                                             mbar_wait(BAR(B_QFULL + it % NSQ), (it / NSQ) & 1, abort_flag));
            if (!ok)
                break;
            tc_fence_after();
            uint32_t sr[2][32];
            tmem_ld32(tS, sr[0]);
            tmem_ld32(tS + 32, sr[1]);
            tmem_wait_ld();
            float p[64];
#pragma unroll
            for (int c = 0; c < 64; c += 4) {
                const float4 l = nl4[c >> 2];
                p[c + 0] = fast_exp2(fmaf(__uint_as_float(sr[c >> 5][(c + 0) & 31]), P.scale_log2, l.x));
                p[c + 1] = fast_exp2(fmaf(__uint_as_float(sr[c >> 5][(c + 1) & 31]), P.scale_log2, l.y));
                p[c + 2] = fast_exp2(fmaf(__uint_as_float(sr[c >> 5][(c + 2) & 31]), P.scale_log2, l.z));
                p[c + 3] = fast_exp2(fmaf(__uint_as_float(sr[c >> 5][(c + 3) & 31]), P.scale_log2, l.w));
            }
            if (!full) {
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
                    const int4 mq = __ldg(mq4 + (c >> 2));
                    if (!allowed_packed(mq.x, mk)) p[c + 0] = 0.f;
                    if (!allowed_packed(mq.y, mk)) p[c + 1] = 0.f;
                    if (!allowed_packed(mq.z, mk)) p[c + 2] = 0.f;
                    if (!allowed_packed(mq.w, mk)) p[c + 3] = 0.f;
                }
            }
            {
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    pk[i] = pack_bf16x2(p[2 * i], p[2 * i + 1]);
                tmem_st32(tS, pk); // packed P^T over the first half of this group's S^T columns
            }
            tmem_wait_st();
            tc_fence_before();
            warp_arrive(BAR(B_PFULL));
            // ---- dS^T
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_DPFULL), it & 1, abort_flag));
            if (!ok)
                break;
            tc_fence_after();
            tmem_ld32(tDP, sr[0]);
            tmem_ld32(tDP + 32, sr[1]);
            tmem_wait_ld();
            tc_fence_before();
            // the dS^T tile is free once dK / dQ of the previous step have run
            if (it > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_DQFULL), (it - 1) & 1, abort_flag));
                if (!ok)
                    break;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) { // 16-byte chunk j = query columns 8j .. 8j+7 of this half
                const float4 d0 = nd4[2 * j], d1 = nd4[2 * j + 1];
                const int c = 8 * j;
                uint4 v;
                v.x = pack_bf16x2(p[c + 0] * (__uint_as_float(sr[c >> 5][(c + 0) & 31]) + d0.x),
                                  p[c + 1] * (__uint_as_float(sr[c >> 5][(c + 1) & 31]) + d0.y));
                v.y = pack_bf16x2(p[c + 2] * (__uint_as_float(sr[c >> 5][(c + 2) & 31]) + d0.z),
                                  p[c + 3] * (__uint_as_float(sr[c >> 5][(c + 3) & 31]) + d0.w));
                v.z = pack_bf16x2(p[c + 4] * (__uint_as_float(sr[c >> 5][(c + 4) & 31]) + d1.x),
                                  p[c + 5] * (__uint_as_float(sr[c >> 5][(c + 5) & 31]) + d1.y));
                v.w = pack_bf16x2(p[c + 6] * (__uint_as_float(sr[c >> 5][(c + 6) & 31]) + d1.z),
                                  p[c + 7] * (__uint_as_float(sr[c >> 5][(c + 7) & 31]) + d1.w));
                *reinterpret_cast<uint4 *>(dsrow + ((j ^ (r & 7)) << 4)) = v;
            }
            fence_proxy_async_smem();
            warp_arrive(BAR(B_DSFULL));
            wk.next();
        }
    }

    // ------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0)
            atomicCAS(P.status, 0, PEAGLE_ERR_TIMEOUT);
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) {
        }
        __syncthreads();
    }
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

int launch_bwd128_main(const CUtensorMap &tmQ, const CUtensorMap &tmdO, const CUtensorMap &tmK,
                       const CUtensorMap &tmV, const CUtensorMap &tmDQ, const BwdParams &P, int n_sm,
                       cudaStream_t s)
{
    // per device, so set before every launch (host time only)
    if (cudaFuncSetAttribute(bwd128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Bwd128Cfg::SMEM_BYTES) != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    bwd128_kernel<<<n_sm, 512, Bwd128Cfg::SMEM_BYTES, s>>>(tmQ, tmdO, tmK, tmV, tmDQ, P);
    return 1;
}

} // namespace peagle
