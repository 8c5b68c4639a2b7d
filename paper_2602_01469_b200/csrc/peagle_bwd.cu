// K2: backward of one query partition on sm_100a (dQ, and fp32 accumulation of dK / dV).
//
// Key-tile-outer formulation.  A work item is one key tile (128 keys) of one KV head together
// with the non-skipped query tiles of one aligned chunk of BWD_CQ query tiles; for each of those
// query tiles the item visits the G query heads of the group (one "step" each).  dK and dV of the
// key tile stay in tensor memory for the whole item and are added to the caller's fp32
// accumulators once at its end; dQ of each step is added to an fp32 staging buffer and rounded to
// bf16 by a last kernel.
//
// All score-shaped matrices are held transposed (lanes = keys, columns = query rows) so that the
// probabilities can feed the dV product straight from tensor memory:
//   S^T  = K Q^T,  dP^T = V dO^T
//   P^T  = exp2(scale*log2e*S^T - LSE*log2e), masked entries 0;  dS^T = P^T o (dP^T - Delta)
//   dV  += P^T dO           P^T from tensor memory (bf16, over S^T), dO from shared memory (MN-major)
//   dK  += dS^T Q           Q MN-major
//   dQ   = dS K             dS^T read from shared memory as an MN-major A operand, K MN-major
// Two kernels with the same structure: bwd64_kernel (head_dim 64, below) and bwd128_kernel
// (head_dim 128, peagle_bwd128.cu).
#include <math_constants.h>

#include "peagle_bwd_common.cuh"

namespace peagle {
using namespace sm100;

int make_bf16_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, int D, int H, int T);
int launch_bwd128_main(const CUtensorMap &tmQ, const CUtensorMap &tmdO, const CUtensorMap &tmK,
                       const CUtensorMap &tmV, const CUtensorMap &tmDQ, const BwdParams &P, int n_sm,
                       cudaStream_t s);

// ---------------------------------------------------------------------------------------------
// head_dim 64.  The MMA warp runs one step ahead of the compute warps
// inside a work item:
//   while the compute warps turn S^T(i) into P^T(i):   dK(i-1), dQ(i-1), dP^T(i)
//   while they turn dP^T(i) into dS^T(i):              dV(i), S^T(i+1)
// K and V of the item sit in tensor memory as bf16 (A operands of S^T and dP^T), dS^T goes both
// over the dP^T columns (A operand of dK) and, swizzled, to shared memory (A operand of dQ).
// The K tile of the next item is prefetched into a second shared-memory stage (V has one stage: it
// is only read when it is copied to tensor memory at the start of its item); Q / dO have three
// stages -- with two, a stage is free only when dK of step i has run, and the reload for step i+2
// can arrive late for S^T(i+2) (3.56 -> 3.53 ms on the headline shape, same GPU, alternating runs); the items come from
// a global cursor through a small queue.  512 threads: warps 0-7 compute, warp 8 issues
// MMAs, warp 9 produces, warps 12-15 drain dQ (through a swizzled fp32 tile in shared memory and
// tiled reduce-adds) and, at the end of an item, dK / dV (global reductions from registers).
// The drain has warps of its own because a thread with reductions in flight stalls on its next
// proxy fence, which the compute warps need once per step for the dS^T hand-over.
// Registers per thread after the roles re-split the CTA's allocation (512 threads x 128): two
// warpgroups of compute warps, the warpgroup of the issuing / producing warps, the drain warpgroup.
// The thread that issues the products wants its descriptors resident: with 56 (head_dim 128: 40)
// registers for its warpgroup the compiler spilled them and re-formed them per product, and the
// kernel was 9 (7) per cent slower than with 88.
#ifndef BWD64_COMPUTE_REGS
#define BWD64_COMPUTE_REGS 160
#define BWD64_ISSUE_REGS 88
#define BWD64_DRAIN_REGS 104
#endif
namespace {
constexpr int COMPUTE_REGS = BWD64_COMPUTE_REGS, ISSUE_REGS = BWD64_ISSUE_REGS, DRAIN_REGS = BWD64_DRAIN_REGS;
static_assert(256 * COMPUTE_REGS + 128 * ISSUE_REGS + 128 * DRAIN_REGS <= 512 * 128,
              "the re-split must fit the launch allocation, or setmaxnreg.inc waits for ever");
} // namespace

struct Bwd64Cfg {
    static constexpr int D = 64;
    static constexpr int NSQ = 3;
    static constexpr int TILE_BYTES = 128 * 128;
    static constexpr int OFF_KV = 0;                              // K stage 0, K stage 1, V (one stage)
    static constexpr int OFF_DS = 3 * TILE_BYTES;                 // 2 panels
    static constexpr int OFF_DQ = OFF_DS + 2 * TILE_BYTES;        // fp32 dQ tile on its way out: 2 panels of 32 columns
    static constexpr int OFF_Q = OFF_DQ + 2 * TILE_BYTES;         // ring of (Q, dO)
    static constexpr int OFF_ROW = OFF_Q + NSQ * 2 * TILE_BYTES;  // ring of (-lse2[128], -delta[128], mq[128])
    static constexpr int ROW_BYTES = 3 * 128 * 4;
    static constexpr int OFF_BAR = OFF_ROW + NSQ * ROW_BYTES;
    static constexpr int N_BAR = 2 * NSQ + 13 + 4;  // the last four: work-queue slots
    static constexpr int OFF_MISC = OFF_BAR + N_BAR * 8; // tensor-memory base, abort flag, work queue
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;
    // tensor memory: S^T | dP^T | dQ | K (bf16) | V (bf16) | dK | dV.  P^T (bf16) overwrites the
    // first half of each group's S^T columns and dS^T (bf16) the first half of its dP^T columns.
    static constexpr int TM_S = 0, TM_DP = 128, TM_DQ = 256, TM_K = 320, TM_V = 352, TM_DK = 384,
                         TM_DV = 448;
};

__global__ void __launch_bounds__(512, 1)
bwd64_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmdO,
             const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
             const __grid_constant__ CUtensorMap tmDQ, const BwdParams P)
{
    using C = Bwd64Cfg;
    constexpr int D = 64, NSQ = C::NSQ, TB = C::TILE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sb = (raw + 1023u) & ~1023u;
    uint8_t *sp = smem_raw + (sb - raw);
    const uint32_t bar0 = sb + C::OFF_BAR;
    auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    constexpr int B_QFULL = 0, B_QEMPTY = NSQ, B_KVFULL = 2 * NSQ, B_KVEMPTY = B_KVFULL + 2,
                  B_SFULL = B_KVFULL + 4, B_DPFULL = B_KVFULL + 5, B_PFULL = B_KVFULL + 6,
                  B_DSFULL = B_KVFULL + 7, B_DQFULL = B_KVFULL + 8, B_KVTFULL = B_KVFULL + 9,
                  B_DQEMPTY = B_KVFULL + 10,
                  B_ACCFREE = B_KVFULL + 12;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(sp + C::OFF_MISC);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 4);
    volatile int *wq = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 16);
    constexpr int B_WQ = 2 * NSQ + 13;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < NSQ; ++s) {
            mbar_init(BAR(B_QFULL + s), 1);
            mbar_init(BAR(B_QEMPTY + s), 1);
        }
        for (int s = 0; s < 4; ++s)
            mbar_init(BAR(B_WQ + s), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(BAR(B_KVFULL + s), 1);
            mbar_init(BAR(B_KVEMPTY + s), 1);
            mbar_init(BAR(B_DQFULL + s), s == 0 ? 1 : 256); // [0] dQ done, [1] = B_KVTFULL
            mbar_init(BAR(B_DQEMPTY + s), 128);              // [0] used
        }
        mbar_init(BAR(B_SFULL), 1);
        mbar_init(BAR(B_DPFULL), 1);
        mbar_init(BAR(B_PFULL), 256);
        mbar_init(BAR(B_DSFULL), 256);
        mbar_init(BAR(B_ACCFREE), 128);
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
        // adds a [32 lanes x 64 columns] block of tensor memory, scaled, to fp32 rows in global
        // memory: row_of(lane) gives the destination row pointer or null
        auto drain_block = [&](uint32_t tcol, float f, auto row_ptr, int barrier) {
            uint32_t o[2][32];
            tmem_ld_16x256b_x8(tmem + lane_base + tcol, o[0]);
            tmem_ld_16x256b_x8(tmem + lane_base + (16u << 16) + tcol, o[1]);
            tmem_wait_ld();
            if (barrier >= 0) {
                tc_fence_before();
                mbar_arrive(BAR(barrier));
            }
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float *ra = row_ptr((warp & 3) * 32 + hf * 16 + sub);
                float *rb = row_ptr((warp & 3) * 32 + hf * 16 + sub + 8);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (ra)
                        red_add_v2(ra + 8 * i + cq, __uint_as_float(o[hf][4 * i]) * f,
                                   __uint_as_float(o[hf][4 * i + 1]) * f);
                    if (rb)
                        red_add_v2(rb + 8 * i + cq, __uint_as_float(o[hf][4 * i + 2]) * f,
                                   __uint_as_float(o[hf][4 * i + 3]) * f);
                }
            }
        };
        for (int it = 0; ok && wk.valid; ++it) {
            if (wk.first())
                ktile = P.ktile[wk.kt];
            const int row0 = P.q_begin + wk.qt() * BM;
            const int h = wk.head();
            const bool last = wk.last();
            ok = mbar_wait(BAR(B_DQFULL), it & 1, abort_flag);
            tc_fence_after();
            // dQ(it): tensor memory -> registers -> swizzled fp32 tile in shared memory -> one
            // tiled reduce-add per 32-column panel.  Whole 256-byte rows reach L2 together, which
            // the L2 takes about 1.6 times faster than the same bytes as scattered 32-byte pieces.
            {
                const int rw = (warp & 3) * 32 + lane; // row of the tile = tensor-memory lane
                uint32_t o[2][32];
                tmem_ld32(tmem + lane_base + C::TM_DQ, o[0]);
                tmem_ld32(tmem + lane_base + C::TM_DQ + 32, o[1]);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(BAR(B_DQEMPTY));
                if (threadIdx.x == 384)
                    bulk_wait_group_read<0>(); // the previous tile has left shared memory
                ok = bar_and(3, 128, ok);      // the four warps go on, or leave, together
                if (!ok)
                    break;
#pragma unroll
                for (int pn = 0; pn < 2; ++pn) {
                    uint8_t *dst = sp + C::OFF_DQ + pn * TB + rw * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 v;
                        v.x = __uint_as_float(o[pn][4 * c]) * P.scale;
                        v.y = __uint_as_float(o[pn][4 * c + 1]) * P.scale;
                        v.z = __uint_as_float(o[pn][4 * c + 2]) * P.scale;
                        v.w = __uint_as_float(o[pn][4 * c + 3]) * P.scale;
                        *reinterpret_cast<float4 *>(dst + ((c ^ (rw & 7)) << 4)) = v;
                    }
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 3, 128;" ::: "memory");
                if (threadIdx.x == 384) {
                    // rows past the partition's end are clipped by the tensor map
                    tma_reduce_add_3d(&tmDQ, sb + C::OFF_DQ, 0, h, row0 - P.q_begin);
                    tma_reduce_add_3d(&tmDQ, sb + C::OFF_DQ + TB, 32, h, row0 - P.q_begin);
                    bulk_commit_group();
                }
            }
            if (last) {
                // every MMA of the work item is complete (the barrier above covers them all)
                const int g = wk.g;
                drain_block(C::TM_DK, P.scale,
                            [&](int i) -> float * {
                                return i < ktile.y
                                           ? P.dK_acc + ((size_t)(ktile.x + i) * P.Hkv + g) * D
                                           : nullptr;
                            },
                            -1);
                drain_block(C::TM_DV, 1.f,
                            [&](int i) -> float * {
                                return i < ktile.y
                                           ? P.dV_acc + ((size_t)(ktile.x + i) * P.Hkv + g) * D
                                           : nullptr;
                            },
                            B_ACCFREE);
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
            auto load_kv = [&](int w, int kt, int g) -> bool {
                bool ok = true;
                if (lane == 0) {
                    const int s = w & 1;
                    ok = mbar_wait(BAR(B_KVEMPTY + s), ((w >> 1) & 1) ^ 1, abort_flag) &&
                         (w == 0 || mbar_wait(BAR(B_KVTFULL), (w - 1) & 1, abort_flag));
                    if (ok) {
                        const int start = P.ktile[kt].x;
                        mbar_arrive_expect_tx(BAR(B_KVFULL + s), 2 * TB);
                        tma_load_3d(sb + C::OFF_KV + s * TB, &tmK, BAR(B_KVFULL + s), 0, g, start);
                        tma_load_3d(sb + C::OFF_KV + 2 * TB, &tmV, BAR(B_KVFULL + s), 0, g, start);
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
                    mbar_arrive_expect_tx(BAR(B_QFULL + st), 2 * TB + C::ROW_BYTES);
                    const uint32_t qa = sb + C::OFF_Q + st * 2 * TB;
                    tma_load_3d(qa, &tmQ, BAR(B_QFULL + st), 0, h, row0);
                    tma_load_3d(qa + TB, &tmdO, BAR(B_QFULL + st), 0, h, row0);
                    const uint32_t ra = sb + C::OFF_ROW + st * C::ROW_BYTES;
                    const size_t ri = (size_t)h * P.q_pad + (size_t)wk.qt() * BM;
                    bulk_load(ra, P.nl2 + ri, 512, BAR(B_QFULL + st));
                    bulk_load(ra + 512, P.nd + ri, 512, BAR(B_QFULL + st));
                    bulk_load(ra + 1024, P.mqp + (size_t)wk.qt() * BM, 512, BAR(B_QFULL + st));
                }
                const bool was_last = wk.last();
                wk.next();
                // the next step's Q / dO tiles start towards L2 one step before their stage is free
                if (wk.valid && lane == 0) {
                    tma_prefetch_3d(&tmQ, 0, wk.head(), P.q_begin + wk.qt() * BM);
                    tma_prefetch_3d(&tmdO, 0, wk.head(), P.q_begin + wk.qt() * BM);
                }
                if (was_last && wk.valid)
                    ok = load_kv(wk.w, wk.kt, wk.g); // next item's K / V into the other stage
            }
        } else if (warp == 8) {
            // -------------------------------------------------------- MMA issue: the whole warp
            // walks the steps and waits, its elected lane issues (see elect_one)
            const uint32_t lead = elect_one();
            constexpr uint32_t IDESC_S = idesc_bf16_f32(128, 128, 0, 0);
            constexpr uint32_t IDESC_KV = idesc_bf16_f32(128, D, 0, 1);
            constexpr uint32_t IDESC_DQ = idesc_bf16_f32(128, D, 1, 1);
            // Lower descriptor words (16-byte units).  "k" = K-major operand, "m" = MN-major.
            const uint32_t ds_k = desc_lo_sw128(sb + C::OFF_DS, 16);
            const uint32_t ds_m = desc_lo_sw128(sb + C::OFF_DS, TB);
            const uint32_t kv_k = desc_lo_sw128(sb + C::OFF_KV, 16);
            const uint32_t kv_m = desc_lo_sw128(sb + C::OFF_KV, TB);
            const uint32_t q_k = desc_lo_sw128(sb + C::OFF_Q, 16);
            const uint32_t q_m = desc_lo_sw128(sb + C::OFF_Q, TB);
            constexpr uint32_t TBU = TB >> 4; // one tile in descriptor units
            // S^T = K Q^T and dP^T = V dO^T: kv / q are the stage offsets in descriptor units
            // S^T = K Q^T and dP^T = V dO^T take K / V from tensor memory (one bf16 copy per
            // work item), so only Q / dO stream from shared memory; q = stage offset in units
            auto issue_s = [&](uint32_t q) {
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    if (lead) mma_ts_lo(tmem + C::TM_S, tmem + C::TM_K + k * 8, q_k + q + k * 2, IDESC_S, k > 0);
            };
            auto issue_dp = [&](uint32_t q) {
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    if (lead) mma_ts_lo(tmem + C::TM_DP, tmem + C::TM_V + k * 8, q_k + q + TBU + k * 2, IDESC_S,
                              k > 0);
            };
            // The issuing thread is a serial instruction stream, so it keeps its bookkeeping
            // minimal: per work item only the number of steps (query tiles x heads).
            const int G = P.Hq / P.Hkv;
            bool ok = true;
            int it = 0, w = 0;
            for (;; ++w) {
                // next (work item, KV head) index from the producer's queue
                if (!mbar_wait(BAR(B_WQ + (w & 3)), (w >> 2) & 1, abort_flag))
                    break;
                const int idx = wq[w & 3];
                if (idx < 0)
                    break;
                const int n_cur = P.bitems[idx / P.Hkv].w * G;
                const int ks = w & 1;
                const uint32_t kvo = ks * TBU;
                // K / V of this item are in tensor memory (and its K tile in shared memory)
                ok = mbar_wait(BAR(B_KVTFULL), w & 1, abort_flag) &&
                     mbar_wait(BAR(B_QFULL + it % 3), (it / 3) & 1, abort_flag);
                if (!ok)
                    break;
                tc_fence_after();
                issue_s((it % 3) * 2 * TBU);
                if (lead) tc_commit(BAR(B_SFULL));
                issue_dp((it % 3) * 2 * TBU);
                if (lead) tc_commit(BAR(B_DPFULL));
                for (int i = 0; ok && i < n_cur; ++i, ++it) {
                    const int st = it % 3, nst = (it + 1) % 3;
                    const uint32_t qo = st * 2 * TBU, nqo = nst * 2 * TBU;
                    const bool first = i == 0, last = i == n_cur - 1;
                    // ---- dV(it) once P^T(it) is in tensor memory, then S^T(it+1)
                    ok = mbar_wait(BAR(B_PFULL), it & 1, abort_flag);
                    if (ok && first)
                        ok = mbar_wait(BAR(B_ACCFREE), (w & 1) ^ 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lead) mma_ts_lo(tmem + C::TM_DV, tmem + C::TM_S + (k / 4) * 64 + (k % 4) * 8,
                                  q_m + qo + TBU + k * 128, IDESC_KV, !first || k > 0);
                    if (!last) {
                        ok = mbar_wait(BAR(B_QFULL + nst), ((it + 1) / 3) & 1, abort_flag);
                        if (!ok)
                            break;
                        tc_fence_after();
                        issue_s(nqo);
                        if (lead) tc_commit(BAR(B_SFULL));
                    }
                    // ---- dK(it), dQ(it) once dS^T(it) is in tensor and shared memory, then
                    // dP^T(it+1); the single dQ accumulator must have been read out
                    ok = mbar_wait(BAR(B_DSFULL), it & 1, abort_flag) &&
                         mbar_wait(BAR(B_DQEMPTY), (it & 1) ^ 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lead) mma_ts_lo(tmem + C::TM_DK, tmem + C::TM_DP + (k / 4) * 64 + (k % 4) * 8,
                                  q_m + qo + k * 128, IDESC_KV, !first || k > 0);
                    if (lead) tc_commit(BAR(B_QEMPTY + st)); // dQ reads neither Q nor dO
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lead) mma_ss_lo(tmem + C::TM_DQ, ds_m + k * 128, kv_m + kvo + k * 128, IDESC_DQ,
                                  k > 0);
                    if (lead) tc_commit(BAR(B_DQFULL));
                    if (last) {
                        if (lead) tc_commit(BAR(B_KVEMPTY + ks));
                    } else {
                        issue_dp(nqo);
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
        const int wg = warp >> 2;
        const int r = threadIdx.x & 127; // key lane for S/dP/dK/dV, query row for dQ
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_sel + C::TM_S + wg * 64;
        const uint32_t tDP = tmem + lane_sel + C::TM_DP + wg * 64;
        uint8_t *dsrow = sp + C::OFF_DS + wg * TB + r * 128;
        BwdWalk wk;
        wk.init(P, wq, BAR(B_WQ), abort_flag, false, lane);
        bool ok = true;
        int32_t mk = META_NONE_K;
        for (int it = 0; ok && wk.valid; ++it) {
            const int st = it % NSQ, ph = (it / NSQ) & 1;
            if (wk.first()) {
                const int2 ktile = P.ktile[wk.kt];
                mk = (r < ktile.y) ? P.meta[ktile.x + r] : META_NONE_K;
                // New work item: a bf16 copy of K (group 0) / V (group 1) goes to tensor memory,
                // one row per thread.  Every S^T / dP^T product of the previous item is complete
                // (their results were consumed in its last step), so the old copy is not in use.
                const int ks = wk.w & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_KVFULL + ks), (wk.w >> 1) & 1, abort_flag));
                if (!ok)
                    break;
                const uint8_t *src = sp + C::OFF_KV + (wg == 0 ? ks : 2) * TB + r * 128;
                uint32_t kvw[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(src + ((c ^ (r & 7)) << 4));
                    kvw[4 * c] = v.x;
                    kvw[4 * c + 1] = v.y;
                    kvw[4 * c + 2] = v.z;
                    kvw[4 * c + 3] = v.w;
                }
                tmem_st32(tmem + lane_sel + (wg == 0 ? C::TM_K : C::TM_V), kvw);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(BAR(B_KVTFULL));
            }
            const bool full = wk.full();
            const float *rowbuf = reinterpret_cast<const float *>(sp + C::OFF_ROW + st * C::ROW_BYTES);
            const float4 *nl4 = reinterpret_cast<const float4 *>(rowbuf + wg * 64);
            const float4 *nd4 = reinterpret_cast<const float4 *>(rowbuf + 128 + wg * 64);
            const int4 *mq4 = reinterpret_cast<const int4 *>(rowbuf + 256 + wg * 64);
            // ---- P^T
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_SFULL), it & 1, abort_flag) &&
                                             mbar_wait(BAR(B_QFULL + st), ph, abort_flag));
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
                float a0, a1, a2, a3;
                fma2(a0, a1, __uint_as_float(sr[c >> 5][(c + 0) & 31]),
                     __uint_as_float(sr[c >> 5][(c + 1) & 31]), P.scale_log2, P.scale_log2, l.x, l.y);
                fma2(a2, a3, __uint_as_float(sr[c >> 5][(c + 2) & 31]),
                     __uint_as_float(sr[c >> 5][(c + 3) & 31]), P.scale_log2, P.scale_log2, l.z, l.w);
                p[c + 0] = fast_exp2(a0);
                p[c + 1] = fast_exp2(a1);
                p[c + 2] = fast_exp2(a2);
                p[c + 3] = fast_exp2(a3);
            }
            if (!full) {
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
                    const int4 mq = mq4[c >> 2];
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
            mbar_arrive(BAR(B_PFULL));
            // ---- dS^T
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_DPFULL), it & 1, abort_flag));
            if (!ok)
                break;
            tc_fence_after();
            tmem_ld32(tDP, sr[0]);
            tmem_ld32(tDP + 32, sr[1]);
            tmem_wait_ld();
            tc_fence_before();
            uint4 dsv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { // 16-byte chunk j = query columns 8j .. 8j+7
                const float4 d0 = nd4[2 * j], d1 = nd4[2 * j + 1];
                const int c = 8 * j;
                float t0, t1, t2, t3, t4, t5, t6, t7;
                add2(t0, t1, __uint_as_float(sr[c >> 5][(c + 0) & 31]), __uint_as_float(sr[c >> 5][(c + 1) & 31]), d0.x, d0.y);
                add2(t2, t3, __uint_as_float(sr[c >> 5][(c + 2) & 31]), __uint_as_float(sr[c >> 5][(c + 3) & 31]), d0.z, d0.w);
                add2(t4, t5, __uint_as_float(sr[c >> 5][(c + 4) & 31]), __uint_as_float(sr[c >> 5][(c + 5) & 31]), d1.x, d1.y);
                add2(t6, t7, __uint_as_float(sr[c >> 5][(c + 6) & 31]), __uint_as_float(sr[c >> 5][(c + 7) & 31]), d1.z, d1.w);
                mul2(t0, t1, t0, t1, p[c + 0], p[c + 1]);
                mul2(t2, t3, t2, t3, p[c + 2], p[c + 3]);
                mul2(t4, t5, t4, t5, p[c + 4], p[c + 5]);
                mul2(t6, t7, t6, t7, p[c + 6], p[c + 7]);
                dsv[j].x = pack_bf16x2(t0, t1);
                dsv[j].y = pack_bf16x2(t2, t3);
                dsv[j].z = pack_bf16x2(t4, t5);
                dsv[j].w = pack_bf16x2(t6, t7);
            }
            // the dS^T buffer is free once dK / dQ of the previous iteration have run
            if (it > 0) {
                ok = __all_sync(0xffffffffu,
                                mbar_wait(BAR(B_DQFULL), (it - 1) & 1, abort_flag));
                if (!ok)
                    break;
            }
            {
                // the same dS^T also goes over this group's dP^T columns: operand of dK
                uint32_t pk[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    pk[4 * j] = dsv[j].x;
                    pk[4 * j + 1] = dsv[j].y;
                    pk[4 * j + 2] = dsv[j].z;
                    pk[4 * j + 3] = dsv[j].w;
                }
                tmem_st32(tDP, pk);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4 *>(dsrow + ((j ^ (r & 7)) << 4)) = dsv[j];
            tmem_wait_st();
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(BAR(B_DSFULL));
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

// Per-row inputs of the backward kernels for the q_pad = n_qt * BM rows the query tiles cover:
// -LSE * log2(e), -Delta with Delta[h][r] = <dO[q,h,:], O[q,h,:]>, and the packed metadata, with
// neutral values for the rows past the partition's end.  Also zeroes the fp32 dQ staging.
template <int D>
__global__ void bwd_prepare(const __nv_bfloat16 *__restrict__ O, const __nv_bfloat16 *__restrict__ dO,
                            const float *__restrict__ LSE, const int32_t *__restrict__ meta,
                            float *__restrict__ nl2, float *__restrict__ nd,
                            int32_t *__restrict__ mqp, float *__restrict__ dq_acc, int q_begin,
                            int q_len, int q_pad, int Hq, int T)
{
    constexpr int TPR = D / 8; // threads per (row, head)
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t n = (size_t)q_pad * Hq * TPR;
    const size_t rh = gid / TPR;
    const size_t r = rh / Hq, h = rh % Hq;
    const bool real = gid < n && r < (size_t)q_len;
    float acc = 0.f;
    if (real) {
        const size_t src = (size_t)q_begin * Hq * D + gid * 8;
        const uint4 a = *reinterpret_cast<const uint4 *>(O + src);
        const uint4 b = *reinterpret_cast<const uint4 *>(dO + src);
        const __nv_bfloat162 *pa = reinterpret_cast<const __nv_bfloat162 *>(&a);
        const __nv_bfloat162 *pb = reinterpret_cast<const __nv_bfloat162 *>(&b);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 x = __bfloat1622float2(pa[i]), y = __bfloat1622float2(pb[i]);
            acc += x.x * y.x + x.y * y.y;
        }
        float4 *z = reinterpret_cast<float4 *>(dq_acc + gid * 8);
        z[0] = make_float4(0.f, 0.f, 0.f, 0.f);
        z[1] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int o = TPR / 2; o > 0; o >>= 1)
        acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (gid < n && (gid % TPR) == 0) {
        float l = -CUDART_INF_F;
        int mq = META_NONE_Q;
        if (real) {
            const float lse = LSE[h * (size_t)T + q_begin + r];
            if (lse != -CUDART_INF_F)
                l = -lse * 1.4426950408889634f;
            mq = meta[q_begin + r];
            if (mq == META_NONE_K)
                mq = META_NONE_Q;
        }
        nl2[h * (size_t)q_pad + r] = l;
        nd[h * (size_t)q_pad + r] = real ? -acc : 0.f;
        if (h == 0)
            mqp[r] = mq;
    }
}

__global__ void bwd_finish_dq(const float *__restrict__ dq_acc, __nv_bfloat16 *__restrict__ dQ,
                              size_t n8)
{
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= n8)
        return;
    const float4 a = reinterpret_cast<const float4 *>(dq_acc)[2 * gid];
    const float4 b = reinterpret_cast<const float4 *>(dq_acc)[2 * gid + 1];
    uint4 v;
    v.x = pack_bf16x2(a.x, a.y);
    v.y = pack_bf16x2(a.z, a.w);
    v.z = pack_bf16x2(b.x, b.y);
    v.w = pack_bf16x2(b.z, b.w);
    reinterpret_cast<uint4 *>(dQ)[gid] = v;
}

__global__ void cast_grads_kernel(const float *__restrict__ a, const float *__restrict__ b,
                                  __nv_bfloat16 *__restrict__ oa, __nv_bfloat16 *__restrict__ ob,
                                  size_t n8)
{
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gid >= 2 * n8)
        return;
    const float *src = gid < n8 ? a : b;
    __nv_bfloat16 *dst = gid < n8 ? oa : ob;
    const size_t i = gid < n8 ? gid : gid - n8;
    const float4 x = reinterpret_cast<const float4 *>(src)[2 * i];
    const float4 y = reinterpret_cast<const float4 *>(src)[2 * i + 1];
    uint4 v;
    v.x = pack_bf16x2(x.x, x.y);
    v.y = pack_bf16x2(x.z, x.w);
    v.z = pack_bf16x2(y.x, y.y);
    v.w = pack_bf16x2(y.z, y.w);
    reinterpret_cast<uint4 *>(dst)[i] = v;
}

template <int D>
static int launch_bwd_t(const Plan &p, const BwdArgs &a, EncodeTiledFn enc, int n_sm, cudaStream_t s,
                        cudaEvent_t ev0, cudaEvent_t ev1)
{
    // Q and dO maps end at the partition's last row so that rows past it read as zeros.
    CUtensorMap tmQ, tmdO, tmK, tmV;
    if (make_bf16_map(enc, &tmQ, a.Q, D, a.Hq, p.q_end) || make_bf16_map(enc, &tmdO, a.dO, D, a.Hq, p.q_end) ||
        make_bf16_map(enc, &tmK, a.K, D, a.Hkv, p.T) || make_bf16_map(enc, &tmV, a.V, D, a.Hkv, p.T))
        return PEAGLE_ERR_CUDA;
    const int q_len = p.q_end - p.q_begin;
    const int q_pad = p.n_qt * BM;
    // fp32 dQ staging [q_len][Hq][D] as a tensor for tiled reduce-adds: 32 columns x 128 rows
    CUtensorMap tmDQ;
    {
        cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)a.Hq, (cuuint64_t)q_len};
        cuuint64_t strides[2] = {(cuuint64_t)D * 4, (cuuint64_t)a.Hq * D * 4};
        cuuint32_t box[3] = {32, 1, 128};
        cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&tmDQ, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, a.dq_acc, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PEAGLE_ERR_CUDA;
    }
    const size_t n_prep = (size_t)q_len * a.Hq * (D / 8);
    const size_t n_prep_pad = (size_t)q_pad * a.Hq * (D / 8);
    // Per-row values and the initial dQ staging: with SINGLE tiles, their backward does both.
    int launches = launch_bwd_single(p, a, s);
    if (launches < 0)
        return launches;
    if (launches == 0 && a.rows_ready) {
        // the forward of this partition left the per-row values; only the staging needs clearing
        if (cudaMemsetAsync(a.dq_acc, 0, (size_t)q_len * a.Hq * D * sizeof(float), s) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
    } else if (launches == 0) {
        bwd_prepare<D><<<(unsigned)((n_prep_pad + 255) / 256), 256, 0, s>>>(
            static_cast<const __nv_bfloat16 *>(a.O), static_cast<const __nv_bfloat16 *>(a.dO), a.LSE,
            p.meta, a.nl2, a.nd, a.mqp, a.dq_acc, p.q_begin, q_len, q_pad, a.Hq, p.T);
        launches = 1;
    }
    if (p.n_kt > 0) {
        BwdParams P;
        P.ktile = p.ktile;
        P.bitems = p.bitems;
        P.counters = p.counters;
        P.cursor = p.counters + 2;
        P.meta = p.meta;
        P.status = p.status;
        P.n_qt = p.n_qt;
        P.q_begin = p.q_begin;
        P.q_end = p.q_end;
        P.T = p.T;
        P.nl2 = a.nl2;
        P.nd = a.nd;
        P.mqp = a.mqp;
        P.q_pad = q_pad;
        P.dq_acc = a.dq_acc;
        P.dK_acc = a.dK_acc;
        P.dV_acc = a.dV_acc;
        P.Hq = a.Hq;
        P.Hkv = a.Hkv;
        P.scale = a.scale;
        P.scale_log2 = a.scale * 1.4426950408889634f;
        // per device, so set before every launch (host time only)
        if (D == 64 && cudaFuncSetAttribute(bwd64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            Bwd64Cfg::SMEM_BYTES) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        if (ev0)
            cudaEventRecord(ev0, s);
        if (D == 64)
            bwd64_kernel<<<n_sm, 512, Bwd64Cfg::SMEM_BYTES, s>>>(tmQ, tmdO, tmK, tmV, tmDQ, P);
        else if (launch_bwd128_main(tmQ, tmdO, tmK, tmV, tmDQ, P, n_sm, s) < 0)
            return PEAGLE_ERR_CUDA;
        if (ev1)
            cudaEventRecord(ev1, s);
        ++launches;
    }
    bwd_finish_dq<<<(unsigned)((n_prep + 255) / 256), 256, 0, s>>>(
        a.dq_acc, static_cast<__nv_bfloat16 *>(a.dQ) + (size_t)p.q_begin * a.Hq * D, n_prep);
    return launches + 1;
}

int launch_bwd(const Plan &p, const BwdArgs &a, EncodeTiledFn enc, int n_sm, cudaStream_t s,
               cudaEvent_t ev0, cudaEvent_t ev1)
{
    if (p.n_qt == 0)
        return 0;
    return a.D == 64 ? launch_bwd_t<64>(p, a, enc, n_sm, s, ev0, ev1)
                     : launch_bwd_t<128>(p, a, enc, n_sm, s, ev0, ev1);
}

// One fp32 array of n elements (a multiple of 8) rounded to bf16.
int launch_cast_one(const float *src, void *dst, size_t n, cudaStream_t s)
{
    const size_t n8 = n / 8;
    if (n8 == 0)
        return 0;
    // the kernel takes two arrays of n8 pieces; here both are the one array, and the grid covers it
    // once (threads past n8 in the last block repeat the first pieces with the same values)
    cast_grads_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, s>>>(
        src, src, static_cast<__nv_bfloat16 *>(dst), static_cast<__nv_bfloat16 *>(dst), n8);
    return 1;
}

int launch_cast_grads(const float *dK_acc, const float *dV_acc, void *dK, void *dV, size_t n,
                      cudaStream_t s)
{
    const size_t n8 = n / 8;
    cast_grads_kernel<<<(unsigned)((2 * n8 + 255) / 256), 256, 0, s>>>(
        dK_acc, dV_acc, static_cast<__nv_bfloat16 *>(dK), static_cast<__nv_bfloat16 *>(dV), n8);
    return 1;
}

} // namespace peagle
