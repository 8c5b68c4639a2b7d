// K1: forward of one query partition on sm_100a.
//
// A work item is one query tile (128 rows) for two query heads of the same KV group (or one head
// when the group size is odd), so both tiles share the K/V tiles staged in shared memory and the
// same mask.  The kernel is persistent: one CTA per SM (it takes all of tensor memory and of the
// register file) draws items from a global counter, longest query tiles first, and its
// barriers, K / V ring and tensor memory carry on from item to item, so that the loads and the
// first S product of the next item run under the last softmax and the epilogue of the current
// one.  Roles (384 threads):
//   warps 0-3  softmax of tile A (one query row per thread; online softmax in the log2 domain,
//              log-sum-exp bookkeeping, final normalisation and store)
//   warps 4-7  softmax of tile B
//              (head_dim 64: the normalised O tile goes to shared memory and leaves by one tiled
//              store per tile instead of 32 scattered 16-byte pieces per store instruction)
//   warp  8    allocates tensor memory; lane 0 issues the MMAs of tile A
//   warp  10   lane 0 issues the MMAs of tile B
//   warp  9    producer: draws the items; TMA loads of Q per item and of the K / V tiles
//              through a ring, plus the packed metadata of each key tile for the implicit mask
// Tensor memory (512 columns x 128 lanes, fp32): S_A | S_B (128 columns each), O_A | O_B
// (head_dim each) and, for head_dim 64, P_A | P_B (bf16 probabilities, 64 columns each) so that
// S(j+1) is computed while the softmax of S(j) runs; for head_dim 128 tensor memory is full and
// the probabilities overwrite the first 64 columns of their own S.
// S = Q K^T takes both operands from shared memory (K-major, 128-byte swizzle); O += P V takes
// P from tensor memory and V from shared memory (MN-major).
// Only tiles the classifier kept are visited; FULL tiles skip the per-element predicate; SINGLE
// tiles (one allowed key per row) pass through the same ring first and are done pair by pair on
// the CUDA cores, their result seeding the running (m, l, O): O in registers at head_dim 64, in
// tensor memory at head_dim 128.
#include <math_constants.h>

#include <algorithm>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

struct FwdParams {
    const int2 *klist;
    const int *kcount;
    const int *qorder;
    const int32_t *meta;
    int *status;
    int *cursor;  // next work item (zero at launch)
    int n_items;  // query tiles x head blocks
    int n_kt, q_begin, q_end, T;
    __nv_bfloat16 *O;
    float *LSE;
    int Hq, Hkv;
    int two; // 1: two heads per CTA
    float scale_log2;
    // SINGLE tiles (one allowed key per row), handled pair by pair before the tile loop
    const int *scount;
    const uint8_t *scs;  // [n_qt][MAX_SINGLE][BM] key column of entry i for row r, or NO_COL
    const int *sbase;    // [n_qt][MAX_SINGLE] first token of entry i's key tile
    const __nv_bfloat16 *Q, *K, *V;
    // Optional hand-over to the backward of the same partition (the driver knows dO when the
    // forward runs): per (head, row) -LSE * log2(e) and -Delta = -<dO, O>, [Hq][q_pad] each, and
    // the rows' packed metadata [q_pad], neutral values for the rows past the partition's end.
    const __nv_bfloat16 *dO; // null: nothing is handed over
    float *nl2, *nd;
    int32_t *mqp;
    int q_pad;
};

// <a, b> of two rows of 64 bf16 held as 32 packed pairs; products are exact in fp32.
__device__ __forceinline__ float dot64_bf16(const uint32_t (&a)[32], const uint4 *b)
{
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint4 v = b[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc = fmaf(__uint_as_float(a[4 * i + k] << 16), __uint_as_float(w[k] << 16), acc);
            acc = fmaf(__uint_as_float(a[4 * i + k] & 0xffff0000u), __uint_as_float(w[k] & 0xffff0000u), acc);
        }
    }
    return acc;
}

template <int D>
struct FwdCfg {
    static constexpr int NS = (D == 64) ? 3 : 2;
    static constexpr int PANELS = D / 64;
    static constexpr int PANEL_BYTES = 128 * 128; // 128 rows of 128 bytes
    static constexpr int TILE_BYTES = PANELS * PANEL_BYTES;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + NS * TILE_BYTES;
    // head_dim 64: the finished O tiles leave through shared memory and a tiled store (a thread
    // that writes its own row puts 32 separate 16-byte pieces into every store instruction of its
    // warp); head_dim 128 has no room for the two staging tiles and stores its rows directly
    static constexpr bool O_STAGED = (D == 64);
    static constexpr int OFF_OST = OFF_V + NS * TILE_BYTES;
    static constexpr int OFF_META = OFF_OST + (O_STAGED ? 2 * TILE_BYTES : 0);
    static constexpr int OFF_BAR = OFF_META + NS * BN * 4;
    static constexpr int N_BAR = 1 + 4 * NS + 8 + 9;
    static constexpr int OFF_MISC = OFF_BAR + N_BAR * 8; // tmem slot, abort flag, item queue
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024; // + slack for 1024-byte alignment
    static constexpr int TM_S = 0;      // S_A at 0, S_B at 128
    static constexpr int TM_O = 256;    // O_A at 256, O_B at 256 + D
    // head_dim 64 leaves 128 columns for the bf16 probabilities (64 columns per tile), so the next
    // S can be computed while the softmax of the current one runs.  head_dim 128 fills tensor
    // memory with S and O, and P overwrites the first 64 columns of its own S.
    static constexpr bool P_SEPARATE = (D == 64);
    static constexpr int TM_P = P_SEPARATE ? 384 : 0;   // P_A, then P_B at + P_STRIDE
    static constexpr int P_STRIDE = P_SEPARATE ? 64 : 128;
};

template <int D>
__global__ void __launch_bounds__(384, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
           const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
           const FwdParams P)
{
    using C = FwdCfg<D>;
    constexpr int NS = C::NS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sb = (raw + 1023u) & ~1023u;
    uint8_t *sp = smem_raw + (sb - raw);

    const uint32_t bar0 = sb + C::OFF_BAR;
    auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    // barrier indices
    constexpr int B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 1 + NS, B_VFULL = 1 + 2 * NS,
                  B_VEMPTY = 1 + 3 * NS, B_SFULL = 1 + 4 * NS, B_PFULL = B_SFULL + 2,
                  B_PVDONE = B_SFULL + 4, B_SREAD = B_SFULL + 6, B_WQFULL = B_SFULL + 8,
                  B_WQFREE = B_WQFULL + 4, B_QEMPTY = B_WQFREE + 4;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(sp + C::OFF_MISC);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 4);
    volatile int *wq = reinterpret_cast<volatile int *>(sp + C::OFF_MISC + 8); // 4 slots
    int32_t *smeta = reinterpret_cast<int32_t *>(sp + C::OFF_META);

    // The warp index read through a shuffle is a value the compiler knows to be the same in every
    // lane, so what depends on it (tensor-memory addresses, barrier addresses) moves to the uniform
    // datapath.  Measured, not reasoned: head_dim 128 0.508 -> 0.482 ms, head_dim 64 1.82 -> 1.89 ms.
    const int warp = D == 128 ? __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0) : (int)(threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int ntile = P.two ? 2 : 1;
    const int n_hb = P.two ? P.Hq / 2 : P.Hq;
    // Work item w of this CTA = (query tile, head block), handed out by a global counter in the
    // order of the schedule (query tiles with the most key tiles first).  The producer warp draws
    // the index and passes it to the other roles through a four-slot queue in shared memory.
    struct Item {
        int qt, h0, g, row0, cnt, n_single;
        const int2 *klist;
    };
    auto decode = [&](int idx) {
        Item it;
        it.qt = P.qorder[idx / n_hb];
        const int hb = idx % n_hb;
        it.h0 = P.two ? 2 * hb : hb;
        it.g = it.h0 / (P.Hq / P.Hkv);
        it.row0 = P.q_begin + it.qt * BM;
        it.cnt = P.kcount[it.qt];
        it.klist = P.klist + (size_t)it.qt * P.n_kt;
        // the result of the SINGLE entries seeds (m, l, O) of the tile loop
        it.n_single = min(P.scount[it.qt], MAX_SINGLE);
        return it;
    };
    // Roles other than the producer: index of item w, or -1 at the end (or when a wait ran out).
    auto take = [&](int w) {
        const int slot = w & 3;
        return mbar_wait(BAR(B_WQFULL + slot), (w >> 2) & 1, abort_flag) ? wq[slot] : -1;
    };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(BAR(B_QFULL), 1);
        for (int s = 0; s < NS; ++s) {
            mbar_init(BAR(B_KFULL + s), 1);
            mbar_init(BAR(B_KEMPTY + s), P.two ? 2 : 1); // one commit per MMA-issuing thread
            mbar_init(BAR(B_VFULL + s), 1);
            mbar_init(BAR(B_VEMPTY + s), P.two ? 2 : 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(BAR(B_SFULL + x), 1);
            mbar_init(BAR(B_PFULL + x), 4);   // one arrival per softmax warp of the tile
            mbar_init(BAR(B_PVDONE + x), 1);
            mbar_init(BAR(B_SREAD + x), 4);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(BAR(B_WQFULL + i), 1);
            mbar_init(BAR(B_WQFREE + i), 4 * ntile); // one arrival per softmax warp
        }
        // Q may be overwritten once the MMA threads are done with it and every softmax warp has
        // read its rows (or has no use for them)
        mbar_init(BAR(B_QEMPTY), 5 * ntile);
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

    // Warps 8-11 hand most of their registers to the eight softmax warps.
    if (warp >= 8)
        reg_dec<56>();
    if (warp == 9) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
        }
        uint32_t kpos = 0; // position in the K / V ring, running over the items
        bool live = true;
        for (int w = 0; live; ++w) {
            // draw the next item once the queue slot's last reader (four items ago) is done
            const int slot = w & 3;
            int idx = -1;
            if (lane == 0 && mbar_wait(BAR(B_WQFREE + slot), ((w >> 2) & 1) ^ 1, abort_flag)) {
                idx = atomicAdd(P.cursor, 1);
                idx = idx < P.n_items ? idx : -1;
                wq[slot] = idx;
                mbar_arrive(BAR(B_WQFULL + slot));
            }
            idx = __shfl_sync(0xffffffffu, idx, 0);
            if (idx < 0)
                break;
            const Item it = decode(idx);
            const int cnt = it.cnt, n_single = it.n_single, g = it.g;
            const int2 *klist = it.klist;
            if (lane == 0) {
                live = mbar_wait(BAR(B_QEMPTY), (w & 1) ^ 1, abort_flag);
                if (live) {
                    mbar_arrive_expect_tx(BAR(B_QFULL), ntile * C::TILE_BYTES);
                    for (int x = 0; x < ntile; ++x)
                        for (int pn = 0; pn < C::PANELS; ++pn)
                            tma_load_3d(sb + C::OFF_Q + x * C::TILE_BYTES + pn * C::PANEL_BYTES, &tmQ,
                                        BAR(B_QFULL), pn * 64, it.h0 + x, it.row0);
                }
            }
            live = __all_sync(0xffffffffu, live);
            // The key tiles of the SINGLE entries go through the same K / V ring first; the softmax
            // warps read their rows from shared memory.
            for (int i = 0; live && i < n_single; ++i) {
                const uint32_t pos = kpos + i;
                const int st = pos % NS, ph = (pos / NS) & 1;
                const int start = P.sbase[it.qt * MAX_SINGLE + i];
                bool ok = true;
                if (lane == 0) {
                    ok = mbar_wait(BAR(B_KEMPTY + st), ph ^ 1, abort_flag) &&
                         mbar_wait(BAR(B_VEMPTY + st), ph ^ 1, abort_flag);
                    if (ok) {
                        mbar_arrive_expect_tx(BAR(B_KFULL + st), C::TILE_BYTES);
                        mbar_arrive_expect_tx(BAR(B_VFULL + st), C::TILE_BYTES);
                        for (int pn = 0; pn < C::PANELS; ++pn) {
                            tma_load_3d(sb + C::OFF_K + st * C::TILE_BYTES + pn * C::PANEL_BYTES,
                                        &tmK, BAR(B_KFULL + st), pn * 64, g, start);
                            tma_load_3d(sb + C::OFF_V + st * C::TILE_BYTES + pn * C::PANEL_BYTES,
                                        &tmV, BAR(B_VFULL + st), pn * 64, g, start);
                        }
                    }
                }
                live = __all_sync(0xffffffffu, ok);
            }
            // List entries and key metadata are fetched one key tile ahead, so that no global
            // load latency sits between a stage becoming free and its TMA loads.
            auto tile_meta = [&](int2 e, int32_t (&mv)[BN / 32]) {
                const int start = e.x, len = e.y & 0xffff;
                const bool need = (e.y >> 16) != TILE_FULL; // FULL tiles skip the predicate
#pragma unroll
                for (int i = 0; i < BN / 32; ++i) {
                    const int t = lane + 32 * i;
                    mv[i] = (need && t < len) ? P.meta[start + t] : META_NONE_K;
                }
            };
            int2 e_cur = cnt > 0 ? klist[0] : make_int2(0, 0);
            int2 e_nxt = cnt > 1 ? klist[1] : e_cur;
            int32_t m_cur[BN / 32], m_nxt[BN / 32];
            if (cnt > 0)
                tile_meta(e_cur, m_cur);
            for (int j = 0; live && j < cnt; ++j) {
                const uint32_t pos = kpos + n_single + j;
                const int st = pos % NS, ph = (pos / NS) & 1;
                const int start = e_cur.x;
                const int2 e_nn = j + 2 < cnt ? klist[j + 2] : e_nxt;
                if (j + 1 < cnt)
                    tile_meta(e_nxt, m_nxt);
                bool ok = true;
                if (lane == 0) {
                    ok = mbar_wait(BAR(B_KEMPTY + st), ph ^ 1, abort_flag);
                    if (ok) {
                        mbar_arrive_expect_tx(BAR(B_KFULL + st), C::TILE_BYTES);
                        for (int pn = 0; pn < C::PANELS; ++pn)
                            tma_load_3d(sb + C::OFF_K + st * C::TILE_BYTES + pn * C::PANEL_BYTES,
                                        &tmK, BAR(B_KFULL + st), pn * 64, g, start);
                    }
                }
                ok = ok && mbar_wait(BAR(B_VEMPTY + st), ph ^ 1, abort_flag);
                live = __all_sync(0xffffffffu, ok);
                if (!live)
                    break;
#pragma unroll
                for (int i = 0; i < BN / 32; ++i)
                    smeta[st * BN + lane + 32 * i] = m_cur[i];
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_expect_tx(BAR(B_VFULL + st), C::TILE_BYTES);
                    for (int pn = 0; pn < C::PANELS; ++pn)
                        tma_load_3d(sb + C::OFF_V + st * C::TILE_BYTES + pn * C::PANEL_BYTES, &tmV,
                                    BAR(B_VFULL + st), pn * 64, g, start);
                }
                e_cur = e_nxt;
                e_nxt = e_nn;
#pragma unroll
                for (int i = 0; i < BN / 32; ++i)
                    m_cur[i] = m_nxt[i];
            }
            kpos += (uint32_t)(n_single + cnt);
        }
    } else if (warp == 8 || warp == 10) {
        // ------------------------------------------------------------ MMA issue
        // Lane 0 of warp 8 issues every MMA of tile A, lane 0 of warp 10 those of tile B: the two
        // tiles are independent instruction streams (they only share the K / V stages, which are
        // released once both threads have committed), and two threads issue twice as fast as one.
        const int x = (warp - 8) >> 1;
        // the whole warp walks the items and waits, its elected lane issues (see elect_one)
        const uint32_t lead = elect_one();
        if (x < ntile) {
            constexpr uint32_t IDESC_S = idesc_bf16_f32(128, BN, 0, 0);
            constexpr uint32_t IDESC_O = idesc_bf16_f32(128, D, 0, 1);
            constexpr uint32_t TU = C::TILE_BYTES >> 4, PU = C::PANEL_BYTES >> 4;
            // lower descriptor words in 16-byte units (see desc_lo_sw128)
            const uint32_t q_lo = desc_lo_sw128(sb + C::OFF_Q, 16) + x * TU;
            const uint32_t k_lo = desc_lo_sw128(sb + C::OFF_K, 16);
            const uint32_t v_lo = desc_lo_sw128(sb + C::OFF_V, C::PANEL_BYTES);
            const uint32_t tS = tmem + C::TM_S + x * 128, tO = tmem + C::TM_O + x * D;
            const uint32_t tP = tmem + C::TM_P + x * C::P_STRIDE;
            auto issue_s = [&](int st) {
                const uint32_t kb = k_lo + st * TU;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * PU + (k % 4) * 2;
                    if (lead) mma_ss_lo(tS, q_lo + off, kb + off, IDESC_S, k > 0);
                }
                if (lead) tc_commit(BAR(B_SFULL + x));
                if (lead) tc_commit(BAR(B_KEMPTY + st));
            };
            auto issue_pv = [&](int st, bool acc) {
                const uint32_t vb = v_lo + st * TU;
                if (lead) mma_ts_lo(tO, tP, vb, IDESC_O, acc);
#pragma unroll
                for (int k = 1; k < BN / 16; ++k)
                    if (lead) mma_ts_lo(tO, tP + k * 8, vb + k * 128, IDESC_O, 1);
                if (lead) tc_commit(BAR(B_PVDONE + x));
                if (lead) tc_commit(BAR(B_VEMPTY + st));
            };
            uint32_t kpos = 0; // position in the K / V ring, running over the items
            uint32_t t = 0;    // key tiles of this thread's tile so far (phases of S, P, PV)
            bool ok = true;
            for (int w = 0; ok; ++w) {
                const int idx = take(w);
                if (idx < 0)
                    break;
                const Item it = decode(idx);
                const int cnt = it.cnt, n_single = it.n_single;
                ok = mbar_wait(BAR(B_QFULL), w & 1, abort_flag);
                // The SINGLE entries come first in the ring.  Their phases are waited for one by
                // one: a parity wait is only meaningful on the phase that follows the last one
                // seen.
                for (int i = 0; ok && i < n_single; ++i) {
                    const uint32_t pos = kpos + i;
                    ok = mbar_wait(BAR(B_KFULL + pos % NS), (pos / NS) & 1, abort_flag) &&
                         mbar_wait(BAR(B_VFULL + pos % NS), (pos / NS) & 1, abort_flag);
                }
                if (ok && cnt == 0)
                    if (lead) mbar_arrive(BAR(B_QEMPTY)); // no product reads this Q
                if (ok && cnt > 0) {
                    const uint32_t p0 = kpos + n_single;
                    // S of the previous item's last key tile must be in the softmax registers
                    ok = mbar_wait(BAR(B_KFULL + p0 % NS), (p0 / NS) & 1, abort_flag) &&
                         (t == 0 || mbar_wait(BAR(B_SREAD + x), (t - 1) & 1, abort_flag));
                    if (ok) {
                        tc_fence_after();
                        issue_s(p0 % NS);
                        if (cnt == 1)
                            if (lead) tc_commit(BAR(B_QEMPTY));
                    }
                }
                for (int j = 0; ok && j < cnt; ++j) {
                    const uint32_t pos = kpos + n_single + j, tt = t + j;
                    const int st = pos % NS, ph = (pos / NS) & 1;
                    const int nst = (pos + 1) % NS, nph = ((pos + 1) / NS) & 1;
                    const bool more = j + 1 < cnt;
                    if constexpr (C::P_SEPARATE) {
                        // S(j+1) as soon as the softmax warps hold S(j) in registers
                        if (more) {
                            ok = mbar_wait(BAR(B_KFULL + nst), nph, abort_flag) &&
                                 mbar_wait(BAR(B_SREAD + x), tt & 1, abort_flag);
                            if (!ok)
                                break;
                            tc_fence_after();
                            issue_s(nst);
                            if (j + 2 == cnt)
                                if (lead) tc_commit(BAR(B_QEMPTY)); // the item's last product with Q
                        }
                    }
                    ok = mbar_wait(BAR(B_VFULL + st), ph, abort_flag) &&
                         mbar_wait(BAR(B_PFULL + x), tt & 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
                    issue_pv(st, j > 0 || n_single > 0);
                    if constexpr (!C::P_SEPARATE) {
                        // P overwrote S(j): S(j+1) can only follow the P V product that reads it
                        if (more) {
                            ok = mbar_wait(BAR(B_KFULL + nst), nph, abort_flag);
                            if (!ok)
                                break;
                            issue_s(nst);
                            if (j + 2 == cnt)
                                if (lead) tc_commit(BAR(B_QEMPTY));
                        }
                    }
                }
                kpos += (uint32_t)(n_single + cnt);
                t += (uint32_t)cnt;
            }
        }
    } else if (warp < 4 * ntile) {
        reg_inc<224>();
        // ------------------------------------------------------------ softmax of tile x
        const int x = warp >> 2;
        const int r = threadIdx.x & 127;
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_sel + C::TM_S + x * 128;
        const uint32_t tO = tmem + lane_sel + C::TM_O + x * D;
        const uint32_t tP = tmem + lane_sel + C::TM_P + x * C::P_STRIDE;
        uint32_t kpos = 0; // position in the K / V ring, running over the items
        uint32_t t = 0;    // key tiles of this tile so far (phases of S, P, PV)
        bool ok = true;
        for (int w = 0; ok; ++w) {
        const int idx = __shfl_sync(0xffffffffu, take(w), 0);
        __syncwarp();
        if (lane == 0 && idx >= 0)
            mbar_arrive(BAR(B_WQFREE + (w & 3))); // this warp has read the queue slot
        if (idx < 0)
            break;
        const Item it = decode(idx);
        const int qt = it.qt, cnt = it.cnt, n_single = it.n_single;
        const int2 *klist = it.klist;
        const int h = it.h0 + x;
        const int row = it.row0 + r;
        const bool row_ok = row < P.q_end;
        int32_t mq = row_ok ? P.meta[row] : META_NONE_Q;
        if (mq == META_NONE_K)
            mq = META_NONE_Q;
        float m = -CUDART_INF_F, l = 0.f;
        if (P.dO && row_ok) { // the epilogue reads this row of dO
            const __nv_bfloat16 *pre = P.dO + ((size_t)row * P.Hq + h) * D;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pre));
            if (D == 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(pre + 64));
        }
        if (n_single == 0 && lane == 0)
            mbar_arrive(BAR(B_QEMPTY)); // no row of Q is read by this warp
        if constexpr (D == 64) {
            if (n_single > 0) {
                // One allowed key per row and tile: the score and the weighted value on the CUDA
                // cores, rows read from the staged K / V tiles, as an online softmax; the result
                // becomes the starting (m, l, O) of the tile loop.
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QFULL), w & 1, abort_flag));
                float qf[64]; // the row of Q, unpacked once
                {
                    const uint8_t *qrow = sp + C::OFF_Q + x * C::TILE_BYTES + r * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(qrow + ((c ^ (r & 7)) << 4));
                        const uint32_t qw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            qf[8 * c + 2 * k] = __uint_as_float(qw[k] << 16);
                            qf[8 * c + 2 * k + 1] = __uint_as_float(qw[k] & 0xffff0000u);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(BAR(B_QEMPTY)); // this warp's rows of Q are in registers
                float o[64];
#pragma unroll
                for (int i = 0; i < 64; ++i)
                    o[i] = 0.f;
                int col_nxt = P.scs[((size_t)qt * MAX_SINGLE) * BM + r];
                for (int i = 0; ok && i < n_single; ++i) {
                    const uint32_t pos = kpos + i;
                    const int st = pos % NS, ph = (pos / NS) & 1;
                    const int col = col_nxt;
                    if (i + 1 < n_single) // requested one entry ahead of its use
                        col_nxt = P.scs[((size_t)qt * MAX_SINGLE + i + 1) * BM + r];
                    ok = mbar_wait(BAR(B_KFULL + st), ph, abort_flag) &&
                         mbar_wait(BAR(B_VFULL + st), ph, abort_flag);
                    if (ok && col != NO_COL && row_ok) {
                        const uint8_t *krow = sp + C::OFF_K + st * C::TILE_BYTES + col * 128;
                        const uint8_t *vrow = sp + C::OFF_V + st * C::TILE_BYTES + col * 128;
                        float acc4[4] = {0.f, 0.f, 0.f, 0.f}; // four chains of dependent adds
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(krow + ((c ^ (col & 7)) << 4));
                            const uint32_t kw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                acc4[k] = fmaf(qf[8 * c + 2 * k], __uint_as_float(kw[k] << 16), acc4[k]);
                                acc4[k] = fmaf(qf[8 * c + 2 * k + 1], __uint_as_float(kw[k] & 0xffff0000u),
                                               acc4[k]);
                            }
                        }
                        const float s2 = ((acc4[0] + acc4[1]) + (acc4[2] + acc4[3])) * P.scale_log2;
                        // As in the tile loop, the running sums move to a new maximum only when it
                        // grew by more than 2^8 (always for the first key, where m is -inf and
                        // the sums are still zero).
                        if (s2 > m + 8.f) {
                            const float alpha = fast_exp2(m - s2); // 0 for the first key
                            l *= alpha;
#pragma unroll
                            for (int e = 0; e < 64; ++e)
                                o[e] *= alpha;
                            m = s2;
                        }
                        const float pr = fast_exp2(s2 - m);
                        l += pr;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(vrow + ((c ^ (col & 7)) << 4));
                            const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                o[8 * c + 2 * k] = fmaf(pr, __uint_as_float(vw[k] << 16), o[8 * c + 2 * k]);
                                o[8 * c + 2 * k + 1] =
                                    fmaf(pr, __uint_as_float(vw[k] & 0xffff0000u), o[8 * c + 2 * k + 1]);
                            }
                        }
                    }
                    // every thread of this tile's four warps is done with the stage (and the four
                    // warps leave together if a wait ran out)
                    ok = bar_and(1 + x, 128, ok);
                    if (!ok)
                        break;
                    if (r == 0) {
                        mbar_arrive(BAR(B_KEMPTY + st));
                        mbar_arrive(BAR(B_VEMPTY + st));
                    }
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t ov[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        ov[i] = __float_as_uint(o[32 * c + i]);
                    tmem_st32(tO + c * 32, ov);
                }
                tmem_wait_st(); // ordered before the first P V product by the P hand-over below
            }
        } else {
            if (n_single > 0) {
                // head_dim 128: the same pair-by-pair online softmax, but a row of O (128 fp32) does
                // not fit beside the row of Q in registers, so O is kept in tensor memory and
                // updated 32 columns at a time (load, scale and add, store).  Tensor-memory
                // accesses are warp-wide, so rows without a key in an entry take part with
                // weight 0.
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_QFULL), w & 1, abort_flag));
                uint32_t qp[64]; // the row of Q as packed bf16 pairs, panel-major
#pragma unroll
                for (int pn = 0; pn < 2; ++pn) {
                    const uint8_t *qrow = sp + C::OFF_Q + x * C::TILE_BYTES + pn * C::PANEL_BYTES + r * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(qrow + ((c ^ (r & 7)) << 4));
                        qp[32 * pn + 4 * c + 0] = v.x;
                        qp[32 * pn + 4 * c + 1] = v.y;
                        qp[32 * pn + 4 * c + 2] = v.z;
                        qp[32 * pn + 4 * c + 3] = v.w;
                    }
                }
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(BAR(B_QEMPTY)); // this warp's rows of Q are in registers
                int col_nxt = P.scs[((size_t)qt * MAX_SINGLE) * BM + r];
                for (int i = 0; ok && i < n_single; ++i) {
                    const uint32_t pos = kpos + i;
                    const int st = pos % NS, ph = (pos / NS) & 1;
                    const int col = col_nxt;
                    if (i + 1 < n_single) // requested one entry ahead of its use
                        col_nxt = P.scs[((size_t)qt * MAX_SINGLE + i + 1) * BM + r];
                    ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_KFULL + st), ph, abort_flag) &&
                                                     mbar_wait(BAR(B_VFULL + st), ph, abort_flag));
                    if (ok) {
                        const bool have = col != NO_COL && row_ok;
                        const int kc = have ? col : 0;
                        const uint8_t *krow = sp + C::OFF_K + st * C::TILE_BYTES + kc * 128;
                        const uint8_t *vrow = sp + C::OFF_V + st * C::TILE_BYTES + kc * 128;
                        float acc4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int pn = 0; pn < 2; ++pn) {
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                const uint4 v = *reinterpret_cast<const uint4 *>(
                                    krow + pn * C::PANEL_BYTES + ((c ^ (kc & 7)) << 4));
                                const uint32_t kw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const uint32_t qw = qp[32 * pn + 4 * c + k];
                                    acc4[k] = fmaf(__uint_as_float(qw << 16), __uint_as_float(kw[k] << 16), acc4[k]);
                                    acc4[k] = fmaf(__uint_as_float(qw & 0xffff0000u),
                                                   __uint_as_float(kw[k] & 0xffff0000u), acc4[k]);
                                }
                            }
                        }
                        const float s2 = ((acc4[0] + acc4[1]) + (acc4[2] + acc4[3])) * P.scale_log2;
                        float alpha = 1.f, pr = 0.f;
                        if (have) {
                            if (s2 > m + 8.f) { // as in the tile loop; always for the row's first key
                                alpha = fast_exp2(m - s2); // 0 for the first key
                                l *= alpha;
                                m = s2;
                            }
                            pr = fast_exp2(s2 - m);
                            l += pr;
                        }
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) { // columns 32 q4 .. 32 q4 + 31 of O
                            uint32_t ov[32];
                            if (i > 0) {
                                tmem_ld32(tO + q4 * 32, ov);
                                tmem_wait_ld();
                            } else {
#pragma unroll
                                for (int e = 0; e < 32; ++e)
                                    ov[e] = 0u;
                            }
                            const uint8_t *vp = vrow + (q4 >> 1) * C::PANEL_BYTES;
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc) {
                                const int c = (q4 & 1) * 4 + cc;
                                const uint4 v = *reinterpret_cast<const uint4 *>(vp + ((c ^ (kc & 7)) << 4));
                                const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const int e = 8 * cc + 2 * k;
                                    ov[e] = __float_as_uint(fmaf(pr, __uint_as_float(vw[k] << 16),
                                                                 alpha * __uint_as_float(ov[e])));
                                    ov[e + 1] = __float_as_uint(fmaf(pr, __uint_as_float(vw[k] & 0xffff0000u),
                                                                     alpha * __uint_as_float(ov[e + 1])));
                                }
                            }
                            tmem_st32(tO + q4 * 32, ov);
                        }
                        tmem_wait_st(); // before the next entry loads these columns, and ordered before
                                        // the first P V product by the P hand-over below
                    }
                    // every thread of this tile's four warps is done with the stage (and the four
                    // warps leave together if a wait ran out)
                    ok = bar_and(1 + x, 128, ok);
                    if (!ok)
                        break;
                    if (r == 0) {
                        mbar_arrive(BAR(B_KEMPTY + st));
                        mbar_arrive(BAR(B_VEMPTY + st));
                    }
                }
            }
        }
        int cls_nxt = cnt > 0 ? klist[0].y >> 16 : 0;
        for (int j = 0; ok && j < cnt; ++j) {
            const uint32_t pos = kpos + n_single + j, tt = t + j;
            const int st = pos % NS, ph = (pos / NS) & 1;
            const int cls = cls_nxt;
            if (j + 1 < cnt)
                cls_nxt = klist[j + 1].y >> 16; // used one key tile later
            ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_SFULL + x), tt & 1, abort_flag));
            if (!ok)
                break;
            tc_fence_after();
            uint32_t xr[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c)
                tmem_ld32(tS + c * 32, xr[c]);
            tmem_wait_ld();
            // S(j) is in registers: its columns may be overwritten by S(j+1)
            tc_fence_before();
            warp_arrive(BAR(B_SREAD + x));
            if (cls != TILE_FULL) {
                ok = __all_sync(0xffffffffu, mbar_wait(BAR(B_VFULL + st), ph, abort_flag));
                if (!ok)
                    break;
                const int4 *mk4 = reinterpret_cast<const int4 *>(smeta + st * BN);
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const int4 mk = mk4[(c * 32 + i) >> 2];
                        if (!allowed_packed(mq, mk.x)) xr[c][i + 0] = 0xff800000u;
                        if (!allowed_packed(mq, mk.y)) xr[c][i + 1] = 0xff800000u;
                        if (!allowed_packed(mq, mk.z)) xr[c][i + 2] = 0xff800000u;
                        if (!allowed_packed(mq, mk.w)) xr[c][i + 3] = 0xff800000u;
                    }
            }
            float mx4[4]; // four independent chains of three-input maxima
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mx4[c] = -CUDART_INF_F;
#pragma unroll
                for (int i = 0; i < 32; i += 2)
                    mx4[c] = max3(mx4[c], __uint_as_float(xr[c][i]), __uint_as_float(xr[c][i + 1]));
            }
            float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            mx *= P.scale_log2; // scale > 0, so the max commutes with the scaling
            const float m_new = fmaxf(m, mx);
            if (j == 0 && n_single == 0) {
                m = m_new;
            } else {
                // P V of the previous key tile must be done before O or P are touched
                if (j > 0) {
                    ok = __all_sync(0xffffffffu,
                                    mbar_wait(BAR(B_PVDONE + x), (tt - 1) & 1, abort_flag));
                    if (!ok)
                        break;
                    tc_fence_after();
                }
                // Rescale the running output only when the maximum grew by more than 2^8; until
                // then the stale maximum keeps every probability below 256.
                const bool grow = m_new > m + 8.f;
                if (__any_sync(0xffffffffu, grow)) {
                    const float alpha = (m_new == -CUDART_INF_F) ? 1.f : fast_exp2(m - m_new);
                    l *= alpha;
                    m = m_new;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tO + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tO + c * 32, o);
                    }
                    tmem_wait_st();
                }
            }
            const float neg_m = (m == -CUDART_INF_F) ? 0.f : -m;
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int c0 = 2 * i + 64 * c; // columns c0, c0+1 of this row
                    const float p0 = fast_exp2(fmaf(__uint_as_float(xr[c0 >> 5][c0 & 31]),
                                                    P.scale_log2, neg_m));
                    // every fourth exponential goes to the FMA pipe: the two softmax groups
                    // together would otherwise keep the exp2 unit busy for 2,048 clocks a step
                    // (a larger share makes instruction issue the limit instead)
                    const float a1 = fmaf(__uint_as_float(xr[(c0 + 1) >> 5][(c0 + 1) & 31]),
                                          P.scale_log2, neg_m);
                    const float p1 = (i & 1) ? exp2_fma(a1) : fast_exp2(a1);
                    sum += p0 + p1;
                    pk[i] = pack_bf16x2(p0, p1);
                }
                tmem_st32(tP + c * 32, pk);
            }
            l += sum;
            tmem_wait_st();
            tc_fence_before();
            warp_arrive(BAR(B_PFULL + x));
        }
        // ---- epilogue: normalise, store O and LSE
        // Delta of the row needs the row of dO: requested here, ahead of the wait for the last
        // P V product (the row was sent towards L2 when the item began)
        const bool want_delta = P.dO != nullptr && row_ok && (cnt > 0 || n_single > 0);
        uint4 dov[D / 8];
        if (want_delta) {
            const uint4 *src = reinterpret_cast<const uint4 *>(P.dO + ((size_t)row * P.Hq + h) * D);
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                dov[i] = __ldg(src + i);
        } else {
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                dov[i] = make_uint4(0, 0, 0, 0);
        }
        // rows of the padded partition are numbered from its first row
        const size_t hand = (size_t)h * P.q_pad + (size_t)(qt * BM + r);
        if (P.dO && x == 0 && (it.h0 == 0))
            P.mqp[qt * BM + r] = mq;
        if (cnt == 0 && n_single == 0) {
            if (row_ok) {
                uint4 z = make_uint4(0, 0, 0, 0);
                uint4 *dst = reinterpret_cast<uint4 *>(P.O + ((size_t)row * P.Hq + h) * D);
                for (int i = 0; i < D / 8; ++i)
                    dst[i] = z;
                P.LSE[(size_t)h * P.T + row] = -CUDART_INF_F;
            }
            if (P.dO) {
                P.nl2[hand] = -CUDART_INF_F;
                P.nd[hand] = 0.f;
            }
        } else if ([&] {
                       bool fin = __all_sync(0xffffffffu,
                                             ok && (cnt == 0 || mbar_wait(BAR(B_PVDONE + x),
                                                                          (t + cnt - 1) & 1, abort_flag)));
                       if constexpr (C::O_STAGED) {
                           // the four warps of the tile go on together (they meet at a barrier
                           // below); before that, the staging tile of the previous item must
                           // have left shared memory
                           if (r == 0)
                               bulk_wait_group_read<0>();
                           fin = bar_and(1 + x, 128, fin);
                       }
                       return fin;
                   }()) {
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            uint4 *dst = reinterpret_cast<uint4 *>(P.O + ((size_t)row * P.Hq + h) * D);
            float delta = 0.f;
            auto dot8 = [&](const uint4 w, const uint32_t *o8) {
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    delta = fmaf(__uint_as_float(ww[k] << 16), __uint_as_float(o8[2 * k]), delta);
                    delta = fmaf(__uint_as_float(ww[k] & 0xffff0000u), __uint_as_float(o8[2 * k + 1]), delta);
                }
            };
            if constexpr (C::O_STAGED) {
                // rows -> swizzled bf16 tile in shared memory -> one tiled store; the map ends at
                // the partition's last row, so rows past it are not written
                uint8_t *orow = sp + C::OFF_OST + x * C::TILE_BYTES + r * 128;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        dot8(dov[c * 4 + (i >> 3)], o + i);
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[i + 0]) * inv, __uint_as_float(o[i + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
                        const int j = c * 4 + (i >> 3); // 16-byte chunk of the row
                        *reinterpret_cast<uint4 *>(orow + ((j ^ (r & 7)) << 4)) = v;
                    }
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(1 + x) : "memory");
                if (r == 0) {
                    tma_store_3d(&tmO, sb + C::OFF_OST + x * C::TILE_BYTES, 0, h, it.row0);
                    bulk_commit_group();
                }
            } else
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        dot8(dov[c * 4 + (i >> 3)], o + i);
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[i + 0]) * inv, __uint_as_float(o[i + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
                        dst[c * 4 + (i >> 3)] = v;
                    }
                }
            }
            const float lse2 = l > 0.f ? m + log2f(l) : -CUDART_INF_F;
            if (row_ok)
                P.LSE[(size_t)h * P.T + row] = lse2 * 0.6931471805599453f;
            if (P.dO) { // the accumulator is not normalised: Delta = inv * <dO, O_acc>
                P.nl2[hand] = (row_ok && l > 0.f) ? -lse2 : -CUDART_INF_F;
                P.nd[hand] = row_ok ? -delta * inv : 0.f;
            }
        } else {
            ok = false; // a wait ran out
        }
        kpos += (uint32_t)(n_single + cnt);
        t += (uint32_t)cnt;
        } // items
    }

    // ------------------------------------------------------------ teardown
    if (C::O_STAGED && warp < 8 && (threadIdx.x & 127) == 0)
        bulk_wait_group<0>(); // this thread's tile stores are complete
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0)
            atomicCAS(P.status, 0, PEAGLE_ERR_TIMEOUT);
        // give copies and MMAs that may still be in flight time to land before the CTA's
        // shared and tensor memory are released
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

static int make_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, int D, int H, int T)
{
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2};
    cuuint32_t box[3] = {64, 1, 128};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

int make_bf16_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, int D, int H, int T)
{
    return make_map(enc, m, base, D, H, T);
}

template <int D>
static int launch_fwd_t(const Plan &p, const FwdArgs &a, EncodeTiledFn enc, int n_sm,
                        cudaStream_t s, cudaEvent_t ev0, cudaEvent_t ev1)
{
    // the O map ends at the partition's last row: a tiled store does not write past it
    CUtensorMap tmQ, tmK, tmV, tmO;
    if (make_map(enc, &tmQ, a.Q, D, a.Hq, p.T) || make_map(enc, &tmK, a.K, D, a.Hkv, p.T) ||
        make_map(enc, &tmV, a.V, D, a.Hkv, p.T) || make_map(enc, &tmO, a.O, D, a.Hq, p.q_end))
        return PEAGLE_ERR_CUDA;
    FwdParams P;
    P.klist = p.klist;
    P.kcount = p.kcount;
    P.qorder = p.qorder;
    P.meta = p.meta;
    P.status = p.status;
    P.cursor = p.counters + 3;
    P.n_kt = p.n_kt;
    P.q_begin = p.q_begin;
    P.q_end = p.q_end;
    P.T = p.T;
    P.O = static_cast<__nv_bfloat16 *>(a.O);
    P.LSE = a.LSE;
    P.Hq = a.Hq;
    P.Hkv = a.Hkv;
    P.two = ((a.Hq / a.Hkv) % 2 == 0) ? 1 : 0;
    P.scale_log2 = a.scale * 1.4426950408889634f;
    P.scount = p.scount;
    P.scs = p.scs;
    P.sbase = p.sbase;
    P.dO = static_cast<const __nv_bfloat16 *>(a.dO);
    P.nl2 = a.nl2;
    P.nd = a.nd;
    P.mqp = a.mqp;
    P.q_pad = p.n_qt * BM;
    P.Q = static_cast<const __nv_bfloat16 *>(a.Q);
    P.K = static_cast<const __nv_bfloat16 *>(a.K);
    P.V = static_cast<const __nv_bfloat16 *>(a.V);
    // the attribute belongs to the current device's copy of the function: set before every launch
    // (host time only), so that a process that drives several GPUs gets it on each of them
    if (cudaFuncSetAttribute(fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             FwdCfg<D>::SMEM_BYTES) != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    const int n_hb = P.two ? a.Hq / 2 : a.Hq;
    P.n_items = p.n_qt * n_hb;
    if (ev0)
        cudaEventRecord(ev0, s);
    fwd_kernel<D><<<std::min(P.n_items, n_sm), 384, FwdCfg<D>::SMEM_BYTES, s>>>(tmQ, tmK, tmV, tmO, P);
    if (ev1)
        cudaEventRecord(ev1, s);
    return 1;
}

int launch_fwd(const Plan &p, const FwdArgs &a, EncodeTiledFn enc, int n_sm, cudaStream_t s,
               cudaEvent_t ev0, cudaEvent_t ev1)
{
    if (p.n_qt == 0)
        return 0;
    return a.D == 64 ? launch_fwd_t<64>(p, a, enc, n_sm, s, ev0, ev1)
                     : launch_fwd_t<128>(p, a, enc, n_sm, s, ev0, ev1);
}

} // namespace peagle
