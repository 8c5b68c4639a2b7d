// Shared by the backward kernels: launch parameters and the walk over a CTA's work items.
#pragma once
#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {

struct BwdParams {
    const int2 *ktile;
    const int4 *bitems;
    const int *counters;
    int *cursor; // device counter, zero at launch: next (work item, KV head) index to hand out
    const int32_t *meta;
    int *status;
    int n_qt, q_begin, q_end, T;
    const float *nl2, *nd; // [Hq][q_pad] -LSE*log2(e) and -Delta, padded rows (-inf, 0)
    const int32_t *mqp;    // [q_pad] packed metadata of the partition's rows
    int q_pad;             // n_qt * BM
    float *dq_acc;         // [q_len][Hq][D]
    float *dK_acc, *dV_acc;
    int Hq, Hkv;
    float scale, scale_log2;
};

// Walks the (work item, query tile, head) iterations of one CTA in execution order.  Work items
// are handed out dynamically: the producer warp takes the next (item, KV head) index from a global
// cursor and publishes it in a four-slot queue in shared memory; the other roles read it there.
// A CTA that falls behind therefore takes fewer items, and the CTAs running at any time work on a
// contiguous window of the chunk-major item list (their shared Q / dO rows and dQ staging rows
// stay in L2), instead of drifting apart as with a static round-robin.
struct BwdWalk {
    const int4 *bitems;
    int *cursor;
    volatile int *wq;
    volatile int *abort;
    uint32_t wqbar;
    int idx, total, Hkv, G, lane;
    bool fetcher;
    int kt, g, c, w;
    unsigned mask, em;
    int hh;
    bool valid;
    __device__ void load()
    {
        const int slot = w & 3;
        if (fetcher) { // the whole producer warp, convergent
            int v = 0;
            if (lane == 0)
                v = atomicAdd(cursor, 1);
            v = __shfl_sync(0xffffffffu, v, 0);
            idx = v < total ? v : -1;
            if (lane == 0) {
                wq[slot] = idx;
                sm100::mbar_arrive(wqbar + 8u * slot);
            }
        } else {
            // slot w & 3 was last used four items ago; no role is more than two items behind
            idx = sm100::mbar_wait(wqbar + 8u * slot, (w >> 2) & 1, abort) ? wq[slot] : -1;
        }
        valid = idx >= 0;
        if (!valid)
            return;
        const int4 item = bitems[idx / Hkv];
        g = idx % Hkv;
        kt = item.x;
        c = item.y;
        mask = (unsigned)item.z;
        em = mask & 0xffu;
        hh = 0;
    }
    __device__ void init(const BwdParams &P, volatile int *queue, uint32_t queue_bar,
                         volatile int *abort_flag, bool is_fetcher, int lane_id)
    {
        bitems = P.bitems;
        cursor = P.cursor;
        wq = queue;
        wqbar = queue_bar;
        abort = abort_flag;
        fetcher = is_fetcher;
        lane = lane_id;
        Hkv = P.Hkv;
        G = P.Hq / P.Hkv;
        total = P.counters[1] * P.Hkv;
        w = 0;
        load();
    }
    __device__ bool first() const { return hh == 0 && em == (mask & 0xffu); }
    __device__ bool last() const { return hh == G - 1 && (em & (em - 1)) == 0; }
    __device__ int qt() const { return c * BWD_CQ + (__ffs(em) - 1); }
    __device__ bool full() const { return (mask >> (8 + __ffs(em) - 1)) & 1u; }
    __device__ int head() const { return g * G + hh; }
    // (query tile, head) of the step after this one, if it belongs to the same work item
    __device__ bool peek(int &qt_next, int &head_next) const
    {
        if (hh + 1 < G) {
            qt_next = qt();
            head_next = g * G + hh + 1;
            return true;
        }
        const unsigned rest = em & (em - 1);
        if (rest == 0)
            return false;
        qt_next = c * BWD_CQ + (__ffs(rest) - 1);
        head_next = g * G;
        return true;
    }
    __device__ void next()
    {
        if (++hh == G) {
            hh = 0;
            em &= em - 1;
            if (em == 0) {
                ++w;
                load();
            }
        }
    }
};

} // namespace peagle
