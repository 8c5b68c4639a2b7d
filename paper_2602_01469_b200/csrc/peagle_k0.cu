// K0: implicit mask evaluator, tile classifier and scheduler.
//
// The parallel-prediction mask (paper Section 3 / 3.2) is a function of per-token metadata only,
// so it is evaluated from a packed word per token (anchor << 8 | depth) and never stored.  For
// one call (a query partition and the key ranges it may see) these kernels
//   1. pack and validate the metadata and lay out the key tiles of the visible ranges,
//   2. summarise every query tile and key tile (min/max anchor and depth),
//   3. classify every (query tile, key tile) pair as SKIP / PARTIAL / FULL -- from the summaries
//      where they decide, else exactly by evaluating the predicate on the tile,
//   4. compact the non-skipped tiles into per-query-tile key lists, order query tiles
//      longest-first, and cut the backward into (key tile, query-tile chunk) work items.
// Everything runs on the caller's stream; nothing returns to the host.
#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {

__device__ __forceinline__ void set_status(int *status, int err)
{
    atomicCAS(status, 0, err);
}

// ---- 1. pack metadata, build key tiles ---------------------------------------------------
__global__ void k0_prepare(Plan p, const int32_t *__restrict__ anchor,
                           const int32_t *__restrict__ depth, int K, int seq_begin, int seq_end,
                           RangeList ranges)
{
    const int t = seq_begin + blockIdx.x * blockDim.x + threadIdx.x;
    if (t < seq_end) {
        const int a = anchor[t], d = depth[t];
        if (a < 0 || a >= (1 << 23) || d < 0 || d >= K) {
            set_status(p.status, PEAGLE_ERR_BAD_META);
            p.meta[t] = META_NONE_K;
        } else {
            p.meta[t] = (a << 8) | d;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        int kt = 0;
        for (int i = 0; i < ranges.n; ++i)
            for (int b = ranges.begin[i]; b < ranges.end[i]; b += BN, ++kt)
                p.ktile[kt] = make_int2(b, min(BN, ranges.end[i] - b));
        for (int i = 0; i < 8; ++i)
            p.counters[i] = 0;
    }
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.n_qt)
        p.scount[i] = 0;
}

// ---- 2. tile summaries -----------------------------------------------------------------
__global__ void k0_summaries(Plan p)
{
    const int tile = blockIdx.x;
    int b, e;
    int4 *out;
    if (tile < p.n_qt) {
        b = p.q_begin + tile * BM;
        e = min(b + BM, p.q_end);
        out = p.qsum + tile;
    } else {
        const int2 kt = p.ktile[tile - p.n_qt];
        b = kt.x;
        e = kt.x + kt.y;
        out = p.ksum + (tile - p.n_qt);
    }
    int a0 = INT_MAX, a1 = -1, d0 = INT_MAX, d1 = -1;
    const int t = b + threadIdx.x;
    if (t < e) {
        const int m = p.meta[t];
        if (m != META_NONE_K) {
            a0 = a1 = m >> 8;
            d0 = d1 = m & 0xff;
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        a0 = min(a0, __shfl_xor_sync(0xffffffffu, a0, o));
        a1 = max(a1, __shfl_xor_sync(0xffffffffu, a1, o));
        d0 = min(d0, __shfl_xor_sync(0xffffffffu, d0, o));
        d1 = max(d1, __shfl_xor_sync(0xffffffffu, d1, o));
    }
    __shared__ int4 part[4];
    if ((threadIdx.x & 31) == 0)
        part[threadIdx.x >> 5] = make_int4(a0, a1, d0, d1);
    __syncthreads();
    if (threadIdx.x == 0) {
        int4 r = part[0];
        for (int w = 1; w < 4; ++w) {
            r.x = min(r.x, part[w].x);
            r.y = max(r.y, part[w].y);
            r.z = min(r.z, part[w].z);
            r.w = max(r.w, part[w].w);
        }
        *out = r;
    }
}

// ---- 3a. classification from summaries ---------------------------------------------------
__global__ void k0_classify_quick(Plan p)
{
    const int kt = blockIdx.x * blockDim.x + threadIdx.x;
    const int qt = blockIdx.y;
    if (kt >= p.n_kt)
        return;
    const int4 q = p.qsum[qt];
    const int4 k = p.ksum[kt];
    const int len = p.ktile[kt].y;
    int c = -1;
    if (k.y < 0 || q.y < 0) {
        c = TILE_SKIP; // a tile with no valid token
    } else if (k.w == 0) { // every key is a depth-0 (real context) token
        if (k.y <= q.x)
            c = (len == BN) ? TILE_FULL : TILE_PARTIAL;
        else if (k.x > q.y)
            c = TILE_SKIP;
    } else if (k.z >= 1) { // no depth-0 key: only same-anchor, not-deeper chain tokens can match
        if (k.x > q.y || k.y < q.x || k.z > q.w)
            c = TILE_SKIP;
    }
    const size_t idx = (size_t)qt * p.n_kt + kt;
    if (c >= 0) {
        p.cls[idx] = (uint8_t)c;
    } else {
        p.cls[idx] = 255;
        p.undecided[atomicAdd(&p.counters[0], 1)] = (int)idx;
    }
}

// ---- 3b. exact classification of the remaining pairs ------------------------------------
__global__ void k0_classify_exact(Plan p)
{
    __shared__ int mk[BN];
    __shared__ int total, most, slot;
    const int n = p.counters[0];
    for (int w = blockIdx.x; w < n; w += gridDim.x) {
        const int idx = p.undecided[w];
        const int qt = idx / p.n_kt, kt = idx % p.n_kt;
        const int2 ktile = p.ktile[kt];
        const int r0 = p.q_begin + qt * BM, r1 = min(r0 + BM, p.q_end);
        __syncthreads();
        mk[threadIdx.x] = ((int)threadIdx.x < ktile.y) ? p.meta[ktile.x + threadIdx.x] : META_NONE_K;
        if (threadIdx.x == 0) {
            total = 0;
            most = 0;
            slot = -1;
        }
        __syncthreads();
        int mine = 0, col = NO_COL;
        if (r0 + (int)threadIdx.x < r1) {
            const int mq = p.meta[r0 + threadIdx.x];
            if (mq != META_NONE_K)
                for (int c = 0; c < BN; ++c)
                    if (allowed_packed(mq, mk[c])) {
                        ++mine;
                        col = c;
                    }
        }
        int cnt = mine, mx = mine;
        for (int o = 16; o > 0; o >>= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        if ((threadIdx.x & 31) == 0) {
            atomicAdd(&total, cnt);
            atomicMax(&most, mx);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint8_t c = TILE_PARTIAL;
            if (total == 0) {
                c = TILE_SKIP;
            } else if (ktile.y == BN && total == (r1 - r0) * BN) {
                c = TILE_FULL;
            } else if (p.allow_single && most <= 1) {
                const int sl = atomicAdd(&p.scount[qt], 1);
                if (sl < MAX_SINGLE) {
                    c = TILE_SINGLE;
                    slot = sl;
                    p.skt[qt * MAX_SINGLE + sl] = kt;
                }
            }
            p.cls[idx] = c;
        }
        __syncthreads();
        if (slot >= 0)
            p.scol[((size_t)qt * MAX_SINGLE + slot) * BM + threadIdx.x] = (uint8_t)col;
    }
}

// ---- 4a. compact lists -------------------------------------------------------------------
// One block per query tile: its non-skipped key tiles, ascending.
__global__ void k0_lists(Plan p)
{
    __shared__ int warp_cnt[4];
    __shared__ int base;
    const int self = blockIdx.x;
    if (threadIdx.x == 0)
        base = 0;
    __syncthreads();
    for (int o0 = 0; o0 < p.n_kt; o0 += blockDim.x) {
        const int o = o0 + threadIdx.x;
        uint8_t c = TILE_SKIP;
        if (o < p.n_kt)
            c = p.cls[(size_t)self * p.n_kt + o];
        if (c == TILE_SINGLE)
            c = TILE_SKIP; // handled outside the tensor-core lists
        const unsigned bal = __ballot_sync(0xffffffffu, c != TILE_SKIP);
        const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
        if (lane == 0)
            warp_cnt[wid] = __popc(bal);
        __syncthreads();
        int off = base;
        for (int w = 0; w < wid; ++w)
            off += warp_cnt[w];
        off += __popc(bal & ((1u << lane) - 1u));
        if (c != TILE_SKIP) {
            const int2 kt = p.ktile[o];
            p.klist[(size_t)self * p.n_kt + off] = make_int2(kt.x, kt.y | ((int)c << 16));
        }
        __syncthreads();
        if (threadIdx.x == 0)
            base += warp_cnt[0] + warp_cnt[1] + warp_cnt[2] + warp_cnt[3];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        p.kcount[self] = base;
        // SINGLE slots were handed out in arrival order: list them by ascending key tile so that
        // the order of the per-pair sums does not change from run to run
        const int ns = min(p.scount[self], MAX_SINGLE);
        uint8_t ord[MAX_SINGLE];
        for (int i = 0; i < ns; ++i) {
            int j = i;
            const int kt = p.skt[self * MAX_SINGLE + i];
            while (j > 0 && p.skt[self * MAX_SINGLE + ord[j - 1]] > kt) {
                ord[j] = ord[j - 1];
                --j;
            }
            ord[j] = (uint8_t)i;
        }
        for (int i = 0; i < ns; ++i) {
            p.sorder[self * MAX_SINGLE + i] = ord[i];
            p.sbase[self * MAX_SINGLE + i] = p.ktile[p.skt[self * MAX_SINGLE + ord[i]]].x;
        }
    }
    __syncthreads();
    {
        const int ns = min(p.scount[self], MAX_SINGLE);
        for (int i = 0; i < ns; ++i) {
            const int slot = p.sorder[self * MAX_SINGLE + i];
            const int col = p.scol[((size_t)self * MAX_SINGLE + slot) * BM + threadIdx.x];
            p.scs[((size_t)self * MAX_SINGLE + i) * BM + threadIdx.x] = (uint8_t)col;
        }
    }
}

// ---- 4b. order query tiles longest-first ----------------------------------------------------
__global__ void k0_schedule(Plan p)
{
    extern __shared__ int cnt[];
    const int n = p.n_qt;
    if (n <= 8192) {
        for (int i = threadIdx.x; i < n; i += blockDim.x)
            cnt[i] = p.kcount[i];
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int ci = cnt[i];
            int rank = 0;
            for (int j = 0; j < n; ++j)
                rank += (cnt[j] > ci) || (cnt[j] == ci && j < i);
            p.qorder[rank] = i;
        }
    } else {
        for (int i = threadIdx.x; i < n; i += blockDim.x)
            p.qorder[i] = n - 1 - i;
    }
    // Order of the SINGLE-tile backward: query tiles by the first token of their lowest SINGLE
    // key tile (tiles without such entries last).  In the depth-major layout the chain tiles of
    // one block of anchors at depths 1, 2, .. then run one after the other, and the fp32 dK / dV
    // rows they all add to are still in L2 (one trip to memory per key row instead of one per depth).
    __syncthreads();
    if (n <= 8192) {
        for (int i = threadIdx.x; i < n; i += blockDim.x)
            cnt[i] = p.scount[i] > 0 ? p.sbase[i * MAX_SINGLE] : INT_MAX;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int ci = cnt[i];
            int rank = 0;
            for (int j = 0; j < n; ++j)
                rank += (cnt[j] < ci) || (cnt[j] == ci && j < i);
            p.sperm[rank] = i;
        }
    } else {
        for (int i = threadIdx.x; i < n; i += blockDim.x)
            p.sperm[i] = i;
    }
}

// ---- 4c. backward work items ------------------------------------------------------------------
// A backward work item is one key tile together with the non-skipped query tiles of one aligned
// group of BWD_CQ consecutive query tiles ("chunk").  Items are laid out chunk-major so that the
// CTAs running at the same time work on the same few query tiles: their Q / dO rows and their
// fp32 dQ staging rows then stay in L2.
// The items with all BWD_CQ query tiles come first, chunk-major; the smaller ones (the chunks on
// the mask's diagonal) follow in descending size, so that the static round-robin over the CTAs
// ends on small items and the CTAs finish together.
// Pass 1, one block per chunk: for every key tile a 16-bit word (bit b: query tile 8c+b is not
// skipped, bit 8+b: it is FULL), and how many key tiles have 1, 2, .. BWD_CQ query tiles.
__global__ void k0_chunk_masks(Plan p)
{
    __shared__ int hist[BWD_CQ];
    const int c = blockIdx.x;
    if (threadIdx.x < BWD_CQ)
        hist[threadIdx.x] = 0;
    __syncthreads();
    for (int kt = threadIdx.x; kt < p.n_kt; kt += blockDim.x) {
        unsigned m = 0;
        for (int b = 0; b < BWD_CQ; ++b) {
            const int qt = c * BWD_CQ + b;
            if (qt < p.n_qt) {
                const uint8_t cl = p.cls[(size_t)qt * p.n_kt + kt];
                if (cl != TILE_SKIP && cl != TILE_SINGLE)
                    m |= 1u << b;
                if (cl == TILE_FULL)
                    m |= 1u << (8 + b);
            }
        }
        p.cmask[(size_t)c * p.n_kt + kt] = (uint16_t)m;
        if (m != 0)
            atomicAdd(&hist[__popc(m & 0xffu) - 1], 1);
    }
    __syncthreads();
    if (threadIdx.x < BWD_CQ)
        p.ccount[c * BWD_CQ + threadIdx.x] = hist[threadIdx.x];
}

// Pass 2, one block per chunk: the items of the chunk go to their size class's region, behind the
// same-size items of all earlier chunks, key tiles ascending.
// item = (key tile, chunk, mask word, query tiles in the item).
__global__ void k0_chunk_items(Plan p)
{
    __shared__ int warp_cnt[4];
    __shared__ int base[BWD_CQ]; // where this chunk's items of each size start
    __shared__ int cursor;
    const int c = blockIdx.x, n_ch = gridDim.x;
    if (threadIdx.x < BWD_CQ) {
        // sizes in output order: BWD_CQ, BWD_CQ-1, .., 1
        const int sz = threadIdx.x; // index = size - 1
        int off = 0;
        for (int s2 = BWD_CQ - 1; s2 > sz; --s2)
            for (int i = 0; i < n_ch; ++i)
                off += p.ccount[i * BWD_CQ + s2];
        for (int i = 0; i < c; ++i)
            off += p.ccount[i * BWD_CQ + sz];
        base[sz] = off;
        if (c == n_ch - 1 && sz == 0)
            p.counters[1] = off + p.ccount[c * BWD_CQ];
    }
    __syncthreads();
    for (int sz = BWD_CQ - 1; sz >= 0; --sz) {
        if (threadIdx.x == 0)
            cursor = base[sz];
        __syncthreads();
        for (int o0 = 0; o0 < p.n_kt; o0 += blockDim.x) {
            const int kt = o0 + threadIdx.x;
            unsigned m = 0;
            if (kt < p.n_kt)
                m = p.cmask[(size_t)c * p.n_kt + kt];
            const bool mine = m != 0 && __popc(m & 0xffu) == sz + 1;
            const unsigned bal = __ballot_sync(0xffffffffu, mine);
            const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
            if (lane == 0)
                warp_cnt[wid] = __popc(bal);
            __syncthreads();
            int off = cursor;
            for (int w = 0; w < wid; ++w)
                off += warp_cnt[w];
            off += __popc(bal & ((1u << lane) - 1u));
            if (mine)
                p.bitems[off] = make_int4(kt, c, (int)m, sz + 1);
            __syncthreads();
            if (threadIdx.x == 0)
                cursor += warp_cnt[0] + warp_cnt[1] + warp_cnt[2] + warp_cnt[3];
            __syncthreads();
        }
    }
}

// ---- test hook: the mask as the device predicate sees it -----------------------------------
__global__ void k0_mask_dense(Plan p, RangeList ranges, uint8_t *out)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int q = p.q_begin + blockIdx.y;
    if (k >= p.T)
        return;
    bool vis = false;
    for (int i = 0; i < ranges.n; ++i)
        vis |= (k >= ranges.begin[i] && k < ranges.end[i]);
    const int mq = p.meta[q], mk = p.meta[k];
    out[(size_t)blockIdx.y * p.T + k] =
        (uint8_t)(vis && mq != META_NONE_K && allowed_packed(mq, mk));
}

// No visible key: every query tile has an empty list.
__global__ void k0_empty(Plan p)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.n_qt) {
        p.kcount[i] = 0;
        p.qorder[i] = i;
        p.sperm[i] = i;
    }
}

int launch_plan(const Plan &p, const int32_t *anchor, const int32_t *depth, int K, int seq_begin,
                int seq_end, const RangeList &ranges, bool for_bwd, int Hkv, cudaStream_t s)
{
    (void)Hkv;
    const int n_seq = seq_end - seq_begin;
    k0_prepare<<<(n_seq + 255) / 256 > 0 ? (n_seq + 255) / 256 : 1, 256, 0, s>>>(
        p, anchor, depth, K, seq_begin, seq_end, ranges);
    if (p.n_qt == 0)
        return 1;
    if (p.n_kt == 0) {
        k0_empty<<<(p.n_qt + 255) / 256, 256, 0, s>>>(p);
        return 2;
    }
    k0_summaries<<<p.n_qt + p.n_kt, 128, 0, s>>>(p);
    k0_classify_quick<<<dim3((p.n_kt + 127) / 128, p.n_qt), 128, 0, s>>>(p);
    k0_classify_exact<<<592, 128, 0, s>>>(p);
    k0_lists<<<p.n_qt, 128, 0, s>>>(p);
    const int smem = (p.n_qt <= 8192 ? p.n_qt : 0) * (int)sizeof(int);
    k0_schedule<<<1, 1024, smem, s>>>(p);
    if (!for_bwd)
        return 6;
    const int n_ch = (p.n_qt + BWD_CQ - 1) / BWD_CQ;
    k0_chunk_masks<<<n_ch, 128, 0, s>>>(p);
    k0_chunk_items<<<n_ch, 128, 0, s>>>(p);
    return 8;
}

// ---- self-test of the bounded waits ----------------------------------------------------------
// One CTA waits, with the kernels' own mbar_wait, on a barrier that nothing ever arrives at; the
// wait gives up after `limit_ns`, the CTA records PEAGLE_ERR_TIMEOUT exactly as the attention
// kernels do, and returns.  Nothing faults and nothing spins without a limit.
__global__ void k0_wait_expiry(int *status, unsigned long long limit_ns, int *reached_end)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    const uint32_t b = sm100::smem_u32(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        sm100::mbar_init(b, 1);
        sm100::fence_mbar_init();
    }
    __syncthreads();
    // every thread waits; the first to run out of time raises the CTA's abort flag, the others
    // leave on seeing it
    const bool ok = sm100::mbar_wait(b, 0, &abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!ok || abort_flag)
            atomicCAS(status, 0, PEAGLE_ERR_TIMEOUT);
        *reached_end = 1;
    }
}

int launch_wait_expiry(int *status, unsigned long long limit_ns, int *reached_end, cudaStream_t s)
{
    k0_wait_expiry<<<1, 64, 0, s>>>(status, limit_ns, reached_end);
    return 1;
}

int launch_mask_dense(const Plan &p, const RangeList &ranges, uint8_t *out, cudaStream_t s)
{
    const int q_len = p.q_end - p.q_begin;
    if (q_len <= 0)
        return 0;
    k0_mask_dense<<<dim3((p.T + 255) / 256, q_len), 256, 0, s>>>(p, ranges, out);
    return 1;
}

} // namespace peagle
