// Backward of the SINGLE tiles (head_dim 64 and 128): tiles in which every query row allows at most one
// key, such as the chain tiles of the depth-major layout.  On the tensor cores such a tile costs a
// full 128 x 128 step for 128 useful pairs, so the pairs are done one by one on the CUDA cores.
// For a pair (query row q of head h, key k of its KV head), with the forward's LSE and
// Delta = <dO, O> (Section 3.2's backward, same formulas as the tile kernel):
//   s = <Q[q,h], K[k]>,  p = exp(scale * s - LSE),  dp = <dO[q,h], V[k]>,  ds = p * (dp - Delta)
//   dQ[q,h] += scale * ds * K[k]      dK[k] += scale * ds * Q[q,h]      dV[k] += p * dO[q,h]
// One kernel, query-major so that no reverse (key -> queries) list is needed: eight lanes per
// (query row, KV head) hold 8 elements of every 64 of the row each; for every head of the group they form the
// row's dQ and add into per-key dK / dV sums kept in registers across the heads (one fp32 add per
// key row at the end).  The kernel runs before the tile kernel and doubles as its preparation
// pass: it reads O and LSE as well, writes -LSE * log2(e), -Delta and the packed metadata of
// every row, and its dQ becomes the initial value of the fp32 staging row (plain stores; zero for
// a row without SINGLE keys), so the staging is never cleared or re-read for these pairs.
#include <math_constants.h>

#include <algorithm>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

struct SingleParams {
    const int *scount;
    const uint8_t *scs;  // [n_qt][MAX_SINGLE][BM] key column of entry i for row r, or NO_COL
    const int *sbase;    // [n_qt][MAX_SINGLE] first token of entry i's key tile
    const int *sperm;    // [n_qt] order in which the blocks take the query tiles
    const __nv_bfloat16 *Q, *K, *V, *O, *dO;
    const float *LSE;      // [Hq][T]
    const int32_t *meta;   // [T] packed metadata
    float *nl2, *nd;       // [Hq][q_pad], written here
    int32_t *mqp;          // [q_pad], written here
    float *dq_acc, *dK_acc, *dV_acc;
    int *status;
    int q_begin, q_end, q_pad, n_qt, Hq, Hkv, T, rows_per_block;
    int rows_ready; // 1: nl2 / nd / mqp were already written by the forward (O and LSE are not read)
    float scale, scale_log2;
};

// A row of D bf16 is spread over 8 consecutive lanes: lane `sub` holds, for each 64-element panel c
// of the row, the 8 elements 64 c + 8 sub .. + 7 (one 16-byte load per panel), so that a warp reads
// four whole rows with every load and dot products finish with three shuffles.
template <int CH>
struct Chunk {
    float v[8 * CH];
};
template <int CH>
__device__ __forceinline__ Chunk<CH> unpack_chunk(const uint4 (&t)[CH])
{
    Chunk<CH> c;
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        const uint32_t w[4] = {t[j].x, t[j].y, t[j].z, t[j].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            c.v[8 * j + 2 * i] = __uint_as_float(w[i] << 16);
            c.v[8 * j + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    return c;
}
template <int CH>
__device__ __forceinline__ Chunk<CH> load_chunk(const __nv_bfloat16 *row, int sub)
{
    uint4 t[CH];
#pragma unroll
    for (int j = 0; j < CH; ++j)
        t[j] = reinterpret_cast<const uint4 *>(row)[sub + 8 * j];
    return unpack_chunk<CH>(t);
}
// adds this lane's pieces of a row (dst = the row's first element) scaled by f
template <int CH>
__device__ __forceinline__ void red_chunk(float *dst, int sub, const float (&x)[8 * CH], float f)
{
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        float *d = dst + 64 * j + 8 * sub;
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(d), "f"(x[8 * j] * f),
                     "f"(x[8 * j + 1] * f), "f"(x[8 * j + 2] * f), "f"(x[8 * j + 3] * f)
                     : "memory");
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(d + 4), "f"(x[8 * j + 4] * f),
                     "f"(x[8 * j + 5] * f), "f"(x[8 * j + 6] * f), "f"(x[8 * j + 7] * f)
                     : "memory");
    }
}

// Block = RB rows of the padded partition x all KV heads; unit (row, KV head g) = 8 lanes.  The
// rows of Q, dO and O (all heads of a row are contiguous) come in by bulk copies, so that the
// memory system sees the block's whole input at once instead of one 16-byte load per lane and
// head; the arithmetic then reads shared memory.  The kernel runs before the tile kernel and
// also prepares what that kernel needs per (row, head), unless the forward already left it:
// -LSE * log2(e), -Delta = -<dO, O>, the row's packed metadata; and always the initial value of
// the fp32 dQ staging row, which is this kernel's own contribution (zero for a row without SINGLE
// keys), written with plain stores.  Keys are taken KEYS at a time so that their dK / dV sums fit
// in registers; a row with more than KEYS keys adds its later groups with reductions.
template <int D, bool FIRST, int KEYS>
__device__ __forceinline__ void single_pass(const SingleParams &P, int i0, int ns, int sub, unsigned um,
                                            int r, int g, int qt, int rr, int G,
                                            const __nv_bfloat16 *sq, const __nv_bfloat16 *sdo,
                                            const __nv_bfloat16 *so, float *snl2, float *snd)
{
    int tok[KEYS];
    bool any = false;
#pragma unroll
    for (int i = 0; i < KEYS; ++i) {
        tok[i] = -1;
        if (i0 + i < ns) {
            const int col = P.scs[((size_t)qt * MAX_SINGLE + i0 + i) * BM + rr];
            if (col != NO_COL)
                tok[i] = P.sbase[qt * MAX_SINGLE + i0 + i] + col;
        }
        any |= tok[i] >= 0;
    }
    if (!any && !FIRST)
        return;
    constexpr int CH = D / 64, E = 8 * CH; // 16-byte pieces and elements of a row per lane
    float dk[KEYS][E], dv[KEYS][E];
    uint4 kp[KEYS][CH], vp[KEYS][CH]; // the keys' elements of this lane, packed bf16
#pragma unroll
    for (int i = 0; i < KEYS; ++i) {
        const size_t kr = ((size_t)(tok[i] >= 0 ? tok[i] : 0) * P.Hkv + g) * D;
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            kp[i][j] = reinterpret_cast<const uint4 *>(P.K + kr)[sub + 8 * j];
            vp[i][j] = reinterpret_cast<const uint4 *>(P.V + kr)[sub + 8 * j];
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            dk[i][e] = 0.f;
            dv[i][e] = 0.f;
        }
    }
    for (int hh = 0; hh < G; ++hh) {
        const int h = g * G + hh;
        const Chunk<CH> q = load_chunk<CH>(sq + (size_t)h * D, sub);
        const Chunk<CH> dO = load_chunk<CH>(sdo + (size_t)h * D, sub);
        float nl2, nd;
        if (FIRST && P.rows_ready) {
            nl2 = snl2[h];
            nd = snd[h];
        } else if (FIRST) {
            const Chunk<CH> o = load_chunk<CH>(so + (size_t)h * D, sub);
            float delta = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e)
                delta = fmaf(dO.v[e], o.v[e], delta);
#pragma unroll
            for (int s = 1; s < 8; s <<= 1)
                delta += __shfl_xor_sync(um, delta, s);
            nd = -delta;
            const float lse = snl2[h]; // holds LSE until here
            nl2 = lse == -CUDART_INF_F ? -CUDART_INF_F : -lse * 1.4426950408889634f;
            __syncwarp(um); // every lane has read the LSE before it is replaced
            if (sub == 0) {
                snl2[h] = nl2;
                snd[h] = nd;
                P.nl2[(size_t)h * P.q_pad + r] = nl2;
                P.nd[(size_t)h * P.q_pad + r] = nd;
            }
        } else {
            nl2 = snl2[h];
            nd = snd[h];
        }
        float dq[E];
#pragma unroll
        for (int e = 0; e < E; ++e)
            dq[e] = 0.f;
#pragma unroll
        for (int i = 0; i < KEYS; ++i) {
            const Chunk<CH> k = unpack_chunk<CH>(kp[i]);
            const Chunk<CH> v = unpack_chunk<CH>(vp[i]);
            float s = 0.f, dp = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                s = fmaf(q.v[e], k.v[e], s);
                dp = fmaf(dO.v[e], v.v[e], dp);
            }
#pragma unroll
            for (int o2 = 1; o2 < 8; o2 <<= 1) {
                s += __shfl_xor_sync(um, s, o2);
                dp += __shfl_xor_sync(um, dp, o2);
            }
            // an absent key takes part with weight zero, so that the keys' chains of dependent
            // instructions interleave instead of branching around each other
            const float p = fast_exp2(fmaf(s, P.scale_log2, tok[i] >= 0 ? nl2 : -CUDART_INF_F)); // nl2 = -inf: p = 0
            const float ds = p * (dp + nd);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                dq[e] = fmaf(ds, k.v[e], dq[e]);
                dk[i][e] = fmaf(ds, q.v[e], dk[i][e]);
                dv[i][e] = fmaf(p, dO.v[e], dv[i][e]);
            }
        }
        float *dst = P.dq_acc + ((size_t)r * P.Hq + h) * D;
        if (FIRST) {
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                float4 *d4 = reinterpret_cast<float4 *>(dst + 64 * j + 8 * sub);
                d4[0] = make_float4(dq[8 * j] * P.scale, dq[8 * j + 1] * P.scale, dq[8 * j + 2] * P.scale,
                                    dq[8 * j + 3] * P.scale);
                d4[1] = make_float4(dq[8 * j + 4] * P.scale, dq[8 * j + 5] * P.scale,
                                    dq[8 * j + 6] * P.scale, dq[8 * j + 7] * P.scale);
            }
        } else {
            red_chunk<CH>(dst, sub, dq, P.scale);
        }
    }
#pragma unroll
    for (int i = 0; i < KEYS; ++i)
        if (tok[i] >= 0) {
            const size_t kr = ((size_t)tok[i] * P.Hkv + g) * D;
            red_chunk<CH>(P.dK_acc + kr, sub, dk[i], P.scale);
            red_chunk<CH>(P.dV_acc + kr, sub, dv[i], 1.f);
        }
}

// head_dim 64 runs in 128 registers: the arithmetic is bound by the latency of its dependent
// chains (dot product, three shuffles, exp2), so more resident warps pay more than fewer passes.
// Shared memory: [3][RB][Hq * D] bf16 rows of Q, dO, O ([2]: no O when the forward left the row
// values), then [2][RB][Hq] fp32 row values.
template <int D>
__global__ void __launch_bounds__(128, D == 64 ? 4 : 2) single_bwd(const SingleParams P)
{
    // Two keys per pass at either head size.  Measured on 8-depth grids as the time of a step
    // outside the two tile kernels: head_dim 64 with four keys and 168 registers 0.76 against
    // 0.66 ms; head_dim 128 with one / two / three keys 0.45 / 0.37 / 0.40 ms.  head_dim 128 holds
    // twice the sums per key and takes up to 255 registers.
    constexpr int KEYS = 2;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    const int RB = P.rows_per_block;
    const int row_elems = P.Hq * D;
    __nv_bfloat16 *sQ = reinterpret_cast<__nv_bfloat16 *>(smem);
    __nv_bfloat16 *sdO = sQ + (size_t)RB * row_elems;
    __nv_bfloat16 *sO = sdO + (size_t)RB * row_elems;
    float *snl2 = reinterpret_cast<float *>(sO + (P.rows_ready ? 0 : (size_t)RB * row_elems));
    float *snd = snl2 + RB * P.Hq;
    // blocks walk the query tiles in the order K0 chose (tiles that share key rows together); RB
    // divides the tile height, so a block's rows lie in one tile
    const int r0 = P.sperm[(blockIdx.x * RB) / BM] * BM + (blockIdx.x * RB) % BM;
    const int n_real = max(0, min(RB, (P.q_end - P.q_begin) - r0)); // rows of the partition
    const uint32_t bar_a = smem_u32(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar_a, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0 && n_real > 0) {
        const uint32_t bytes = (uint32_t)(n_real * row_elems * 2);
        mbar_arrive_expect_tx(bar_a, (P.rows_ready ? 2 : 3) * bytes);
        const size_t off = (size_t)(P.q_begin + r0) * row_elems;
        bulk_load(smem_u32(sQ), P.Q + off, bytes, bar_a);
        bulk_load(smem_u32(sdO), P.dO + off, bytes, bar_a);
        if (!P.rows_ready)
            bulk_load(smem_u32(sO), P.O + off, bytes, bar_a);
    }
    if (P.rows_ready) {
        for (int i = threadIdx.x; i < n_real * P.Hq; i += blockDim.x) {
            const size_t ri = (size_t)(i % P.Hq) * P.q_pad + r0 + i / P.Hq;
            snl2[i] = P.nl2[ri];
            snd[i] = P.nd[ri];
        }
    } else {
        for (int i = threadIdx.x; i < n_real * P.Hq; i += blockDim.x)
            snl2[i] = P.LSE[(size_t)(i % P.Hq) * P.T + P.q_begin + r0 + i / P.Hq];
    }
    __syncthreads();

    const int sub = threadIdx.x & 7;
    const unsigned um = 0xffu << (threadIdx.x & 24); // the lanes of this unit
    const int unit = threadIdx.x >> 3;
    const int rl = unit / P.Hkv, g = unit % P.Hkv;
    const int r = r0 + rl;
    const int G = P.Hq / P.Hkv;
    const bool real = rl < n_real;
    if (rl < RB && r < P.q_pad && !real && !P.rows_ready) { // padded row: seen by nobody
        if (sub == 0) {
            for (int hh = 0; hh < G; ++hh) {
                P.nl2[(size_t)(g * G + hh) * P.q_pad + r] = -CUDART_INF_F;
                P.nd[(size_t)(g * G + hh) * P.q_pad + r] = 0.f;
            }
            if (g == 0)
                P.mqp[r] = META_NONE_Q;
        }
    }
    if (n_real == 0)
        return;
    // every thread waits for the rows (bounded); the units of padded rows then leave
    if (!mbar_wait(bar_a, 0, &abort_flag)) {
        if (threadIdx.x == 0)
            atomicCAS(P.status, 0, PEAGLE_ERR_TIMEOUT);
        return;
    }
    if (!real)
        return; // the 8 lanes of a unit leave together
    const int row = P.q_begin + r;
    if (g == 0 && sub == 0 && !P.rows_ready) {
        const int32_t mq = P.meta[row];
        P.mqp[r] = mq == META_NONE_K ? META_NONE_Q : mq;
    }
    const __nv_bfloat16 *sq = sQ + (size_t)rl * row_elems, *sdo = sdO + (size_t)rl * row_elems,
                        *so = sO + (size_t)rl * row_elems;
    float *rnl2 = snl2 + rl * P.Hq, *rnd = snd + rl * P.Hq;
    const int qt = r / BM, rr = r % BM;
    const int ns = min(P.scount[qt], MAX_SINGLE);
    single_pass<D, true, KEYS>(P, 0, ns, sub, um, r, g, qt, rr, G, sq, sdo, so, rnl2, rnd);
    for (int i0 = KEYS; i0 < ns; i0 += KEYS) {
        __syncwarp(um); // lane 0's row values are visible to the unit's later passes
        single_pass<D, false, KEYS>(P, i0, ns, sub, um, r, g, qt, rr, G, sq, sdo, so, rnl2, rnd);
    }
}

int launch_bwd_single(const Plan &p, const BwdArgs &a, cudaStream_t s)
{
    if (!p.allow_single || p.n_qt == 0 || (a.D != 64 && a.D != 128))
        return 0;
    SingleParams P;
    P.scount = p.scount;
    P.scs = p.scs;
    P.sbase = p.sbase;
    P.sperm = p.sperm;
    P.Q = static_cast<const __nv_bfloat16 *>(a.Q);
    P.K = static_cast<const __nv_bfloat16 *>(a.K);
    P.V = static_cast<const __nv_bfloat16 *>(a.V);
    P.O = static_cast<const __nv_bfloat16 *>(a.O);
    P.dO = static_cast<const __nv_bfloat16 *>(a.dO);
    P.LSE = a.LSE;
    P.meta = p.meta;
    P.nl2 = a.nl2;
    P.nd = a.nd;
    P.mqp = a.mqp;
    P.dq_acc = a.dq_acc;
    P.dK_acc = a.dK_acc;
    P.dV_acc = a.dV_acc;
    P.q_begin = p.q_begin;
    P.q_end = p.q_end;
    P.q_pad = p.n_qt * BM;
    P.n_qt = p.n_qt;
    P.Hq = a.Hq;
    P.Hkv = a.Hkv;
    P.T = p.T;
    P.scale = a.scale;
    P.scale_log2 = a.scale * 1.4426950408889634f;
    P.status = p.status;
    P.rows_ready = a.rows_ready ? 1 : 0;
    // rows per block: up to 16 units of 8 lanes within 48 KB of shared memory (the headline shape,
    // 64 heads: one row, 25 KB, 64 threads; two rows per block measured the same)
    const size_t row_bytes = (size_t)a.Hq * ((a.rows_ready ? 2 : 3) * a.D * 2 + 8);
    int rb = 1; // a power of two, so that it divides the tile height
    while (2 * rb * a.Hkv <= 16 && 2 * rb * row_bytes <= 48 * 1024)
        rb *= 2;
    const size_t smem = rb * row_bytes;
    const int threads = rb * a.Hkv * 8;
    if (threads > 128 || smem > 200 * 1024)
        return PEAGLE_ERR_BAD_SHAPE;
    P.rows_per_block = rb;
    // per device, so set before every launch (host time only)
    void (*kern)(const SingleParams) = a.D == 64 ? single_bwd<64> : single_bwd<128>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    kern<<<(unsigned)((P.q_pad + rb - 1) / rb), threads, smem, s>>>(P);
    return 1;
}

} // namespace peagle
