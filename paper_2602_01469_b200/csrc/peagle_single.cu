// Backward of the SINGLE tiles (head_dim 64): tiles in which every query row allows at most one
// key, such as the chain tiles of the depth-major layout.  On the tensor cores such a tile costs a
// full 128 x 128 step for 128 useful pairs, so the pairs are done one by one on the CUDA cores.
// For a pair (query row q of head h, key k of its KV head), with the forward's LSE and
// Delta = <dO, O> (Section 3.2's backward, same formulas as the tile kernel):
//   s = <Q[q,h], K[k]>,  p = exp(scale * s - LSE),  dp = <dO[q,h], V[k]>,  ds = p * (dp - Delta)
//   dQ[q,h] += scale * ds * K[k]      dK[k] += scale * ds * Q[q,h]      dV[k] += p * dO[q,h]
// Two kernels, both query-major so that no reverse (key -> queries) list is needed:
//   single_dq   one thread per (query row, head): dQ over the row's SINGLE keys, one fp32 add to
//               the dQ staging row;
//   single_dkv  one thread per (query row, SINGLE slot, KV head): dK / dV of the row's key summed
//               over the heads of the group in registers, one fp32 add per key row.
#include <math_constants.h>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

struct SingleParams {
    const int *scount, *skt;
    const uint8_t *sorder, *scol;
    const int2 *ktile;
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *nl2, *nd; // [Hq][q_pad]
    float *dq_acc, *dK_acc, *dV_acc;
    int q_begin, q_end, q_pad, n_qt, Hq, Hkv;
    float scale, scale_log2;
};

__device__ __forceinline__ void load_row64(const __nv_bfloat16 *src, uint32_t (&v)[32])
{
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint4 t = s4[i];
        v[4 * i] = t.x;
        v[4 * i + 1] = t.y;
        v[4 * i + 2] = t.z;
        v[4 * i + 3] = t.w;
    }
}
__device__ __forceinline__ float lo_bf16(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_bf16(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float dot64(const uint32_t (&a)[32], const uint32_t (&b)[32])
{
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        acc = fmaf(lo_bf16(a[i]), lo_bf16(b[i]), acc);
        acc = fmaf(hi_bf16(a[i]), hi_bf16(b[i]), acc);
    }
    return acc;
}

// Thread (row r of the partition, head h); threads of a block share the row's query tile.
__global__ void __launch_bounds__(128) single_dq(const SingleParams P)
{
    const int per_row = P.Hq;
    const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int r = (int)(gid / per_row), h = (int)(gid % per_row);
    const int row = P.q_begin + r;
    if (row >= P.q_end)
        return;
    const int qt = r / BM, rr = r % BM;
    const int ns = min(P.scount[qt], MAX_SINGLE);
    if (ns == 0)
        return;
    const int g = h / (P.Hq / P.Hkv);
    const float nl2 = P.nl2[(size_t)h * P.q_pad + r], nd = P.nd[(size_t)h * P.q_pad + r];
    uint32_t q[32], dO[32];
    load_row64(P.Q + ((size_t)row * P.Hq + h) * 64, q);
    load_row64(P.dO + ((size_t)row * P.Hq + h) * 64, dO);
    float dq[64];
#pragma unroll
    for (int i = 0; i < 64; ++i)
        dq[i] = 0.f;
    bool any = false;
    for (int i = 0; i < ns; ++i) {
        const int slot = P.sorder[qt * MAX_SINGLE + i];
        const int col = P.scol[((size_t)qt * MAX_SINGLE + slot) * BM + rr];
        if (col == NO_COL)
            continue;
        any = true;
        const size_t tok = (size_t)P.ktile[P.skt[qt * MAX_SINGLE + slot]].x + col;
        uint32_t k[32], v[32];
        load_row64(P.K + (tok * P.Hkv + g) * 64, k);
        load_row64(P.V + (tok * P.Hkv + g) * 64, v);
        const float p = fast_exp2(fmaf(dot64(q, k), P.scale_log2, nl2)); // nl2 = -inf: p = 0
        const float ds = p * (dot64(dO, v) + nd);
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            dq[2 * c] = fmaf(ds, lo_bf16(k[c]), dq[2 * c]);
            dq[2 * c + 1] = fmaf(ds, hi_bf16(k[c]), dq[2 * c + 1]);
        }
    }
    if (!any)
        return;
    float *dst = P.dq_acc + ((size_t)r * P.Hq + h) * 64;
#pragma unroll
    for (int c = 0; c < 64; c += 4)
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + c),
                     "f"(dq[c] * P.scale), "f"(dq[c + 1] * P.scale), "f"(dq[c + 2] * P.scale),
                     "f"(dq[c + 3] * P.scale)
                     : "memory");
}

// Block (query tile qt, slot index i, KV head g), thread = row of the tile.
__global__ void __launch_bounds__(128) single_dkv(const SingleParams P)
{
    const int g = blockIdx.x % P.Hkv;
    const int i = (blockIdx.x / P.Hkv) % MAX_SINGLE;
    const int qt = blockIdx.x / (P.Hkv * MAX_SINGLE);
    if (i >= min(P.scount[qt], MAX_SINGLE))
        return;
    const int rr = threadIdx.x, r = qt * BM + rr, row = P.q_begin + r;
    if (row >= P.q_end)
        return;
    const int slot = P.sorder[qt * MAX_SINGLE + i];
    const int col = P.scol[((size_t)qt * MAX_SINGLE + slot) * BM + rr];
    if (col == NO_COL)
        return;
    const size_t tok = (size_t)P.ktile[P.skt[qt * MAX_SINGLE + slot]].x + col;
    uint32_t k[32], v[32];
    load_row64(P.K + (tok * P.Hkv + g) * 64, k);
    load_row64(P.V + (tok * P.Hkv + g) * 64, v);
    float dk[64], dv[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) {
        dk[c] = 0.f;
        dv[c] = 0.f;
    }
    const int G = P.Hq / P.Hkv;
    for (int hh = 0; hh < G; ++hh) {
        const int h = g * G + hh;
        const float nl2 = P.nl2[(size_t)h * P.q_pad + r], nd = P.nd[(size_t)h * P.q_pad + r];
        uint32_t t[32];
        load_row64(P.Q + ((size_t)row * P.Hq + h) * 64, t);
        const float s = dot64(t, k);
        const float p = fast_exp2(fmaf(s, P.scale_log2, nl2));
        uint32_t u[32];
        load_row64(P.dO + ((size_t)row * P.Hq + h) * 64, u);
        const float ds = p * (dot64(u, v) + nd);
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            dk[2 * c] = fmaf(ds, lo_bf16(t[c]), dk[2 * c]);
            dk[2 * c + 1] = fmaf(ds, hi_bf16(t[c]), dk[2 * c + 1]);
            dv[2 * c] = fmaf(p, lo_bf16(u[c]), dv[2 * c]);
            dv[2 * c + 1] = fmaf(p, hi_bf16(u[c]), dv[2 * c + 1]);
        }
    }
    float *dkd = P.dK_acc + (tok * P.Hkv + g) * 64, *dvd = P.dV_acc + (tok * P.Hkv + g) * 64;
#pragma unroll
    for (int c = 0; c < 64; c += 4) {
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dkd + c),
                     "f"(dk[c] * P.scale), "f"(dk[c + 1] * P.scale), "f"(dk[c + 2] * P.scale),
                     "f"(dk[c + 3] * P.scale)
                     : "memory");
        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dvd + c), "f"(dv[c]),
                     "f"(dv[c + 1]), "f"(dv[c + 2]), "f"(dv[c + 3])
                     : "memory");
    }
}

int launch_bwd_single(const Plan &p, const BwdArgs &a, cudaStream_t s)
{
    if (!p.allow_single || p.n_qt == 0 || a.D != 64)
        return 0;
    SingleParams P;
    P.scount = p.scount;
    P.skt = p.skt;
    P.sorder = p.sorder;
    P.scol = p.scol;
    P.ktile = p.ktile;
    P.Q = static_cast<const __nv_bfloat16 *>(a.Q);
    P.K = static_cast<const __nv_bfloat16 *>(a.K);
    P.V = static_cast<const __nv_bfloat16 *>(a.V);
    P.dO = static_cast<const __nv_bfloat16 *>(a.dO);
    P.nl2 = a.nl2;
    P.nd = a.nd;
    P.dq_acc = a.dq_acc;
    P.dK_acc = a.dK_acc;
    P.dV_acc = a.dV_acc;
    P.q_begin = p.q_begin;
    P.q_end = p.q_end;
    P.q_pad = p.n_qt * BM;
    P.n_qt = p.n_qt;
    P.Hq = a.Hq;
    P.Hkv = a.Hkv;
    P.scale = a.scale;
    P.scale_log2 = a.scale * 1.4426950408889634f;
    const size_t n_dq = (size_t)(p.q_end - p.q_begin) * a.Hq;
    single_dq<<<(unsigned)((n_dq + 127) / 128), 128, 0, s>>>(P);
    single_dkv<<<(unsigned)((size_t)p.n_qt * MAX_SINGLE * a.Hkv), 128, 0, s>>>(P);
    return 2;
}

} // namespace peagle
