// Backward of the SINGLE tiles (head_dim 64): tiles in which every query row allows at most one
// key, such as the chain tiles of the depth-major layout.  On the tensor cores such a tile costs a
// full 128 x 128 step for 128 useful pairs, so the pairs are done one by one on the CUDA cores.
// For a pair (query row q of head h, key k of its KV head), with the forward's LSE and
// Delta = <dO, O> (Section 3.2's backward, same formulas as the tile kernel):
//   s = <Q[q,h], K[k]>,  p = exp(scale * s - LSE),  dp = <dO[q,h], V[k]>,  ds = p * (dp - Delta)
//   dQ[q,h] += scale * ds * K[k]      dK[k] += scale * ds * Q[q,h]      dV[k] += p * dO[q,h]
// One kernel, query-major so that no reverse (key -> queries) list is needed: eight lanes per
// (query row, KV head) hold 8 of the 64 elements each; for every head of the group they form the
// row's dQ (one fp32 add to the staging row per head) and add into per-key dK / dV sums kept in
// registers across the heads (one fp32 add per key row at the end).
#include <math_constants.h>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

struct SingleParams {
    const int *scount;
    const uint8_t *scs;  // [n_qt][MAX_SINGLE][BM] key column of entry i for row r, or NO_COL
    const int *sbase;    // [n_qt][MAX_SINGLE] first token of entry i's key tile
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *nl2, *nd; // [Hq][q_pad]
    float *dq_acc, *dK_acc, *dV_acc;
    int q_begin, q_end, q_pad, n_qt, Hq, Hkv;
    float scale, scale_log2;
};

// A row of 64 bf16 is spread over 8 consecutive lanes, 8 elements (one 16-byte load) per lane, so
// that a warp reads four whole rows with every load and dot products finish with three shuffles.
struct Chunk {
    float v[8];
};
__device__ __forceinline__ Chunk unpack_chunk(const uint4 t)
{
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
    Chunk c;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c.v[2 * i] = __uint_as_float(w[i] << 16);
        c.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return c;
}
__device__ __forceinline__ Chunk load_chunk(const __nv_bfloat16 *row, int sub)
{
    const uint4 t = reinterpret_cast<const uint4 *>(row)[sub];
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
    Chunk c;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c.v[2 * i] = __uint_as_float(w[i] << 16);
        c.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return c;
}
__device__ __forceinline__ void red_chunk(float *dst, const float (&x)[8], float f)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(x[0] * f),
                 "f"(x[1] * f), "f"(x[2] * f), "f"(x[3] * f)
                 : "memory");
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4), "f"(x[4] * f),
                 "f"(x[5] * f), "f"(x[6] * f), "f"(x[7] * f)
                 : "memory");
}

// Unit (row r of the partition, KV head g) = 8 lanes; a block of 128 threads holds 16 units.
// Keys are taken KEYS at a time so that their dK / dV sums fit in registers.
__global__ void __launch_bounds__(128) single_bwd(const SingleParams P)
{
    constexpr int KEYS = 4;
    const int sub = threadIdx.x & 7;
    const unsigned um = 0xffu << (threadIdx.x & 24); // the lanes of this unit
    const size_t unit = (size_t)blockIdx.x * 16 + (threadIdx.x >> 3);
    const int r = (int)(unit / P.Hkv), g = (int)(unit % P.Hkv);
    const int row = P.q_begin + r;
    if (row >= P.q_end)
        return; // the 8 lanes of a unit leave together
    const int qt = r / BM, rr = r % BM;
    const int ns = min(P.scount[qt], MAX_SINGLE);
    const int G = P.Hq / P.Hkv;
    for (int i0 = 0; i0 < ns; i0 += KEYS) {
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
        if (!any)
            continue;
        float dk[KEYS][8], dv[KEYS][8];
        uint4 kp[KEYS], vp[KEYS]; // the keys' elements of this lane, packed bf16
#pragma unroll
        for (int i = 0; i < KEYS; ++i) {
            const size_t kr = ((size_t)(tok[i] >= 0 ? tok[i] : 0) * P.Hkv + g) * 64;
            kp[i] = reinterpret_cast<const uint4 *>(P.K + kr)[sub];
            vp[i] = reinterpret_cast<const uint4 *>(P.V + kr)[sub];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                dk[i][e] = 0.f;
                dv[i][e] = 0.f;
            }
        }
        // the rows of the next head are requested before this head's arithmetic
        const size_t qoff = ((size_t)row * P.Hq + (size_t)g * G) * 64;
        uint4 qn = reinterpret_cast<const uint4 *>(P.Q + qoff)[sub];
        uint4 dn = reinterpret_cast<const uint4 *>(P.dO + qoff)[sub];
        float nl2n = P.nl2[(size_t)(g * G) * P.q_pad + r], ndn = P.nd[(size_t)(g * G) * P.q_pad + r];
        for (int hh = 0; hh < G; ++hh) {
            const int h = g * G + hh;
            const float nl2 = nl2n, nd = ndn;
            const Chunk q = unpack_chunk(qn);
            const Chunk dO = unpack_chunk(dn);
            if (hh + 1 < G) {
                qn = reinterpret_cast<const uint4 *>(P.Q + qoff + (size_t)(hh + 1) * 64)[sub];
                dn = reinterpret_cast<const uint4 *>(P.dO + qoff + (size_t)(hh + 1) * 64)[sub];
                nl2n = P.nl2[(size_t)(h + 1) * P.q_pad + r];
                ndn = P.nd[(size_t)(h + 1) * P.q_pad + r];
            }
            float dq[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < KEYS; ++i) {
                if (tok[i] < 0)
                    continue; // same for the 8 lanes of the unit
                const Chunk k = unpack_chunk(kp[i]);
                const Chunk v = unpack_chunk(vp[i]);
                float s = 0.f, dp = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    s = fmaf(q.v[e], k.v[e], s);
                    dp = fmaf(dO.v[e], v.v[e], dp);
                }
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) {
                    s += __shfl_xor_sync(um, s, o);
                    dp += __shfl_xor_sync(um, dp, o);
                }
                const float p = fast_exp2(fmaf(s, P.scale_log2, nl2)); // nl2 = -inf: p = 0
                const float ds = p * (dp + nd);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    dq[e] = fmaf(ds, k.v[e], dq[e]);
                    dk[i][e] = fmaf(ds, q.v[e], dk[i][e]);
                    dv[i][e] = fmaf(p, dO.v[e], dv[i][e]);
                }
            }
            red_chunk(P.dq_acc + ((size_t)r * P.Hq + h) * 64 + sub * 8, dq, P.scale);
        }
#pragma unroll
        for (int i = 0; i < KEYS; ++i)
            if (tok[i] >= 0) {
                const size_t kr = ((size_t)tok[i] * P.Hkv + g) * 64 + sub * 8;
                red_chunk(P.dK_acc + kr, dk[i], P.scale);
                red_chunk(P.dV_acc + kr, dv[i], 1.f);
            }
    }
}

int launch_bwd_single(const Plan &p, const BwdArgs &a, cudaStream_t s)
{
    if (!p.allow_single || p.n_qt == 0 || a.D != 64)
        return 0;
    SingleParams P;
    P.scount = p.scount;
    P.scs = p.scs;
    P.sbase = p.sbase;
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
    const size_t units = (size_t)(p.q_end - p.q_begin) * a.Hkv; // of 8 lanes each
    single_bwd<<<(unsigned)((units + 15) / 16), 128, 0, s>>>(P);
    return 1;
}

} // namespace peagle
