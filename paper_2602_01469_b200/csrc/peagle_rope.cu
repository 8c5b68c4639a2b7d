// Rotary prologue of the drafter layer and its backward (Section 2: a LLaMA-3-style layer with
// rotary position embeddings; a token with anchor a and depth d stands at position p = a + d).
//
// Forward: one fused projection row per token, [Hq query heads | Hkv key heads | Hkv value heads]
// of D bf16 elements each, is split into the three tensors the attention kernels read, Q and K
// rotated by R_p, V copied.  R_p turns the pair (x[i], x[i + D/2]) of a head by the angle
// p * base^(-2i/D).  Backward: the gradients of Q and K are turned back by R_{-p} and the three
// are packed into the gradient of the fused row.
//
// The work is one read and one write of every element (HBM-bound).  A block walks over tokens;
// for each token D/2 threads first form cos and sin of its angles in shared memory, with the angle
// and its range reduction in fp64 (p * frequency reaches 3e4 rad, where an fp32 product is already
// off by 1e-3 rad); then every thread takes pairs of 16-byte pieces, elements 8c .. 8c+7 and their
// partners D/2 further on, so that loads and stores are whole 16-byte vectors of contiguous rows.
#include <math_constants.h>

#include <algorithm>
#include <cmath>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

namespace {

constexpr int ROPE_THREADS = 256;

struct RopeParams {
    const __nv_bfloat16 *fused_in;          // forward: [T][(Hq + 2 Hkv) * D]
    __nv_bfloat16 *fused_out;               // backward: the same layout
    const __nv_bfloat16 *q_in, *k_in, *v_in; // backward: gradients of Q, K, V
    __nv_bfloat16 *q_out, *k_out, *v_out;    // forward
    const int32_t *anchor, *depth;
    int T, Hq, Hkv;
    double log2_base;
};

__device__ __forceinline__ void unpack8(const uint4 v, float (&f)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                      pack_bf16x2(f[6], f[7]));
}

// BACKWARD = false: fused row -> Q, K, V.  BACKWARD = true: dQ, dK, dV -> gradient of the row.
template <int D, bool BACKWARD>
__global__ void __launch_bounds__(ROPE_THREADS) rope_kernel(const RopeParams P)
{
    constexpr int HALF = D / 2;
    constexpr int CH = D / 16; // 16-byte pieces per half head = tasks per head
    constexpr int ROPE_TOKENS = ROPE_THREADS / HALF; // tokens per iteration: a table entry per thread
    __shared__ float s_cos[ROPE_TOKENS][HALF], s_sin[ROPE_TOKENS][HALF];
    const int heads = P.Hq + 2 * P.Hkv;
    const int tasks = heads * CH; // per token
    const int W = heads * D;
    // frequency of this thread's pair, once: base^(-2i/D) in fp64
    const int fi = threadIdx.x % HALF, ft = threadIdx.x / HALF;
    const double inv_freq = exp2(-(double)(2 * fi) / (double)D * P.log2_base);
    for (int t0 = blockIdx.x * ROPE_TOKENS; t0 < P.T; t0 += gridDim.x * ROPE_TOKENS) {
        __syncthreads(); // the previous tokens' tables are no longer read
        if (ft < ROPE_TOKENS && t0 + ft < P.T) {
            const int p = P.anchor[t0 + ft] + P.depth[t0 + ft];
            double sn, cs;
            sincos((double)p * inv_freq, &sn, &cs);
            s_cos[ft][fi] = (float)cs;
            s_sin[ft][fi] = BACKWARD ? -(float)sn : (float)sn;
        }
        __syncthreads();
        for (int task = threadIdx.x; task < ROPE_TOKENS * tasks; task += ROPE_THREADS) {
            const int tt = task / tasks, rem = task % tasks;
            const int t = t0 + tt;
            if (t >= P.T)
                break;
            const int hh = rem / CH, c = rem % CH; // head within the fused row, piece of the half
            // where this head lives outside the fused row
            const __nv_bfloat16 *src;
            __nv_bfloat16 *dst;
            const size_t fused_off = (size_t)t * W + (size_t)hh * D;
            size_t split_off;
            const __nv_bfloat16 *split_in;
            __nv_bfloat16 *split_out;
            if (hh < P.Hq) {
                split_off = ((size_t)t * P.Hq + hh) * D;
                split_in = P.q_in;
                split_out = P.q_out;
            } else if (hh < P.Hq + P.Hkv) {
                split_off = ((size_t)t * P.Hkv + (hh - P.Hq)) * D;
                split_in = P.k_in;
                split_out = P.k_out;
            } else {
                split_off = ((size_t)t * P.Hkv + (hh - P.Hq - P.Hkv)) * D;
                split_in = P.v_in;
                split_out = P.v_out;
            }
            if (BACKWARD) {
                src = split_in + split_off;
                dst = P.fused_out + fused_off;
            } else {
                src = P.fused_in + fused_off;
                dst = split_out + split_off;
            }
            const uint4 lo = reinterpret_cast<const uint4 *>(src)[c];
            const uint4 hi = reinterpret_cast<const uint4 *>(src)[c + CH];
            if (hh >= P.Hq + P.Hkv) { // value heads pass through
                reinterpret_cast<uint4 *>(dst)[c] = lo;
                reinterpret_cast<uint4 *>(dst)[c + CH] = hi;
                continue;
            }
            float a[8], b[8], ya[8], yb[8];
            unpack8(lo, a);
            unpack8(hi, b);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float cs = s_cos[tt][8 * c + e], sn = s_sin[tt][8 * c + e];
                ya[e] = fmaf(a[e], cs, -b[e] * sn);
                yb[e] = fmaf(b[e], cs, a[e] * sn);
            }
            reinterpret_cast<uint4 *>(dst)[c] = pack8(ya);
            reinterpret_cast<uint4 *>(dst)[c + CH] = pack8(yb);
        }
    }
}

template <int D, bool BACKWARD>
int launch_rope_t(const RopeParams &P, int n_sm, cudaStream_t s)
{
    constexpr int ROPE_TOKENS = ROPE_THREADS / (D / 2);
    const int blocks = std::min((P.T + ROPE_TOKENS - 1) / ROPE_TOKENS, n_sm * 8);
    rope_kernel<D, BACKWARD><<<blocks, ROPE_THREADS, 0, s>>>(P);
    return 1;
}

} // namespace

int launch_rope(bool backward, const void *fused_in, void *fused_out, const void *q_in,
                const void *k_in, const void *v_in, void *q_out, void *k_out, void *v_out,
                const int32_t *anchor, const int32_t *depth, int T, int Hq, int Hkv, int D,
                float base, int n_sm, cudaStream_t s)
{
    if (T == 0)
        return 0;
    RopeParams P;
    P.fused_in = static_cast<const __nv_bfloat16 *>(fused_in);
    P.fused_out = static_cast<__nv_bfloat16 *>(fused_out);
    P.q_in = static_cast<const __nv_bfloat16 *>(q_in);
    P.k_in = static_cast<const __nv_bfloat16 *>(k_in);
    P.v_in = static_cast<const __nv_bfloat16 *>(v_in);
    P.q_out = static_cast<__nv_bfloat16 *>(q_out);
    P.k_out = static_cast<__nv_bfloat16 *>(k_out);
    P.v_out = static_cast<__nv_bfloat16 *>(v_out);
    P.anchor = anchor;
    P.depth = depth;
    P.T = T;
    P.Hq = Hq;
    P.Hkv = Hkv;
    P.log2_base = std::log2((double)base);
    if (D == 64)
        return backward ? launch_rope_t<64, true>(P, n_sm, s) : launch_rope_t<64, false>(P, n_sm, s);
    return backward ? launch_rope_t<128, true>(P, n_sm, s) : launch_rope_t<128, false>(P, n_sm, s);
}

} // namespace peagle
