// Dense bf16 projection products of the drafter layer on sm_100a (Section 2: a LLaMA-3-style layer;
// Section 3.2: every segment runs the layer on its own tokens and on the depth-0 tokens before
// it, so the K / V projections of those tokens are recomputed per segment).
//
//   C[m][n] (+)= sum_k A(m, k) * B(n, k),   bf16 operands, fp32 accumulation in tensor memory
//
// Each operand is either stored with k contiguous ("K-major": A[m][k], B[n][k]) or transposed
// ("MN-major": A[k][m], B[k][n]); the three products of a linear layer are
//   forward      Y  = X W^T      A = X  [rows][d_in]  K-major,  B = W [d_out][d_in] K-major
//   input grad   dX = dY W       A = dY [rows][d_out] K-major,  B = W [d_out][d_in] MN-major (k = d_out)
//   weight grad  dW = dY^T X     A = dY [rows][d_out] MN-major, B = X [rows][d_in]  MN-major (k = rows)
// Persistent CTAs take 128 x 128 or 128 x 256 tiles of C in turn: warp 0 loads 64-wide k slabs of A
// and B by TMA into a ring of stages (128-byte swizzle), warp 1 lane 0 issues tcgen05.mma (four
// k = 16 products per slab) into one of two accumulators in tensor memory and releases the stages
// by commits, warps 2-5 read an accumulator when its last commit arrives, hand it back as soon as
// it is in registers, and either store bf16 rows or add into an fp32 C (tiles of one launch are
// disjoint and launches on a stream are ordered, so the addition is a plain load-add-store).
#include <cstdint>

#include "peagle_internal.h"
#include "sm100_ptx.cuh"

namespace peagle {
using namespace sm100;

namespace {

constexpr int GT = 128;      // rows of a tile of C
constexpr int GK = 64;       // k slab
constexpr int G_TILE_BYTES = GT * GK * 2; // 16 KB: 128 rows of an operand, one stage
// A tile of C is 128 x NT.  NT = 128: three stages, two CTAs per SM (one's epilogue under the
// other's products).  NT = 256: the products are twice as wide, so the A operand and the
// instruction stream are shared by twice the work and a product moves 12 instead of 16 KB of
// shared memory per 128 columns; four stages of 48 KB, one CTA per SM.
template <int NT>
struct GemmCfg {
    static constexpr int STAGES = NT == 128 ? 3 : 4;
    static constexpr int B_BYTES = (NT / GT) * G_TILE_BYTES;
    static constexpr int STAGE_BYTES = G_TILE_BYTES + B_BYTES;
    static constexpr int OFF_BAR = STAGES * STAGE_BYTES;
    static constexpr int N_BAR = 2 * STAGES + 4; // + two accumulators: full, empty
    static constexpr int SMEM = OFF_BAR + N_BAR * 8 + 32 + 1024;
    static constexpr int CTAS = NT == 128 ? 2 : 1;
};

struct GemmParams {
    int M, N, K;
    int a_t, b_t;  // 1: operand stored transposed (MN-major)
    int c_f32_add; // 0: C bf16, stored; 1: C fp32, added to
    void *C;
    long long ldc;
    int *status;
};

template <int NT>
__global__ void __launch_bounds__(192, GemmCfg<NT>::CTAS)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const GemmParams P)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sb = (raw + 1023u) & ~1023u;
    uint8_t *sp = smem_raw + (sb - raw);
    using C = GemmCfg<NT>;
    constexpr int G_STAGES = C::STAGES, G_OFF_BAR = C::OFF_BAR;
    const uint32_t bar0 = sb + G_OFF_BAR;
    auto FULL = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto EMPTY = [&](int s) { return bar0 + 8u * (uint32_t)(G_STAGES + s); };
    auto ACCFULL = [&](int b) { return bar0 + 8u * (uint32_t)(2 * G_STAGES + b); };
    auto ACCEMPTY = [&](int b) { return bar0 + 8u * (uint32_t)(2 * G_STAGES + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(sp + G_OFF_BAR + C::N_BAR * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sp + G_OFF_BAR + C::N_BAR * 8 + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_k = (P.K + GK - 1) / GK;
    // The CTA is persistent: it takes the tiles blockIdx.x, + gridDim.x, ... in row-major order of C
    // (CTAs running together then share a few row blocks of A, and B stays in L2), with two
    // accumulators in tensor memory so that the epilogue of a tile runs under the next one's
    // products.
    const int tiles_n = (P.N + NT - 1) / NT;
    const int n_tiles = tiles_n * ((P.M + GT - 1) / GT);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < G_STAGES; ++s) {
            mbar_init(FULL(s), 1);
            mbar_init(EMPTY(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(ACCFULL(b), 1);
            mbar_init(ACCEMPTY(b), 4); // one arrival per epilogue warp
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), 2 * NT);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            bool live = true;
            int it = 0; // k slabs loaded so far, over all tiles of this CTA
            for (int t = blockIdx.x; live && t < n_tiles; t += gridDim.x) {
            const int m0 = (t / tiles_n) * GT, n0 = (t % tiles_n) * NT;
            for (int i = 0; i < n_k; ++i, ++it) {
                const int s = it % G_STAGES;
                if (!mbar_wait(EMPTY(s), ((it / G_STAGES) & 1) ^ 1, abort_flag)) {
                    live = false;
                    break;
                }
                mbar_arrive_expect_tx(FULL(s), C::STAGE_BYTES);
                const uint32_t a = sb + s * C::STAGE_BYTES, b = a + G_TILE_BYTES;
                const int k0 = i * GK;
                if (!P.a_t) {
                    tma_load_2d(a, &tmA, FULL(s), k0, m0); // [128 m][64 k]
                } else {                                    // two panels [64 k][64 m]
                    tma_load_2d(a, &tmA, FULL(s), m0, k0);
                    tma_load_2d(a + G_TILE_BYTES / 2, &tmA, FULL(s), m0 + 64, k0);
                }
                if (!P.b_t) {
                    tma_load_2d(b, &tmB, FULL(s), k0, n0); // [NT n][64 k]
                } else {                                    // NT / 64 panels [64 k][64 n]
#pragma unroll
                    for (int pn = 0; pn < NT / 64; ++pn)
                        tma_load_2d(b + pn * (G_TILE_BYTES / 2), &tmB, FULL(s), n0 + 64 * pn, k0);
                }
            }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue (whole warp
        // converged, elected lane issues: see elect_one)
        const uint32_t lead = elect_one();
        {
            const uint32_t idesc = idesc_bf16_f32(GT, NT, P.a_t, P.b_t);
            // K-major: a k = 16 slice is 32 bytes further inside the 128-byte rows; MN-major: 16
            // rows (2,048 bytes) further, the second 64-wide panel half a tile on
            const uint32_t a_step = P.a_t ? 128u : 2u, b_step = P.b_t ? 128u : 2u;
            bool ok = true;
            int it = 0, j = 0; // k slabs and tiles done so far
            for (int t = blockIdx.x; ok && t < n_tiles; t += gridDim.x, ++j) {
            const int buf = j & 1;
            // the epilogue has read this accumulator's previous tile
            ok = mbar_wait(ACCEMPTY(buf), ((j >> 1) & 1) ^ 1, abort_flag);
            if (!ok)
                break;
            tc_fence_after();
            for (int i = 0; ok && i < n_k; ++i, ++it) {
                const int s = it % G_STAGES;
                ok = mbar_wait(FULL(s), (it / G_STAGES) & 1, abort_flag);
                if (!ok)
                    break;
                tc_fence_after();
                const uint32_t a = sb + s * C::STAGE_BYTES, b = a + G_TILE_BYTES;
                const uint32_t a_lo = desc_lo_sw128(a, P.a_t ? G_TILE_BYTES / 2 : 16);
                const uint32_t b_lo = desc_lo_sw128(b, P.b_t ? G_TILE_BYTES / 2 : 16);
#pragma unroll
                for (int k = 0; k < GK / 16; ++k)
                    if (lead) mma_ss_lo(tmem + buf * NT, a_lo + k * a_step, b_lo + k * b_step, idesc,
                              (i > 0 || k > 0) ? 1u : 0u);
                if (lead) tc_commit(EMPTY(s));
            }
            if (ok)
                if (lead) tc_commit(ACCFULL(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2-5)
        const int q = warp & 3; // tensor-memory lane quarter this warp may read
        int j = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++j) {
            const int buf = j & 1;
            const int m0 = (t / tiles_n) * GT, n0 = (t % tiles_n) * NT;
            const int m = m0 + q * 32 + lane;
            if (!__all_sync(0xffffffffu, mbar_wait(ACCFULL(buf), (j >> 1) & 1, abort_flag)))
                break;
            tc_fence_after();
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + buf * NT;
#pragma unroll 1
            for (int c = 0; c < NT / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(trow + c * 32, o);
                tmem_wait_ld();
                if (c == NT / 32 - 1) { // the accumulator is in registers: the next tile may take it
                    tc_fence_before();
                    warp_arrive(ACCEMPTY(buf));
                }
                const int n = n0 + c * 32;
                if (m >= P.M)
                    continue;
                if (!P.c_f32_add) {
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(P.C) + (size_t)m * P.ldc + n;
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        if (n + i < P.N) { // N is a multiple of 8
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(o[i + 0]), __uint_as_float(o[i + 1]));
                            v.y = pack_bf16x2(__uint_as_float(o[i + 2]), __uint_as_float(o[i + 3]));
                            v.z = pack_bf16x2(__uint_as_float(o[i + 4]), __uint_as_float(o[i + 5]));
                            v.w = pack_bf16x2(__uint_as_float(o[i + 6]), __uint_as_float(o[i + 7]));
                            *reinterpret_cast<uint4 *>(dst + i) = v;
                        }
                    }
                } else {
                    float *dst = static_cast<float *>(P.C) + (size_t)m * P.ldc + n;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        if (n + i < P.N) {
                            float4 v = *reinterpret_cast<float4 *>(dst + i);
                            v.x += __uint_as_float(o[i + 0]);
                            v.y += __uint_as_float(o[i + 1]);
                            v.z += __uint_as_float(o[i + 2]);
                            v.w += __uint_as_float(o[i + 3]);
                            *reinterpret_cast<float4 *>(dst + i) = v;
                        }
                    }
                }
            }
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
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, 2 * NT);
    }
}

// ---- the same product by pairs of CTAs (a cluster of two, tcgen05 cta_group::2) -------------
// A pair takes 256 x 256 tiles of C: each CTA loads its own 128 rows of A and its own half (128
// of the 256 columns) of B, one thread of the pair's first CTA issues M = 256 products that read
// both CTAs' shared memory and write both CTAs' tensor memory, and each CTA's epilogue warps read
// their own 128 rows of the accumulator.  Per 128 x 256 of C a CTA now stages 32 KB per k slab
// instead of 48.  No load is multicast: every CTA's TMA writes its own shared memory; the bytes
// of both CTAs are counted on the first CTA's barrier of the stage (the cta_group::2 form of the
// load lets the second CTA name it), and stages and accumulators are handed back to both CTAs by
// multicast commits.
struct Gemm2Cfg {
    static constexpr int NT = 256;
    static constexpr int STAGES = 6;
    static constexpr int STAGE_BYTES = 2 * G_TILE_BYTES; // A: 128 m x 64 k, B half: 128 n x 64 k
    static constexpr int OFF_BAR = STAGES * STAGE_BYTES;
    static constexpr int N_BAR = 2 * STAGES + 4; // full, empty per stage; accumulator full / empty x 2
    // two 128 x 32 fp32 tiles through which an accumulate-mode C leaves by tiled reduce-adds
    static constexpr int OFF_OUT = OFF_BAR + 1024;
    static constexpr int OUT_BYTES = GT * 32 * 4;
    static constexpr int SMEM = OFF_OUT + 2 * OUT_BYTES + 1024;
    static_assert(N_BAR * 8 + 32 <= 1024 && SMEM <= 227 * 1024, "shared memory of one CTA");
};

__global__ void __launch_bounds__(192, 1)
gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const __grid_constant__ CUtensorMap tmC, const GemmParams P)
{
    using C = Gemm2Cfg;
    constexpr int NT = C::NT, ST = C::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sb = (raw + 1023u) & ~1023u; // the same offset in both CTAs of the pair
    uint8_t *sp = smem_raw + (sb - raw);
    const uint32_t bar0 = sb + C::OFF_BAR;
    auto FULL = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto EMPTY = [&](int s) { return bar0 + 8u * (uint32_t)(ST + s); };
    auto ACCFULL = [&](int b) { return bar0 + 8u * (uint32_t)(2 * ST + b); };
    auto ACCEMPTY = [&](int b) { return bar0 + 8u * (uint32_t)(2 * ST + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(sp + C::OFF_BAR + C::N_BAR * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sp + C::OFF_BAR + C::N_BAR * 8 + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(); // 0: issues the products
    const int n_k = (P.K + GK - 1) / GK;
    const int tiles_n = (P.N + NT - 1) / NT;
    const int n_tiles = tiles_n * ((P.M + 2 * GT - 1) / (2 * GT));
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < ST; ++s) {
            mbar_init(FULL(s), 1);  // used in the first CTA: one arrival, the bytes of both CTAs
            mbar_init(EMPTY(s), 1); // one multicast commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(ACCFULL(b), 1);
            mbar_init(ACCEMPTY(b), 8); // used in the first CTA: four epilogue warps of each CTA
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_slot)), 2 * NT);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all(); // both CTAs' barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;


    if (warp == 0) {
        // ------------------------------------------------------------ producer (each CTA its own)
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmB);
            bool live = true;
            int it = 0;
            for (int t = pair; live && t < n_tiles; t += n_pairs) {
                const int m0 = (t / tiles_n) * 2 * GT + (int)rank * GT;
                const int nb = (t % tiles_n) * NT + (int)rank * (NT / 2); // this CTA's half of B
                for (int i = 0; i < n_k; ++i, ++it) {
                    const int s = it % ST;
                    if (!mbar_wait_cluster(EMPTY(s), ((it / ST) & 1) ^ 1, abort_flag)) {
                        live = false;
                        break;
                    }
                    if (rank == 0)
                        mbar_arrive_expect_tx(FULL(s), 2 * C::STAGE_BYTES); // both CTAs' slabs
                    const uint32_t full = cluster_map(FULL(s), 0);
                    const uint32_t a = sb + s * C::STAGE_BYTES, b = a + G_TILE_BYTES;
                    const int k0 = i * GK;
                    if (!P.a_t) {
                        tma_load_2d_pair(a, &tmA, full, k0, m0);
                    } else {
                        tma_load_2d_pair(a, &tmA, full, m0, k0);
                        tma_load_2d_pair(a + G_TILE_BYTES / 2, &tmA, full, m0 + 64, k0);
                    }
                    if (!P.b_t) {
                        tma_load_2d_pair(b, &tmB, full, k0, nb);
                    } else {
                        tma_load_2d_pair(b, &tmB, full, nb, k0);
                        tma_load_2d_pair(b + G_TILE_BYTES / 2, &tmB, full, nb + 64, k0);
                    }
                }
            }
        }
    } else if (warp == 1) {
        const uint32_t lead = elect_one();
        if (rank == 0) {
            // ---------------------------------------- first CTA: the pair's products (whole warp
            // converged, elected lane issues: see elect_one)
            const uint32_t idesc = idesc_bf16_f32(2 * GT, NT, P.a_t, P.b_t);
            const uint32_t a_step = P.a_t ? 128u : 2u, b_step = P.b_t ? 128u : 2u;
            bool ok = true;
            int it = 0, j = 0;
            for (int t = pair; ok && t < n_tiles; t += n_pairs, ++j) {
                const int buf = j & 1;
                ok = mbar_wait_cluster(ACCEMPTY(buf), ((j >> 1) & 1) ^ 1, abort_flag);
                if (!ok)
                    break;
                tc_fence_after();
                for (int i = 0; ok && i < n_k; ++i, ++it) {
                    const int s = it % ST;
                    ok = mbar_wait_cluster(FULL(s), (it / ST) & 1, abort_flag);
                    if (!ok)
                        break;
                    tc_fence_after();
                    const uint32_t a = sb + s * C::STAGE_BYTES, b = a + G_TILE_BYTES;
                    const uint32_t a_lo = desc_lo_sw128(a, P.a_t ? G_TILE_BYTES / 2 : 16);
                    const uint32_t b_lo = desc_lo_sw128(b, P.b_t ? G_TILE_BYTES / 2 : 16);
#pragma unroll
                    for (int k = 0; k < GK / 16; ++k)
                        if (lead) mma_ss_lo_pair(tmem + buf * NT, a_lo + k * a_step, b_lo + k * b_step, idesc,
                                       (i > 0 || k > 0) ? 1u : 0u);
                    if (lead) tc_commit_pair(EMPTY(s));
                }
                if (ok)
                    if (lead) tc_commit_pair(ACCFULL(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2-5, each CTA)
        const int q = warp & 3;
        int j = 0, piece = 0;
        for (int t = pair; t < n_tiles; t += n_pairs, ++j) {
            const int buf = j & 1;
            const int m = (t / tiles_n) * 2 * GT + (int)rank * GT + q * 32 + lane;
            const int n0 = (t % tiles_n) * NT;
            // the four warps go on, or leave, together (they meet at named barriers below)
            if (!bar_and(2, 128, mbar_wait_cluster(ACCFULL(buf), (j >> 1) & 1, abort_flag)))
                break;
            tc_fence_after();
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + buf * NT;
#pragma unroll 1
            for (int c = 0; c < NT / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(trow + c * 32, o);
                tmem_wait_ld();
                if (c == NT / 32 - 1) { // in registers: the first CTA may reuse the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0)
                        mbar_arrive_remote(ACCEMPTY(buf), 0);
                }
                const int n = n0 + c * 32;
                if (P.c_f32_add) {
                    // fp32 C: the 128 x 32 piece goes through a swizzled tile in shared memory and
                    // is added to C by one tiled reduce-add (whole 128-byte rows reach L2 together;
                    // rows and columns past the matrix are clipped by the tensor map).  Two tiles
                    // alternate: a tile is rewritten once the reduce-add issued two pieces ago has
                    // read it.
                    const uint32_t ob = sb + C::OFF_OUT + (uint32_t)(piece & 1) * C::OUT_BYTES;
                    if (threadIdx.x == 64)
                        bulk_wait_group_read<1>();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    const int rw = q * 32 + lane;
                    uint8_t *dst = sp + C::OFF_OUT + (piece & 1) * C::OUT_BYTES + rw * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4 *>(dst + ((i ^ (rw & 7)) << 4)) =
                            make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (threadIdx.x == 64) {
                        const int row0 = (t / tiles_n) * 2 * GT + (int)rank * GT;
                        if (n < P.N && row0 < P.M) // a piece wholly outside C is not sent at all
                            tma_reduce_add_2d(&tmC, ob, n, row0);
                        bulk_commit_group();
                    }
                    ++piece;
                    continue;
                }
                if (m >= P.M)
                    continue;
                if (!P.c_f32_add) {
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(P.C) + (size_t)m * P.ldc + n;
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        if (n + i < P.N) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(o[i + 0]), __uint_as_float(o[i + 1]));
                            v.y = pack_bf16x2(__uint_as_float(o[i + 2]), __uint_as_float(o[i + 3]));
                            v.z = pack_bf16x2(__uint_as_float(o[i + 4]), __uint_as_float(o[i + 5]));
                            v.w = pack_bf16x2(__uint_as_float(o[i + 6]), __uint_as_float(o[i + 7]));
                            *reinterpret_cast<uint4 *>(dst + i) = v;
                        }
                    }
                }
            }
        }
        if (threadIdx.x == 64)
            bulk_wait_group<0>(); // the last reduce-adds have left shared memory and reached C
    }

    // ------------------------------------------------------------ teardown
    // Both CTAs meet before either frees tensor memory or leaves: the first CTA's products and
    // commits reach into the second, and remote arrivals into the first.  Every wait above is
    // bounded, so both get here.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (*abort_flag && threadIdx.x == 0)
        atomicCAS(P.status, 0, PEAGLE_ERR_TIMEOUT);
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem, 2 * NT);
    }
}

// Tensor map of a row-major bf16 matrix [rows][cols] with leading dimension ld (elements).
int matrix_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, long long rows, long long cols,
               long long ld, int box_cols, int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS
               ? 0
               : -1;
}

} // namespace

// Returns the number of kernels launched (1), 0 for an empty product, or a negative status.
int launch_gemm(EncodeTiledFn enc, const void *A, long long lda, int a_t, const void *B, long long ldb,
                int b_t, void *C, long long ldc, int c_f32_add, int M, int N, int K, int *status,
                cudaStream_t s)
{
    if (M <= 0 || N <= 0)
        return 0;
    if (K <= 0 || (N % 8) || (lda % 8) || (ldb % 8) || (ldc % (c_f32_add ? 4 : 8)))
        return PEAGLE_ERR_BAD_SHAPE;
    CUtensorMap tmA, tmB;
    // K-major operand [R][K]: boxes of 64 k x 128 rows; transposed [K][R]: boxes of 64 r x 64 k
    const int ra = a_t ? matrix_map(enc, &tmA, A, K, M, lda, 64, 64) : matrix_map(enc, &tmA, A, M, K, lda, 64, GT);
    // wide tiles where they do not waste much of the last column of tiles
    const bool wide = N >= 1024 && ((N + 255) / 256) * 256 <= N + N / 8;
    const int NT = wide ? 256 : 128;
    // pairs of CTAs where there are at least two row blocks to pair
#ifndef PEAGLE_GEMM_PAIRS
#define PEAGLE_GEMM_PAIRS 1
#endif
    const bool pairs = PEAGLE_GEMM_PAIRS && wide && M > GT;
    const int rb = b_t ? matrix_map(enc, &tmB, B, K, N, ldb, 64, 64)
                       : matrix_map(enc, &tmB, B, N, K, ldb, 64, pairs ? GT : NT);
    if (ra || rb)
        return PEAGLE_ERR_CUDA;
    GemmParams P;
    P.M = M;
    P.N = N;
    P.K = K;
    P.a_t = a_t ? 1 : 0;
    P.b_t = b_t ? 1 : 0;
    P.c_f32_add = c_f32_add ? 1 : 0;
    P.C = C;
    P.ldc = ldc;
    P.status = status;
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    if (pairs) {
        if (cudaFuncSetAttribute(gemm2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 Gemm2Cfg::SMEM) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        cfg.blockDim = dim3(192);
        cfg.dynamicSmemBytes = Gemm2Cfg::SMEM;
        cfg.stream = s;
        cfg.gridDim = dim3((unsigned)(n_sm & ~1));
        int fit = 0; // pairs that can be resident at once
        if (cudaOccupancyMaxActiveClusters(&fit, gemm2_kernel, &cfg) != cudaSuccess || fit < 1)
            return PEAGLE_ERR_CUDA;
        const long long tiles2 = (long long)((N + 255) / 256) * ((M + 255) / 256);
        const long long n_pairs = tiles2 < fit ? tiles2 : fit;
        cfg.gridDim = dim3((unsigned)(2 * n_pairs));
        // fp32 C as a tensor for the tiled reduce-adds: 32 columns (128 bytes) x 128 rows
        CUtensorMap tmC = tmA;
        if (c_f32_add) {
            if (reinterpret_cast<uintptr_t>(C) & 15)
                return PEAGLE_ERR_ALIGN;
            cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
            cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
            cuuint32_t box[2] = {32, (cuuint32_t)GT};
            cuuint32_t estr[2] = {1, 1};
            if (enc(&tmC, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return PEAGLE_ERR_CUDA;
        }
        if (cudaLaunchKernelEx(&cfg, gemm2_kernel, tmA, tmB, tmC, P) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        return 1;
    }
    const long long n_tiles = (long long)((N + NT - 1) / NT) * ((M + GT - 1) / GT);
    const long long resident = (long long)n_sm * (wide ? GemmCfg<256>::CTAS : GemmCfg<128>::CTAS);
    const unsigned grid = (unsigned)(n_tiles < resident ? n_tiles : resident);
    if (wide) {
        if (cudaFuncSetAttribute(gemm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 GemmCfg<256>::SMEM) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        gemm_kernel<256><<<grid, 192, GemmCfg<256>::SMEM, s>>>(tmA, tmB, P);
    } else {
        if (cudaFuncSetAttribute(gemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 GemmCfg<128>::SMEM) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        gemm_kernel<128><<<grid, 192, GemmCfg<128>::SMEM, s>>>(tmA, tmB, P);
    }
    return 1;
}

} // namespace peagle
