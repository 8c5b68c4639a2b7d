// Internal declarations shared by the translation units of libpeagle.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/peagle.h"

namespace peagle {

constexpr int BM = 128;          // query rows per tile
constexpr int BN = 128;          // keys per tile
constexpr int MAX_KRANGES = 32;  // visible key ranges per partition
#ifndef PEAGLE_BWD_CQ
#define PEAGLE_BWD_CQ 4 // measured: 2 / 4 / 8 give 3.33 / 3.27 / 3.38 ms for the head_dim 64 main kernel
#endif
constexpr int BWD_CQ = PEAGLE_BWD_CQ; // query tiles per backward work item (aligned chunk; at most 8)
static_assert(BWD_CQ >= 1 && BWD_CQ <= 8, "the chunk's mask word has eight bits per field");
constexpr int32_t META_NONE_Q = -1;         // packed metadata of a row outside the partition (sees nothing)
constexpr int32_t META_NONE_K = 0x7fffffff; // packed metadata of a key outside the batch (seen by nobody)

// TILE_SINGLE is internal: a PARTIAL tile in which every query row allows at most one key (the
// chain tiles of the depth-major layout: one allowed pair per row).  Such tiles are taken out of
// the tensor-core lists and handled pair by pair.  The test hook reports them as PARTIAL.
enum TileClass : uint8_t { TILE_SKIP = 0, TILE_PARTIAL = 1, TILE_FULL = 2, TILE_SINGLE = 3 };
constexpr int MAX_SINGLE = 16;   // SINGLE tiles kept per query tile; further ones stay PARTIAL
constexpr int NO_COL = 255;      // "this row allows no key of the tile"

// Visible key ranges of one call, passed to kernels by value.
struct RangeList {
    int n;
    int begin[MAX_KRANGES];
    int end[MAX_KRANGES];
};

// Everything the mask evaluator / tile classifier / scheduler (K0) produces for one call.
// All pointers are device memory inside the context's scratch buffer.
struct Plan {
    int T;                 // tokens in the batch
    int q_begin, q_end;    // query rows of the call
    int n_qt, n_kt;        // tile counts
    int32_t *meta;         // [T] packed (anchor << 8 | depth)
    int2 *ktile;           // [n_kt] (first token, length)
    int4 *qsum;            // [n_qt] (min anchor, max anchor, min depth, max depth)
    int4 *ksum;            // [n_kt]
    uint8_t *cls;          // [n_qt][n_kt] tile classes
    int *undecided;        // [n_qt*n_kt] pairs the quick test could not decide
    int *counters;         // [8] device counters (0: undecided, 1: bwd items, 2: bwd work cursor, 3: fwd cursor)
    int2 *klist;           // [n_qt][n_kt] compact non-skip key tiles per query tile: (first token, len | cls<<16)
    int *kcount;           // [n_qt]
    int *qorder;           // [n_qt] query tiles, most key tiles first
    uint16_t *cmask;       // [n_ch][n_kt] per chunk of BWD_CQ query tiles: bit b not skipped, bit 8+b FULL
    int *ccount;           // [n_ch][BWD_CQ] key tiles whose word has 1, 2, .. BWD_CQ query tiles
    int4 *bitems;          // [n_ch * n_kt] backward work items (key tile, chunk, mask word, query tiles)
    int allow_single;      // 1: the kernels of this shape take SINGLE tiles pair by pair
    int *scount;           // [n_qt] SINGLE tiles found per query tile (may exceed MAX_SINGLE: clamp)
    int *skt;              // [n_qt][MAX_SINGLE] key tile of a slot
    uint8_t *sorder;       // [n_qt][MAX_SINGLE] slots by ascending key tile
    uint8_t *scol;         // [n_qt][MAX_SINGLE][BM] per row: the one allowed key column, or NO_COL
    int *sbase;            // [n_qt][MAX_SINGLE] first token of entry i's key tile
    uint8_t *scs;          // [n_qt][MAX_SINGLE][BM] what the kernels read: entry i (slots by ascending
                           // key tile) of row r is its key's column in that tile, or NO_COL
    int *sperm;            // [n_qt] query tiles in the order the SINGLE-tile backward takes them:
                           // by the first key tile of their SINGLE entries, so that the query
                           // tiles that add to the same key rows run close together in time
    int *status;           // device status word
};

struct FwdArgs {
    const void *Q, *K, *V;
    void *O;
    float *LSE;
    int Hq, Hkv, D;
    float scale;
    // optional hand-over to the backward of the same partition (all null when not wanted):
    // dO and the backward's per-row scratch, which the forward's epilogue then fills
    const void *dO = nullptr;
    float *nl2 = nullptr, *nd = nullptr;
    int32_t *mqp = nullptr;
};

struct BwdArgs {
    const void *Q, *K, *V, *O, *dO;
    const float *LSE;
    void *dQ;
    float *dK_acc, *dV_acc;
    // per-row scratch of the call, q_pad = query tiles * BM rows, rows past the partition padded
    float *nl2;     // [Hq][q_pad] -LSE * log2(e); -inf for a padded row or a row that saw no key
    float *nd;      // [Hq][q_pad] -Delta = -<dO, O>; 0 for a padded row
    int32_t *mqp;   // [q_pad] packed metadata of the partition's rows; META_NONE_Q when padded
    float *dq_acc;  // [q_len][Hq][D] scratch, fp32
    int Hq, Hkv, D;
    float scale;
    bool rows_ready = false; // nl2 / nd / mqp were written by the forward of this partition
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// K0: mask evaluator, tile classifier, scheduler.  Returns the number of kernels launched.
int launch_plan(const Plan &p, const int32_t *anchor, const int32_t *depth, int K, int seq_begin,
                int seq_end, const RangeList &ranges, bool for_bwd, int Hkv, cudaStream_t s);
int launch_mask_dense(const Plan &p, const RangeList &ranges, uint8_t *out, cudaStream_t s);
// One CTA whose bounded wait runs out after limit_ns: records PEAGLE_ERR_TIMEOUT in *status.
int launch_wait_expiry(int *status, unsigned long long limit_ns, int *reached_end, cudaStream_t s);

// K1 / K2.  Return the number of kernels launched, or a negative peagle_status.
// ev0/ev1 (may be null) are recorded on the stream right before / after the main kernel.
int launch_fwd(const Plan &p, const FwdArgs &a, EncodeTiledFn enc, int n_sm, cudaStream_t s,
               cudaEvent_t ev0, cudaEvent_t ev1);
int launch_bwd(const Plan &p, const BwdArgs &a, EncodeTiledFn enc, int n_sm, cudaStream_t s,
               cudaEvent_t ev0, cudaEvent_t ev1);
// Backward of the SINGLE tiles (head_dim 64 with SINGLE tiles enabled, else returns 0): adds to
// dK_acc / dV_acc, and prepares the tile kernel's per-row values and the initial dQ staging.
int launch_bwd_single(const Plan &p, const BwdArgs &a, cudaStream_t s);
int launch_cast_grads(const float *dK_acc, const float *dV_acc, void *dK, void *dV, size_t n,
                      cudaStream_t s);
int launch_cast_one(const float *src, void *dst, size_t n, cudaStream_t s);

// Rotary prologue (backward = false: fused row -> Q, K, V) and its backward (dQ, dK, dV -> gradient
// of the fused row).  Returns the number of kernels launched.
int launch_rope(bool backward, const void *fused_in, void *fused_out, const void *q_in,
                const void *k_in, const void *v_in, void *q_out, void *k_out, void *v_out,
                const int32_t *anchor, const int32_t *depth, int T, int Hq, int Hkv, int D,
                float base, int n_sm, cudaStream_t s);

// C[m][n] (+)= sum_k A(m,k) B(n,k) in bf16 with fp32 accumulation (peagle_gemm.cu).  a_t / b_t: the
// operand is stored transposed ([k][m] / [k][n]); c_f32_add: C is fp32 and added to, else bf16 and
// stored.  Leading dimensions in elements.  Returns kernels launched or a negative status.
int launch_gemm(EncodeTiledFn enc, const void *A, long long lda, int a_t, const void *B, long long ldb,
                int b_t, void *C, long long ldc, int c_f32_add, int M, int N, int K, int *status,
                cudaStream_t s);

// Packed-metadata form of the attention predicate: m = anchor << 8 | depth.
// (depth_k == 0 and anchor_k <= anchor_q) or (anchor_k == anchor_q and depth_k <= depth_q)
__host__ __device__ inline bool allowed_packed(int32_t mq, int32_t mk)
{
    return (mk <= mq) && (((mk & 0xff) == 0) || ((mk ^ mq) < 256));
}

} // namespace peagle
