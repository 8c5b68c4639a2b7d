// C ABI of libpeagle: context, argument validation, scratch memory, and the drivers that chain
// K0 (mask evaluator / tile classifier / scheduler), K1 (forward) and K2 (backward).
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "peagle_internal.h"

using namespace peagle;

struct DevBuf {
    void *ptr = nullptr;
    size_t bytes = 0;
};

struct peagle_ctx {
    int device = 0;
    int n_sm = 0;
    EncodeTiledFn encode = nullptr;
    int *status = nullptr; // device status word
    DevBuf plan_buf, bwd_buf, acc_buf, host_buf, layer_buf;
    int64_t launches = 0;
    char cuda_err[256] = {0};
    bool timing = false;
    std::vector<cudaEvent_t> ev[2]; // recorded (start, stop) pairs: [0] forward, [1] backward
    size_t ev_used[2] = {0, 0};
    // host entry point: copy-in / compute / copy-out streams and their hand-over events
    cudaStream_t hs[3] = {nullptr, nullptr, nullptr};
    std::vector<cudaEvent_t> hev;
};

namespace {

// SINGLE tiles are taken out of the backward's tensor-core lists when the kernel that does them
// pair by pair fits: a block of at most 16 KV heads x 8 lanes, a query row of all heads (Q, dO, O
// and two fp32 values per head) within its shared memory.  Otherwise such tiles stay PARTIAL.
bool single_tiles_ok(const peagle_problem_t *prob)
{
    return prob->n_kv_heads <= 16 && (size_t)prob->n_q_heads * (6 * prob->head_dim + 8) <= 200 * 1024;
}

int cuda_fail(peagle_ctx *ctx, cudaError_t e, const char *what)
{
    if (ctx)
        snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return PEAGLE_ERR_CUDA;
}

#define CK(call)                                        \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess)                          \
            return cuda_fail(ctx, e_, #call);           \
    } while (0)

// Grows a scratch buffer.  The old buffer may still be in use by work queued earlier, so the
// stream is drained before it is freed.
int ensure(peagle_ctx *ctx, DevBuf &b, size_t bytes, cudaStream_t s)
{
    if (bytes <= b.bytes)
        return PEAGLE_OK;
    if (b.ptr) {
        CK(cudaStreamSynchronize(s));
        CK(cudaFree(b.ptr));
        b.ptr = nullptr;
        b.bytes = 0;
    }
    const size_t want = bytes + bytes / 8 + 4096;
    if (cudaMalloc(&b.ptr, want) != cudaSuccess) {
        cudaGetLastError();
        b.ptr = nullptr;
        return PEAGLE_ERR_WORKSPACE;
    }
    b.bytes = want;
    return PEAGLE_OK;
}

// Next (start, stop) event pair of a kind, or nulls when timing is off or the pool is full.
void next_events(peagle_ctx *ctx, int kind, cudaEvent_t *e0, cudaEvent_t *e1)
{
    *e0 = *e1 = nullptr;
    if (!ctx->timing || ctx->ev_used[kind] >= 2 * 4096)
        return;
    std::vector<cudaEvent_t> &v = ctx->ev[kind];
    while (v.size() < ctx->ev_used[kind] + 2) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess)
            return;
        v.push_back(e);
    }
    *e0 = v[ctx->ev_used[kind]];
    *e1 = v[ctx->ev_used[kind] + 1];
    ctx->ev_used[kind] += 2;
}

struct Carver {
    uint8_t *base;
    size_t off = 0;
    explicit Carver(void *p) : base(static_cast<uint8_t *>(p)) {}
    template <class T>
    T *take(size_t n)
    {
        off = (off + 255) & ~size_t(255);
        T *r = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return r;
    }
};

void carve_plan(Plan &p, void *base, size_t *bytes_out)
{
    Carver c(base);
    const size_t nq = (size_t)(p.n_qt > 0 ? p.n_qt : 1), nk = (size_t)(p.n_kt > 0 ? p.n_kt : 1);
    p.meta = c.take<int32_t>((size_t)p.T);
    p.ktile = c.take<int2>(nk);
    p.qsum = c.take<int4>(nq);
    p.ksum = c.take<int4>(nk);
    p.cls = c.take<uint8_t>(nq * nk);
    p.undecided = c.take<int>(nq * nk);
    p.counters = c.take<int>(8);
    p.klist = c.take<int2>(nq * nk);
    p.kcount = c.take<int>(nq);
    p.qorder = c.take<int>(nq);
    const size_t nch = (nq + BWD_CQ - 1) / BWD_CQ;
    p.cmask = c.take<uint16_t>(nch * nk);
    p.ccount = c.take<int>(nch * BWD_CQ);
    p.bitems = c.take<int4>(nch * nk);
    p.scount = c.take<int>(nq);
    p.skt = c.take<int>(nq * MAX_SINGLE);
    p.sorder = c.take<uint8_t>(nq * MAX_SINGLE);
    p.scol = c.take<uint8_t>(nq * MAX_SINGLE * BM);
    p.scs = c.take<uint8_t>(nq * MAX_SINGLE * BM);
    p.sbase = c.take<int>(nq * MAX_SINGLE);
    p.sperm = c.take<int>(nq);
    if (bytes_out)
        *bytes_out = c.off + 256;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Call {
    Plan plan;
    RangeList ranges;
    int seq_begin, seq_end;
};

int validate_problem(const peagle_problem_t *prob)
{
    if (!prob || !prob->cu_seqlens)
        return PEAGLE_ERR_NULL;
    if (prob->num_seqs < 1 || prob->total_tokens < 0)
        return PEAGLE_ERR_BAD_SHAPE;
    if (prob->head_dim != 64 && prob->head_dim != 128)
        return PEAGLE_ERR_BAD_SHAPE;
    if (prob->n_q_heads < 1 || prob->n_kv_heads < 1 || prob->n_q_heads % prob->n_kv_heads != 0)
        return PEAGLE_ERR_BAD_SHAPE;
    if (prob->K < 1 || prob->K > 255)
        return PEAGLE_ERR_BAD_SHAPE;
    if (!(prob->softmax_scale > 0.f))
        return PEAGLE_ERR_BAD_SHAPE;
    if (prob->cu_seqlens[0] != 0 || prob->cu_seqlens[prob->num_seqs] != prob->total_tokens)
        return PEAGLE_ERR_BAD_SHAPE;
    for (int i = 0; i < prob->num_seqs; ++i)
        if (prob->cu_seqlens[i + 1] < prob->cu_seqlens[i])
            return PEAGLE_ERR_BAD_SHAPE;
    if (prob->total_tokens > 0 && (!prob->anchor || !prob->depth))
        return PEAGLE_ERR_NULL;
    return PEAGLE_OK;
}

// Host-side checks of one partition; fills tile counts and the visible ranges.
int validate_partition(const peagle_problem_t *prob, const peagle_partition_t *part, Call &c)
{
    if (!part)
        return PEAGLE_ERR_NULL;
    if (part->seq < 0 || part->seq >= prob->num_seqs)
        return PEAGLE_ERR_BAD_RANGE;
    const int sb = prob->cu_seqlens[part->seq], se = prob->cu_seqlens[part->seq + 1];
    if (part->q.begin > part->q.end || part->q.begin < sb || part->q.end > se)
        return PEAGLE_ERR_BAD_RANGE;
    if (part->nk < 0 || (part->nk > 0 && !part->k))
        return part->nk < 0 ? PEAGLE_ERR_BAD_RANGE : PEAGLE_ERR_NULL;
    if (part->nk > MAX_KRANGES)
        return PEAGLE_ERR_TOO_LARGE;
    c.seq_begin = sb;
    c.seq_end = se;
    c.ranges.n = 0;
    if (part->nk == 0) {
        if (se > sb) {
            c.ranges.n = 1;
            c.ranges.begin[0] = sb;
            c.ranges.end[0] = se;
        }
    } else {
        int prev = sb;
        for (int i = 0; i < part->nk; ++i) {
            const peagle_range_t r = part->k[i];
            if (r.begin >= r.end || r.begin < prev || r.end > se)
                return PEAGLE_ERR_BAD_RANGE;
            prev = r.end;
            c.ranges.begin[i] = r.begin;
            c.ranges.end[i] = r.end;
        }
        c.ranges.n = part->nk;
    }
    Plan &p = c.plan;
    memset(&p, 0, sizeof(p));
    p.T = prob->total_tokens;
    p.q_begin = part->q.begin;
    p.q_end = part->q.end;
    p.n_qt = (p.q_end - p.q_begin + BM - 1) / BM;
    p.n_kt = 0;
    for (int i = 0; i < c.ranges.n; ++i)
        p.n_kt += (c.ranges.end[i] - c.ranges.begin[i] + BN - 1) / BN;
    return PEAGLE_OK;
}

// Runs K0 for one call.  On return c.plan points into ctx->plan_buf.
int plan_call(peagle_ctx *ctx, const peagle_problem_t *prob, const peagle_partition_t *part,
              bool for_bwd, cudaStream_t s, Call &c)
{
    int rc = validate_partition(prob, part, c);
    if (rc != PEAGLE_OK)
        return rc;
    size_t bytes = 0;
    carve_plan(c.plan, nullptr, &bytes);
    rc = ensure(ctx, ctx->plan_buf, bytes, s);
    if (rc != PEAGLE_OK)
        return rc;
    carve_plan(c.plan, ctx->plan_buf.ptr, nullptr);
    c.plan.status = ctx->status;
    c.plan.allow_single = single_tiles_ok(prob) ? 1 : 0;
    if (c.plan.n_qt == 0)
        return PEAGLE_OK;
    ctx->launches += launch_plan(c.plan, prob->anchor, prob->depth, prob->K, c.seq_begin, c.seq_end,
                                 c.ranges, for_bwd, prob->n_kv_heads, s);
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

// Scratch of one backward call inside ctx->bwd_buf: per-row values and the fp32 dQ staging.
int bwd_scratch(peagle_ctx *ctx, const peagle_problem_t *prob, const Call &c, cudaStream_t s,
                BwdArgs &a)
{
    const size_t q_len = (size_t)(c.plan.q_end - c.plan.q_begin);
    const size_t Hq = (size_t)prob->n_q_heads, D = (size_t)prob->head_dim;
    const size_t q_pad = (size_t)c.plan.n_qt * BM;
    const size_t row_bytes = ((2 * Hq + 1) * q_pad * 4 + 255) / 256 * 256;
    const size_t dq_bytes = q_len * Hq * D * 4;
    int rc = ensure(ctx, ctx->bwd_buf, row_bytes + dq_bytes + 256, s);
    if (rc != PEAGLE_OK)
        return rc;
    a.nl2 = static_cast<float *>(ctx->bwd_buf.ptr);
    a.nd = a.nl2 + Hq * q_pad;
    a.mqp = reinterpret_cast<int32_t *>(a.nd + Hq * q_pad);
    a.dq_acc = reinterpret_cast<float *>(static_cast<uint8_t *>(ctx->bwd_buf.ptr) + row_bytes);
    return PEAGLE_OK;
}

// `hand`: when the caller already knows dO (the partition driver), the backward's row scratch
// that the forward's epilogue fills (-LSE * log2 e, -Delta, packed metadata); else null.
int run_fwd(peagle_ctx *ctx, const peagle_problem_t *prob, const Call &c, const void *Q,
            const void *K, const void *V, void *O, float *LSE, cudaStream_t s,
            const void *dO = nullptr, const BwdArgs *hand = nullptr)
{
    if (c.plan.n_qt == 0)
        return PEAGLE_OK;
    FwdArgs a;
    if (hand) {
        a.dO = dO;
        a.nl2 = hand->nl2;
        a.nd = hand->nd;
        a.mqp = hand->mqp;
    }
    a.Q = Q;
    a.K = K;
    a.V = V;
    a.O = O;
    a.LSE = LSE;
    a.Hq = prob->n_q_heads;
    a.Hkv = prob->n_kv_heads;
    a.D = prob->head_dim;
    a.scale = prob->softmax_scale;
    cudaEvent_t e0, e1;
    next_events(ctx, 0, &e0, &e1);
    const int n = launch_fwd(c.plan, a, ctx->encode, ctx->n_sm, s, e0, e1);
    if (n < 0)
        return n;
    ctx->launches += n;
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int run_bwd(peagle_ctx *ctx, const peagle_problem_t *prob, const Call &c, const void *Q,
            const void *K, const void *V, const void *O, const void *dO, const float *LSE,
            void *dQ, float *dK_acc, float *dV_acc, cudaStream_t s, bool rows_ready = false)
{
    if (c.plan.n_qt == 0)
        return PEAGLE_OK;
    BwdArgs a;
    int rc = bwd_scratch(ctx, prob, c, s, a);
    if (rc != PEAGLE_OK)
        return rc;
    a.rows_ready = rows_ready;
    a.Q = Q;
    a.K = K;
    a.V = V;
    a.O = O;
    a.dO = dO;
    a.LSE = LSE;
    a.dQ = dQ;
    a.dK_acc = dK_acc;
    a.dV_acc = dV_acc;
    a.Hq = prob->n_q_heads;
    a.Hkv = prob->n_kv_heads;
    a.D = prob->head_dim;
    a.scale = prob->softmax_scale;
    cudaEvent_t e0, e1;
    next_events(ctx, 1, &e0, &e1);
    const int n = launch_bwd(c.plan, a, ctx->encode, ctx->n_sm, s, e0, e1);
    if (n < 0)
        return n;
    ctx->launches += n;
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

} // namespace

// ---- scratch of peagle_attn_fwd_static ------------------------------------------------------
// Lives in the library image: every GPU that loads the library holds these bytes until the
// process exits.  Layout: the K0 plan (carve_plan) from byte 0, a fallback status word in the
// last 256 bytes.
constexpr size_t STATIC_SCRATCH_BYTES = size_t(4) << 20;
constexpr int STATIC_MAX_TOKENS = 32768;
constexpr int STATIC_MAX_TILE_PAIRS = 65536;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

namespace {

struct StaticDevice {
    bool ready = false;
    unsigned char *scratch = nullptr; // device address of g_static_scratch on this device
    EncodeTiledFn encode = nullptr;
    int n_sm = 0;
};
constexpr int STATIC_MAX_DEVICES = 64;
StaticDevice g_static_dev[STATIC_MAX_DEVICES];
std::mutex g_static_mutex;

// One-time set-up of a device for peagle_attn_fwd_static; `device` is current.  In host code
// `g_static_scratch` is only a handle for the runtime, so the array's real device address is
// looked up here and that pointer is what the kernels get.
int static_setup(int device, StaticDevice **out)
{
    if (device < 0 || device >= STATIC_MAX_DEVICES)
        return PEAGLE_ERR_TOO_LARGE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice &d = g_static_dev[device];
    if (!d.ready) {
        int major = 0, n_sm = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return PEAGLE_ERR_CUDA;
        if (major != 10)
            return PEAGLE_ERR_UNSUPPORTED_ARCH;
        void *addr = nullptr;
        if (cudaGetSymbolAddress((void **)&addr, g_static_scratch) != cudaSuccess || !addr) {
            cudaGetLastError();
            return PEAGLE_ERR_CUDA;
        }
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
                cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return PEAGLE_ERR_CUDA;
        d.scratch = static_cast<unsigned char *>(addr);
        d.encode = reinterpret_cast<EncodeTiledFn>(fn);
        d.n_sm = n_sm;
        d.ready = true;
    }
    *out = &d;
    return PEAGLE_OK;
}

} // namespace

extern "C" {

int peagle_create(peagle_ctx **out, int device)
{
    if (!out)
        return PEAGLE_ERR_NULL;
    *out = nullptr;
    peagle_ctx *ctx = new peagle_ctx();
    ctx->device = device;
    cudaDeviceProp prop;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess)
        e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) {
        delete ctx;
        return PEAGLE_ERR_CUDA;
    }
    if (prop.major != 10) {
        delete ctx;
        return PEAGLE_ERR_UNSUPPORTED_ARCH;
    }
    ctx->n_sm = prop.multiProcessorCount;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        delete ctx;
        return PEAGLE_ERR_CUDA;
    }
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
    if (cudaMalloc(&ctx->status, 256) != cudaSuccess || cudaMemset(ctx->status, 0, 256) != cudaSuccess) {
        delete ctx;
        return PEAGLE_ERR_WORKSPACE;
    }
    *out = ctx;
    return PEAGLE_OK;
}

int peagle_destroy(peagle_ctx *ctx)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    DevBuf *bufs[5] = {&ctx->plan_buf, &ctx->bwd_buf, &ctx->acc_buf, &ctx->host_buf, &ctx->layer_buf};
    for (DevBuf *b : bufs)
        if (b->ptr)
            cudaFree(b->ptr);
    if (ctx->status)
        cudaFree(ctx->status);
    for (int k = 0; k < 2; ++k)
        for (cudaEvent_t e : ctx->ev[k])
            cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->hev)
        cudaEventDestroy(e);
    for (cudaStream_t st : ctx->hs)
        if (st)
            cudaStreamDestroy(st);
    delete ctx;
    return PEAGLE_OK;
}

const char *peagle_status_string(int status)
{
    switch (status) {
    case PEAGLE_OK: return "ok";
    case PEAGLE_ERR_NULL: return "null pointer";
    case PEAGLE_ERR_BAD_SHAPE: return "bad shape";
    case PEAGLE_ERR_BAD_RANGE: return "bad range";
    case PEAGLE_ERR_BAD_META: return "bad token metadata";
    case PEAGLE_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    case PEAGLE_ERR_WORKSPACE: return "scratch allocation failed";
    case PEAGLE_ERR_TIMEOUT: return "device-side wait timed out";
    case PEAGLE_ERR_TOO_LARGE: return "request exceeds a limit";
    case PEAGLE_ERR_CUDA: return "CUDA error";
    case PEAGLE_ERR_ALIGN: return "tensor not 16-byte aligned";
    default: return "unknown status";
    }
}

const char *peagle_last_cuda_error(const peagle_ctx *ctx) { return ctx ? ctx->cuda_err : ""; }

int peagle_tile_shape(const peagle_ctx *ctx, int head_dim, int *bm, int *bn)
{
    (void)ctx;
    if (!bm || !bn)
        return PEAGLE_ERR_NULL;
    if (head_dim != 64 && head_dim != 128)
        return PEAGLE_ERR_BAD_SHAPE;
    *bm = BM;
    *bn = BN;
    return PEAGLE_OK;
}

int peagle_poll_status(peagle_ctx *ctx, void *stream)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 0;
    CK(cudaStreamSynchronize(s));
    CK(cudaMemcpy(&st, ctx->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (st != 0)
        CK(cudaMemset(ctx->status, 0, sizeof(int)));
    return st;
}

int64_t peagle_launch_count(const peagle_ctx *ctx) { return ctx ? ctx->launches : 0; }

int peagle_timing_enable(peagle_ctx *ctx, int on)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    ctx->timing = on != 0;
    return PEAGLE_OK;
}

int peagle_timing_read(peagle_ctx *ctx, double *ms_out, int64_t *n_out)
{
    if (!ctx || !ms_out || !n_out)
        return PEAGLE_ERR_NULL;
    CK(cudaSetDevice(ctx->device));
    CK(cudaDeviceSynchronize());
    for (int k = 0; k < 2; ++k) {
        double total = 0.0;
        for (size_t i = 0; i + 1 < ctx->ev_used[k]; i += 2) {
            float ms = 0.f;
            CK(cudaEventElapsedTime(&ms, ctx->ev[k][i], ctx->ev[k][i + 1]));
            total += ms;
        }
        ms_out[k] = total;
        n_out[k] = (int64_t)(ctx->ev_used[k] / 2);
        ctx->ev_used[k] = 0;
    }
    return PEAGLE_OK;
}

int peagle_attn_fwd(peagle_ctx *ctx, const peagle_problem_t *prob, const peagle_partition_t *part,
                    const void *Q, const void *K, const void *V, void *O, float *LSE, void *stream)
{
    if (!ctx || !Q || !K || !V || !O || !LSE)
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O))
        return PEAGLE_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CK(cudaSetDevice(ctx->device));
    Call c;
    rc = plan_call(ctx, prob, part, false, s, c);
    if (rc != PEAGLE_OK)
        return rc;
    return run_fwd(ctx, prob, c, Q, K, V, O, LSE, s);
}

static int rope_args_ok(int32_t T, int32_t Hq, int32_t Hkv, int32_t D, float base)
{
    if (T < 0 || Hq <= 0 || Hkv <= 0 || (D != 64 && D != 128) || !(base > 1.f))
        return PEAGLE_ERR_BAD_SHAPE;
    return PEAGLE_OK;
}

int peagle_rope_qkv_fwd(peagle_ctx *ctx, const void *qkv, const int32_t *anchor, const int32_t *depth,
                        int32_t total_tokens, int32_t n_q_heads, int32_t n_kv_heads,
                        int32_t head_dim, float rope_base, void *Q, void *K, void *V, void *stream)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    const int rc = rope_args_ok(total_tokens, n_q_heads, n_kv_heads, head_dim, rope_base);
    if (rc != PEAGLE_OK)
        return rc;
    if (total_tokens == 0)
        return PEAGLE_OK; // nothing to do, pointers not looked at
    if (!qkv || !anchor || !depth || !Q || !K || !V)
        return PEAGLE_ERR_NULL;
    if (!aligned16(qkv) || !aligned16(Q) || !aligned16(K) || !aligned16(V))
        return PEAGLE_ERR_ALIGN;
    CK(cudaSetDevice(ctx->device));
    ctx->launches += launch_rope(false, qkv, nullptr, nullptr, nullptr, nullptr, Q, K, V, anchor, depth,
                                 total_tokens, n_q_heads, n_kv_heads, head_dim, rope_base,
                                 ctx->n_sm, static_cast<cudaStream_t>(stream));
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_rope_qkv_bwd(peagle_ctx *ctx, const void *dQ, const void *dK, const void *dV,
                        const int32_t *anchor, const int32_t *depth, int32_t total_tokens,
                        int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float rope_base,
                        void *d_qkv, void *stream)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    const int rc = rope_args_ok(total_tokens, n_q_heads, n_kv_heads, head_dim, rope_base);
    if (rc != PEAGLE_OK)
        return rc;
    if (total_tokens == 0)
        return PEAGLE_OK;
    if (!dQ || !dK || !dV || !anchor || !depth || !d_qkv)
        return PEAGLE_ERR_NULL;
    if (!aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(d_qkv))
        return PEAGLE_ERR_ALIGN;
    CK(cudaSetDevice(ctx->device));
    ctx->launches += launch_rope(true, nullptr, d_qkv, dQ, dK, dV, nullptr, nullptr, nullptr, anchor,
                                 depth, total_tokens, n_q_heads, n_kv_heads, head_dim, rope_base,
                                 ctx->n_sm, static_cast<cudaStream_t>(stream));
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_attn_fwd_static(int device, const peagle_problem_t *prob,
                           const peagle_partition_t *part, const void *Q, const void *K,
                           const void *V, void *O, float *LSE, int32_t *dev_status, void *stream)
{
    if (!Q || !K || !V || !O || !LSE)
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O))
        return PEAGLE_ERR_ALIGN;
    Call c;
    rc = validate_partition(prob, part, c);
    if (rc != PEAGLE_OK)
        return rc;
    // The limits are checked before anything touches the device.
    if (prob->total_tokens > STATIC_MAX_TOKENS ||
        (int64_t)c.plan.n_qt * (int64_t)c.plan.n_kt > STATIC_MAX_TILE_PAIRS)
        return PEAGLE_ERR_TOO_LARGE;
    size_t plan_bytes = 0;
    carve_plan(c.plan, nullptr, &plan_bytes);
    if (plan_bytes + 256 > STATIC_SCRATCH_BYTES)
        return PEAGLE_ERR_TOO_LARGE;
    if (cudaSetDevice(device) != cudaSuccess) {
        cudaGetLastError();
        return PEAGLE_ERR_CUDA;
    }
    StaticDevice *dev = nullptr;
    rc = static_setup(device, &dev);
    if (rc != PEAGLE_OK)
        return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    carve_plan(c.plan, dev->scratch, nullptr);
    int *status = dev_status ? dev_status
                             : reinterpret_cast<int *>(dev->scratch + STATIC_SCRATCH_BYTES - 256);
    c.plan.status = status;
    c.plan.allow_single = single_tiles_ok(prob) ? 1 : 0;
    // The array keeps whatever the previous call left.  The status word is cleared here; the
    // plan's counters are cleared by the first K0 kernel; every other plan field this call
    // reads is written by this call's K0 kernels first.
    if (cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess) {
        cudaGetLastError();
        return PEAGLE_ERR_CUDA;
    }
    if (c.plan.n_qt == 0)
        return PEAGLE_OK;
    launch_plan(c.plan, prob->anchor, prob->depth, prob->K, c.seq_begin, c.seq_end, c.ranges,
                false, prob->n_kv_heads, s);
    if (cudaGetLastError() != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    FwdArgs a;
    a.Q = Q;
    a.K = K;
    a.V = V;
    a.O = O;
    a.LSE = LSE;
    a.Hq = prob->n_q_heads;
    a.Hkv = prob->n_kv_heads;
    a.D = prob->head_dim;
    a.scale = prob->softmax_scale;
    const int n = launch_fwd(c.plan, a, dev->encode, dev->n_sm, s, nullptr, nullptr);
    if (n < 0)
        return n;
    if (cudaGetLastError() != cudaSuccess)
        return PEAGLE_ERR_CUDA;
    return PEAGLE_OK;
}

int peagle_attn_bwd(peagle_ctx *ctx, const peagle_problem_t *prob, const peagle_partition_t *part,
                    const void *Q, const void *K, const void *V, const void *O, const void *dO,
                    const float *LSE, void *dQ, float *dK_acc, float *dV_acc, void *stream)
{
    if (!ctx || !Q || !K || !V || !O || !dO || !LSE || !dQ || !dK_acc || !dV_acc)
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK_acc) || !aligned16(dV_acc))
        return PEAGLE_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CK(cudaSetDevice(ctx->device));
    Call c;
    rc = plan_call(ctx, prob, part, true, s, c);
    if (rc != PEAGLE_OK)
        return rc;
    return run_bwd(ctx, prob, c, Q, K, V, O, dO, LSE, dQ, dK_acc, dV_acc, s);
}

// Runs forward + backward of the given partitions in order, adding into fp32 dK / dV accumulators.
static int run_partitions(peagle_ctx *ctx, const peagle_problem_t *prob,
                          const peagle_partition_t *parts, int32_t nparts, const void *Q,
                          const void *K, const void *V, const void *dO, void *O, float *LSE,
                          void *dQ, float *dK_acc, float *dV_acc, cudaStream_t s)
{
    for (int i = 0; i < nparts; ++i) {
        Call c;
        int rc = plan_call(ctx, prob, &parts[i], true, s, c);
        if (rc != PEAGLE_OK)
            return rc;
        // dO is known here, so the forward's epilogue leaves the backward's per-row values
        // (the separate peagle_attn_bwd forms them itself from O, dO and LSE)
        BwdArgs hand;
        if (c.plan.n_qt > 0) {
            rc = bwd_scratch(ctx, prob, c, s, hand);
            if (rc != PEAGLE_OK)
                return rc;
        }
        rc = run_fwd(ctx, prob, c, Q, K, V, O, LSE, s, dO, &hand);
        if (rc != PEAGLE_OK)
            return rc;
        rc = run_bwd(ctx, prob, c, Q, K, V, O, dO, LSE, dQ, dK_acc, dV_acc, s, true);
        if (rc != PEAGLE_OK)
            return rc;
    }
    return PEAGLE_OK;
}

static int check_partitioned_args(const peagle_problem_t *prob, const peagle_partition_t *parts,
                                  int32_t nparts)
{
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    if (nparts < 0)
        return PEAGLE_ERR_BAD_RANGE;
    Call tmp; // check every partition before anything is launched
    for (int i = 0; i < nparts; ++i) {
        rc = validate_partition(prob, &parts[i], tmp);
        if (rc != PEAGLE_OK)
            return rc;
    }
    return PEAGLE_OK;
}

int peagle_attn_partitioned(peagle_ctx *ctx, const peagle_problem_t *prob,
                            const peagle_partition_t *parts, int32_t nparts, const void *Q,
                            const void *K, const void *V, const void *dO, void *O, float *LSE,
                            void *dQ, void *dK, void *dV, void *stream)
{
    if (!ctx || !Q || !K || !V || !dO || !O || !LSE || !dQ || !dK || !dV || (nparts > 0 && !parts))
        return PEAGLE_ERR_NULL;
    int rc = check_partitioned_args(prob, parts, nparts);
    if (rc != PEAGLE_OK)
        return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return PEAGLE_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CK(cudaSetDevice(ctx->device));
    const size_t n_kv = (size_t)prob->total_tokens * prob->n_kv_heads * prob->head_dim;
    if (n_kv == 0)
        return PEAGLE_OK;
    rc = ensure(ctx, ctx->acc_buf, 2 * n_kv * sizeof(float), s);
    if (rc != PEAGLE_OK)
        return rc;
    float *dK_acc = static_cast<float *>(ctx->acc_buf.ptr);
    float *dV_acc = dK_acc + n_kv;
    CK(cudaMemsetAsync(dK_acc, 0, 2 * n_kv * sizeof(float), s));
    rc = run_partitions(ctx, prob, parts, nparts, Q, K, V, dO, O, LSE, dQ, dK_acc, dV_acc, s);
    if (rc != PEAGLE_OK)
        return rc;
    ctx->launches += launch_cast_grads(dK_acc, dV_acc, dK, dV, n_kv, s);
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_attn_partitioned_acc(peagle_ctx *ctx, const peagle_problem_t *prob,
                                const peagle_partition_t *parts, int32_t nparts, const void *Q,
                                const void *K, const void *V, const void *dO, void *O, float *LSE,
                                void *dQ, float *dK_acc, float *dV_acc, void *stream)
{
    if (!ctx || !Q || !K || !V || !dO || !O || !LSE || !dQ || !dK_acc || !dV_acc ||
        (nparts > 0 && !parts))
        return PEAGLE_ERR_NULL;
    int rc = check_partitioned_args(prob, parts, nparts);
    if (rc != PEAGLE_OK)
        return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(dO) ||
        !aligned16(dQ) || !aligned16(dK_acc) || !aligned16(dV_acc))
        return PEAGLE_ERR_ALIGN;
    CK(cudaSetDevice(ctx->device));
    return run_partitions(ctx, prob, parts, nparts, Q, K, V, dO, O, LSE, dQ, dK_acc, dV_acc,
                          static_cast<cudaStream_t>(stream));
}

int peagle_cast_grads(peagle_ctx *ctx, const float *dK_acc, const float *dV_acc, int64_t count,
                      void *dK, void *dV, void *stream)
{
    if (!ctx || !dK_acc || !dV_acc || !dK || !dV)
        return PEAGLE_ERR_NULL;
    if (count < 0 || count % 8 != 0)
        return PEAGLE_ERR_BAD_SHAPE;
    if (!aligned16(dK_acc) || !aligned16(dV_acc) || !aligned16(dK) || !aligned16(dV))
        return PEAGLE_ERR_ALIGN;
    if (count == 0)
        return PEAGLE_OK;
    CK(cudaSetDevice(ctx->device));
    ctx->launches += launch_cast_grads(dK_acc, dV_acc, dK, dV, (size_t)count,
                                       static_cast<cudaStream_t>(stream));
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_gemm_bf16(peagle_ctx *ctx, const void *A, int64_t lda, int a_transposed, const void *B,
                     int64_t ldb, int b_transposed, void *C, int64_t ldc, int c_fp32_accumulate,
                     int32_t M, int32_t N, int32_t K, void *stream)
{
    if (!ctx || !A || !B || !C)
        return PEAGLE_ERR_NULL;
    if (M < 0 || N < 0 || K <= 0)
        return PEAGLE_ERR_BAD_SHAPE;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C))
        return PEAGLE_ERR_ALIGN;
    CK(cudaSetDevice(ctx->device));
    const int n = launch_gemm(ctx->encode, A, lda, a_transposed, B, ldb, b_transposed, C, ldc,
                              c_fp32_accumulate, M, N, K, ctx->status, static_cast<cudaStream_t>(stream));
    if (n < 0)
        return n;
    ctx->launches += n;
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_layer_partitioned(peagle_ctx *ctx, const peagle_problem_t *prob,
                             const peagle_partition_t *parts, int32_t nparts, const void *X,
                             const void *W, int32_t d_model, float rope_base, const void *dO, void *O,
                             float *LSE, void *dX, void *dW, void *stream)
{
    if (!ctx || !X || !W || !dO || !O || !LSE || !dX || !dW || (nparts > 0 && !parts))
        return PEAGLE_ERR_NULL;
    int rc = check_partitioned_args(prob, parts, nparts);
    if (rc != PEAGLE_OK)
        return rc;
    if (d_model < 8 || d_model % 8 != 0 || !(rope_base > 1.f))
        return PEAGLE_ERR_BAD_SHAPE;
    if (!aligned16(X) || !aligned16(W) || !aligned16(dO) || !aligned16(O) || !aligned16(dX) || !aligned16(dW))
        return PEAGLE_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CK(cudaSetDevice(ctx->device));
    const size_t T = (size_t)prob->total_tokens;
    const int Hq = prob->n_q_heads, Hkv = prob->n_kv_heads, D = prob->head_dim;
    const size_t nq = (size_t)Hq * D, nkv = (size_t)Hkv * D, nqkv = nq + 2 * nkv, dm = (size_t)d_model;
    if (T == 0)
        return PEAGLE_OK;
    // scratch: fused rows (projection output, later its gradient), the same for key-only tokens,
    // Q K V and their gradients, fp32 sums of a segment's dK / dV, fp32 sums of dX and dW
    auto up = [](size_t b) { return (b + 255) & ~size_t(255); };
    const size_t b_fused = up(T * nqkv * 2), b_fkv = up(T * 2 * nkv * 2), b_q = up(T * nq * 2),
                 b_kv = up(T * nkv * 2), b_acc = up(T * nkv * 4), b_dx = up(T * dm * 4),
                 b_dw = up(nqkv * dm * 4);
    rc = ensure(ctx, ctx->layer_buf, b_fused + b_fkv + 2 * b_q + 4 * b_kv + 2 * b_acc + b_dx + b_dw + 256, s);
    if (rc != PEAGLE_OK)
        return rc;
    uint8_t *b = static_cast<uint8_t *>(ctx->layer_buf.ptr);
    auto take = [&](size_t n) { uint8_t *r = b; b += n; return r; };
    uint8_t *fused = take(b_fused), *fkv = take(b_fkv), *Qb = take(b_q), *dQb = take(b_q);
    uint8_t *Kb = take(b_kv), *Vb = take(b_kv), *dKb = take(b_kv), *dVb = take(b_kv);
    float *dK_acc = reinterpret_cast<float *>(take(b_acc)), *dV_acc = reinterpret_cast<float *>(take(b_acc));
    float *dX_acc = reinterpret_cast<float *>(take(b_dx)), *dW_acc = reinterpret_cast<float *>(take(b_dw));
    CK(cudaMemsetAsync(dX_acc, 0, T * dm * 4, s));
    CK(cudaMemsetAsync(dW_acc, 0, nqkv * dm * 4, s));
    const uint8_t *Xb = static_cast<const uint8_t *>(X), *Wb = static_cast<const uint8_t *>(W);
    const uint8_t *Wkv = Wb + nq * dm * 2; // rows of W that make the key and value heads
    auto gemm = [&](const void *A, long long lda, int a_t, const void *B, long long ldb, int b_t, void *C,
                    long long ldc, int acc, size_t M, size_t N, size_t K) {
        const int n = launch_gemm(ctx->encode, A, lda, a_t, B, ldb, b_t, C, ldc, acc, (int)M, (int)N, (int)K,
                                  ctx->status, s);
        if (n > 0)
            ctx->launches += n;
        return n < 0 ? n : PEAGLE_OK;
    };
    for (int i = 0; i < nparts; ++i) {
        Call c;
        rc = validate_partition(prob, &parts[i], c);
        if (rc != PEAGLE_OK)
            return rc;
        const int qb = parts[i].q.begin, qe = parts[i].q.end;
        if (qe <= qb)
            continue;
        // the visible tokens outside the segment's own block: keys only (Algorithm 1, phase 3)
        int kb[2 * MAX_KRANGES], ke[2 * MAX_KRANGES], nko = 0;
        for (int r = 0; r < c.ranges.n; ++r) {
            const int rb = c.ranges.begin[r], re = c.ranges.end[r];
            if (rb < qb) { kb[nko] = rb; ke[nko] = re < qb ? re : qb; ++nko; }
            if (re > qe) { kb[nko] = rb > qe ? rb : qe; ke[nko] = re; ++nko; }
        }
        const size_t rows = (size_t)(qe - qb);
        // ---- forward: projection and rotary prologue of the segment's tokens ...
        rc = gemm(Xb + (size_t)qb * dm * 2, dm, 0, Wb, dm, 0, fused + (size_t)qb * nqkv * 2, nqkv, 0, rows, nqkv, dm);
        if (rc != PEAGLE_OK)
            return rc;
        ctx->launches += launch_rope(false, fused + (size_t)qb * nqkv * 2, nullptr, nullptr, nullptr, nullptr,
                                     Qb + (size_t)qb * nq * 2, Kb + (size_t)qb * nkv * 2, Vb + (size_t)qb * nkv * 2,
                                     prob->anchor + qb, prob->depth + qb, (int)rows, Hq, Hkv, D, rope_base,
                                     ctx->n_sm, s);
        // ... and, again in this segment, K / V of the earlier depth-0 tokens it sees
        for (int r = 0; r < nko; ++r) {
            const size_t o = (size_t)kb[r], n = (size_t)(ke[r] - kb[r]);
            rc = gemm(Xb + o * dm * 2, dm, 0, Wkv, dm, 0, fkv + o * 2 * nkv * 2, 2 * nkv, 0, n, 2 * nkv, dm);
            if (rc != PEAGLE_OK)
                return rc;
            ctx->launches += launch_rope(false, fkv + o * 2 * nkv * 2, nullptr, nullptr, nullptr, nullptr, Qb,
                                         Kb + o * nkv * 2, Vb + o * nkv * 2, prob->anchor + o, prob->depth + o,
                                         (int)n, 0, Hkv, D, rope_base, ctx->n_sm, s);
        }
        CK(cudaGetLastError());
        // ---- attention forward and backward of the segment; dK / dV sums of this segment only
        for (int r = 0; r < c.ranges.n; ++r) {
            const size_t o = (size_t)c.ranges.begin[r] * nkv, n = (size_t)(c.ranges.end[r] - c.ranges.begin[r]) * nkv;
            CK(cudaMemsetAsync(dK_acc + o, 0, n * 4, s));
            CK(cudaMemsetAsync(dV_acc + o, 0, n * 4, s));
        }
        rc = plan_call(ctx, prob, &parts[i], true, s, c);
        if (rc != PEAGLE_OK)
            return rc;
        BwdArgs hand;
        rc = bwd_scratch(ctx, prob, c, s, hand);
        if (rc != PEAGLE_OK)
            return rc;
        rc = run_fwd(ctx, prob, c, Qb, Kb, Vb, O, LSE, s, dO, &hand);
        if (rc != PEAGLE_OK)
            return rc;
        rc = run_bwd(ctx, prob, c, Qb, Kb, Vb, O, dO, LSE, dQb, dK_acc, dV_acc, s, true);
        if (rc != PEAGLE_OK)
            return rc;
        for (int r = 0; r < c.ranges.n; ++r) {
            const size_t o = (size_t)c.ranges.begin[r] * nkv, n = (size_t)(c.ranges.end[r] - c.ranges.begin[r]) * nkv;
            ctx->launches += launch_cast_grads(dK_acc + o, dV_acc + o, dKb + o * 2, dVb + o * 2, n, s);
        }
        // ---- backward of the rotary prologue and of the projection, gradients added up over
        // the segments (within-sequence gradient accumulation)
        ctx->launches += launch_rope(true, nullptr, fused + (size_t)qb * nqkv * 2, dQb + (size_t)qb * nq * 2,
                                     dKb + (size_t)qb * nkv * 2, dVb + (size_t)qb * nkv * 2, nullptr, nullptr,
                                     nullptr, prob->anchor + qb, prob->depth + qb, (int)rows, Hq, Hkv, D,
                                     rope_base, ctx->n_sm, s);
        rc = gemm(fused + (size_t)qb * nqkv * 2, nqkv, 0, Wb, dm, 1, dX_acc + (size_t)qb * dm, dm, 1, rows, dm, nqkv);
        if (rc == PEAGLE_OK)
            rc = gemm(fused + (size_t)qb * nqkv * 2, nqkv, 1, Xb + (size_t)qb * dm * 2, dm, 1, dW_acc, dm, 1, nqkv, dm, rows);
        for (int r = 0; rc == PEAGLE_OK && r < nko; ++r) {
            const size_t o = (size_t)kb[r], n = (size_t)(ke[r] - kb[r]);
            ctx->launches += launch_rope(true, nullptr, fkv + o * 2 * nkv * 2, dQb, dKb + o * nkv * 2,
                                         dVb + o * nkv * 2, nullptr, nullptr, nullptr, prob->anchor + o,
                                         prob->depth + o, (int)n, 0, Hkv, D, rope_base, ctx->n_sm, s);
            rc = gemm(fkv + o * 2 * nkv * 2, 2 * nkv, 0, Wkv, dm, 1, dX_acc + o * dm, dm, 1, n, dm, 2 * nkv);
            if (rc == PEAGLE_OK)
                rc = gemm(fkv + o * 2 * nkv * 2, 2 * nkv, 1, Xb + o * dm * 2, dm, 1, dW_acc + nq * dm, dm, 1,
                          2 * nkv, dm, n);
        }
        if (rc != PEAGLE_OK)
            return rc;
        CK(cudaGetLastError());
    }
    ctx->launches += launch_cast_one(dX_acc, dX, T * dm, s);
    ctx->launches += launch_cast_one(dW_acc, dW, nqkv * dm, s);
    CK(cudaGetLastError());
    return PEAGLE_OK;
}

int peagle_attn_partitioned_host(peagle_ctx *ctx, const peagle_problem_t *prob,
                                 const peagle_partition_t *parts, int32_t nparts, const void *Q,
                                 const void *K, const void *V, const void *dO, void *O, float *LSE,
                                 void *dQ, void *dK, void *dV)
{
    if (!ctx || !Q || !K || !V || !dO || !O || !LSE || !dQ || !dK || !dV || (nparts > 0 && !parts))
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    if (nparts < 0)
        return PEAGLE_ERR_BAD_RANGE;
    CK(cudaSetDevice(ctx->device));
    cudaStream_t s = nullptr;
    const size_t T = (size_t)prob->total_tokens;
    const size_t nq = T * prob->n_q_heads * prob->head_dim * 2;  // bytes of a bf16 query-side tensor
    const size_t nkv = T * prob->n_kv_heads * prob->head_dim * 2;
    const size_t nlse = T * prob->n_q_heads * 4;
    const size_t nmeta = T * 4;
    auto up = [](size_t b) { return (b + 255) & ~size_t(255); };
    const size_t total = 4 * up(nq) + 4 * up(nkv) + up(nlse) + 2 * up(nmeta) + 256;
    rc = ensure(ctx, ctx->host_buf, total, s);
    if (rc != PEAGLE_OK)
        return rc;
    uint8_t *b = static_cast<uint8_t *>(ctx->host_buf.ptr);
    uint8_t *dQin = b;            b += up(nq);
    uint8_t *ddO = b;             b += up(nq);
    uint8_t *dOout = b;           b += up(nq);
    uint8_t *ddQ = b;             b += up(nq);
    uint8_t *dKin = b;            b += up(nkv);
    uint8_t *dVin = b;            b += up(nkv);
    uint8_t *ddK = b;             b += up(nkv);
    uint8_t *ddV = b;             b += up(nkv);
    uint8_t *dLSE = b;            b += up(nlse);
    uint8_t *danchor = b;         b += up(nmeta);
    uint8_t *ddepth = b;
    if (T == 0)
        return PEAGLE_OK;
    // Three streams: rows of Q / dO go in, partitions are computed, rows of O / LSE / dQ come
    // back, each query range cut into slices of HOST_SLICE rows so that the copies of one slice
    // overlap the arithmetic of another (the slices are query partitions like any other: K / V
    // and the dK / dV accumulators are shared, exactly Section 3.2's within-sequence scheme).
    {
        Call tmp;
        for (int i = 0; i < nparts; ++i) {
            rc = validate_partition(prob, &parts[i], tmp);
            if (rc != PEAGLE_OK)
                return rc;
        }
    }
    for (cudaStream_t &st : ctx->hs)
        if (!st)
            CK(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    cudaStream_t s_in = ctx->hs[0], s_c = ctx->hs[1], s_out = ctx->hs[2];
    // From here on copies into the caller's host buffers may be in flight: every error exit
    // drains the three streams first, so that nothing writes O / LSE / dQ after the return.
    auto drained = [&](int status) {
        cudaStreamSynchronize(s_in);
        cudaStreamSynchronize(s_c);
        cudaStreamSynchronize(s_out);
        return status;
    };
#define CKD(call)                                          \
    do {                                                   \
        cudaError_t e_ = (call);                           \
        if (e_ != cudaSuccess)                             \
            return drained(cuda_fail(ctx, e_, #call));     \
    } while (0)
    size_t ev_next = 0;
    auto event = [&]() -> cudaEvent_t {
        if (ev_next == ctx->hev.size()) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess)
                return nullptr;
            ctx->hev.push_back(e);
        }
        return ctx->hev[ev_next++];
    };
    const size_t row_q = (size_t)prob->n_q_heads * prob->head_dim * 2; // bytes of one Q / O row
    const size_t n_kv = T * prob->n_kv_heads * prob->head_dim;
    rc = ensure(ctx, ctx->acc_buf, 2 * n_kv * sizeof(float), s);
    if (rc != PEAGLE_OK)
        return rc;
    float *dK_acc = static_cast<float *>(ctx->acc_buf.ptr), *dV_acc = dK_acc + n_kv;
    CKD(cudaMemcpyAsync(dKin, K, nkv, cudaMemcpyHostToDevice, s_in));
    CKD(cudaMemcpyAsync(dVin, V, nkv, cudaMemcpyHostToDevice, s_in));
    CKD(cudaMemcpyAsync(danchor, prob->anchor, nmeta, cudaMemcpyHostToDevice, s_in));
    CKD(cudaMemcpyAsync(ddepth, prob->depth, nmeta, cudaMemcpyHostToDevice, s_in));
    CKD(cudaMemsetAsync(dK_acc, 0, 2 * n_kv * sizeof(float), s_c));
    peagle_problem_t dprob = *prob;
    dprob.anchor = reinterpret_cast<const int32_t *>(danchor);
    dprob.depth = reinterpret_cast<const int32_t *>(ddepth);
    constexpr int HOST_SLICE = 16 * BM;
    for (int i = 0; i < nparts; ++i) {
        for (int b0 = parts[i].q.begin; b0 < parts[i].q.end; b0 += HOST_SLICE) {
            const int b1 = b0 + HOST_SLICE < parts[i].q.end ? b0 + HOST_SLICE : parts[i].q.end;
            const size_t off = (size_t)b0 * row_q, len = (size_t)(b1 - b0) * row_q;
            peagle_partition_t sl = parts[i];
            sl.q.begin = b0;
            sl.q.end = b1;
            CKD(cudaMemcpyAsync(dQin + off, static_cast<const uint8_t *>(Q) + off, len,
                               cudaMemcpyHostToDevice, s_in));
            CKD(cudaMemcpyAsync(ddO + off, static_cast<const uint8_t *>(dO) + off, len,
                               cudaMemcpyHostToDevice, s_in));
            cudaEvent_t e_in = event(), e_c = event();
            if (!e_in || !e_c)
                return drained(PEAGLE_ERR_CUDA);
            CKD(cudaEventRecord(e_in, s_in));
            CKD(cudaStreamWaitEvent(s_c, e_in, 0));
            Call c;
            rc = plan_call(ctx, &dprob, &sl, true, s_c, c);
            BwdArgs hand;
            if (rc == PEAGLE_OK && c.plan.n_qt > 0)
                rc = bwd_scratch(ctx, &dprob, c, s_c, hand);
            if (rc == PEAGLE_OK)
                rc = run_fwd(ctx, &dprob, c, dQin, dKin, dVin, dOout, reinterpret_cast<float *>(dLSE), s_c,
                             ddO, &hand);
            if (rc == PEAGLE_OK)
                rc = run_bwd(ctx, &dprob, c, dQin, dKin, dVin, dOout, ddO,
                             reinterpret_cast<float *>(dLSE), ddQ, dK_acc, dV_acc, s_c, true);
            if (rc != PEAGLE_OK)
                return drained(rc);
            CKD(cudaEventRecord(e_c, s_c));
            CKD(cudaStreamWaitEvent(s_out, e_c, 0));
            CKD(cudaMemcpyAsync(static_cast<uint8_t *>(O) + off, dOout + off, len, cudaMemcpyDeviceToHost, s_out));
            CKD(cudaMemcpyAsync(static_cast<uint8_t *>(dQ) + off, ddQ + off, len, cudaMemcpyDeviceToHost, s_out));
            CKD(cudaMemcpy2DAsync(LSE + b0, T * 4, reinterpret_cast<float *>(dLSE) + b0, T * 4,
                                 (size_t)(b1 - b0) * 4, (size_t)prob->n_q_heads,
                                 cudaMemcpyDeviceToHost, s_out));
        }
    }
    ctx->launches += launch_cast_grads(dK_acc, dV_acc, ddK, ddV, n_kv, s_c);
    CKD(cudaGetLastError());
    cudaEvent_t e_done = event();
    if (!e_done)
        return drained(PEAGLE_ERR_CUDA);
    CKD(cudaEventRecord(e_done, s_c));
    CKD(cudaStreamWaitEvent(s_out, e_done, 0));
    CKD(cudaMemcpyAsync(dK, ddK, nkv, cudaMemcpyDeviceToHost, s_out));
    CKD(cudaMemcpyAsync(dV, ddV, nkv, cudaMemcpyDeviceToHost, s_out));
    CKD(cudaStreamSynchronize(s_in));
    CKD(cudaStreamSynchronize(s_c));
    CKD(cudaStreamSynchronize(s_out));
    return PEAGLE_OK;
#undef CKD
}

int peagle_assign_segments(const int32_t *anchor, const int32_t *depth, int32_t count, int32_t K,
                           const int32_t *boundaries, int32_t S, int32_t *segment_out)
{
    if (!anchor || !depth || !boundaries || !segment_out)
        return PEAGLE_ERR_NULL;
    if (S < 1 || K < 1 || count < 0)
        return PEAGLE_ERR_BAD_SHAPE;
    const int n = boundaries[S];
    if (boundaries[0] != 0 || n < 0)
        return PEAGLE_ERR_BAD_RANGE;
    for (int s = 0; s < S; ++s)
        if (boundaries[s + 1] < boundaries[s])
            return PEAGLE_ERR_BAD_RANGE;
    // seg_of[d][a] for the tokens present, -1 elsewhere; filled depth by depth.
    std::vector<std::vector<int32_t>> seg_of((size_t)K, std::vector<int32_t>((size_t)n, -1));
    for (int i = 0; i < count; ++i)
        if (depth[i] < 0 || depth[i] >= K || anchor[i] < 0 || anchor[i] >= n)
            return PEAGLE_ERR_BAD_META;
    auto by_position = [&](int pos) {
        int s = 0;
        while (s + 1 <= S && boundaries[s + 1] <= pos)
            ++s; // largest s with boundaries[s] <= pos
        return s < S ? s : S - 1;
    };
    for (int d = 0; d < K; ++d)
        for (int i = 0; i < count; ++i) {
            if (depth[i] != d)
                continue;
            int s;
            if (d <= 1) {
                s = by_position(anchor[i] + d);
            } else {
                s = seg_of[(size_t)d - 1][(size_t)anchor[i]];
                if (s < 0)
                    return PEAGLE_ERR_BAD_META;
            }
            seg_of[(size_t)d][(size_t)anchor[i]] = s;
            segment_out[i] = s;
        }
    return PEAGLE_OK;
}

int peagle_classify_tiles(peagle_ctx *ctx, const peagle_problem_t *prob,
                          const peagle_partition_t *part, uint8_t *host_out, int32_t *n_qtiles,
                          int32_t *n_ktiles)
{
    if (!ctx || !n_qtiles || !n_ktiles)
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    CK(cudaSetDevice(ctx->device));
    Call c;
    if (!host_out) {
        rc = validate_partition(prob, part, c);
        if (rc != PEAGLE_OK)
            return rc;
        *n_qtiles = c.plan.n_qt;
        *n_ktiles = c.plan.n_kt;
        return PEAGLE_OK;
    }
    rc = plan_call(ctx, prob, part, true, nullptr, c);
    if (rc != PEAGLE_OK)
        return rc;
    *n_qtiles = c.plan.n_qt;
    *n_ktiles = c.plan.n_kt;
    CK(cudaStreamSynchronize(nullptr));
    if (c.plan.n_qt > 0 && c.plan.n_kt > 0)
        CK(cudaMemcpy(host_out, c.plan.cls, (size_t)c.plan.n_qt * c.plan.n_kt, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < (size_t)c.plan.n_qt * c.plan.n_kt; ++i)
        if (host_out[i] == TILE_SINGLE)
            host_out[i] = TILE_PARTIAL; // an internal refinement of PARTIAL
    return PEAGLE_OK;
}

int peagle_selftest_wait_expiry(peagle_ctx *ctx, int32_t limit_ms, void *stream)
{
    if (!ctx)
        return PEAGLE_ERR_NULL;
    if (limit_ms < 1 || limit_ms > 1000)
        return PEAGLE_ERR_BAD_SHAPE;
    CK(cudaSetDevice(ctx->device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int *flag = ctx->status + 8; // a spare word of the status allocation
    CK(cudaMemsetAsync(flag, 0, sizeof(int), s));
    ctx->launches += launch_wait_expiry(ctx->status, (unsigned long long)limit_ms * 1000000ull, flag, s);
    CK(cudaGetLastError());
    int reached = 0;
    CK(cudaMemcpyAsync(&reached, flag, sizeof(int), cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    return reached == 1 ? PEAGLE_OK : PEAGLE_ERR_CUDA;
}

int peagle_mask_dense(peagle_ctx *ctx, const peagle_problem_t *prob,
                      const peagle_partition_t *part, uint8_t *host_out)
{
    if (!ctx || !host_out)
        return PEAGLE_ERR_NULL;
    int rc = validate_problem(prob);
    if (rc != PEAGLE_OK)
        return rc;
    CK(cudaSetDevice(ctx->device));
    Call c;
    rc = validate_partition(prob, part, c);
    if (rc != PEAGLE_OK)
        return rc;
    const size_t q_len = (size_t)(c.plan.q_end - c.plan.q_begin);
    const size_t n = q_len * (size_t)c.plan.T;
    if (n > (size_t(1) << 26))
        return PEAGLE_ERR_TOO_LARGE;
    if (n == 0)
        return PEAGLE_OK;
    rc = plan_call(ctx, prob, part, false, nullptr, c);
    if (rc != PEAGLE_OK)
        return rc;
    uint8_t *dev = nullptr;
    if (cudaMalloc(&dev, n) != cudaSuccess) {
        cudaGetLastError();
        return PEAGLE_ERR_WORKSPACE;
    }
    ctx->launches += launch_mask_dense(c.plan, c.ranges, dev, nullptr);
    cudaError_t e = cudaMemcpy(host_out, dev, n, cudaMemcpyDeviceToHost);
    cudaFree(dev);
    if (e != cudaSuccess)
        return cuda_fail(ctx, e, "cudaMemcpy(mask)");
    return PEAGLE_OK;
}

} // extern "C"
