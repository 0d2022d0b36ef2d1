// Host side of the C ABI declared in include/weave_moe.h: argument checks, workspace layout,
// TMA descriptor encoding, the single cooperative launch per layer, and the small query calls.
// No device memory is allocated here; everything lives in the caller's workspace.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/weave_moe.h"
#include "weave_kernel.cuh"

using namespace weave;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr int kWaitLogSlots = 1024 * 8;      // one slot per warp of up to 1024 CTAs

struct Layout {
    size_t ctl, fcnt, xe_ready, h_ready, wait_log, zero_end;       // [0, zero_end) is zeroed at create / recovery
    size_t hist, topk, gates, row_of, token_of, counts, offsets, bw, tf, uniq_mask, xs;
    size_t xe, hbuf, y, st_x, st_logits, st_out, st2_x, st2_logits, st2_out, total;
    int nmb_max, nblk_max, p_max;
};

bool shape_ok(const weave_moe_config *c)
{
    if (!c) return false;
    if (c->hidden < 128 || c->hidden % 128 || c->ffn < 128 || c->ffn % 128) return false;
    if (c->hidden > 16384) return false;     // one bf16 row must fit a 32 KB movement buffer
    if (c->num_experts < 1 || c->num_shared < 0 || c->num_experts + c->num_shared > kMaxEE) return false;
    if (c->top_k < 1 || c->top_k > c->num_experts || c->top_k > kMaxTopK || c->num_shared > 8) return false;
    if (c->max_tokens < 1 || c->max_tokens > (1 << 20)) return false;
    // row and weight-row coordinates of the TMA descriptors are 32-bit
    const long long rows_w = (long long)(c->num_experts + c->num_shared) * 2 * c->ffn;
    const long long rows_d = (long long)(c->num_experts + c->num_shared) * c->hidden;
    const long long p_max = (long long)c->max_tokens * (c->top_k + c->num_shared);
    if (rows_w >= (1ll << 31) || rows_d >= (1ll << 31) || p_max >= (1ll << 30)) return false;
    return true;
}

Layout make_layout(const weave_moe_config *c)
{
    Layout L{};
    const int EE = c->num_experts + c->num_shared;
    const int ks = c->top_k + c->num_shared;
    const size_t T = (size_t)c->max_tokens;
    L.p_max = (int)(T * ks);
    L.nblk_max = (int)((T + kRouteBlock - 1) / kRouteBlock);
    L.nmb_max = (L.p_max + kBM - 1) / kBM + EE * kFine;
    size_t o = 0;
    auto take = [&](size_t bytes, size_t al) { o = align_up(o, al); size_t r = o; o += bytes; return r; };
    L.ctl = take(sizeof(Ctl), 256);
    L.fcnt = take(sizeof(unsigned) * kFine * kMaxEE, 256);
    L.xe_ready = take(sizeof(unsigned) * L.nmb_max, 256);
    L.h_ready = take(sizeof(unsigned) * L.nmb_max, 256);
    L.wait_log = take(sizeof(int4) * kWaitLogSlots, 256);     // written by failed waits only, cleared by the host
    L.zero_end = align_up(o, 256);
    L.hist = take(sizeof(int) * (size_t)L.nblk_max * kMaxEE, 256);
    L.topk = take(sizeof(int) * T * c->top_k, 256);
    L.gates = take(sizeof(float) * T * c->top_k, 256);
    L.row_of = take(sizeof(int) * T * c->top_k, 256);
    L.token_of = take(sizeof(int) * (size_t)L.p_max, 256);
    L.counts = take(sizeof(int) * EE, 256);
    L.offsets = take(sizeof(int) * (EE + 1), 256);
    L.bw = take(sizeof(float) * 1024, 256);
    L.tf = take(sizeof(float) * 1024, 256);
    L.uniq_mask = take(sizeof(unsigned long long) * (size_t)L.nblk_max, 256);
    L.xs = take(T * c->hidden * 2, 1024);       // expert-parallel share: staged copies of remote tokens
    L.xe = take((size_t)L.p_max * c->hidden * 2, 1024);
    L.hbuf = take((size_t)L.p_max * c->ffn * 2, 1024);
    L.y = take((size_t)L.p_max * c->hidden * 2, 1024);
    L.st_x = take(T * c->hidden * 2, 1024);
    L.st_logits = take(T * c->num_experts * 4, 1024);
    L.st_out = take(T * c->hidden * 2, 1024);
    L.st2_x = take(T * c->hidden * 2, 1024);          // second staging slot of the pipelined host path
    L.st2_logits = take(T * c->num_experts * 4, 1024);
    L.st2_out = take(T * c->hidden * 2, 1024);
    L.total = align_up(o, 1024);
    return L;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct weave_moe {
    weave_moe_config cfg;
    Layout L;
    uint8_t *ws;
    int n_sm;      // SMs of the device
    int n_cta;     // persistent CTAs = SMs rounded down to whole pairs
    int device;
    int mode, fixed_c, fixed_K, fixed_steal;
    int c_min, c_max, c_step;
    float alpha, eff[4];
    int timeout_ms;
    int withhold_mb;
    int last_T;
    cudaStream_t last_stream;
    int last_cuda_error;
    int last_timeout_where;
    std::vector<int32_t> *wait_log;     // records of the last failed launch: {cta, warp, wait id, object, wanted, how}
    int kinds;         // plan kinds AUTO may choose (bit mask)
    int elastic;       // -1 = on under AUTO only, 0 = off, 1 = on
    const float *bw_dev, *tf_dev;     // cost tables on the device (in the workspace unless set otherwise)
    void *trace;
    int trace_cap;
    int ep_rank, ep_size;
    // pipelined host path: copy streams and per-slot events, created on first use
    bool pipe_ready;
    unsigned long long pipe_calls;
    cudaStream_t pipe_h2d, pipe_d2h;
    cudaEvent_t pipe_in_ready[2], pipe_k_done[2], pipe_out_done[2];
    TmaMaps tm;
};

namespace {

int cuda_fail(weave_moe *h, cudaError_t e)
{
    if (h) h->last_cuda_error = (int)e;
    return WEAVE_ERR_CUDA;
}

// bf16 matrix [rows][cols] row-major, box = 64 columns (128 bytes) x 128 rows, 128-byte swizzle
int encode_map(EncodeTiledFn fn, CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols, bool weights,
               uint32_t box_rows = kBM)
{
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {kBK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : (int)r;
}

int encode_maps(EncodeTiledFn fn, TmaMaps *m, const void *xe, const void *hbuf, const void *gate_up, const void *down,
                uint64_t p_max, uint64_t EE, uint64_t hidden, uint64_t ffn)
{
    int r = 0;
    r |= encode_map(fn, &m->xe, xe, p_max, hidden, false);
    r |= encode_map(fn, &m->wgu, gate_up, EE * 2 * ffn, hidden, true);
    r |= encode_map(fn, &m->h, hbuf, p_max, ffn, false);
    r |= encode_map(fn, &m->wd, down, EE * hidden, ffn, true);
    r |= encode_map(fn, &m->wgu64, gate_up, EE * 2 * ffn, hidden, true, 64);
    for (int i = 0; i < 4; ++i) {
        r |= encode_map(fn, &m->xe_n[i], xe, p_max, hidden, false, 8u << i);
        r |= encode_map(fn, &m->h_n[i], hbuf, p_max, ffn, false, 8u << i);
    }
    return r;
}

void default_tables(int n_sm, std::vector<float> &bw, std::vector<float> &tf)
{
    // Curves measured with the calibration tool on a B200 (148 SMs, power-limited clocks), of the
    // shape the paper's Figure 4 describes: movement bandwidth grows linearly with the number of
    // movement SMs (about 42 GB/s of dispatch payload per SM, no saturation up to half the SMs),
    // GEMM throughput is sub-linear in the number of GEMM SMs (close to a square root: with fewer
    // busy tensor cores the clocks rise).  Units: byte/us and FLOP/us.  weave_moe_set_cost_tables()
    // replaces them with curves measured for a particular layer shape.
    bw.assign(n_sm + 1, 0.f);
    tf.assign(n_sm + 1, 0.f);
    for (int i = 1; i <= n_sm; ++i) {
        bw[i] = 42.0e3f * (float)i;
        tf[i] = 1.30e9f * sqrtf((float)i / (float)n_sm);
    }
    bw[0] = bw[1];
    tf[0] = tf[1];
}

int upload_tables(weave_moe *h, const float *bw, const float *tf)
{
    cudaError_t e = cudaMemcpy(h->ws + h->L.bw, bw, sizeof(float) * (h->n_sm + 1), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail(h, e);
    e = cudaMemcpy(h->ws + h->L.tf, tf, sizeof(float) * (h->n_sm + 1), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return WEAVE_OK;
}

}  // namespace

extern "C" {

size_t weave_moe_workspace_bytes(const weave_moe_config *cfg)
{
    if (!shape_ok(cfg)) return 0;
    return make_layout(cfg).total;
}

int weave_moe_create(const weave_moe_config *cfg, weave_moe_t *out)
{
    if (!out) return WEAVE_ERR_INVALID_ARG;
    *out = nullptr;
    if (!shape_ok(cfg)) return WEAVE_ERR_INVALID_ARG;
    if (!cfg->gate_up || !cfg->down || !cfg->workspace) return WEAVE_ERR_INVALID_ARG;
    if (((uintptr_t)cfg->gate_up & 15) || ((uintptr_t)cfg->down & 15) || ((uintptr_t)cfg->workspace & 1023))
        return WEAVE_ERR_INVALID_ARG;
    Layout L = make_layout(cfg);
    if (cfg->workspace_bytes < L.total) return WEAVE_ERR_WORKSPACE;

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return WEAVE_ERR_CUDA;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return WEAVE_ERR_CUDA;
    if (prop.major != 10 || !prop.cooperativeLaunch) return WEAVE_ERR_UNSUPPORTED_DEVICE;
    if ((int)prop.sharedMemPerBlockOptin < kSmemBytes) return WEAVE_ERR_UNSUPPORTED_DEVICE;
    if (prop.multiProcessorCount + 1 > 1024 || prop.multiProcessorCount < 4) return WEAVE_ERR_UNSUPPORTED_DEVICE;

    weave_moe *h = new (std::nothrow) weave_moe();
    if (!h) return WEAVE_ERR_INVALID_ARG;
    h->cfg = *cfg;
    h->L = L;
    h->ws = static_cast<uint8_t *>(cfg->workspace);
    h->n_sm = prop.multiProcessorCount & ~1;     // the scheduler counts SMs in whole CTA pairs
    h->n_cta = h->n_sm;
    h->device = dev;
    h->mode = WEAVE_SCHED_AUTO;
    h->fixed_c = (h->n_sm * 15 / 100 + 1) & ~1;
    h->fixed_K = 1;
    h->fixed_steal = 0;
    h->c_min = 2;
    h->c_max = h->n_sm / 2;
    h->c_step = 2;
    h->alpha = 0.8f;
    h->eff[0] = 1.0f; h->eff[1] = 0.83f; h->eff[2] = 0.62f; h->eff[3] = 0.43f;     // measured (calibration tool)
    h->timeout_ms = 4000;
    h->withhold_mb = -1;
    h->last_T = 0;
    h->last_stream = nullptr;
    h->last_cuda_error = 0;
    h->last_timeout_where = 0;
    h->wait_log = new (std::nothrow) std::vector<int32_t>();
    h->kinds = 7;       // split, dispatch-all, phased; the rejoin kind is opt-in (weave_moe_set_model_options)
    h->elastic = -1;
    h->bw_dev = reinterpret_cast<const float *>(h->ws + L.bw);
    h->tf_dev = reinterpret_cast<const float *>(h->ws + L.tf);
    h->trace = nullptr;
    h->trace_cap = 0;
    h->ep_rank = 0;
    h->ep_size = 1;
    h->pipe_ready = false;
    h->pipe_calls = 0;

    e = cudaFuncSetAttribute(weave_moe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) { int rc = cuda_fail(h, e); delete h; return rc; }
    e = cudaFuncSetAttribute(weave_moe_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 0);
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, weave_moe_kernel, kThreads, kSmemBytes);
    if (e != cudaSuccess || occ < 1) { delete h; return WEAVE_ERR_UNSUPPORTED_DEVICE; }
    {
        cudaLaunchConfig_t lc;
        memset(&lc, 0, sizeof(lc));
        lc.gridDim = dim3(h->n_cta); lc.blockDim = dim3(kThreads); lc.dynamicSmemBytes = (size_t)kSmemBytes;
        lc.attrs = nullptr; lc.numAttrs = 0;      // the cluster shape (2,1,1) is compiled into the kernel
        int ncl = 0;
        e = cudaOccupancyMaxActiveClusters(&ncl, (const void *)weave_moe_kernel, &lc);
        if (e != cudaSuccess || ncl * 2 < h->n_cta) { delete h; return WEAVE_ERR_UNSUPPORTED_DEVICE; }
    }

    void *fnp = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres);
    if (e != cudaSuccess || !fnp || qres != cudaDriverEntryPointSuccess) { delete h; return WEAVE_ERR_UNSUPPORTED_DEVICE; }
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fnp);
    const int EE = cfg->num_experts + cfg->num_shared;
    int r = 0;
    r = encode_maps(enc, &h->tm, h->ws + L.xe, h->ws + L.hbuf, cfg->gate_up, cfg->down, (uint64_t)L.p_max, (uint64_t)EE,
                    (uint64_t)cfg->hidden, (uint64_t)cfg->ffn);
    if (r) { h->last_cuda_error = r; delete h; return WEAVE_ERR_CUDA; }

    e = cudaMemset(h->ws, 0, L.zero_end);
    if (e != cudaSuccess) { int rc = cuda_fail(h, e); delete h; return rc; }
    std::vector<float> bw, tf;
    default_tables(h->n_sm, bw, tf);
    int rc = upload_tables(h, bw.data(), tf.data());
    if (rc) { delete h; return rc; }
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { rc = cuda_fail(h, e); delete h; return rc; }
    *out = h;
    return WEAVE_OK;
}

int weave_moe_forward(weave_moe_t h, const void *x, const float *logits, void *out, int T, void *stream)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return WEAVE_ERR_INVALID_ARG;
    if (T == 0) return WEAVE_OK;
    if (!x || !logits || !out) return WEAVE_ERR_INVALID_ARG;
    if (((uintptr_t)x & 15) || ((uintptr_t)logits & 15) || ((uintptr_t)out & 15)) return WEAVE_ERR_INVALID_ARG;

    const weave_moe_config &c = h->cfg;
    const Layout &L = h->L;
    KParams p;
    memset(&p, 0, sizeof(p));
    p.T = T; p.H = c.hidden; p.I = c.ffn; p.E = c.num_experts; p.S = c.num_shared; p.k = c.top_k;
    p.EE = c.num_experts + c.num_shared;
    p.nblk = (T + kRouteBlock - 1) / kRouteBlock;
    p.mode = h->mode; p.fixed_c = h->fixed_c; p.fixed_K = h->fixed_K; p.fixed_steal = h->fixed_steal;
    p.nt0 = c.ffn / kTN0;
    p.nt1 = (c.hidden + 255) / 256;
    p.nmb_max = L.nmb_max;
    p.withhold_mb = h->withhold_mb;
    p.elastic_steal = h->elastic < 0 ? ((h->mode == WEAVE_SCHED_AUTO) ? 1 : 0) : h->elastic;
    p.kinds = h->kinds;
    p.c_min = h->c_min; p.c_max = h->c_max; p.c_step = h->c_step;
    p.alpha = h->alpha;
    for (int i = 0; i < 4; ++i) p.eff[i] = h->eff[i];
    p.timeout_ns = (unsigned long long)h->timeout_ms * 1000000ull;
    p.x = static_cast<const __nv_bfloat16 *>(x);
    p.logits = logits;
    p.out = static_cast<__nv_bfloat16 *>(out);
    uint8_t *ws = h->ws;
    p.ctl = reinterpret_cast<Ctl *>(ws + L.ctl);
    p.fcnt = reinterpret_cast<unsigned *>(ws + L.fcnt);
    p.hist = reinterpret_cast<int *>(ws + L.hist);
    p.topk_idx = reinterpret_cast<int *>(ws + L.topk);
    p.gates = reinterpret_cast<float *>(ws + L.gates);
    p.row_of = reinterpret_cast<int *>(ws + L.row_of);
    p.token_of = reinterpret_cast<int *>(ws + L.token_of);
    p.counts = reinterpret_cast<int *>(ws + L.counts);
    p.offsets = reinterpret_cast<int *>(ws + L.offsets);
    p.xe = reinterpret_cast<__nv_bfloat16 *>(ws + L.xe);
    p.hbuf = reinterpret_cast<__nv_bfloat16 *>(ws + L.hbuf);
    p.y = reinterpret_cast<__nv_bfloat16 *>(ws + L.y);
    p.xe_ready = reinterpret_cast<unsigned *>(ws + L.xe_ready);
    p.h_ready = reinterpret_cast<unsigned *>(ws + L.h_ready);
    p.bw = h->bw_dev;
    p.tf = h->tf_dev;
    p.ep_rank = h->ep_rank;
    p.ep_size = h->ep_size;
    p.ep_tshard = (T + h->ep_size - 1) / h->ep_size;
    p.xs = reinterpret_cast<__nv_bfloat16 *>(ws + L.xs);
    p.uniq_mask = reinterpret_cast<unsigned long long *>(ws + L.uniq_mask);
    p.trace = reinterpret_cast<uint4 *>(h->trace);
    p.trace_cap = h->trace_cap;
    p.wait_log = reinterpret_cast<int4 *>(ws + L.wait_log);

    void *args[] = {&p, &h->tm};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // one CTA per SM; the kernel is compiled with a cluster shape of two neighbouring CTAs (the GEMM
    // phase's CTA pairs); cooperative, so that all CTAs are co-resident for the in-kernel grid
    // barrier and flag waits
    cudaError_t e = cudaLaunchCooperativeKernel((const void *)weave_moe_kernel, dim3(h->n_cta), dim3(kThreads), args,
                                                (size_t)kSmemBytes, st);
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->last_T = T;
    h->last_stream = st;
    return WEAVE_OK;
}

int weave_moe_forward_host(weave_moe_t h, const void *x_host, const float *logits_host, void *out_host, int T,
                           void *stream)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return WEAVE_ERR_INVALID_ARG;
    if (T == 0) return WEAVE_OK;
    if (!x_host || !logits_host || !out_host) return WEAVE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const weave_moe_config &c = h->cfg;
    uint8_t *ws = h->ws;
    const size_t xb = (size_t)T * c.hidden * 2, lb = (size_t)T * c.num_experts * 4;
    cudaError_t e = cudaMemcpyAsync(ws + h->L.st_x, x_host, xb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(h, e);
    e = cudaMemcpyAsync(ws + h->L.st_logits, logits_host, lb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(h, e);
    int rc = weave_moe_forward(h, ws + h->L.st_x, reinterpret_cast<const float *>(ws + h->L.st_logits),
                               ws + h->L.st_out, T, stream);
    if (rc) return rc;
    e = cudaMemcpyAsync(out_host, ws + h->L.st_out, xb, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return WEAVE_OK;
}

/* Throughput-oriented host path: the copies run on two internal copy streams and two staging
 * slots alternate, so that the H2D copy of call i+1 and the D2H copy of call i-1 overlap the
 * kernel of call i (the kernels themselves stay ordered on the caller's stream). */
int weave_moe_forward_host_pipelined(weave_moe_t h, const void *x_host, const float *logits_host, void *out_host,
                                     int T, void *stream)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return WEAVE_ERR_INVALID_ARG;
    if (T == 0) return WEAVE_OK;
    if (!x_host || !logits_host || !out_host) return WEAVE_ERR_INVALID_ARG;
    cudaError_t e;
    if (!h->pipe_ready) {
        if ((e = cudaStreamCreateWithFlags(&h->pipe_h2d, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(h, e);
        if ((e = cudaStreamCreateWithFlags(&h->pipe_d2h, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(h, e);
        for (int i = 0; i < 2; ++i) {
            if ((e = cudaEventCreateWithFlags(&h->pipe_in_ready[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(h, e);
            if ((e = cudaEventCreateWithFlags(&h->pipe_k_done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(h, e);
            if ((e = cudaEventCreateWithFlags(&h->pipe_out_done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(h, e);
        }
        h->pipe_ready = true;
        h->pipe_calls = 0;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const weave_moe_config &c = h->cfg;
    const Layout &L = h->L;
    uint8_t *ws = h->ws;
    const int slot = (int)(h->pipe_calls & 1ull);
    uint8_t *sx = ws + (slot ? L.st2_x : L.st_x), *sl = ws + (slot ? L.st2_logits : L.st_logits),
            *so = ws + (slot ? L.st2_out : L.st_out);
    const size_t xb = (size_t)T * c.hidden * 2, lb = (size_t)T * c.num_experts * 4;
    // the slot's inputs may be overwritten once the kernel that read them (two calls ago) is done
    if (h->pipe_calls >= 2 && (e = cudaStreamWaitEvent(h->pipe_h2d, h->pipe_k_done[slot], 0)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaMemcpyAsync(sx, x_host, xb, cudaMemcpyHostToDevice, h->pipe_h2d)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaMemcpyAsync(sl, logits_host, lb, cudaMemcpyHostToDevice, h->pipe_h2d)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaEventRecord(h->pipe_in_ready[slot], h->pipe_h2d)) != cudaSuccess) return cuda_fail(h, e);
    // the kernel needs its inputs, and its output slot must have been copied out (two calls ago)
    if ((e = cudaStreamWaitEvent(st, h->pipe_in_ready[slot], 0)) != cudaSuccess) return cuda_fail(h, e);
    if (h->pipe_calls >= 2 && (e = cudaStreamWaitEvent(st, h->pipe_out_done[slot], 0)) != cudaSuccess) return cuda_fail(h, e);
    int rc = weave_moe_forward(h, sx, reinterpret_cast<const float *>(sl), so, T, stream);
    if (rc) return rc;
    if ((e = cudaEventRecord(h->pipe_k_done[slot], st)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaStreamWaitEvent(h->pipe_d2h, h->pipe_k_done[slot], 0)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaMemcpyAsync(out_host, so, xb, cudaMemcpyDeviceToHost, h->pipe_d2h)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaEventRecord(h->pipe_out_done[slot], h->pipe_d2h)) != cudaSuccess) return cuda_fail(h, e);
    h->pipe_calls += 1;
    return WEAVE_OK;
}

int weave_moe_host_wait(weave_moe_t h)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (!h->pipe_ready || h->pipe_calls == 0) return WEAVE_OK;
    cudaError_t e = cudaStreamSynchronize(h->pipe_d2h);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return WEAVE_OK;
}

int weave_moe_destroy(weave_moe_t h)
{
    if (h && h->pipe_ready) {
        cudaStreamSynchronize(h->pipe_d2h);
        cudaStreamSynchronize(h->pipe_h2d);
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(h->pipe_in_ready[i]);
            cudaEventDestroy(h->pipe_k_done[i]);
            cudaEventDestroy(h->pipe_out_done[i]);
        }
        cudaStreamDestroy(h->pipe_h2d);
        cudaStreamDestroy(h->pipe_d2h);
    }
    if (h) delete h->wait_log;
    delete h;
    return WEAVE_OK;
}

int weave_moe_set_schedule(weave_moe_t h, int mode, int c, int K, int steal)
{
    if (!h || mode < WEAVE_SCHED_AUTO || mode > WEAVE_SCHED_SERIAL) return WEAVE_ERR_INVALID_ARG;
    if (mode == WEAVE_SCHED_FIXED) {
        if (c < 1 || (K != 1 && K != 2 && K != 4 && K != 8) || steal < 0) return WEAVE_ERR_INVALID_ARG;
        h->fixed_c = c; h->fixed_K = K; h->fixed_steal = steal;
    }
    h->mode = mode;
    return WEAVE_OK;
}

int weave_moe_set_cost_tables(weave_moe_t h, const float *bw, const float *tflops, const float *eff_chunk,
                              float alpha, int c_min, int c_max, int c_step)
{
    if (!h || !bw || !tflops || !eff_chunk) return WEAVE_ERR_INVALID_ARG;
    if (!(alpha >= 0.f && alpha < 1.f) || c_min < 2 || c_step < 2 || c_max < c_min) return WEAVE_ERR_INVALID_ARG;
    if ((c_min & 1) || (c_step & 1)) return WEAVE_ERR_INVALID_ARG;     // movement SMs come in CTA pairs
    if ((c_max - c_min) / c_step + 1 > 64) return WEAVE_ERR_INVALID_ARG;      // one candidate c per four threads
    for (int i = 1; i <= h->n_sm; ++i)
        if (!(bw[i] > 0.f) || !(tflops[i] > 0.f)) return WEAVE_ERR_INVALID_ARG;
    for (int i = 0; i < 4; ++i)
        if (!(eff_chunk[i] > 0.f && eff_chunk[i] <= 1.f)) return WEAVE_ERR_INVALID_ARG;
    if (h->last_stream || h->last_T) cudaStreamSynchronize(h->last_stream);
    int rc = upload_tables(h, bw, tflops);
    if (rc) return rc;
    for (int i = 0; i < 4; ++i) h->eff[i] = eff_chunk[i];
    h->alpha = alpha; h->c_min = c_min; h->c_max = c_max; h->c_step = c_step;
    return WEAVE_OK;
}

int weave_moe_get_plan(weave_moe_t h, int *c, int *K, int *n_steal, float *t_total_us)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    Ctl ctl;
    e = cudaMemcpy(&ctl, h->ws + h->L.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (c) *c = ctl.plan_c;
    if (K) *K = ctl.plan_K;
    if (n_steal) *n_steal = ctl.plan_steal;
    if (t_total_us) *t_total_us = ctl.plan_t;
    return WEAVE_OK;
}

int weave_moe_get_plan_kind(weave_moe_t h, int *kind)
{
    if (!h || !kind) return WEAVE_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    Ctl ctl;
    e = cudaMemcpy(&ctl, h->ws + h->L.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    *kind = ctl.plan_kind;
    return WEAVE_OK;
}

int weave_moe_set_model_options(weave_moe_t h, int kinds_mask, int elastic)
{
    if (!h || (kinds_mask & 15) == 0 || (kinds_mask & ~15) || elastic < -1 || elastic > 1) return WEAVE_ERR_INVALID_ARG;
    h->kinds = kinds_mask;
    h->elastic = elastic;
    return WEAVE_OK;
}

int weave_moe_get_geometry(weave_moe_t h, int *n_sm, int *block_m, int *tile_n0, int *tile_n1, int *route_block,
                           int *combine_tile, int *gemm_tile_m)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (n_sm) *n_sm = h->n_sm;
    if (block_m) *block_m = kBM;
    if (tile_n0) *tile_n0 = kTN0;
    if (tile_n1) *tile_n1 = 256;
    if (gemm_tile_m) *gemm_tile_m = 2 * kBM;
    if (route_block) *route_block = kRouteBlock;
    if (combine_tile) *combine_tile = kCombTile;
    return WEAVE_OK;
}

int weave_moe_get_routing(weave_moe_t h, const int32_t **topk_idx, const float **gates, const int32_t **counts,
                          const int32_t **offsets, const int32_t **row_of, const int32_t **token_of)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    const Layout &L = h->L;
    if (topk_idx) *topk_idx = reinterpret_cast<const int32_t *>(h->ws + L.topk);
    if (gates) *gates = reinterpret_cast<const float *>(h->ws + L.gates);
    if (counts) *counts = reinterpret_cast<const int32_t *>(h->ws + L.counts);
    if (offsets) *offsets = reinterpret_cast<const int32_t *>(h->ws + L.offsets);
    if (row_of) *row_of = reinterpret_cast<const int32_t *>(h->ws + L.row_of);
    if (token_of) *token_of = reinterpret_cast<const int32_t *>(h->ws + L.token_of);
    return WEAVE_OK;
}

int weave_moe_get_intermediates(weave_moe_t h, const void **xe, const void **hbuf, const void **y)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (xe) *xe = h->ws + h->L.xe;
    if (hbuf) *hbuf = h->ws + h->L.hbuf;
    if (y) *y = h->ws + h->L.y;
    return WEAVE_OK;
}

int weave_moe_status(weave_moe_t h)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    Ctl ctl;
    e = cudaMemcpy(&ctl, h->ws + h->L.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    int st = ctl.status;
    if (st != 0) {
        // keep what the failed waits wrote down, for weave_moe_debug_wait_log()
        if (h->wait_log) {
            std::vector<int4> raw(kWaitLogSlots);
            h->wait_log->clear();
            if (cudaMemcpy(raw.data(), h->ws + h->L.wait_log, sizeof(int4) * kWaitLogSlots, cudaMemcpyDeviceToHost) == cudaSuccess)
                for (int i = 0; i < kWaitLogSlots; ++i)
                    if (raw[i].w != 0) {
                        const int32_t rec[6] = {i / 8, i % 8, raw[i].x, raw[i].y, raw[i].z, raw[i].w};
                        h->wait_log->insert(h->wait_log->end(), rec, rec + 6);
                    }
        }
        // a failed launch may have left flags behind: start from a clean slate
        e = cudaMemset(h->ws, 0, h->L.zero_end);
        if (e != cudaSuccess) return cuda_fail(h, e);
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return cuda_fail(h, e);
        h->last_timeout_where = st == WEAVE_ERR_TIMEOUT ? ctl.timeout_where : 0;
    } else {
        h->last_timeout_where = 0;
    }
    return st;
}

int weave_moe_set_expert_parallel(weave_moe_t h, int ep_rank, int ep_size)
{
    if (!h || ep_size < 1 || ep_rank < 0 || ep_rank >= ep_size) return WEAVE_ERR_INVALID_ARG;
    if (ep_size > 1 && (h->cfg.num_experts % ep_size != 0 || h->cfg.num_shared != 0)) return WEAVE_ERR_INVALID_ARG;
    h->ep_rank = ep_rank;
    h->ep_size = ep_size;
    return WEAVE_OK;
}

int weave_moe_get_ep_descriptors(weave_moe_t h, long long *x_local, long long *x_in, long long *x_in_uniq)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize(h->last_stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    Ctl ctl;
    e = cudaMemcpy(&ctl, h->ws + h->L.ctl, sizeof(Ctl), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (x_local) *x_local = ctl.ep_x_local;
    if (x_in) *x_in = ctl.ep_x_in;
    if (x_in_uniq) *x_in_uniq = ctl.ep_x_in_uniq;
    return WEAVE_OK;
}

int weave_moe_set_sm_count(weave_moe_t h, int n_sm)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (n_sm < 4 || (n_sm & 1) || n_sm > h->n_sm) return WEAVE_ERR_INVALID_ARG;
    h->n_cta = n_sm;
    return WEAVE_OK;
}

int weave_moe_set_timeout_ms(weave_moe_t h, int ms)
{
    if (!h || ms < 1) return WEAVE_ERR_INVALID_ARG;
    h->timeout_ms = ms;
    return WEAVE_OK;
}

int weave_moe_debug_withhold_flag(weave_moe_t h, int m_block)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    h->withhold_mb = m_block;
    return WEAVE_OK;
}

int weave_moe_set_trace(weave_moe_t h, void *buf, int events_per_cta)
{
    if (!h) return WEAVE_ERR_INVALID_ARG;
    if (buf && (events_per_cta < 2 || ((uintptr_t)buf & 15))) return WEAVE_ERR_INVALID_ARG;
    h->trace = buf;
    h->trace_cap = buf ? events_per_cta : 0;
    return WEAVE_OK;
}

int weave_moe_last_cuda_error(weave_moe_t h) { return h ? h->last_cuda_error : 0; }

int weave_moe_last_timeout_where(weave_moe_t h) { return h ? h->last_timeout_where : 0; }

int weave_moe_debug_wait_log(weave_moe_t h, int32_t *out, int max_records)
{
    if (!h || max_records < 0 || (max_records > 0 && !out)) return WEAVE_ERR_INVALID_ARG;
    if (!h->wait_log) return 0;
    const int n = (int)(h->wait_log->size() / 6);
    for (int i = 0; i < n && i < max_records; ++i)
        for (int j = 0; j < 6; ++j) out[i * 6 + j] = (*h->wait_log)[(size_t)i * 6 + j];
    return n;
}

int weave_moe_debug_gemm_queue(const int32_t *rows, int num_segments, int num_chunks, int nt0, int nt1, int32_t *out,
                               int max_tiles)
{
    if (!rows || num_segments < 1 || nt0 < 1 || nt1 < 1) return WEAVE_ERR_INVALID_ARG;
    if (num_chunks != 1 && num_chunks != 2 && num_chunks != 4 && num_chunks != 8) return WEAVE_ERR_INVALID_ARG;
    if (num_segments * num_chunks > kMaxSeg) return WEAVE_ERR_INVALID_ARG;
    // the tables the kernel's set-up builds in shared memory, built here the same way
    std::vector<unsigned char> raw(sizeof(SmemTail), 0);
    SmemTail &S = *reinterpret_cast<SmemTail *>(raw.data());
    KParams p;
    memset(&p, 0, sizeof(p));
    p.EE = num_segments; p.nt0 = nt0; p.nt1 = nt1; p.H = kBK; p.I = kBK;
    int mb = 0, pt = 0, row = 0;
    for (int j = 0; j < num_chunks; ++j) {
        S.chunk_mb0[j] = mb; S.chunk_pt0[j] = pt; S.chunk_tile0[j] = pt * (nt0 + nt1);
        int nodd = 0;
        for (int e = 0; e < num_segments; ++e) {
            const int r = rows[j * num_segments + e];
            if (r < 0) return WEAVE_ERR_INVALID_ARG;
            const int mbs = (r + kBM - 1) / kBM;
            S.seg_mb0[j * num_segments + e] = mb; S.seg_pt0[j * num_segments + e] = pt;
            S.seg_row0[j * num_segments + e] = row; S.seg_rows[j * num_segments + e] = r;
            mb += mbs; pt += (mbs + 1) / 2; row += r; nodd += mbs & 1;
        }
        S.chunk_nswap[j] = nodd;
    }
    S.seg_mb0[num_chunks * num_segments] = mb; S.seg_pt0[num_chunks * num_segments] = pt;
    S.chunk_mb0[num_chunks] = mb; S.chunk_pt0[num_chunks] = pt; S.chunk_tile0[num_chunks] = pt * (nt0 + nt1);
    S.K = num_chunks;
    const int n = pt * (nt0 + nt1);
    for (int g = 0; g < n && g < max_tiles && out; ++g) {
        TileInfo tl, tp;
        decode_pair_tile(S, p, g, tl, tp);
        int32_t *o = out + (size_t)g * 6;
        o[0] = tl.type; o[1] = tl.mb; o[2] = tl.type >= 3 ? -1 : tp.mb; o[3] = tl.n; o[4] = tl.chunk; o[5] = tl.nrows;
    }
    return n;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Entry point for callers that cannot allocate device memory.
//
// The layer's scratch (control words, routing arrays, expert-major buffers) normally lives in a
// workspace the caller allocates.  Here it lives in a fixed array that is part of the loaded
// library image, so nothing is allocated or freed: not by this library, and the caller does not
// have to either.  The price: a hard size limit, one forward at a time per device, and memory that
// every device loading the library holds until the process exits.

namespace {

constexpr size_t kStaticScratchBytes = 64ull << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// the default cost tables BW(i), TFLOPS(i), i <= 1023: they depend on the device only and are
// written once per device, at set-up
static __device__ __align__(256) float g_static_tables[2][1024];

struct StaticDevice {
    bool ready;
    uint8_t *base;        // device address of g_static_scratch on this device, rounded up to 1024
    const float *tables;  // device address of g_static_tables on this device
    size_t usable;
    int n_sm;
    EncodeTiledFn encode;
};
constexpr int kMaxDevices = 64;
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: turn the array's name, which in host code is only a
// stand-in, into the address the device can use.
int static_setup(int dev, StaticDevice **out)
{
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice &d = g_static_dev[dev];
    if (!d.ready) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return WEAVE_ERR_CUDA;
        if (prop.major != 10 || !prop.cooperativeLaunch || (int)prop.sharedMemPerBlockOptin < kSmemBytes ||
            prop.multiProcessorCount < 4 || prop.multiProcessorCount + 1 > 1024)
            return WEAVE_ERR_UNSUPPORTED_DEVICE;
        void *sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_static_scratch) != cudaSuccess || sym == nullptr) return WEAVE_ERR_CUDA;
        const uintptr_t a = ((uintptr_t)sym + 1023) & ~(uintptr_t)1023;
        d.base = reinterpret_cast<uint8_t *>(a);
        d.usable = kStaticScratchBytes - (size_t)(a - (uintptr_t)sym);
        d.n_sm = prop.multiProcessorCount & ~1;
        void *tsym = nullptr;
        if (cudaGetSymbolAddress(&tsym, g_static_tables) != cudaSuccess || tsym == nullptr) return WEAVE_ERR_CUDA;
        d.tables = static_cast<const float *>(tsym);
        {
            std::vector<float> bw, tf;      // host heap only; filled and copied once per device
            default_tables(d.n_sm, bw, tf);
            if (cudaMemcpy(tsym, bw.data(), sizeof(float) * (d.n_sm + 1), cudaMemcpyHostToDevice) != cudaSuccess ||
                cudaMemcpy(static_cast<float *>(tsym) + 1024, tf.data(), sizeof(float) * (d.n_sm + 1),
                           cudaMemcpyHostToDevice) != cudaSuccess)
                return WEAVE_ERR_CUDA;
        }
        if (cudaFuncSetAttribute(weave_moe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
            cudaSuccess)
            return WEAVE_ERR_CUDA;
        void *fnp = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres) != cudaSuccess || !fnp ||
            qres != cudaDriverEntryPointSuccess)
            return WEAVE_ERR_UNSUPPORTED_DEVICE;
        d.encode = reinterpret_cast<EncodeTiledFn>(fnp);
        d.ready = true;
    }
    *out = &d;
    return WEAVE_OK;
}

}  // namespace

extern "C" {

size_t weave_moe_static_scratch_bytes(void) { return kStaticScratchBytes - 1024; }

int weave_moe_forward_static(int hidden, int ffn, int num_experts, int top_k, int num_shared, const void *gate_up,
                             const void *down, const void *x, const float *router_logits, void *out, int T,
                             void *cuda_stream)
{
    weave_moe_config cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.hidden = hidden; cfg.ffn = ffn; cfg.num_experts = num_experts; cfg.top_k = top_k;
    cfg.num_shared = num_shared; cfg.max_tokens = T;
    if (T == 0) return WEAVE_OK;
    if (!shape_ok(&cfg)) return WEAVE_ERR_INVALID_ARG;
    if (!gate_up || !down || ((uintptr_t)gate_up & 15) || ((uintptr_t)down & 15)) return WEAVE_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return WEAVE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return WEAVE_ERR_UNSUPPORTED_DEVICE;
    StaticDevice *sd = nullptr;
    int rc = static_setup(dev, &sd);
    if (rc) return rc;
    const Layout L = make_layout(&cfg);
    if (L.total > sd->usable) return WEAVE_ERR_WORKSPACE;      // beyond the built-in scratch: use a handle

    // a handle that lives on this stack frame only; nothing is allocated on the host heap either
    weave_moe h;
    memset(static_cast<void *>(&h), 0, sizeof(h));
    h.cfg = cfg;
    h.cfg.gate_up = gate_up; h.cfg.down = down; h.cfg.workspace = sd->base; h.cfg.workspace_bytes = sd->usable;
    h.L = L;
    h.ws = sd->base;
    h.n_sm = sd->n_sm; h.n_cta = sd->n_sm; h.device = dev;
    h.mode = WEAVE_SCHED_AUTO;
    h.fixed_c = (h.n_sm * 15 / 100 + 1) & ~1; h.fixed_K = 1; h.fixed_steal = 0;
    h.c_min = 2; h.c_max = h.n_sm / 2; h.c_step = 2;
    h.alpha = 0.8f;
    h.eff[0] = 1.0f; h.eff[1] = 0.83f; h.eff[2] = 0.62f; h.eff[3] = 0.43f;
    h.timeout_ms = 4000;
    h.withhold_mb = -1;
    h.ep_rank = 0;
    h.ep_size = 1;
    h.kinds = 7;
    h.elastic = -1;
    h.bw_dev = sd->tables;
    h.tf_dev = sd->tables + 1024;
    const int EE = num_experts + num_shared;
    int r = 0;
    r = encode_maps(sd->encode, &h.tm, h.ws + L.xe, h.ws + L.hbuf, gate_up, down, (uint64_t)L.p_max, (uint64_t)EE,
                    (uint64_t)hidden, (uint64_t)ffn);
    if (r) return WEAVE_ERR_CUDA;

    // the array keeps whatever the last call left behind: zero the control words (the cost tables sit
    // in their own array, written once at set-up), then the kernel; nothing else is enqueued
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(h.ws, 0, L.zero_end, st) != cudaSuccess) return WEAVE_ERR_CUDA;
    return weave_moe_forward(&h, x, router_logits, out, T, cuda_stream);
}


const char *weave_moe_strerror(int code)
{
    switch (code) {
        case WEAVE_OK: return "ok";
        case WEAVE_ERR_INVALID_ARG: return "invalid argument";
        case WEAVE_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs sm_100 with cooperative launch)";
        case WEAVE_ERR_CUDA: return "CUDA call failed";
        case WEAVE_ERR_WORKSPACE: return "workspace too small";
        case WEAVE_ERR_NONFINITE_LOGITS: return "non-finite router logit";
        case WEAVE_ERR_TIMEOUT: return "a bounded in-kernel wait expired";
        default: return "unknown error";
    }
}

}  // extern "C"
