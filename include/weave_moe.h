/*
 * weave_moe.h - C ABI of a single-GPU Mixture-of-Experts layer that runs as ONE persistent
 * sm_100a kernel: top-k routing, dispatch (token-major -> expert-major rows), grouped expert
 * SwiGLU GEMMs, combine (gate-weighted reduction back to token order), with an in-kernel cost
 * model that splits the SMs between data-movement workers and GEMM workers and a tile-level
 * ready-flag scheduler (chunk pipeline, bubble stealing).
 *
 * Conventions for every entry point
 *   - Plain C, no exceptions.  Return value: 0 = WEAVE_OK, negative = error
 *     (weave_moe_strerror() names it).  The handle-based calls keep no global state: everything
 *     lives in the handle and in the caller's workspace.  (The one exception is documented with
 *     weave_moe_forward_static(), which keeps a per-device record and a built-in scratch array.)
 *   - "device pointer" = address in the memory of the CUDA device that is current when
 *     weave_moe_create() is called; "host pointer" = ordinary (ideally pinned) host memory.
 *   - The caller owns every buffer (weights, workspace, inputs, outputs) and keeps the weights
 *     and the workspace alive and untouched until weave_moe_destroy().  The handle owns only
 *     host state.  The library never allocates or frees device memory.
 *   - One forward call per handle may be in flight at a time; calls are asynchronous on the
 *     given stream unless stated otherwise.
 *   - bf16 = IEEE-like bfloat16 bit patterns (upper 16 bits of an fp32).  All matrices are
 *     row-major and dense.
 */
#ifndef WEAVE_MOE_H
#define WEAVE_MOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct weave_moe *weave_moe_t;

enum {
    WEAVE_OK = 0,
    WEAVE_ERR_INVALID_ARG = -1,        /* null / misaligned pointer, bad shape, T > max_tokens, ...   */
    WEAVE_ERR_UNSUPPORTED_DEVICE = -2, /* not an sm_100 device, or cooperative launch unavailable     */
    WEAVE_ERR_CUDA = -3,               /* a CUDA runtime/driver call failed (see weave_moe_last_cuda_error) */
    WEAVE_ERR_WORKSPACE = -4,          /* workspace_bytes smaller than weave_moe_workspace_bytes()    */
    WEAVE_ERR_NONFINITE_LOGITS = -5,   /* device status: a router logit was NaN or +-inf               */
    WEAVE_ERR_TIMEOUT = -6             /* device status: a bounded in-kernel wait expired              */
};

/* Scheduling modes (the paper's ablation, Section 5.6):
 *   AUTO   - full method: the cost model of Section 3.3 (Eq. 15-16) picks the number of movement
 *            SMs c and the chunk count K from the routing result, Eq. 11-14 give the steal count.
 *            (Besides the paper's split the model also costs two plan kinds that only make sense
 *            where movement is a local copy: see weave_moe_set_model_options().)
 *   FIXED  - the given c, K and steal count are used as they are ("w/o T" when K = 1, steal = 0).
 *   SERIAL - dispatch, GEMMs and combine run one after the other on all SMs ("w/o S+T").       */
enum { WEAVE_SCHED_AUTO = 0, WEAVE_SCHED_FIXED = 1, WEAVE_SCHED_SERIAL = 2 };

typedef struct weave_moe_config {
    int hidden;       /* H: model width, multiple of 128, at most 16384                           */
    int ffn;          /* I: per-expert intermediate width, multiple of 128                         */
    int num_experts;  /* E: routed experts, >= 1                                                  */
    int top_k;        /* k: experts per token, 1 <= k <= min(E, 16)                               */
    int num_shared;   /* S: always-on experts applied to every token with weight 1; E + S <= 256  */
    int max_tokens;   /* largest T a forward call may pass (sizes the workspace)                  */
    const void *gate_up; /* device, bf16 [E+S][2I][H]: rows [0,I) gate projection (gets SiLU),
                            rows [I,2I) up projection; 16-byte aligned                            */
    const void *down;    /* device, bf16 [E+S][H][I]; 16-byte aligned                             */
    void *workspace;     /* device scratch of at least weave_moe_workspace_bytes(); 1024-byte aligned */
    size_t workspace_bytes;
} weave_moe_config;

/* Bytes of device scratch a handle with this config needs.  Pure host arithmetic (reads only the
 * six integer fields).  Returns 0 if the shape is invalid. */
size_t weave_moe_workspace_bytes(const weave_moe_config *cfg);

/* Validates the config, encodes the TMA descriptors of the weight and scratch matrices, zeroes
 * the control words in the workspace (synchronous), installs default cost-model tables.
 * The layer computed is the five-stage MoE forward of the paper's Section 2.1 / Figure 3, with the
 * router added in front:  idx[t,0..k) = the k largest fp32 logits of token t (ties to the lowest
 * expert index, listed by descending logit);  gate[t,j] = softmax over those k logits;
 *   out[t] = sum_j gate[t,j] * Wd[e_j] ( silu(Wg[e_j] x[t]) (.) Wu[e_j] x[t] )  +  sum_s (same, shared
 * expert s, weight 1).  Intermediates h and y are rounded to bf16; accumulation is fp32. */
int weave_moe_create(const weave_moe_config *cfg, weave_moe_t *out_handle);

/* One layer.  x: device bf16 [T][H];  router_logits: device fp32 [T][E];  out: device bf16 [T][H]
 * (fully overwritten).  All three 16-byte aligned, not aliasing each other or the workspace.
 * 0 <= T <= max_tokens (T = 0 is a no-op).  cuda_stream: a cudaStream_t (NULL = default stream).
 * Launches exactly one kernel; returns once it is enqueued.  Device-side failures
 * (WEAVE_ERR_NONFINITE_LOGITS, WEAVE_ERR_TIMEOUT) are reported by weave_moe_status().
 * The call makes no other CUDA call (no allocation, copy, memset or synchronisation: the kernel
 * re-zeroes its own control words), so a sequence of layers may be captured into a CUDA graph on
 * `cuda_stream`; the replay reads the arguments and the schedule settings given at capture time. */
int weave_moe_forward(weave_moe_t h, const void *x, const float *router_logits, void *out, int T,
                      void *cuda_stream);

/* Same layer with HOST buffers: copies x and router_logits into staging areas of the workspace,
 * runs weave_moe_forward, copies out back; all enqueued on the stream (asynchronous only if the
 * host buffers are pinned). */
int weave_moe_forward_host(weave_moe_t h, const void *x_host, const float *router_logits_host,
                           void *out_host, int T, void *cuda_stream);

/* Throughput variant of weave_moe_forward_host for back-to-back calls: the copies run on two
 * internal copy streams (created on first use, destroyed with the handle) and two staging slots
 * alternate, so the H2D copy of call i+1 and the D2H copy of call i-1 overlap the kernel of call
 * i; the kernels stay ordered on cuda_stream.  out_host of a call is complete once
 * weave_moe_host_wait() returns (or after two further pipelined calls have been waited for);
 * synchronising cuda_stream alone does NOT cover the last D2H copy.  Host buffers must be pinned
 * and stay valid until then. */
int weave_moe_forward_host_pipelined(weave_moe_t h, const void *x_host, const float *router_logits_host,
                                     void *out_host, int T, void *cuda_stream);

/* Blocks until the output copies of all pipelined calls made so far have arrived in host memory. */
int weave_moe_host_wait(weave_moe_t h);

/* Releases host state.  Does not touch device memory. */
int weave_moe_destroy(weave_moe_t h);

/* ---- scheduling surface (Section 3; ablation of Section 5.6) -------------------------------- */

/* mode: WEAVE_SCHED_*.  For FIXED: c = number of movement SMs (rounded up to whole SM pairs and
 * clamped to [2, n_sm-2]), K = chunk count in {1,2,4,8} (lowered until K*(E+S) <= 1024), steal =
 * GEMM tiles each movement SM pair takes after dispatch (Section 3.2.2).  Takes effect at the
 * next forward. */
int weave_moe_set_schedule(weave_moe_t h, int mode, int c, int K, int steal);

/* One expert-parallel rank's share of the layer (the paper's setting, Sections 2.1 and 3.1, modelled
 * on one GPU): with ep_size > 1 the handle acts as rank ep_rank of ep_size.  It hosts experts
 * [ep_rank*E/ep_size, (ep_rank+1)*E/ep_size) (weights of all E experts are still passed; the others
 * are not touched) and owns token shard ep_rank, shard s = tokens [s*Ts, (s+1)*Ts), Ts =
 * ceil(T/ep_size); the other shards play the remote ranks' tokens, held in local HBM.  Routing stays
 * global (gates normalised over all k experts).  Every remote token with at least one expert here
 * is copied once into a staging buffer and all its local experts read that copy (dispatch-side
 * deduplication, Section 4); out[t] = the partial sum over t's experts hosted here (zero if none) -
 * summing the outputs of all ranks gives the full layer.  row_of is -1 for slots whose expert
 * lives elsewhere.  The cost model then uses Eq. 1-3 literally (X_local, X_in, X_in^uniq).
 * Needs E % ep_size == 0 and no shared experts.  ep_size = 1 switches it off (the default). */
int weave_moe_set_expert_parallel(weave_moe_t h, int ep_rank, int ep_size);

/* The workload descriptors of Section 3.1 counted by the most recent forward in expert-parallel
 * mode: pairs with an own-shard token, pairs with a remote token, distinct remote tokens.
 * Synchronises the last stream. */
int weave_moe_get_ep_descriptors(weave_moe_t h, long long *x_local, long long *x_in, long long *x_in_uniq);

/* Number of SMs (= persistent CTAs) the kernel occupies from the next forward on: even, at least 4,
 * at most the device's SM count rounded down to even (the default).  Leaves the other SMs to
 * concurrent work (or to a profiler).  The cost tables keep being indexed by SM count, so the
 * model's candidate c must stay below the new count. */
int weave_moe_set_sm_count(weave_moe_t h, int n_sm);

/* Hardware input of the cost model (Figure 7): bw[i] = bytes/us moved by i movement SMs,
 * tflops[i] = FLOP/us of i GEMM SMs, i in [0, n_sm] (host arrays of n_sm+1 floats, entry 0
 * ignored); eff_chunk[4] = Eq. 9's correction factor for K = 1,2,4,8; alpha = Section 3.1's
 * overlap ratio in [0,1); candidate grid c = c_min, c_min+c_step, ... <= c_max (at most 64
 * values; c_min and c_step even, c_min >= 2).  A candidate (c, K) is skipped when K*(E+S) > 1024
 * (the kernel's table of (chunk, expert) segments).  Synchronous copy to the device. */
int weave_moe_set_cost_tables(weave_moe_t h, const float *bw, const float *tflops,
                              const float *eff_chunk, float alpha, int c_min, int c_max, int c_step);

/* Plan of the most recent forward (Section 3.3: SM split, chunk count, steal count) and the
 * model's predicted layer time in us.  Synchronises the handle's last stream. */
int weave_moe_get_plan(weave_moe_t h, int *c, int *K, int *n_steal, float *t_total_us);

/* Plan kinds.  SPLIT is the paper's execution plan (Section 3.3, Eq. 15): c movement SMs next to
 * N - c GEMM SMs from the first tile on.  The paper's movement crosses NVLink; here it is a copy
 * inside one GPU's memory that all SMs can do at full speed, so AUTO's arg-min (Eq. 16) also ranges
 * over three kinds the paper has no use for, costed from the same tables BW(.), TFLOPS(.), eff_chunk,
 * alpha:
 *   DISPATCH_ALL  every SM dispatches, then c SMs combine chunk by chunk while N - c run the GEMMs:
 *                 T = W_disp/BW(N) + max(T_comp(c,K) + T_tail(c,K), W_comb/BW(c))
 *   PHASED        no roles: every SM dispatches, then takes GEMM tiles until the queue is empty,
 *                 then combines (tile-level ready flags, no grid barrier between the phases):
 *                 T = W_disp/BW(N) + W_comp/TFLOPS(N) + (1-alpha) * W_comb/BW(N);  reported as
 *                 c = n_sm, K = 1, n_steal = 0.
 *   REJOIN        the split in which the c movement SMs return to the GEMM queue for good once the
 *                 dispatch is done (they take GEMM tiles whenever no combine chunk is ready; no
 *                 quota) and every GEMM CTA dispatches one m-block before its first tile; K = 1:
 *                 t_d = W_disp/BW(c), W_during = min(t_d * TFLOPS(N-c), 2/3 W_comp)  (the work done
 *                 meanwhile, as Eq. 12, capped at the gate/up tiles' share, which the queue runs first),
 *                 T = t_d + max(0, W_comp - W_during)/TFLOPS(N) + (1-alpha) * W_comb/BW(N).
 * Ties go to SPLIT, then DISPATCH_ALL, PHASED, REJOIN, then to the smaller c, then to the smaller K.  The steal quota of Eq. 11-14
 * belongs to SPLIT; the other kinds report n_steal = 0.  FIXED always runs SPLIT; SERIAL reports
 * PHASED (it is the same order of work with a grid barrier between the phases). */
enum { WEAVE_PLAN_SPLIT = 0, WEAVE_PLAN_DISPATCH_ALL = 1, WEAVE_PLAN_PHASED = 2, WEAVE_PLAN_REJOIN = 3 };

/* Kind of the plan of the most recent forward.  Synchronises the handle's last stream. */
int weave_moe_get_plan_kind(weave_moe_t h, int *kind);

/* kinds_mask: which plan kinds AUTO's arg-min may choose (bit 1 << WEAVE_PLAN_*; default 7 = SPLIT,
 * DISPATCH_ALL and PHASED; 15 adds REJOIN, which measured no better than PHASED on this hardware;
 * 1 = the paper's split only; must be non-zero).  elastic: whether movement SM pairs keep
 * taking GEMM tiles beyond their steal quota while no combine chunk is ready, and GEMM CTAs
 * dispatch one m-block before their first GEMM tile: 1 = on, 0 = off, -1 = the default (on under
 * AUTO, off under FIXED, so that FIXED is the plain static split of the paper's ablation).
 * Takes effect at the next forward. */
int weave_moe_set_model_options(weave_moe_t h, int kinds_mask, int elastic);

/* Geometry the scheduler works with: number of SMs used (= persistent CTAs; an even number,
 * because the GEMM phase runs on pairs of neighbouring SMs), rows per m-block (the unit of the
 * dispatch queue and of the ready flags), h-columns per gemm0 tile, out-columns per gemm1 tile,
 * tokens per routing block, tokens per combine tile (the largest size: a batch that would give
 * fewer tiles than SMs is cut into tiles of half that size, repeatedly, down to one token), rows
 * per GEMM tile (two m-blocks of one expert segment; a segment with an odd number of m-blocks ends
 * in a half-empty tile).
 * Any pointer may be NULL. */
int weave_moe_get_geometry(weave_moe_t h, int *n_sm, int *block_m, int *tile_n0, int *tile_n1,
                           int *route_block, int *combine_tile, int *gemm_tile_m);

/* ---- verification surface ------------------------------------------------------------------- */

/* Device pointers INTO THE WORKSPACE holding the routing result of the most recent forward:
 * topk_idx int32 [T][k], gates fp32 [T][k], counts int32 [E+S], offsets int32 [E+S+1],
 * row_of int32 [T][k] (routed slots; the row of shared expert s is offsets[E+s] + t),
 * token_of int32 [T*(k+S)].  Valid until the next forward.  Any pointer may be NULL. */
int weave_moe_get_routing(weave_moe_t h, const int32_t **topk_idx, const float **gates,
                          const int32_t **counts, const int32_t **offsets, const int32_t **row_of,
                          const int32_t **token_of);

/* Device pointers into the workspace of the expert-major intermediates of the most recent
 * forward: xe bf16 [P][H] (dispatched rows), h bf16 [P][I], y bf16 [P][H], P = T*(k+S). */
int weave_moe_get_intermediates(weave_moe_t h, const void **xe, const void **hbuf, const void **y);

/* Synchronises the last stream, returns the device status word of the last forward
 * (WEAVE_OK, WEAVE_ERR_NONFINITE_LOGITS, WEAVE_ERR_TIMEOUT) and clears it; after a failure it
 * also re-zeroes the control words so that the handle is usable again. */
int weave_moe_status(weave_moe_t h);

/* After weave_moe_status() returned WEAVE_ERR_TIMEOUT: a small integer naming the wait that gave
 * up first (1-3 grid barriers, 10-16 dispatch, 20-24 combine, 30-57 GEMM phase); 0 otherwise.
 * Diagnostic only. */
int weave_moe_last_timeout_where(weave_moe_t h);

/* Post-mortem of the launch whose failure the last weave_moe_status() reported.  Every bounded wait
 * that ended without success - its own limit ran out, or it saw the abort word another wait had raised -
 * left a record in its warp's slot.  Copies up to max_records records of six ints to `out` (host):
 * {CTA, warp, wait id (as weave_moe_last_timeout_where), the object waited on (for a shared-memory
 * barrier its address, whose low 10 bits are the barrier's byte offset among the CTA's barriers; for
 * a ready flag the low 32 bits of its device address), the parity or count waited for, 1 = this
 * wait's limit ran out / 2 = cut short by the abort word}.  Returns the number of records there
 * are (may exceed max_records), 0 when the last status was clean.  Diagnostic only: which warps
 * waited for what when the launch stopped.  (A device-side wait that fails is the only failure
 * injected or observed on the GPU; nothing traps or faults.) */
int weave_moe_debug_wait_log(weave_moe_t h, int32_t *out, int max_records);

/* Upper bound, in milliseconds, for any single in-kernel wait (grid barrier, ready flag,
 * mbarrier); after it the kernel records WEAVE_ERR_TIMEOUT and every CTA returns.  Default 4000. */
int weave_moe_set_timeout_ms(weave_moe_t h, int ms);

/* Test hook for the give-up path: the m-block with this index never publishes its
 * "dispatched" flag (-1 = off), so its consumer's bounded wait expires.  Host-side injection
 * only; nothing faults or traps. */
int weave_moe_debug_withhold_flag(weave_moe_t h, int m_block);

/* Optional in-kernel timeline (our analogue of the utilisation profile of the paper's Section 5.4).
 * buf: device memory of at least n_sm * events_per_cta * 16 bytes, caller-owned, or NULL to switch
 * tracing off.  Each CTA writes up to events_per_cta - 1 records {start ns, end ns (low 32 bits of
 * the global nanosecond timer), kind << 24 | id, extra} into its slice; the slice's last record
 * holds the number written.  Kinds: 1 routing, 2 set-up, 3 permutation fix-up, 4 dispatch tile,
 * 5 GEMM tile scheduled (claim until its inputs were ready), 6 GEMM tile epilogue (id = m-block,
 * extra = type << 16 | ns spent before the release), 7 combine tile, 8 wait for a chunk's gemm1,
 * 9 grid barrier (the one behind the routing; a batch of at most 64 tokens is routed by every CTA for itself
 * and has none), 11 GEMM tile main loop on the MMA issuer (id = type << 16 | rows, extra = ns spent
 * waiting for a free accumulator). */
int weave_moe_set_trace(weave_moe_t h, void *buf, int events_per_cta);

/* HOST-ONLY (no GPU needed, no handle): the order in which the kernel's GEMM schedulers claim pair
 * tiles (Section 4: the queues follow the dependency order of the chunk pipeline), for `num_chunks` chunks of
 * `num_segments` expert segments whose row counts are rows[chunk * num_segments + expert], n-tile
 * counts nt0 (gemm0) and nt1 (gemm1).  Writes up to max_tiles records of
 * 6 ints {type (0 gemm0, 1 gemm1, +3 when the operands are swapped), leader m-block, peer m-block
 * (-1 for a swapped tile), n-tile, chunk, rows of the leader m-block} to `out` (host memory, may be
 * NULL) and returns the total number of tiles, or a negative error for bad arguments (chunks not
 * in {1,2,4,8}, more than 1024 segments in total, non-positive tile counts).  This is the same
 * decoding routine the device runs; tests use it to check that every tile a gemm1 tile waits for
 * comes earlier in the queue. */
int weave_moe_debug_gemm_queue(const int32_t *rows, int num_segments, int num_chunks, int nt0, int nt1,
                               int32_t *out, int max_tiles);

/* ---- for callers that cannot allocate ---------------------------------------------------------
 *
 * (No counterpart in the paper: this is a packaging variant of the same kernel.)
 * Some callers of this library may not allocate device memory at the point where they need a
 * layer: code that runs while a memory pool is frozen, plugins handed a fixed arena by their host
 * application, latency-critical serving loops whose allocator must stay untouched.  For them this
 * entry point runs weave_moe_forward's kernel with its scratch placed in a fixed array built into
 * the library image instead of a caller-provided workspace.  It takes no handle and calls no
 * cudaMalloc / cudaFree or any other allocating routine; the caller still passes weights, inputs
 * and the output.
 *
 *   - Limit: the layer's scratch (what weave_moe_workspace_bytes() reports for this shape with
 *     max_tokens = T) must fit weave_moe_static_scratch_bytes() (64 MiB minus alignment); larger
 *     calls fail with WEAVE_ERR_WORKSPACE and must use a handle.  Every GPU on which the library
 *     is loaded holds those 64 MiB until the process exits.
 *   - The first call on each device performs a one-time set-up with that device current (it looks
 *     up the device addresses of the built-in arrays, fills the built-in cost tables with a
 *     synchronous copy, raises the kernel's shared-memory limit and resolves the TMA descriptor
 *     encoder).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents; every
 *     call enqueues one memset of the control words and then the kernel.  Calls that overlap on the
 *     GPU (different streams, no ordering between them) race on the array: order them.
 *   - Scheduling is AUTO with the default cost tables.  Arguments, layouts and alignment as for
 *     weave_moe_create() / weave_moe_forward(); asynchronous on the stream; a device-side failure
 *     of this call (non-finite logits, an expired wait) is not reported - use a handle when the
 *     status word is needed. */
int weave_moe_forward_static(int hidden, int ffn, int num_experts, int top_k, int num_shared,
                             const void *gate_up, const void *down, const void *x,
                             const float *router_logits, void *out, int T, void *cuda_stream);

/* Size limit of the built-in scratch used by weave_moe_forward_static(). */
size_t weave_moe_static_scratch_bytes(void);

int weave_moe_last_cuda_error(weave_moe_t h);
const char *weave_moe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* WEAVE_MOE_H */
