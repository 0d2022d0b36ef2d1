// The persistent MoE-layer megakernel: one CTA per SM, one launch per layer.
//
//   phase R  (all CTAs)   top-k routing of 64-token blocks (four threads per token, lists merged by
//                         shuffles), per-block expert bitmasks -> in-block ranks and a
//                         [block][expert] histogram; grid barrier (bounded)
//   set-up   (every CTA, redundantly) counts, offsets, candidate tile counts, cost model -> plan
//                         (c, K, n_steal), segment tables of the chosen K; permutation fix-up
//   phase A  (movement CTAs: blockIdx < c)  dispatch tiles: gather x rows into expert-major Xe
//   phase B  (GEMM CTA pairs until the queue is empty; movement pairs for n_steal tiles)
//                         two neighbouring CTAs (a cluster of 2) share a 256-row tile: a scheduler
//                         warp claims tiles and waits for their inputs, TMA producers feed a
//                         6-stage smem ring, one thread issues tcgen05.mma.cta_group::2 into TMEM,
//                         four epilogue warps per CTA drain it through a staged, coalesced store,
//                         and a releasing warp makes the tiles' arrivals on the ready counters
//   phase C  (every CTA once it has nothing else)  combine tiles, chunk by chunk as the chunk's
//                         gemm1 tiles complete
//
// Stage list, roles, queue order, steal placement and the all-SM final combine follow the paper's
// Sections 3 and 4; the cost model is Section 3's Eq. 1-16.
#pragma once
#include <cuda.h>

#include "weave_ptx.cuh"

namespace weave {

constexpr int kThreads = 256;
constexpr int kBM = 128;        // rows per GEMM m-block (UMMA M)
constexpr int kBK = 64;         // K elements per pipeline stage: 128 bytes of bf16 = one swizzle row
constexpr int kTN0 = 128;       // h columns per gemm0 tile; the MMA is N = 256 (gate | up)
constexpr int kStages = 6;
constexpr int kStageA = kBM * kBK * 2;                  // 16 KB: this CTA's 128 rows of A
constexpr int kStageB = 128 * kBK * 2;                  // 16 KB: this CTA's half (128 rows) of the 256-row B tile
constexpr int kStageBytes = kStageA + kStageB;          // 32 KB
constexpr int kEpiStageBytes = 4 * 2 * 32 * 64;         // epilogue staging: per warp two buffers of 32 rows x 64 bytes
constexpr int kRouteBlock = 64;  // tokens per routing block (one 64-bit mask per expert)
constexpr int kLocalBlocks = 1;  // a batch of at most this many routing blocks is routed by every CTA for itself
                                 // (measured at two blocks: routing both in every CTA costs more than the grid barrier saves)
constexpr int kCombTile = 16;    // tokens per combine tile (fewer when the batch would give fewer tiles than SMs)
constexpr int kMaxEE = 256;      // routed + shared experts
constexpr int kMaxTopK = 16;
constexpr int kFine = 8;         // fine chunks = largest chunk count K
constexpr int kMaxSeg = 1024;     // (chunk, expert) segments: K * (E+S) <= 1024 bounds the chunk count
constexpr int kTinfo = 4;        // tile-descriptor ring between the producer and its consumers
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 4;     // warps 4..7
constexpr int kRel = 3;          // mailbox ring between the epilogue warps and the releasing warp (warp 3)
constexpr unsigned kRelEnd = 0xFFFFFFFFu;
constexpr int kPairGroup = 8;    // 256-row pair tiles (= 16 m-blocks) kept L2-resident while all n-tiles pass

constexpr int kErrNonFinite = -5;
constexpr int kErrTimeout = -6;

enum { kModeAuto = 0, kModeFixed = 1, kModeSerial = 2 };

// Control words in global memory.  The first kCtlZeroWords words are zero at kernel entry and are
// re-zeroed by the last CTA to leave, so no memset precedes a launch.
struct Ctl {
    unsigned bar_count;   // grid-barrier arrivals
    unsigned q_disp;      // next dispatch tile
    unsigned q_gemm;      // next GEMM tile (chunk-pipeline DAG order)
    unsigned q_comb;      // next combine tile
    unsigned fix_done;    // routing blocks whose rows are final
    unsigned exit_count;
    unsigned abort;       // set by the first wait that gives up; every wait polls it
    unsigned pad0;
    unsigned y_done[kFine];  // per chunk: epilogue-warp arrivals of finished gemm1 tiles
    unsigned q_pull;      // expert-parallel share: next block of remote tokens to stage
    unsigned pull_done;   // ... blocks staged
    unsigned x_local, x_in, x_in_uniq;   // ... the workload descriptors of Section 3.1, counted while routing
    unsigned pad1[3];
    // ---- not re-zeroed: results for the host
    int status;
    int timeout_where;
    int plan_c, plan_K, plan_steal;
    float plan_t;
    int plan_nmb, plan_ngemm;
    unsigned ep_x_local, ep_x_in, ep_x_in_uniq;
    int plan_kind;
};
constexpr int kCtlZeroWords = 24;

// Plan kinds of the cost model.  kPlanSplit is the paper's (Eq. 15): c movement SMs beside N - c GEMM
// SMs from the start.  The other two exist because on one GPU the movement is an HBM copy that all
// SMs can do at full speed: kPlanDispatchAll lets every SM dispatch before the roles split (only the
// combine is left to the movement SMs), kPlanPhased has no roles at all (every SM dispatches, then
// runs GEMM tiles until the queue is empty, then combines; the ready flags still order the tiles,
// no grid barrier separates the phases).  kPlanRejoin is the split in which the movement SMs come back to
// the GEMM queue for good once the dispatch is done (no steal quota: they take GEMM tiles whenever no
// combine chunk is ready) and every GEMM CTA dispatches one m-block before its first tile; K = 1.
enum { kPlanSplit = 0, kPlanDispatchAll = 1, kPlanPhased = 2, kPlanRejoin = 3 };

struct KParams {
    int T, H, I, E, S, k, EE;
    int nblk;             // routing blocks = ceil(T / 64)
    int mode, fixed_c, fixed_K, fixed_steal;
    int nt0, nt1;         // n-tiles per m-block: I / 128, ceil(H / 256)
    int nmb_max;          // allocated length of the per-m-block flag arrays
    int ep_rank, ep_size; // expert-parallel share (ep_size <= 1: off): this rank hosts experts
                          // [ep_rank*E/ep_size, (ep_rank+1)*E/ep_size) and owns token shard ep_rank
    int ep_tshard;        // tokens per shard = ceil(T / ep_size)
    __nv_bfloat16 *xs;    // [T][H] staging of remote tokens (each unique one is copied once)
    unsigned long long *uniq_mask;   // [nblk] remote tokens of the block that have a local expert
    int elastic_steal;    // movement pairs keep stealing past their quota while no combine chunk is ready
    int kinds;            // bit mask of the plan kinds the cost model may choose (bit kPlanSplit, ...)
    int withhold_mb;      // test hook: this m-block's "dispatched" flag is never published (-1 = off)
    int c_min, c_max, c_step;
    float alpha;
    float eff[4];
    unsigned long long timeout_ns;
    const __nv_bfloat16 *x;
    const float *logits;
    __nv_bfloat16 *out;
    Ctl *ctl;
    unsigned *fcnt;       // [8][256] rows per (fine chunk, expert); zero at entry
    int *hist;            // [nblk][256]
    int *topk_idx;        // [T][k]
    float *gates;         // [T][k]
    int *row_of;          // [T][k]
    int *token_of;        // [P]
    int *counts;          // [EE]
    int *offsets;         // [EE+1]
    __nv_bfloat16 *xe;    // [P][H]
    __nv_bfloat16 *hbuf;  // [P][I]
    __nv_bfloat16 *y;     // [P][H]
    unsigned *xe_ready;   // [nmb_max] 1 when the m-block's rows are dispatched; zero at entry
    unsigned *h_ready;    // [nmb_max] epilogue-warp arrivals of the m-block's gemm0 tiles; zero at entry
    const float *bw;      // [n_sm+1] byte/us
    const float *tf;      // [n_sm+1] FLOP/us
    uint4 *trace;         // optional [n_sm][trace_cap] event records (nullptr = off)
    int trace_cap;
    int4 *wait_log;       // [n_sm][8 warps]: written only by a wait that gives up or is cut short by the abort word
};

struct TileInfo {
    int type;   // 0 gemm0 (+SwiGLU), 1 gemm1, 2 no more tiles; 3 / 4 = gemm0 / gemm1 of a single m-block
                // with the operands swapped (weights on the MMA's M axis, the m-block's rows on N)
    int mb;     // this CTA's m-block (-1: the pair tile has no second half)
    int row0;   // first row of this CTA's 128 rows of A
    int nrows;  // valid rows (0 for a missing half)
    int e, n, chunk, nkb;
};

// what one movement buffer (a 32 KB stage) currently holds
struct MvDesc {
    int a;      // dispatch: first destination row        combine: token
    int b;      // dispatch: rows in the buffer            combine: first column
    int c;      // dispatch: m-block                       combine: columns
    int d;      // dispatch: 1 = last buffer of its tile;  2 = no more work (both phases);
                // 3 / 4 = staging of remote tokens (rows go to xs[tok[i]]; 4 = last buffer of the block)
    int n;      // combine: rows gathered (0: the token has no expert here, the piece is zero)
    float g[kMaxTopK + 8];   // combine: weight of each gathered row
    int tok[32];             // staging: destination token of each row in the buffer
};
constexpr int kMvBuf = kStageBytes;     // 32 KB
constexpr int kCombWarps = 6;           // warps 2..7 reduce

struct SmemTail {
    uint64_t full[kStages], empty[kStages];
    uint64_t tmem_full[2], tmem_empty[2];
    uint64_t ti_full[kTinfo], ti_empty[kTinfo];
    uint64_t dv_full[kStages], dv_empty[kStages];   // dispatch: loader -> storer ring over the stage buffers
    uint64_t cb_full[kStages], cb_empty[kStages];   // combine: loader -> reducing warps
    uint64_t xg_full, xg_empty;                     // swapped gemm0 epilogue: up warps -> gate warps
    uint64_t rel_full[kRel], rel_empty[kRel];       // epilogue warps -> releasing warp: a tile's stores are issued
    unsigned *rel_flag[kRel];                       // the ready counter that tile arrives on, and by how much
    unsigned rel_cnt[kRel];
    TileInfo ti[kTinfo];
    uint32_t tmem_base;
    int bcast[3];
    int red_i[8][4];
    float red_f[8];
    int scan_w[8];
    int scan_total;
    int c, K, steal, nmb, n_gemm, n_comb;
    int elastic;                 // this launch: movement pairs take GEMM tiles beyond their quota, GEMM CTAs dispatch one m-block first
    int comb_tok;                // tokens per combine tile of this launch: 16, 8, 4, 2 or 1
    unsigned trace_n;
    int chunk_mb0[kFine + 1];
    int chunk_pt0[kFine + 1];
    int chunk_nswap[kFine];      // per chunk: segments with an odd number of m-blocks
    int chunk_tile0[kFine + 1];
    int offsets[kMaxEE + 1];
    int seg_mb0[kMaxSeg + 1];
    int seg_pt0[kMaxSeg + 1];    // prefix of pair tiles: ceil(m-blocks / 2) per segment
    int seg_row0[kMaxSeg];
    int seg_rows[kMaxSeg];
};

// Scratch of the movement phases (dispatch, combine).  A CTA is in one phase at a time, so it shares
// its space with the second half of the GEMM epilogue's staging area.
struct MoveScratch {
    MvDesc mv[kStages];
    int tok[kBM];
    int crow[kCombTile][kMaxTopK + 8];
    float cgate[kCombTile][kMaxTopK + 8];
};
static_assert(sizeof(MoveScratch) <= kEpiStageBytes / 2, "movement scratch must fit half of the staging area");
static_assert(kLocalBlocks * (kMaxEE + 1) * 8 <= kEpiStageBytes / 2, "the routing masks must fit the other half");
static_assert(kFine == 8, "chunk of a fine chunk = f >> (3 - log2 K)");
__device__ __forceinline__ MoveScratch &move_scratch(uint8_t *stages)
{
    return *reinterpret_cast<MoveScratch *>(stages + kStages * kStageBytes + kEpiStageBytes / 2);
}

constexpr int kSmemBytes = kStages * kStageBytes + kEpiStageBytes + (int)sizeof(SmemTail) + 1024;
static_assert(kSmemBytes <= 232448, "exceeds the 227 KB a CTA may opt into");

// ------------------------------------------------------------------------------------ waits

__device__ __noinline__ void give_up(Ctl *ctl, int where)
{
    if (atomicCAS(&ctl->status, 0, kErrTimeout) == 0) ctl->timeout_where = where;
    atomicExch(&ctl->abort, 1u);
}

// Post-mortem of a failed launch: every wait that ends without success (its own limit ran out, or it saw
// the abort word another wait had raised) leaves {wait id, what it waited on (shared-memory address of the
// barrier or low bits of the flag's address), the parity or target it waited for, 1 = timed out / 2 = cut
// short} in its warp's slot (the warp's first such wait only).  Together the slots show who was waiting
// for whom when the launch stopped.
__device__ __noinline__ void note_failed_wait(int4 *log, int where, unsigned what, unsigned want, int how)
{
    // the first failed wait of a warp is the one that tells where it stood; what it runs into afterwards,
    // on its way out with the abort word set, is not recorded
    if (log && log[blockIdx.x * 8 + (threadIdx.x >> 5)].w == 0)
        log[blockIdx.x * 8 + (threadIdx.x >> 5)] = make_int4(where, (int)what, (int)want, how);
}

// Optional timeline: one 16-byte record {start ns, end ns, kind<<24 | id, extra} per event, per CTA.
enum { kEvRoute = 1, kEvSetup = 2, kEvFixup = 3, kEvDispatch = 4, kEvGemmLoad = 5, kEvGemmEpi = 6,
       kEvCombine = 7, kEvWaitChunk = 8, kEvBarrier = 9, kEvMma = 11 };
__device__ __forceinline__ void trace_ev(const KParams &p, SmemTail &S, int kind, unsigned id,
                                         unsigned long long t0, unsigned long long t1, unsigned extra)
{
    if (p.trace == nullptr) return;
    const unsigned i = atomicAdd(&S.trace_n, 1u);
    if (i + 1u < (unsigned)p.trace_cap)
        p.trace[(size_t)blockIdx.x * p.trace_cap + i] =
            make_uint4((unsigned)t0, (unsigned)t1, ((unsigned)kind << 24) | (id & 0xFFFFFFu), extra);
}
__device__ __forceinline__ unsigned long long trace_now(const KParams &p)
{
    return p.trace ? globaltimer_ns() : 0ull;
}
// the same for the CTA-wide phases, whose records thread 0 writes: the other threads do not read the timer
__device__ __forceinline__ unsigned long long trace_now_t0(const KParams &p)
{
    return (p.trace && threadIdx.x == 0) ? globaltimer_ns() : 0ull;
}

// Every wait is bounded: it polls the global abort word and a wall-clock limit, and returns false
// instead of spinning forever.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, const KParams &p, int where)
{
    if (mbar_try_wait(bar, parity)) return true;
    // the clock is read only every 32 polls (the first reading starts the limit): a reading costs far
    // more than a poll, and most waits end within a few polls.  The abort word is looked at one round
    // late: its load (an L2 round trip on a line that every SM's queue claims hit) is issued here and its
    // value used 32 polls later, so the waiting thread is never stalled on it when the barrier completes.
    unsigned long long t0 = 0;
    unsigned it = 0;
    unsigned ab = 0u;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 31u) == 0u) {
            if (ab) { note_failed_wait(p.wait_log, where, smem_u32(bar), parity, 2); return false; }
            ab = ld_relaxed_u32(&p.ctl->abort);
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if ((long long)(now - t0) > (long long)p.timeout_ns) {     // signed: a timer that steps back is not a time-out
                give_up(p.ctl, where);
                note_failed_wait(p.wait_log, where, smem_u32(bar), parity, 1);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ bool flag_wait_ge(const unsigned *flag, unsigned target, const KParams &p, int where)
{
    if (ld_acquire_u32(flag) >= target) return true;
    unsigned long long t0 = 0;
    unsigned it = 0;
    while (ld_acquire_u32(flag) < target) {
        __nanosleep(40);
        if ((++it & 31u) == 0u) {
            if (ld_relaxed_u32(&p.ctl->abort)) {
                note_failed_wait(p.wait_log, where, (unsigned)(size_t)flag, target, 2);
                return false;
            }
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if ((long long)(now - t0) > (long long)p.timeout_ns) {
                give_up(p.ctl, where);
                note_failed_wait(p.wait_log, where, (unsigned)(size_t)flag, target, 1);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void linger_after_abort()
{
    // lets copies and MMAs that are already in flight land before this CTA can leave
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 50000ull) __nanosleep(1000);
}

// All CTAs are co-resident (cooperative launch); arrivals accumulate over the barriers of a launch.
// Three exclusive scans in one pass: v = a | b << 24 | c << 48 with a, b < 2^24 and c < 2^16 in total.
__device__ __forceinline__ unsigned long long block_excl_scan_packed(unsigned long long v, SmemTail &S, unsigned long long &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) { S.red_i[warp][0] = (int)(unsigned)inc; S.red_i[warp][1] = (int)(unsigned)(inc >> 32); }
    __syncthreads();
    unsigned long long wbase = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        const unsigned long long sw = (unsigned long long)(unsigned)S.red_i[w][0] | ((unsigned long long)(unsigned)S.red_i[w][1] << 32);
        if (w < warp) wbase += sw;
        tot += sw;
    }
    total = tot;
    return wbase + inc - v;
}

// the two halves of a grid barrier, for a caller that has work to do between arriving and waiting
__device__ __forceinline__ void grid_barrier_arrive(const KParams &p)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        red_release_add_u32(&p.ctl->bar_count, 1u);
    }
}
__device__ __forceinline__ bool grid_barrier_wait(const KParams &p, SmemTail &S, unsigned target, int where)
{
    if (threadIdx.x == 0) S.bcast[2] = flag_wait_ge(&p.ctl->bar_count, target, p, where) ? 1 : 0;
    __syncthreads();
    return S.bcast[2] != 0;
}
__device__ __forceinline__ bool grid_barrier(const KParams &p, SmemTail &S, unsigned target, int where)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        red_release_add_u32(&p.ctl->bar_count, 1u);
        S.bcast[2] = flag_wait_ge(&p.ctl->bar_count, target, p, where) ? 1 : 0;
    }
    __syncthreads();
    return S.bcast[2] != 0;
}

// ------------------------------------------------------------------------------------ block helpers

__device__ __forceinline__ int block_excl_scan(int v, SmemTail &S, int &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) S.scan_w[warp] = inc;
    __syncthreads();
    int wbase = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        int s = S.scan_w[w];
        if (w < warp) wbase += s;
        tot += s;
    }
    total = tot;
    return wbase + inc - v;
}

// ------------------------------------------------------------------------------------ phase R

// Four threads route one token, so a CTA's 256 threads take a whole 64-token block at once and every
// warp instruction serves eight tokens (a prologue of eight warps per SM is bound by the instructions each
// warp has to issue, not by their latencies).  The block's logits are staged in shared memory (row stride
// = 4 mod 32 words, so the 32 lanes of a warp - eight tokens x four threads - hit 32 different banks).
// Thread q of a quad holds experts q, q+4, ... as order keys in registers; the k selections are k rounds of
// arg-max over the quad.  Order: larger logit first, equal logits by lower expert index (-0 == +0);
// gates = softmax over the selected k.

// fp32 -> uint32 that orders like the float (finite values; -0 has been folded into +0)
__device__ __forceinline__ unsigned float_order_key(float v)
{
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(unsigned k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ int route_row_stride(int E) { return ((E + 27) / 32) * 32 + 4; }

// cooperative copy of the block's logit rows into shared memory, coalesced; all copies are in flight
// together (one memory round trip).  The caller waits (cp_async_wait_all) and publishes them
// (__syncthreads) when it needs them, and may do other work in between.
__device__ __forceinline__ void stage_logits_issue(const KParams &p, int b, float *lg_s)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ntok = min(kRouteBlock, p.T - b * kRouteBlock);
    const int stride = route_row_stride(p.E);
    if ((p.E & 3) == 0) {      // rows are 16-byte multiples: both sides of every copy are 16-byte aligned
        const int per_row = p.E >> 2;
        for (int i = threadIdx.x; i < ntok * per_row; i += kThreads) {
            const int r = i / per_row, c = (i - r * per_row) << 2;
            cp_async_16(smem_u32(lg_s + r * stride + c), p.logits + (size_t)(b * kRouteBlock + r) * p.E + c);
        }
    } else {
        for (int r = warp; r < ntok; r += kThreads / 32) {
            const float *src = p.logits + (size_t)(b * kRouteBlock + r) * p.E;
            for (int c = lane; c < p.E; c += 32) cp_async_4(smem_u32(lg_s + r * stride + c), src + c);
        }
    }
}

// Top-k selection of routing block b by k rounds of arg-max.  Thread q of a quad owns experts q, q+4, ...
// of its token.  A first pass turns the staged logits into order keys IN PLACE (shared memory) and finds
// the thread's best (largest key, lowest expert index among equals).  A round: the quad's best of the four
// bests (two shuffle steps; equal keys go to the lower expert index) is slot j; its owner writes a zero over
// that key and rescans its keys.  The keys live in shared memory rather than in registers so that both
// passes are short ROLLED loops: this code runs once or twice per launch, at the speed of instruction
// fetch, and a loop body is fetched once (the unrolled register version issued fewer instructions and
// took twice as long).  The scratch arrays come as 32-bit shared-memory addresses.  r_mask[e] (64 bits):
// bit tl set when token tl of the block selected expert e (an expert hosted here); r_idx[tl][j]: the
// expert of slot j, -1 when another rank hosts it; r_cnt: local / remote (token, expert) pairs of the
// block (expert-parallel share only); r_p: [64][16] floats of scratch for the exponentials (the sum is
// only known once all k slots are chosen).  write_out: this CTA is the one that writes the block's selections
// and gates to global memory (every CTA routes a small batch for itself, one of them writes it down).
// Its shared-memory accesses name the shared space, so that it could also be compiled out of line (a function
// that is not inlined sees generic pointers, and generic atomics that land in shared memory take a slow
// path); inlined it is 1-3 us per layer faster on the small batches.
struct RouteArgs {
    int T, E, k, ep_size, ep_rank, ep_tshard;
    int *status;
    int *topk_idx;
    float *gates;
};
__device__ __forceinline__ void route_block_quads(int T, int E, int k, int ep_size, int ep_rank, int ep_tshard, int *status,
                                               int *topk_idx, float *gates, int b, uint32_t lg_s, uint32_t r_mask,
                                               uint32_t r_idx, uint32_t r_cnt, uint32_t r_p, bool write_out)
{
    static_assert(kThreads == 4 * kRouteBlock, "four threads per token of a routing block");
    const int tl = threadIdx.x >> 2, q = threadIdx.x & 3;
    const int t = b * kRouteBlock + tl;
    const bool valid = t < T;
    const int e_lo = ep_size > 1 ? ep_rank * (E / ep_size) : 0;
    const int e_hi = ep_size > 1 ? e_lo + E / ep_size : E;
    const uint32_t row = lg_s + 4u * (uint32_t)(tl * route_row_stride(E));      // this token's logits, then keys

    // keys: 0 = nothing there; every finite logit maps to a key >= 1 that orders like the float
    // (a token past the end keeps all-zero keys: its quad then selects nothing and writes nothing)
    unsigned bk = 0u;
    int be = 0x7fffffff;      // expert of this thread's best key
    bool bad = false;
#pragma unroll 2
    for (int e = q; e < E; e += 4) {
        float x = ld_shared_f32(row + 4u * (uint32_t)e);
        const bool nf = !(fabsf(x) <= 3.402823466e38f);      // NaN or +-inf: flag it, keep indices in range
        bad = bad || (valid && nf);
        x = nf ? -3.402823466e38f : x;
        x = __fadd_rn(x, 0.0f);                              // folds -0 into +0, leaves everything else alone
        const unsigned c = valid ? float_order_key(x) : 0u;
        st_shared_u32(row + 4u * (uint32_t)e, c);
        if (c > bk) { bk = c; be = e; }                      // strict: the lower expert index stays
    }
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicCAS(status, 0, kErrNonFinite);

    float vmax = 0.f, sum = 0.f;
    int nloc = 0;
    for (int j = 0; j < k; ++j) {
        unsigned hk = bk;
        int hi = bk ? be : 0x7fffffff;
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {
            const unsigned ok = __shfl_xor_sync(0xffffffffu, hk, o);
            const int oi = __shfl_xor_sync(0xffffffffu, hi, o);
            if (ok > hk || (ok == hk && oi < hi)) { hk = ok; hi = oi; }
        }
        // every thread of the quad knows slot j now; thread j mod 4 writes it down
        const float v = float_from_order_key(hk);
        if (j == 0) vmax = v;
        const float pj = expf(v - vmax);
        sum += pj;                                   // slot order
        // expert-parallel share: only the experts hosted here get rows; the gates stay normalised over
        // all k selected experts
        const bool local = hi >= e_lo && hi < e_hi;
        nloc += local ? 1 : 0;
        if (valid && (j & 3) == q) {
            st_shared_u32(r_p + 4u * (uint32_t)(tl * kMaxTopK + j), __float_as_uint(pj));
            if (write_out) {
                topk_idx[(size_t)t * k + j] = hi;
                st_shared_u32(r_idx + 4u * (uint32_t)(tl * kMaxTopK + j), (uint32_t)(local ? hi : -1));
            }
            if (local) red_shared_or_u32(r_mask + 8u * (uint32_t)hi + 4u * (uint32_t)(tl >> 5), 1u << (tl & 31));
        }
        // the owner takes its winner out and looks for its next best
        if ((hi & 3) == q && hk != 0u) {
            st_shared_u32(row + 4u * (uint32_t)hi, 0u);
            bk = 0u; be = 0x7fffffff;
#pragma unroll 4
            for (int e = q; e < E; e += 4) {
                const unsigned c = ld_shared_u32(row + 4u * (uint32_t)e);
                if (c > bk) { bk = c; be = e; }
            }
        }
    }
    __syncwarp();
    if (valid) {
        if (write_out)
            for (int j = q; j < k; j += 4)
                gates[(size_t)t * k + j] = __fdiv_rn(__uint_as_float(ld_shared_u32(r_p + 4u * (uint32_t)(tl * kMaxTopK + j))), sum);
        if (ep_size > 1 && q == 0 && nloc) {
            if (t / ep_tshard == ep_rank) red_shared_add_u32(r_cnt, (uint32_t)nloc);
            else {
                red_shared_add_u32(r_cnt + 4u, (uint32_t)nloc);
                red_shared_or_u32(r_mask + 8u * (uint32_t)kMaxEE + 4u * (uint32_t)(tl >> 5), 1u << (tl & 31));
            }
        }
    }
}

// ------------------------------------------------------------------------------------ cost model

// Eq. 15 for one candidate, in the same fp32 operation order as the CPU restatement:
// T_comp = W_comp / (TFLOPS(N-c) * eff_chunk(K))  (Eq. 9),  T_comm = (W_disp + W_comb) / BW(c)  (Eq. 5),
// T_tail = (1 - alpha) * W_comb / (BW(c) * K)  (Eq. 10),  T_total = max(T_comp + T_tail, T_comm).
// bw = BW(c), tf = TFLOPS(N - c): the candidate's two table entries
template <class PB>
__device__ __forceinline__ float model_t_total(const PB &p, float bw, float tf, int ki, float w_comp, float w_disp,
                                               float w_comb)
{
    const float Kf = (float)(1 << ki);
    const float t_comp = __fdiv_rn(w_comp, __fmul_rn(tf, p.eff[ki]));
    const float t_comm = __fdiv_rn(__fadd_rn(w_disp, w_comb), bw);
    const float t_tail = __fmul_rn(__fsub_rn(1.0f, p.alpha), __fdiv_rn(w_comb, __fmul_rn(bw, Kf)));
    return fmaxf(__fadd_rn(t_comp, t_tail), t_comm);
}

// Plan kind "dispatch on all SMs, then split": W_disp / BW(N), then Eq. 15 with only the combine left as
// communication.  bw_n = BW(N).
template <class PB>
__device__ __forceinline__ float model_t_dispatch_all(const PB &p, float bw, float tf, float bw_n, int ki, float w_comp,
                                                      float w_disp, float w_comb)
{
    const float Kf = (float)(1 << ki);
    const float t_disp = __fdiv_rn(w_disp, bw_n);
    const float t_comp = __fdiv_rn(w_comp, __fmul_rn(tf, p.eff[ki]));
    const float t_tail = __fmul_rn(__fsub_rn(1.0f, p.alpha), __fdiv_rn(w_comb, __fmul_rn(bw, Kf)));
    const float t_comb = __fdiv_rn(w_comb, bw);
    return __fadd_rn(t_disp, fmaxf(__fadd_rn(t_comp, t_tail), t_comb));
}

// Plan kind "phased": dispatch, GEMMs and combine one after the other, each on all N SMs.
template <class PB>
__device__ __forceinline__ float model_t_phased(const PB &p, float bw_n, float tf_n, float w_comp, float w_disp, float w_comb)
{
    return __fadd_rn(__fadd_rn(__fdiv_rn(w_disp, bw_n), __fdiv_rn(w_comp, tf_n)),
                     __fmul_rn(__fsub_rn(1.0f, p.alpha), __fdiv_rn(w_comb, bw_n)));
}

// Plan kind "split with rejoin": while c SMs dispatch (W_disp / BW(c)), N - c SMs run GEMM tiles (the work
// done meanwhile as in Eq. 12, but no more than the gate/up tiles of the layer, 4HI of the 6HI FLOPs per
// row: the queue runs them first and a down tile needs its m-block's gate/up tiles, so a dispatch that
// outlasts them holds the GEMM SMs up); what is left then runs on all N SMs; the final combine is on all
// N SMs.
template <class PB>
__device__ __forceinline__ float model_t_rejoin(const PB &p, float bw, float tf, float bw_n, float tf_n, float w_comp,
                                                float w_disp, float w_comb)
{
    const float t_disp = __fdiv_rn(w_disp, bw);
    const float w_during = fminf(__fmul_rn(t_disp, tf), __fmul_rn(w_comp, 0.6666667f));
    const float w_rest = fmaxf(0.0f, __fsub_rn(w_comp, w_during));
    return __fadd_rn(__fadd_rn(t_disp, __fdiv_rn(w_rest, tf_n)),
                     __fmul_rn(__fsub_rn(1.0f, p.alpha), __fdiv_rn(w_comb, bw_n)));
}

// Eq. 11-14 with W_tile = W_comp / n_tiles (the mean GEMM tile of this layer).
__device__ __forceinline__ int model_n_steal(int n_sm, float bw, float tf, float w_comp, float w_disp,
                                             float w_comb, int n_tiles)
{
    if (n_tiles <= 0) return 0;
    const float t_comm = __fdiv_rn(__fadd_rn(w_disp, w_comb), bw);
    const float w_partial = __fmul_rn(t_comm, tf);
    const float w_steal = fmaxf(0.0f, __fsub_rn(w_comp, w_partial));
    const float w_tile = __fdiv_rn(w_comp, (float)n_tiles);
    if (!(w_tile > 0.0f)) return 0;
    // a GEMM worker is a CTA pair: W_steal is shared by n_sm / 2 workers (Eq. 14's N)
    const float ns = __fdiv_rn(w_steal, __fmul_rn((float)(n_sm / 2), w_tile));
    int r = (int)floorf(__fadd_rn(ns, 0.5f));
    return max(0, min(r, n_tiles));
}

// Eq. 16: the arg-min of the modelled layer time over the candidate plans, evaluated by the whole CTA (every
// CTA evaluates it for itself and gets the same answer).  Thread tid owns the split candidate
// (c, K) = (c_min + (tid >> 2) * c_step, 1 << (tid & 3)) and its "dispatch on all SMs first" and "rejoin"
// variants; thread 0 also owns the phased plan.  Candidate order = (kind, c ascending, K ascending),
// index = kind * 256 + thread; the phased plan is index 512, the rejoin plans follow it; ties go to the
// smaller index.  Contains one __syncthreads(); S.red_f and S.red_i[.][0] carry the reduction.
struct PlanPick { int c, ki, kind; float t; };
struct ModelArgs { float alpha, eff[4]; int kinds, c_min, c_step; };     // by value, see RouteArgs
__device__ __noinline__ PlanPick model_pick(const ModelArgs p, SmemTail &S, int n_sm, float w_comp, float w_disp, float w_comb,
                                            bool cm_ok, float cm_bw, float cm_tf, float cm_bw_n, float cm_tf_n)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cm_ki = tid & 3;
    float t = __int_as_float(0x7f800000);
    int bi = tid;
    if (cm_ok && (p.kinds & (1 << kPlanSplit))) t = model_t_total(p, cm_bw, cm_tf, cm_ki, w_comp, w_disp, w_comb);
    if (cm_ok && (p.kinds & (1 << kPlanDispatchAll))) {
        const float t1 = model_t_dispatch_all(p, cm_bw, cm_tf, cm_bw_n, cm_ki, w_comp, w_disp, w_comb);
        if (t1 < t) { t = t1; bi = kThreads + tid; }
    }
    if (tid == 0 && (p.kinds & (1 << kPlanPhased))) {
        const float t2 = model_t_phased(p, cm_bw_n, cm_tf_n, w_comp, w_disp, w_comb);
        if (t2 < t) { t = t2; bi = 2 * kThreads; }
    }
    if (cm_ok && cm_ki == 0 && (p.kinds & (1 << kPlanRejoin))) {      // K = 1 only
        const float t3 = model_t_rejoin(p, cm_bw, cm_tf, cm_bw_n, cm_tf_n, w_comp, w_disp, w_comb);
        if (t3 < t) { t = t3; bi = 3 * kThreads + tid; }
    }
    // (rolled loops: this code runs once per launch, at the speed of instruction fetch)
#pragma unroll 1
    for (int o = 16; o > 0; o >>= 1) {
        const float ot = __shfl_xor_sync(0xffffffffu, t, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ot < t || (ot == t && oi < bi)) { t = ot; bi = oi; }
    }
    if (lane == 0) { S.red_f[warp] = t; S.red_i[warp][0] = bi; }
    __syncthreads();
    t = S.red_f[0]; bi = S.red_i[0][0];
#pragma unroll 1
    for (int w = 1; w < kThreads / 32; ++w) {
        const float ot = S.red_f[w];
        const int oi = S.red_i[w][0];
        if (ot < t || (ot == t && oi < bi)) { t = ot; bi = oi; }
    }
    PlanPick r;
    r.kind = bi / kThreads;
    const int bt = bi % kThreads;      // the thread that evaluated the winner
    r.c = r.kind == kPlanPhased ? n_sm : p.c_min + (bt >> 2) * p.c_step;
    r.ki = r.kind == kPlanPhased ? 0 : (bt & 3);
    r.t = t;
    return r;
}

// ------------------------------------------------------------------------------------ tile decoding

// largest s in [lo, hi) with (seg_mb0[s] - base) * mul <= key   (empty segments share a start)
__device__ __forceinline__ int seg_search(const SmemTail &S, int lo, int hi, int base, int mul, int key)
{
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if ((S.seg_mb0[mid] - base) * mul <= key) lo = mid; else hi = mid;
    }
    return lo;
}

// m-block -> its rows; seg = the (chunk, expert) segment it belongs to (index chunk * EE + expert)
__device__ __forceinline__ void decode_mblock(const SmemTail &S, int EE, int mb, int &row0, int &nrows, int &seg)
{
    const int s = seg_search(S, 0, S.K * EE, 0, 1, mb);
    seg = s;
    const int m = mb - S.seg_mb0[s];
    row0 = S.seg_row0[s] + m * kBM;
    nrows = min(kBM, S.seg_rows[s] - m * kBM);
}

// GEMM queue order (the chunk-pipeline DAG order): chunk by chunk; inside a chunk all gemm0 tiles,
// then all gemm1 tiles (every gemm0 tile a gemm1 tile waits for comes earlier in the queue and waits
// only for dispatch, which keeps the in-order schedulers free of deadlock); inside those
// expert-major, then groups of kPairGroup pair tiles, n-tile, pair tile fastest: consecutive tiles
// share a weight panel, and a group's rows stay in L2 while all its n-tiles pass.  A pair tile = two
// consecutive m-blocks of one segment; a segment's last, unpaired m-block is a member of its group
// like any other pair tile (operands swapped), so it reads each weight panel right beside the
// expert's regular tiles.  `lead` describes the leader CTA's half, `peer` the other CTA's.
// Two other orders were measured and dropped: spreading the swapped tiles evenly over the queue
// (no faster, and a large expert's panels were fetched a second time for its last m-block: +27 %
// DRAM traffic on the Mixtral-shaped layer), and alternating gemm1 with gemm0 units (+1 % at
// I = 512, -9 % on the Qwen3-235B-shaped stack: two weight working sets in L2).
// Host-callable so that the order can be checked without a GPU.
__host__ __device__ __forceinline__ void decode_pair_tile(const SmemTail &S, const KParams &p, int g, TileInfo &lead,
                                                          TileInfo &peer)
{
    int j = 0;
    while (j + 1 < S.K && g >= S.chunk_tile0[j + 1]) ++j;
    int local = g - S.chunk_tile0[j];
    const int cpt0 = S.chunk_pt0[j];
    const int nptj = S.chunk_pt0[j + 1] - cpt0;
    int type = 0, nt = p.nt0;
    if (local >= nptj * p.nt0) { type = 1; local -= nptj * p.nt0; nt = p.nt1; }
    // largest s of the chunk with (seg_pt0[s] - cpt0) * nt <= local (empty segments share a start)
    int lo = j * p.EE, hi = (j + 1) * p.EE;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((S.seg_pt0[mid] - cpt0) * nt <= local) lo = mid; else hi = mid;
    }
    const int s = lo;
    const int pts = S.seg_pt0[s + 1] - S.seg_pt0[s];
    const int within = local - (S.seg_pt0[s] - cpt0) * nt;
    const int gi = within / (kPairGroup * nt);
    const int wg = within - gi * kPairGroup * nt;
    const int gsize = (pts - gi * kPairGroup) < kPairGroup ? (pts - gi * kPairGroup) : kPairGroup;
    const int n = wg / gsize;
    const int m0 = 2 * (gi * kPairGroup + (wg - n * gsize));
    const int rows = S.seg_rows[s];
    lead.type = peer.type = type;
    lead.e = peer.e = s - j * p.EE;
    lead.n = peer.n = n;
    lead.chunk = peer.chunk = j;
    lead.nkb = peer.nkb = (type == 0 ? p.H : p.I) / kBK;
    lead.mb = S.seg_mb0[s] + m0;
    lead.row0 = S.seg_row0[s] + m0 * kBM;
    lead.nrows = (rows - m0 * kBM) < kBM ? (rows - m0 * kBM) : kBM;
    if (rows - (m0 + 1) * kBM <= 0) {
        // the segment's last, unpaired m-block: both CTAs work on it with the operands swapped,
        // so the MMA costs ceil(nrows/16)*16 columns instead of a half-empty 256-row tile
        lead.type = type + 3;
        peer = lead;
        return;
    }
    peer.nrows = (rows - (m0 + 1) * kBM) < kBM ? (rows - (m0 + 1) * kBM) : kBM;
    peer.mb = lead.mb + 1;
    peer.row0 = lead.row0 + kBM;
}

// epilogue-warp arrivals on y_done[j] when all gemm1 tiles of chunk j are finished: 4 per (m-block,
// n-tile); an m-block processed as a swapped tile is finished by both CTAs of the pair (8)
__device__ __forceinline__ unsigned y_done_target(const SmemTail &S, const KParams &p, int j)
{
    return (unsigned)(((S.chunk_mb0[j + 1] - S.chunk_mb0[j]) + S.chunk_nswap[j]) * p.nt1 * kEpiWarps);
}

// ------------------------------------------------------------------------------------ phase A: dispatch

// Tile = one m-block: Xe[row0 + r] = x[token_of[row0 + r]].  The copy engine does the moving: warp 0
// gathers the source rows with bulk loads into a ring of 32 KB buffers, one thread of warp 1
// writes each full buffer to its (contiguous) destination rows with one bulk store.  About 96 KB
// of loads and as much of stores are in flight per SM.  The m-block's ready flag is released once
// its last store has completed.
// n_disp = number of CTAs that take part in the dispatch of this launch: CTA i's first tile is m-block i
// (no queue round trip before the first copy), later claims go through the queue, which starts at n_disp.
// local_route (a small batch that every CTA routed for itself): this CTA's copy of the routing blocks'
// expert masks, [nblk][kMaxEE + 1], sits at the start of the epilogue staging area; the source tokens of a
// tile are looked up there and nothing is read from the routing outputs in global memory.
__device__ __forceinline__ int nth_set_bit(unsigned long long m, int r)
{
    const unsigned lo = (unsigned)m, hi = (unsigned)(m >> 32);
    const int cl = __popc(lo);
    return r < cl ? (int)__fns(lo, 0u, r + 1) : 32 + (int)__fns(hi, 0u, r - cl + 1);
}
__device__ __forceinline__ void dispatch_phase(const KParams &p, SmemTail &S, uint8_t *stages, int max_tiles, int n_disp,
                                               bool local_route)
{
    const unsigned long long *lmask = local_route ? reinterpret_cast<const unsigned long long *>(stages + kStages * kStageBytes) : nullptr;
    MoveScratch &M = move_scratch(stages);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    fence_proxy_async();      // the buffers held routing scratch written with ordinary stores
    __syncthreads();
    const uint32_t rowb = (uint32_t)p.H * 2u;
    const int R = max(1, kMvBuf / (int)rowb);     // rows per buffer
    if (warp == 0) {
        // ---- loader
        int b = 0;
        uint32_t ph = 0;
        bool ok = true;
        if (lane == 0 && lmask == nullptr) ok = flag_wait_ge(&p.ctl->fix_done, (unsigned)p.nblk, p, 10);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (p.ep_size > 1) {
            // expert-parallel share: first every remote token that has an expert here is copied ONCE
            // into the staging buffer xs (the dispatch-side deduplication of the paper's Section 4);
            // the rows of all its local experts are then gathered from that copy.  One tile per
            // 64-token routing block, taken by whoever comes first.
            while (ok) {
                int blk = 0;
                if (lane == 0) blk = (int)atomicAdd(&p.ctl->q_pull, 1u);
                blk = __shfl_sync(0xffffffffu, blk, 0);
                if (blk >= p.nblk) break;
                const unsigned long long um = lmask ? lmask[blk * (kMaxEE + 1) + kMaxEE] : __ldcg(p.uniq_mask + blk);
                const int n = __popcll(um);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int bit = lane + 32 * hh;
                    if ((um >> bit) & 1ull) M.tok[__popcll(um & ((1ull << bit) - 1ull))] = blk * kRouteBlock + bit;
                }
                __syncwarp();
                if (lane == 0) {
                    if (n == 0) {
                        red_release_add_u32(&p.ctl->pull_done, 1u);
                    } else {
                        const int Rp = min(R, 32);
                        for (int r0 = 0; r0 < n; r0 += Rp) {
                            const int nr = min(Rp, n - r0);
                            if (!mbar_wait(&S.dv_empty[b], ph ^ 1u, p, 14)) { ok = false; break; }
                            M.mv[b].a = 0; M.mv[b].b = nr; M.mv[b].c = blk; M.mv[b].d = (r0 + nr >= n) ? 4 : 3;
                            for (int i = 0; i < nr; ++i) M.mv[b].tok[i] = M.tok[r0 + i];
                            mbar_arrive_expect_tx(&S.dv_full[b], (uint32_t)nr * rowb);
                            const uint32_t dst = smem_u32(stages + b * kMvBuf);
                            for (int i = 0; i < nr; ++i)
                                bulk_load(dst + (uint32_t)i * rowb, p.x + (size_t)M.tok[r0 + i] * p.H, rowb, &S.dv_full[b]);
                            if (++b == kStages) { b = 0; ph ^= 1u; }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                __syncwarp();
            }
            // rows may be gathered from xs only when every block has been staged: have the storer
            // complete and publish what it still holds back (d = 5), then wait for everybody's blocks
            if (lane == 0 && ok) {
                if (mbar_wait(&S.dv_empty[b], ph ^ 1u, p, 16)) {
                    M.mv[b].d = 5;
                    mbar_arrive(&S.dv_full[b]);
                    if (++b == kStages) { b = 0; ph ^= 1u; }
                } else ok = false;
            }
            if (lane == 0 && ok && max_tiles > 0) ok = flag_wait_ge(&p.ctl->pull_done, (unsigned)p.nblk, p, 15);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            // only lane 0 walked the ring so far; from here on every lane addresses the buffers
            b = __shfl_sync(0xffffffffu, b, 0);
            ph = __shfl_sync(0xffffffffu, ph, 0);
        }
        for (int taken = 0; ok && taken < max_tiles; ++taken) {
            int mb = (int)blockIdx.x;
            if (taken > 0) {
                if (lane == 0) mb = n_disp + (int)atomicAdd(&p.ctl->q_disp, 1u);
                mb = __shfl_sync(0xffffffffu, mb, 0);
            }
            if (mb >= S.nmb) { if (taken > 0) break; else continue; }
            int row0, nrows, seg;
            decode_mblock(S, p.EE, mb, row0, nrows, seg);
            if (lmask == nullptr) {
                for (int i = lane; i < nrows; i += 32) M.tok[i] = __ldcg(p.token_of + row0 + i);
            } else {
                // row r of expert e = the r-th token that selected it, in token order; a shared expert's
                // row r is token r
                const int e = seg % p.EE;
                for (int i = lane; i < nrows; i += 32) {
                    int rank = row0 + i - S.offsets[e];
                    int tok = rank;
                    if (e < p.E) {
                        tok = 0;
                        for (int bb = 0; bb < p.nblk; ++bb) {
                            const unsigned long long mk = lmask[bb * (kMaxEE + 1) + e];
                            const int c = __popcll(mk);
                            if (rank < c) { tok = bb * kRouteBlock + nth_set_bit(mk, rank); break; }
                            rank -= c;
                        }
                    }
                    M.tok[i] = tok;
                }
            }
            __syncwarp();
            for (int r0 = 0; r0 < nrows && ok; r0 += R) {
                const int nr = min(R, nrows - r0);
                if (lane == 0) {
                    if (!mbar_wait(&S.dv_empty[b], ph ^ 1u, p, 11)) ok = false;
                    else {
                        M.mv[b].a = row0 + r0; M.mv[b].b = nr; M.mv[b].c = mb; M.mv[b].d = (r0 + nr >= nrows) ? 1 : 0;
                        mbar_arrive_expect_tx(&S.dv_full[b], (uint32_t)nr * rowb);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                // the expected byte count is registered; the lanes issue the row copies side by side
                const uint32_t dst = smem_u32(stages + b * kMvBuf);
                for (int i = lane; i < nr; i += 32) {
                    const int tk = M.tok[r0 + i];
                    // a remote token (another rank's shard) is read from its staged copy
                    const __nv_bfloat16 *src = (p.ep_size > 1 && tk / p.ep_tshard != p.ep_rank) ? p.xs : p.x;
                    bulk_load(dst + (uint32_t)i * rowb, src + (size_t)tk * p.H, rowb, &S.dv_full[b]);
                }
                if (++b == kStages) { b = 0; ph ^= 1u; }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            __syncwarp();
        }
        if (lane == 0 && ok && mbar_wait(&S.dv_empty[b], ph ^ 1u, p, 12)) {
            M.mv[b].d = 2;
            mbar_arrive(&S.dv_full[b]);
        }
        // a wait gave up (or the abort word was seen): copies this warp issued may still be landing in
        // this CTA's buffers; let them land before the CTA can leave
        if (!ok && lane == 0) linger_after_abort();
        __syncwarp();
    } else if (warp == 1) {
        // ---- storer: one bulk store per buffer.  A buffer is handed back as soon as the store has
        // read it; an m-block's flag is published once the stores up to its last one have completed
        // (checked with a lag of kFlagLag stores, so the copy engine never drains).
        if (lane == 0) {
            constexpr int kFlagLag = 4, kPend = 8;
            int b = 0, n = 0;
            uint32_t ph = 0;
            int prev_buf = -1;
            int pe_idx[kPend], pe_mb[kPend], pe_rows[kPend];      // tile ends not yet published (mb < 0: a staged block)
            unsigned long long pe_t0[kPend];
            for (int i = 0; i < kPend; ++i) { pe_idx[i] = 0; pe_mb[i] = 0; pe_rows[i] = 0; pe_t0[i] = 0ull; }
            int pe_head = 0, pe_tail = 0;
            auto publish_upto = [&](int done_idx) {      // stores with index <= done_idx have completed
                bool fenced = false;
                while (pe_head != pe_tail && pe_idx[pe_head % kPend] <= done_idx) {
                    const int s8 = pe_head % kPend;
                    // (the bulk stores have completed; the release below orders them for whoever acquires the flag)
                    if (!fenced) { fence_proxy_async_global(); fenced = true; }
                    if (pe_mb[s8] < 0) {
                        red_release_add_u32(&p.ctl->pull_done, 1u);      // a block of remote tokens is staged
                    } else {
                        if (pe_mb[s8] != p.withhold_mb) st_release_u32(&p.xe_ready[pe_mb[s8]], 1u);
                        trace_ev(p, S, kEvDispatch, (unsigned)pe_mb[s8], pe_t0[s8], trace_now(p), (unsigned)pe_rows[s8]);
                    }
                    ++pe_head;
                }
            };
            unsigned long long tile_t0 = trace_now(p);
            for (;;) {
                if (!mbar_wait(&S.dv_full[b], ph, p, 13)) break;
                const int da = M.mv[b].a, db = M.mv[b].b, dc = M.mv[b].c, dd = M.mv[b].d;
                if (dd == 2) break;
                if (dd == 5) {      // flush: everything stored so far becomes visible and is published
                    bulk_wait<0>();
                    if (prev_buf >= 0) { mbar_arrive(&S.dv_empty[prev_buf]); prev_buf = -1; }
                    publish_upto(n);
                    mbar_arrive(&S.dv_empty[b]);
                    if (++b == kStages) { b = 0; ph ^= 1u; }
                    continue;
                }
                if (dd >= 3) {      // staged remote tokens: one store per row, to the token's own slot of xs
                    for (int i = 0; i < db; ++i)
                        bulk_store(p.xs + (size_t)M.mv[b].tok[i] * p.H, smem_u32(stages + b * kMvBuf) + (uint32_t)i * rowb, rowb);
                } else {
                    bulk_store(p.xe + (size_t)da * p.H, smem_u32(stages + b * kMvBuf), (uint32_t)db * rowb);
                }
                bulk_commit();
                if (prev_buf >= 0) { bulk_wait_read<1>(); mbar_arrive(&S.dv_empty[prev_buf]); }
                prev_buf = b;
                if (dd == 1 || dd == 4) {
                    if (pe_tail - pe_head == kPend) { bulk_wait<0>(); publish_upto(n); }
                    const int s8 = pe_tail % kPend;
                    pe_idx[s8] = n; pe_mb[s8] = dd == 4 ? -1 : dc; pe_rows[s8] = db; pe_t0[s8] = tile_t0;
                    ++pe_tail;
                    tile_t0 = trace_now(p);
                }
                if (n >= kFlagLag && pe_head != pe_tail) { bulk_wait<kFlagLag>(); publish_upto(n - kFlagLag); }
                ++n;
                if (++b == kStages) { b = 0; ph ^= 1u; }
            }
            bulk_wait<0>();
            if (prev_buf >= 0) mbar_arrive(&S.dv_empty[prev_buf]);
            publish_upto(n);
        }
        __syncwarp();
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------ phase C: combine

// Tile = 16 tokens.  out[t] = sum_j gate[t,j] * y[row_of[t,j]] in slot order, then the shared
// experts with weight 1; fp32 accumulate, bf16 store.  Warp 0 gathers, per token and per piece of
// W columns, the k+S source rows with bulk loads into a ring of 32 KB buffers; warps 2..7 reduce
// each full buffer from shared memory and write the output row piece with coalesced stores.
__device__ __forceinline__ void combine_phase(const KParams &p, SmemTail &S, uint8_t *stages)
{
    MoveScratch &M = move_scratch(stages);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    fence_proxy_async();
    __syncthreads();
    const int kk = p.k + p.S;
    const int W = min(p.H, ((kMvBuf / (2 * kk)) / 64) * 64);     // columns per piece (128-byte multiple)
    const int g = kFine / S.K;
    if (warp == 0) {
        // ---- loader
        int b = 0;
        uint32_t ph = 0;
        int ready_upto = -1;     // chunks [0, ready_upto] are known complete
        bool perm_final = false; // the permutation's rows (row_of, gates) are known final
        bool ok = true;
        for (;;) {
            int q = 0;
            if (lane == 0) q = (int)atomicAdd(&p.ctl->q_comb, 1u);
            q = __shfl_sync(0xffffffffu, q, 0);
            if (q >= S.n_comb) break;
            const int t0 = q * S.comb_tok;
            const int chunk = (((t0 / kRouteBlock) * kFine) / p.nblk) / g;
            const int ntok = min(S.comb_tok, p.T - t0);
            // the tile's rows and gates are final once the permutation is; they are fetched before the wait for
            // the chunk's last GEMM tile, so that only the row copies themselves follow that wait
            if (!perm_final) {
                if (lane == 0) ok = flag_wait_ge(&p.ctl->fix_done, (unsigned)p.nblk, p, 20);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                perm_final = true;
            }
            for (int i = lane; i < ntok * kk; i += 32) {
                const int tt = i / kk, j = i - tt * kk, t = t0 + tt;
                M.crow[tt][j] = j < p.k ? __ldcg(p.row_of + (size_t)t * p.k + j) : S.offsets[p.E + (j - p.k)] + t;
                M.cgate[tt][j] = j < p.k ? __ldcg(p.gates + (size_t)t * p.k + j) : 1.0f;
            }
            __syncwarp();
            if (chunk > ready_upto) {
                if (lane == 0) {
                    const unsigned long long tw0 = trace_now(p);
                    for (int j = ready_upto + 1; ok && j <= chunk; ++j) {
                        ok = flag_wait_ge(&p.ctl->y_done[j], y_done_target(S, p, j), p, 21);
                    }
                    trace_ev(p, S, kEvWaitChunk, (unsigned)chunk, tw0, trace_now(p), 0u);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                ready_upto = chunk;
            }
            const unsigned long long tc0 = trace_now(p);
            for (int tt = 0; tt < ntok && ok; ++tt) {
                // lane j owns slot j of the token: its rank among the slots that have a row here (slots
                // whose expert lives on another rank have row -1 and are skipped)
                const int myrow = lane < kk ? M.crow[tt][lane] : -1;
                const unsigned vmask = __ballot_sync(0xffffffffu, myrow >= 0);
                const int nv = __popc(vmask), mypos = __popc(vmask & ((1u << lane) - 1u));
                // a token with few rows here (expert-parallel share) takes wider pieces: as many columns
                // as fit the buffer with the rows it really has
                const int Wt = nv >= kk ? W : min(p.H, ((kMvBuf / (2 * max(nv, 1))) / 64) * 64);
                for (int col0 = 0; col0 < p.H && ok; col0 += Wt) {
                    const int w = min(Wt, p.H - col0);
                    if (lane == 0) {
                        if (!mbar_wait(&S.cb_empty[b], ph ^ 1u, p, 22)) ok = false;
                        else {
                            M.mv[b].a = t0 + tt; M.mv[b].b = col0; M.mv[b].c = w; M.mv[b].d = 0; M.mv[b].n = nv;
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (myrow >= 0) M.mv[b].g[mypos] = M.cgate[tt][lane];
                    __syncwarp();
                    if (lane == 0) {
                        if (nv > 0) mbar_arrive_expect_tx(&S.cb_full[b], (uint32_t)(nv * w * 2));
                        else mbar_arrive(&S.cb_full[b]);
                    }
                    __syncwarp();
                    // the byte count is registered; the lanes issue the row copies side by side
                    if (myrow >= 0)
                        bulk_load(smem_u32(stages + b * kMvBuf) + (uint32_t)(mypos * w * 2),
                                  p.y + (size_t)myrow * p.H + col0, (uint32_t)(w * 2), &S.cb_full[b]);
                    if (++b == kStages) { b = 0; ph ^= 1u; }
                }
            }
            if (lane == 0) trace_ev(p, S, kEvCombine, (unsigned)q, tc0, trace_now(p), 0u);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            __syncwarp();
        }
        if (lane == 0 && ok && mbar_wait(&S.cb_empty[b], ph ^ 1u, p, 23)) {
            M.mv[b].d = 2;
            mbar_arrive(&S.cb_full[b]);
        }
        if (!ok && lane == 0) linger_after_abort();      // as in the dispatch loader
        __syncwarp();
    } else if (warp >= 2) {
        // ---- reducers
        const int ctid = tid - 64;
        int b = 0;
        uint32_t ph = 0;
        for (;;) {
            bool ok = mbar_wait(&S.cb_full[b], ph, p, 24);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const MvDesc &d = M.mv[b];
            if (d.d == 2) break;
            const int w = d.c, nv = w >> 3, nrow = d.n;
            const uint32_t src = smem_u32(stages + b * kMvBuf);
            __nv_bfloat16 *dst = p.out + (size_t)d.a * p.H + d.b;
            for (int v = ctid; v < nv; v += kCombWarps * 32) {
                float a0[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) a0[i] = 0.f;
                for (int j = 0; j < nrow; ++j) {
                    const uint4 q4 = ld_shared_v4(src + (uint32_t)(j * w * 2 + v * 16));
                    const float gw = d.g[j];
                    a0[0] = fmaf(gw, bf16lo_to_f32(q4.x), a0[0]); a0[1] = fmaf(gw, bf16hi_to_f32(q4.x), a0[1]);
                    a0[2] = fmaf(gw, bf16lo_to_f32(q4.y), a0[2]); a0[3] = fmaf(gw, bf16hi_to_f32(q4.y), a0[3]);
                    a0[4] = fmaf(gw, bf16lo_to_f32(q4.z), a0[4]); a0[5] = fmaf(gw, bf16hi_to_f32(q4.z), a0[5]);
                    a0[6] = fmaf(gw, bf16lo_to_f32(q4.w), a0[6]); a0[7] = fmaf(gw, bf16hi_to_f32(q4.w), a0[7]);
                }
                st_cs_v4(dst + v * 8, make_uint4(pack_bf16x2(a0[0], a0[1]), pack_bf16x2(a0[2], a0[3]),
                                                 pack_bf16x2(a0[4], a0[5]), pack_bf16x2(a0[6], a0[7])));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.cb_empty[b]);
            if (++b == kStages) { b = 0; ph ^= 1u; }
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------ phase B: GEMM

// Tensor maps of the GEMM operands: bf16 matrices, boxes of 64 columns (one 128-byte swizzle row) by
// 128 rows (64 rows for the gate and up halves of a swapped tile's weight operand; 8, 16, 32 or 64
// rows for a swapped tile's row operand, whichever covers its half of the m-block's rows).
struct TmaMaps { CUtensorMap xe, wgu, h, wd, wgu64, xe_n[4], h_n[4]; };

struct PipeState {     // per-role ring positions; they persist across the tiles of a phase
    int stage = 0;  uint32_t stage_phase = 0;
    int acc = 0;    uint32_t acc_phase = 0;
    int slot = 0;   uint32_t slot_phase = 0;
    __device__ __forceinline__ void next_stage() { if (++stage == kStages) { stage = 0; stage_phase ^= 1u; } }
    __device__ __forceinline__ void next_acc() { if (++acc == 2) { acc = 0; acc_phase ^= 1u; } }
    __device__ __forceinline__ void next_slot() { if (++slot == kTinfo) { slot = 0; slot_phase ^= 1u; } }
    int rel = 0;    uint32_t rel_phase = 0;
    __device__ __forceinline__ void next_rel() { if (++rel == kRel) { rel = 0; rel_phase ^= 1u; } }
};

__device__ __forceinline__ float silu_mul(float g, float u)
{
    return __fdividef(g, 1.0f + __expf(-g)) * u;
}

// A consumer of the tile-descriptor ring hands its slot back with a barrier arrival, after which the
// scheduler (for the peer CTA: a thread of ANOTHER CTA, through remote stores) may overwrite the slot.
// The copy of the descriptor must have LANDED in this thread's registers by then.  Program order alone
// does not say so: the arrival has CTA scope (a cluster-scope release would wait for the thread's
// global stores, ~1000 cycles) and no instruction reads the loaded words before it is issued, so the
// shared-memory loads can still be in flight when the slot is rewritten.  Storing a fold of all eight
// words to a scratch word makes the hardware wait for them here: a store cannot issue before its
// operand has arrived, and the arrival is issued after the store.  (An empty asm statement that
// merely names the words generates no instruction and therefore no wait.)
// Seen without it, about once in 300 000 launches and only in the peer CTA: warps reading different
// row counts for one swapped tile, the up/gate exchange of its epilogue running out of step, the
// accumulator never handed back, a bounded wait running out.
__device__ __forceinline__ void tile_info_landed(const TileInfo &ti, int *scratch)
{
    *reinterpret_cast<volatile int *>(scratch) = ti.type ^ ti.mb ^ ti.row0 ^ ti.nrows ^ ti.e ^ ti.n ^ ti.chunk ^ ti.nkb;
}

// bounded wait on a barrier whose guarded data may come from the peer CTA
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, const KParams &p, int where)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    unsigned long long t0 = 0;
    unsigned it = 0;
    unsigned ab = 0u;      // looked at one round late, see mbar_wait
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((++it & 31u) == 0u) {
            if (ab) { note_failed_wait(p.wait_log, where, smem_u32(bar), parity, 2); return false; }
            ab = ld_relaxed_u32(&p.ctl->abort);
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if ((long long)(now - t0) > (long long)p.timeout_ns) {
                give_up(p.ctl, where);
                note_failed_wait(p.wait_log, where, smem_u32(bar), parity, 1);
                return false;
            }
        }
    }
    return true;
}

// 32 rows x 32 columns of bf16 held one row per thread (16 packed words each) go out through the
// warp's own 2 KB of shared memory, so that every store instruction writes 16 rows x 64 contiguous
// bytes (two lanes per row) instead of 32 rows x 32 bytes.  An SM retires st.global at 32 B per
// cycle but at most one 128-byte line every two cycles: one row per thread is 15.8 B/clk per SM,
// two lanes per row 31 B/clk (measured with a store-only probe, alone or on all SMs).
// Shared-memory layout: row r at r*64, its 16-byte chunk c at position c ^ ((r >> 1) & 3): the
// row-per-thread writes and the two-lanes-per-row reads are both free of bank conflicts.
// dst = first of the warp's 32 rows (this batch's first column), pitch in elements.
__device__ __forceinline__ void staged_store_32(const uint32_t (&o)[16], uint32_t stage, __nv_bfloat16 *dst, int pitch,
                                                int rows_valid, int lane)
{
    const uint32_t wbase = stage + (uint32_t)lane * 64u, wsw = (uint32_t)((lane >> 1) & 3);
#pragma unroll
    for (int c = 0; c < 4; ++c)
        st_shared_v4(wbase + (((uint32_t)c ^ wsw) << 4), make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]));
    __syncwarp();
    const int half = lane & 1;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int r = 16 * j + (lane >> 1);
        const uint32_t rbase = stage + (uint32_t)r * 64u, rsw = (uint32_t)((r >> 1) & 3);
        const uint4 q0 = ld_shared_v4(rbase + (((uint32_t)(2 * half) ^ rsw) << 4));
        const uint4 q1 = ld_shared_v4(rbase + (((uint32_t)(2 * half + 1) ^ rsw) << 4));
        if (r < rows_valid) {
            const uint32_t v[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
            st_v8(dst + (size_t)r * pitch + half * 16, v);
        }
    }
    __syncwarp();      // the region is rewritten by the next batch
}

// budget = how many pair tiles this CTA pair may claim (the steal count for a movement pair).
// Called by both CTAs of a pair with the same arguments.
__device__ __forceinline__ void gemm_phase(const KParams &p, SmemTail &S, uint8_t *stages, uint32_t tmem_base,
                                           const TmaMaps *tm, int budget, PipeState &ps)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();      // 0 = leader (issues the MMAs), 1 = peer
    fence_proxy_async();     // the stage buffers were last touched by ordinary stores (routing scratch)
    __syncthreads();

    if (warp == 2 && rank == 0) {
        // ---------------- scheduler (leader only): claims pair tiles in queue order, waits until their
        // inputs are ready, then publishes the tile to both CTAs' descriptor rings.  Runs up to
        // kTinfo tiles ahead of the MMAs, so claim and flag latencies stay off the critical path.
        if (lane == 0) {
            int taken = 0;
            int g_next = (budget > 0 || S.elastic) ? (int)atomicAdd(&p.ctl->q_gemm, 1u) : 0x7fffffff;
            for (;;) {
                const int g = g_next;
                const unsigned long long tp0 = trace_now(p);
                TileInfo tl, tp;
                if (g >= S.n_gemm) { tl.type = tp.type = 2; tl.mb = tp.mb = -1; tl.nrows = tp.nrows = 0; }
                else decode_pair_tile(S, p, g, tl, tp);
                if (!mbar_wait(&S.ti_empty[ps.slot], ps.slot_phase ^ 1u, p, 30)) break;
                S.ti[ps.slot] = tl;
                {
                    const uint32_t dst = mapa_u32(smem_u32(&S.ti[ps.slot]), 1u);
                    const uint32_t *src = reinterpret_cast<const uint32_t *>(&tp);
#pragma unroll
                    for (int w = 0; w < (int)(sizeof(TileInfo) / 4); ++w) st_cluster_u32(dst + 4 * w, src[w]);
                }
                if (tl.type != 2) {
                    ++taken;
                    bool more = taken < budget;
                    if (!more && S.elastic) {
                        // the steal quota is used up: keep taking GEMM tiles for as long as the next
                        // combine chunk has not been produced yet (nothing else to do meanwhile)
                        const unsigned qc = ld_relaxed_u32(&p.ctl->q_comb);
                        if (qc >= (unsigned)S.n_comb) more = true;
                        else {
                            const int ch = ((((int)qc * S.comb_tok / kRouteBlock) * kFine) / p.nblk) / (kFine / S.K);
                            more = ld_acquire_u32(&p.ctl->y_done[ch]) < y_done_target(S, p, ch);
                        }
                    }
                    g_next = more ? (int)atomicAdd(&p.ctl->q_gemm, 1u) : 0x7fffffff;
                    bool ok;
                    const bool two = tp.mb != tl.mb;         // a regular pair tile has two m-blocks
                    if (tl.type == 0 || tl.type == 3) {
                        ok = flag_wait_ge(&p.xe_ready[tl.mb], 1u, p, 31);
                        if (ok && two) ok = flag_wait_ge(&p.xe_ready[tp.mb], 1u, p, 31);
                    } else {
                        const unsigned need = (unsigned)(p.nt0 * kEpiWarps);
                        ok = flag_wait_ge(&p.h_ready[tl.mb], need, p, 32);
                        if (ok && two) ok = flag_wait_ge(&p.h_ready[tp.mb], need, p, 32);
                    }
                    if (!ok) break;
                    // the tile's input rows may have been written with ordinary stores on other SMs and
                    // are read by TMA next: the cross-proxy fence sits here, after the acquire and before
                    // the hand-over to the producers, off their critical path
                    fence_proxy_async_global();
                    trace_ev(p, S, kEvGemmLoad, (unsigned)g, tp0, trace_now(p), 0u);
                }
                mbar_arrive(&S.ti_full[ps.slot]);
                mbar_arrive_cluster(mapa_u32(smem_u32(&S.ti_full[ps.slot]), 1u));
                ps.next_slot();
                if (tl.type == 2) break;
            }
        }
        __syncwarp();
    } else if (warp == 0) {
        // ---------------- TMA producer (both CTAs): this CTA's 128 rows of A and its half of B;
        // lane 0 issues the loads, the warp stays together tile by tile
        bool dead = false;
        while (!dead) {
            bool ok = true;
            if (lane == 0) ok = mbar_wait_cluster(&S.ti_full[ps.slot], ps.slot_phase, p, 35);
            if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
            const TileInfo ti = S.ti[ps.slot];
            tile_info_landed(ti, &S.scan_w[warp]);
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(mapa_u32(smem_u32(&S.ti_empty[ps.slot]), 0u));
            ps.next_slot();
            if (ti.type == 2) break;
            bool dead_l = false;
            if (lane == 0) {
                const CUtensorMap *tma_a, *tma_b;
                int arow, brow, arow2 = -1;
                // swapped tiles: rows per CTA on the N axis (the MMA's N, a multiple of 16, split in two)
                const int nhalf = (((ti.nrows + 15) >> 4) << 4) >> 1;
                // ... fetched with the smallest box that covers them (the copy engine takes in a fixed
                // number of rows per cycle, so rows nobody reads cost as much as the others)
                const int bi = nhalf <= 8 ? 0 : nhalf <= 16 ? 1 : nhalf <= 32 ? 2 : 3;
                uint32_t tx = 2u * kStageBytes;                  // bytes landing in both CTAs per k-step
                if (ti.type == 0) {      // leader holds the gate rows of the n-tile, peer the up rows
                    tma_a = &tm->xe; tma_b = &tm->wgu;
                    arow = ti.row0;
                    brow = ti.e * 2 * p.I + ti.n * kTN0 + (int)rank * p.I;
                } else if (ti.type == 1) {   // 256 output columns: leader the first 128 weight rows, peer the rest
                    tma_a = &tm->h; tma_b = &tm->wd;
                    arow = ti.row0;
                    brow = ti.e * p.H + ti.n * 256 + (int)rank * 128;
                } else if (ti.type == 3) {   // M axis: 64 gate rows then 64 up rows of this CTA's 64 h-columns
                    tma_a = &tm->wgu64; tma_b = &tm->xe_n[bi];
                    tx = 2u * (kStageA + (1024u << bi));
                    arow = ti.e * 2 * p.I + ti.n * kTN0 + (int)rank * 64;
                    arow2 = arow + p.I;
                    brow = ti.row0 + (int)rank * nhalf;
                } else {                     // M axis: this CTA's 128 of the n-tile's 256 out-columns
                    tma_a = &tm->wd; tma_b = &tm->h_n[bi];
                    tx = 2u * (kStageA + (1024u << bi));
                    arow = ti.e * p.H + ti.n * 256 + (int)rank * 128;
                    brow = ti.row0 + (int)rank * nhalf;
                }
                for (int kb = 0; kb < ti.nkb; ++kb) {
                    if (!mbar_wait(&S.empty[ps.stage], ps.stage_phase ^ 1u, p, 33)) { dead_l = true; break; }
                    uint8_t *sa = stages + ps.stage * kStageBytes;
                    const uint32_t lbar = mapa_u32(smem_u32(&S.full[ps.stage]), 0u);
                    if (rank == 0) mbar_arrive_expect_tx(&S.full[ps.stage], tx);
                    tma_load_2d_pair(sa, tma_a, kb * kBK, arow, lbar);
                    if (arow2 >= 0) tma_load_2d_pair(sa + kStageA / 2, tma_a, kb * kBK, arow2, lbar);
                    tma_load_2d_pair(sa + kStageA, tma_b, kb * kBK, brow, lbar);
                    ps.next_stage();
                }
            }
            dead = __any_sync(0xffffffffu, dead_l);
        }
        if (dead && lane == 0) linger_after_abort();
        __syncwarp();
    } else if (warp == 1 && rank == 0) {
        // ---------------- MMA issuer (leader only): one elected thread drives both SMs' tensor cores.
        // The whole warp walks the loop so that control flow and operands stay warp-uniform; lane 0
        // does the waiting, the elected lane the issuing.
        bool dead = false;
        const uint64_t desc0 = umma_desc_sw128(smem_u32(stages));      // stage 0, A operand, first 16 of K
        while (!dead) {
            bool ok = true;
            if (lane == 0) ok = mbar_wait(&S.ti_full[ps.slot], ps.slot_phase, p, 40);
            if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
            const TileInfo ti = S.ti[ps.slot];
            tile_info_landed(ti, &S.scan_w[warp]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.ti_empty[ps.slot]);
            ps.next_slot();
            if (ti.type == 2) break;
            // regular tiles: 256 rows x 256 columns; swapped tiles: 256 weight rows x (rows rounded up to 16)
            const uint32_t idesc = umma_idesc_bf16(2 * kBM, ti.type >= 3 ? (uint32_t)(((ti.nrows + 15) >> 4) << 4) : 256u);
            // timeline record of this tile: extra = time spent waiting for a free accumulator (ns)
            const unsigned long long tm0 = trace_now(p);
            if (lane == 0) ok = mbar_wait_cluster(&S.tmem_empty[ps.acc], ps.acc_phase ^ 1u, p, 41);
            if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
            tc_fence_after();
            const unsigned long long tm1 = trace_now(p);
            const uint32_t d = tmem_base + (uint32_t)ps.acc * 256u;
            for (int kb = 0; kb < ti.nkb; ++kb) {
                // The operands were written by TMA (either CTA's, into its own shared memory) and are
                // read by the tensor cores only: the barrier's completion is all the ordering needed.
                // A wait that gives up has raised the abort flag: the following ones return at once,
                // and the tile's (meaningless) MMAs only touch memory this pair owns.
                if (lane == 0) ok = mbar_wait(&S.full[ps.stage], ps.stage_phase, p, 42) && ok;
                __syncwarp();
                const uint64_t da = desc0 + (uint64_t)(ps.stage * (kStageBytes >> 4));
                tc_mma_kstep_pair(d, da, da + (uint64_t)(kStageA >> 4), idesc, (uint32_t)(kb != 0), &S.empty[ps.stage], 3);
                ps.next_stage();
            }
            if (elect_one()) tc_commit_pair(&S.tmem_full[ps.acc], 3);        // accumulators complete in both CTAs
            if (lane == 0)
                trace_ev(p, S, kEvMma, (unsigned)(ti.type << 16 | min(ti.nrows, 65535)), tm0, trace_now(p),
                         (unsigned)min(0xFFFFFFFFull, tm1 - tm0));
            ps.next_acc();
            if (!__all_sync(0xffffffffu, ok)) { dead = true; break; }
        }
        if (dead && lane == 0) linger_after_abort();
        __syncwarp();
    } else if (warp >= 4) {
        // ---------------- epilogue (both CTAs): TMEM -> registers -> (SwiGLU) -> bf16 -> staged store
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        bool dead = false;
        uint32_t xg_phase = 0;
        // A release at GPU scope waits until the thread's stores are performed, ~2 us for a tile's
        // worth.  The epilogue warps do not wait: once a tile's stores are issued they tell warp 3,
        // through a shared-memory barrier (which orders their stores before whatever warp 3 does
        // next), which counter the tile arrives on, and go on to the next tile; warp 3 does the
        // release.  Warp q = 0 fills the mailbox, all four warps arrive on it.
        auto post = [&](unsigned *flag, unsigned cnt) -> bool {
            bool ok = true;
            if (lane == 0) {
                if (q == 0) {
                    ok = mbar_wait(&S.rel_empty[ps.rel], ps.rel_phase ^ 1u, p, 56);
                    S.rel_flag[ps.rel] = flag;
                    S.rel_cnt[ps.rel] = cnt;
                }
                mbar_arrive(&S.rel_full[ps.rel]);
            }
            ps.next_rel();
            return !__any_sync(0xffffffffu, !ok);
        };
        while (!dead) {
            if (!mbar_wait_cluster(&S.ti_full[ps.slot], ps.slot_phase, p, 50)) { dead = true; }
            dead = __any_sync(0xffffffffu, dead);
            if (dead) break;
            const TileInfo ti = S.ti[ps.slot];
            tile_info_landed(ti, &S.scan_w[warp]);
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(mapa_u32(smem_u32(&S.ti_empty[ps.slot]), 0u));
            ps.next_slot();
            if (ti.type == 2) { post(nullptr, kRelEnd); break; }
            if (!mbar_wait(&S.tmem_full[ps.acc], ps.acc_phase, p, 51)) { dead = true; }
            dead = __any_sync(0xffffffffu, dead);
            if (dead) break;
            tc_fence_after();
            const unsigned long long te0 = trace_now(p);
            const int rows_valid = ti.nrows - q * 32;          // rows of this warp's quadrant that exist
            const uint32_t epi_stage = smem_u32(stages + kStages * kStageBytes) + (uint32_t)q * 4096u;   // this warp's staging (2 x 2 KB)
            bool acc_released = false;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)ps.acc * 256u;
            if (ti.type == 3) {
                // swapped gemm0: lanes 0..63 hold the gate projection of this CTA's 64 h-columns, lanes
                // 64..127 the up projection; TMEM columns are the m-block's rows.  The up warps hand
                // their values to the gate warps through the staging buffer, 16 rows at a time.
                // each up warp (q = 2, 3) writes into its OWN 2 KB staging region, [32][16] fp32, and gate
                // warp q - 2 reads it; a warp's region is never written by anybody else, so a warp that
                // is still busy with the previous tile cannot be overrun
                const uint32_t xs = smem_u32(stages + kStages * kStageBytes) + (uint32_t)(2 + (q & 1)) * 4096u;
                const int col = ti.n * kTN0 + (int)rank * 64 + (q & 1) * 32 + lane;      // this thread's h-column
                const int nch = (ti.nrows + 15) >> 4;
                for (int c = 0; c < nch && !dead; ++c) {
                    uint32_t v[16];
                    tmem_ld_32x16(taddr + c * 16, v);
                    tmem_ld_wait16(v);
                    if (q >= 2) {
                        if (!mbar_wait(&S.xg_empty, xg_phase ^ 1u, p, 52)) dead = true;
                        dead = __any_sync(0xffffffffu, dead);
                        if (dead) break;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            st_shared_v4(xs + (uint32_t)(lane * 64 + i * 16),
                                         make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&S.xg_full);
                    } else {
                        if (!mbar_wait(&S.xg_full, xg_phase, p, 53)) dead = true;
                        dead = __any_sync(0xffffffffu, dead);
                        if (dead) break;
                        uint32_t u[16];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint4 t4 = ld_shared_v4(xs + (uint32_t)(lane * 64 + i * 16));
                            u[4 * i] = t4.x; u[4 * i + 1] = t4.y; u[4 * i + 2] = t4.z; u[4 * i + 3] = t4.w;
                        }
                        // the four vector loads have landed before the region is handed back to the up warp
                        // (see tile_info_landed: the values are not used until after the arrival)
                        *reinterpret_cast<volatile int *>(&S.scan_w[warp]) = (int)(u[0] ^ u[4] ^ u[8] ^ u[12]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&S.xg_empty);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int tok = c * 16 + j;
                            if (tok < ti.nrows)
                                p.hbuf[(size_t)(ti.row0 + tok) * p.I + col] =
                                    __float2bfloat16_rn(silu_mul(__uint_as_float(v[j]), __uint_as_float(u[j])));
                        }
                    }
                    xg_phase ^= 1u;
                }
                if (dead) break;
                // an up warp may reuse its staging region in the next tile only after the gate warps
                // have read the last chunk
                if (q >= 2) {
                    if (!mbar_wait(&S.xg_empty, xg_phase ^ 1u, p, 54)) dead = true;
                    dead = __any_sync(0xffffffffu, dead);
                    if (dead) break;
                }
            } else if (ti.type == 4) {
                // swapped gemm1: lane = one of this CTA's 128 out-columns, TMEM columns = the m-block's rows
                const int col = ti.n * 256 + (int)rank * 128 + q * 32 + lane;
                const int nch = (ti.nrows + 15) >> 4;
                if (ti.n * 256 + (int)rank * 128 < p.H) {
                    for (int c = 0; c < nch; ++c) {
                        uint32_t v[16];
                        tmem_ld_32x16(taddr + c * 16, v);
                        tmem_ld_wait16(v);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int tok = c * 16 + j;
                            if (tok < ti.nrows)
                                p.y[(size_t)(ti.row0 + tok) * p.H + col] = __float2bfloat16_rn(__uint_as_float(v[j]));
                        }
                    }
                }
            } else if (rows_valid > 0) {
                // TMEM loads run one (half-)chunk ahead of the conversion and the stores; the
                // accumulator is handed back to the MMA issuer as soon as the last load has landed
                if (ti.type == 0) {
                    // batches of 32 h-columns (32 gate + 32 up accumulator columns), double-buffered:
                    // a TMEM load takes several hundred cycles while the tensor core is busy, so
                    // the next batch is in flight while this one is converted and stored
                    __nv_bfloat16 *dst = p.hbuf + (size_t)(ti.row0 + q * 32) * p.I + (size_t)ti.n * kTN0;
                    uint32_t gr[2][32], ur[2][32], o[16];
                    tmem_ld_32x32(taddr, gr[0]);
                    tmem_ld_32x32(taddr + 128, ur[0]);
#pragma unroll
                    for (int c = 0; c < kTN0 / 32; ++c) {
                        tmem_ld_wait32(gr[c & 1]);
                        reg_fence32(ur[c & 1]);
                        if (c + 1 < kTN0 / 32) {
                            tmem_ld_32x32(taddr + (c + 1) * 32, gr[(c + 1) & 1]);
                            tmem_ld_32x32(taddr + 128 + (c + 1) * 32, ur[(c + 1) & 1]);
                        } else {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_remote(mapa_u32(smem_u32(&S.tmem_empty[ps.acc]), 0u));
                            acc_released = true;
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            o[i] = pack_bf16x2(silu_mul(__uint_as_float(gr[c & 1][2 * i]), __uint_as_float(ur[c & 1][2 * i])),
                                               silu_mul(__uint_as_float(gr[c & 1][2 * i + 1]), __uint_as_float(ur[c & 1][2 * i + 1])));
                        staged_store_32(o, epi_stage, dst + c * 32, p.I, rows_valid, lane);
                    }
                } else {
                    // batches of 64 out-columns in two register buffers.  A TMEM load takes most of a
                    // microsecond while the tensor core works on the next tile, and a wait covers every
                    // load in flight, so the tile's epilogue is a chain of load latencies: the batches
                    // are fetched two at a time (two latencies instead of four before the accumulator
                    // can be handed back).
                    __nv_bfloat16 *dst = p.y + (size_t)(ti.row0 + q * 32) * p.H + (size_t)ti.n * 256;
                    const int nb = min(256, p.H - ti.n * 256) / 64;   // the last n-tile may be half wide
                    uint32_t ar[2][64], o[16];
                    tmem_ld_32x64(taddr, ar[0]);
                    if (nb > 1) tmem_ld_32x64(taddr + 64, ar[1]);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if (c < nb) {
                            if ((c & 1) == 0) {              // an odd batch lands together with the one before it
                                tmem_ld_wait64(ar[0]);
                                reg_fence64(ar[1]);
                            }
                            if (c + 2 >= nb && !acc_released) {      // every load of the tile has landed
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive_remote(mapa_u32(smem_u32(&S.tmem_empty[ps.acc]), 0u));
                                acc_released = true;
                            }
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    o[i] = pack_bf16x2(__uint_as_float(ar[c & 1][hh * 32 + 2 * i]),
                                                       __uint_as_float(ar[c & 1][hh * 32 + 2 * i + 1]));
                                staged_store_32(o, epi_stage, dst + c * 64 + hh * 32, p.H, rows_valid, lane);
                            }
                            // this buffer is free again: fetch the batch after next into it
                            if (c + 2 < nb) tmem_ld_32x64(taddr + (c + 2) * 64, ar[c & 1]);
                        }
                    }
                }
            }
            // the accumulator may be overwritten by the next-but-one tile; the rows just stored are read
            // by TMA (gemm1) or by ordinary loads (combine) on other SMs once the counter says so
            const unsigned long long te1 = trace_now(p);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (!acc_released) mbar_arrive_remote(mapa_u32(smem_u32(&S.tmem_empty[ps.acc]), 0u));
                if (q == 0) trace_ev(p, S, kEvGemmEpi, (unsigned)(ti.mb & 0xFFFFFF), te0, trace_now(p),
                                     (unsigned)(ti.type << 16 | (int)min(65535ull, te1 - te0)));
            }
            // a swapped gemm0 tile is stored by the two gate warps of each CTA (4 arrivals per m-block
            // and n-tile over the pair, like a regular tile); a swapped gemm1 tile by all 8 warps
            const bool g0 = ti.type == 0 || ti.type == 3;
            if (!post(g0 ? &p.h_ready[ti.mb] : &p.ctl->y_done[ti.chunk], ti.type == 3 ? 2u : (unsigned)kEpiWarps)) dead = true;
            ps.next_acc();
        }
    } else if (warp == 3) {
        // ---------------- releasing warp (both CTAs): makes the tiles' arrivals on the ready counters
        int rs = 0;
        uint32_t rph = 0;
        while (true) {
            if (!mbar_wait(&S.rel_full[rs], rph, p, 57)) break;
            unsigned *flag = S.rel_flag[rs];
            const unsigned cnt = S.rel_cnt[rs];
            // both words have landed before the slot goes back (see tile_info_landed)
            *reinterpret_cast<volatile int *>(&S.scan_w[warp]) = (int)cnt ^ (int)(size_t)flag;
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.rel_empty[rs]);
            if (cnt == kRelEnd) break;
            if (lane == 0) {
                fence_proxy_async_global();
                red_release_add_u32(flag, cnt);
            }
            if (++rs == kRel) { rs = 0; rph ^= 1u; }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // nobody targets the other CTA's shared memory or barriers after this
    tc_fence_after();
}

// ------------------------------------------------------------------------------------ the kernel

constexpr int kErrNoPairs = -2;     // reported as "unsupported device"

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
weave_moe_kernel(const __grid_constant__ KParams p, const __grid_constant__ TmaMaps tm)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // [stage ring | epilogue staging | SmemTail]
    SmemTail &S = *reinterpret_cast<SmemTail *>(stages + kStages * kStageBytes + kEpiStageBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_sm = (int)gridDim.x;
    const int EE = p.EE;

    // The GEMM phase addresses the neighbouring CTA's shared memory and barriers.  If a launch path
    // ever drops the cluster shape, say so and leave before anything is sent to a peer that is
    // not there (every CTA takes the same branch).
    if (cluster_nctarank() != 2u) {
        if (threadIdx.x == 0) atomicCAS(&p.ctl->status, 0, kErrNoPairs);
        return;
    }

    // The logits of this CTA's first routing block start on their way before anything else: the copy needs
    // no barrier, and the set-up of the barriers and of tensor memory (~1 us) hides part of its latency.
    float *lg_s = reinterpret_cast<float *>(stages + 2048 + kLocalBlocks * kRouteBlock * kMaxTopK * 4);   // [64][route_row_stride(E)]
    {
        const int b_first = p.nblk <= kLocalBlocks ? 0 : (int)blockIdx.x;
        if (b_first < p.nblk) stage_logits_issue(p, b_first, lg_s);
    }

    if (tid == 0) {
        // (rolled loops: code that runs once per launch runs at the speed of instruction fetch)
#pragma unroll 1
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&S.full[i], 1); mbar_init(&S.empty[i], 1);
            mbar_init(&S.dv_full[i], 1); mbar_init(&S.dv_empty[i], 1);
            mbar_init(&S.cb_full[i], 1); mbar_init(&S.cb_empty[i], kCombWarps);
        }
        // accumulator free: 4 epilogue warps in each CTA of the pair arrive on the leader's barrier
#pragma unroll 1
        for (int i = 0; i < 2; ++i) { mbar_init(&S.tmem_full[i], 1); mbar_init(&S.tmem_empty[i], 2 * kEpiWarps); }
        // tile descriptor consumed: leader's producer + MMA + 4 epilogue warps, peer's producer + 4 warps
#pragma unroll 1
        for (int i = 0; i < kTinfo; ++i) { mbar_init(&S.ti_full[i], 1); mbar_init(&S.ti_empty[i], 3 + 2 * kEpiWarps); }
        mbar_init(&S.xg_full, 2); mbar_init(&S.xg_empty, 2);
#pragma unroll 1
        for (int i = 0; i < kRel; ++i) { mbar_init(&S.rel_full[i], kEpiWarps); mbar_init(&S.rel_empty[i], 1); }
        fence_mbar_init();
        tma_prefetch_desc(&tm.xe); tma_prefetch_desc(&tm.wgu); tma_prefetch_desc(&tm.h); tma_prefetch_desc(&tm.wd);
        tma_prefetch_desc(&tm.wgu64);
#pragma unroll 1
        for (int i = 0; i < 4; ++i) { tma_prefetch_desc(&tm.xe_n[i]); tma_prefetch_desc(&tm.h_n[i]); }
    }
    if (warp == 1) { tmem_alloc_pair(&S.tmem_base, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // the peer's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = S.tmem_base;
    if (tid == 0) S.trace_n = 0u;
    const unsigned long long tk0 = trace_now_t0(p);

    // Routing scratch.  The expert masks of the routing blocks sit in the first half of the epilogue staging
    // area: a small batch's masks are still needed while its dispatch copies run through all the stage
    // buffers.  Everything else lives in the (not yet used) stage buffers.
    unsigned long long *lmask = reinterpret_cast<unsigned long long *>(stages + kStages * kStageBytes);   // [kLocalBlocks][256 + 1 (remote tokens)]
    int *r_base = reinterpret_cast<int *>(stages);                                         // [256]
    int *r_cnt = r_base + kMaxEE;                                                          // [kLocalBlocks][2] local / remote pairs
    int *r_idx = reinterpret_cast<int *>(stages + 2048);                                   // [kLocalBlocks][64][16]; the logits follow (lg_s)
    float *r_p = reinterpret_cast<float *>(stages + 96 * 1024);                            // [64][16] exponentials of the selected logits

    // A batch of at most kLocalBlocks routing blocks is routed by every CTA for itself: no grid barrier and
    // no round trip through global memory stand between the logits and the first dispatch copy.  CTA b
    // writes block b's results down for the combine and the host.  Larger batches: block b is routed by
    // CTA b mod N, the counts meet in global memory behind a grid barrier.
    const bool local_route = p.nblk <= kLocalBlocks;
    const bool ep = p.ep_size > 1;

    // The cost tables do not depend on the routing: this thread's candidate (c, K) asks for its two
    // entries first of all, and (without an expert-parallel share, whose workload descriptors are counted
    // while routing) the plan is chosen where it costs nothing: behind the grid barrier's latency, or, in a
    // batch that has no barrier, while the logits are on their way.
    const int cm_ki = tid & 3, cm_c = p.c_min + (tid >> 2) * p.c_step;
    const bool cm_ok = p.mode == kModeAuto && cm_c >= 2 && cm_c <= p.c_max && cm_c <= n_sm - 2 && (EE << cm_ki) <= kMaxSeg;
    float cm_bw = 0.f, cm_tf = 0.f, cm_bw_n = 0.f, cm_tf_n = 0.f;
    if (cm_ok) { cm_bw = p.bw[cm_c]; cm_tf = p.tf[n_sm - cm_c]; }
    if (p.mode == kModeAuto) { cm_bw_n = p.bw[n_sm]; cm_tf_n = p.tf[n_sm]; }
    const int P = p.T * (p.k + p.S);
    // Eq. 1-3 (single-GPU reading: every pair moves through HBM)
    const float B = (float)(2 * p.H);
    float w_comp = __fmul_rn(__fmul_rn(__fmul_rn((float)P, 6.0f), (float)p.H), (float)p.I);
    float w_disp = __fmul_rn((float)(p.T + P), B);
    float w_comb = __fmul_rn((float)(P + p.T), B);
    ModelArgs ma;
    ma.alpha = p.alpha; ma.eff[0] = p.eff[0]; ma.eff[1] = p.eff[1]; ma.eff[2] = p.eff[2]; ma.eff[3] = p.eff[3];
    ma.kinds = p.kinds; ma.c_min = p.c_min; ma.c_step = p.c_step;
    RouteArgs ra;
    ra.T = p.T; ra.E = p.E; ra.k = p.k; ra.ep_size = p.ep_size; ra.ep_rank = p.ep_rank; ra.ep_tshard = p.ep_tshard;
    ra.status = &p.ctl->status; ra.topk_idx = p.topk_idx; ra.gates = p.gates;
    PlanPick pick;
    pick.c = n_sm; pick.ki = 0; pick.kind = kPlanSplit; pick.t = 0.f;
    bool picked = false;

    // ================= phase R: routing
    for (int it = 0;; ++it) {
        const int b = local_route ? it : (int)blockIdx.x + it * n_sm;
        if (b >= p.nblk) break;
        const int slot = local_route ? b : 0;
        unsigned long long *r_mask = lmask + slot * (kMaxEE + 1);
        const bool writer = !local_route || b == (int)blockIdx.x;
        for (int e = tid; e < EE; e += kThreads) r_mask[e] = 0ull;
        if (tid == 0) { r_mask[kMaxEE] = 0ull; r_cnt[2 * slot] = 0; r_cnt[2 * slot + 1] = 0; }
        if (it > 0) stage_logits_issue(p, b, lg_s);      // (the first block's copy was issued at kernel entry)
        if (local_route && !ep && p.mode == kModeAuto) {      // (no barrier to hide it behind: the logits' way in will do)
            pick = model_pick(ma, S, n_sm, w_comp, w_disp, w_comb, cm_ok, cm_bw, cm_tf, cm_bw_n, cm_tf_n);
            picked = true;
        }
        cp_async_wait_all();
        __syncthreads();
        int *idx_b = r_idx + slot * kRouteBlock * kMaxTopK;
        {
            const uint32_t a0 = smem_u32(lg_s), a1 = smem_u32(r_mask), a2 = smem_u32(idx_b), a3 = smem_u32(r_cnt + 2 * slot),
                           a4 = smem_u32(r_p);
            route_block_quads(ra.T, ra.E, ra.k, ra.ep_size, ra.ep_rank, ra.ep_tshard, ra.status, ra.topk_idx, ra.gates, b, a0, a1, a2, a3, a4, writer);
        }
        __syncthreads();
        if (p.nblk > n_sm) {
            // this CTA routes several blocks and its scratch is reused: the in-block rank of each (token,
            // slot) - tokens before it in the block that chose the same expert - goes out to global memory
            for (int pi = tid; pi < kRouteBlock * p.k; pi += kThreads) {
                const int tl = pi / p.k, j = pi - tl * p.k;
                const int t = b * kRouteBlock + tl;
                if (t < p.T) {
                    const int e = idx_b[tl * kMaxTopK + j];     // -1: the expert lives on another rank
                    p.row_of[(size_t)t * p.k + j] = e >= 0 ? __popcll(r_mask[e] & ((1ull << tl) - 1ull)) : -1;
                }
            }
        }
        if (ep && writer && tid == 0) p.uniq_mask[b] = r_mask[kMaxEE];
        if (!local_route) {
            if (ep && tid == 0) {
                const unsigned long long um = r_mask[kMaxEE];
                if (r_cnt[0]) atomicAdd(&p.ctl->x_local, (unsigned)r_cnt[0]);
                if (r_cnt[1]) atomicAdd(&p.ctl->x_in, (unsigned)r_cnt[1]);
                if (um) atomicAdd(&p.ctl->x_in_uniq, (unsigned)__popcll(um));
            }
            const int ntok = min(kRouteBlock, p.T - b * kRouteBlock);
            const int f = (b * kFine) / p.nblk;
            for (int e = tid; e < EE; e += kThreads) {
                const int cnt = e < p.E ? __popcll(r_mask[e]) : ntok;
                p.hist[(size_t)b * kMaxEE + e] = cnt;
                if (cnt) atomicAdd(&p.fcnt[f * kMaxEE + e], (unsigned)cnt);
            }
            __syncthreads();      // the scratch is reused by this CTA's next block
        }
    }
    const unsigned long long tk1 = trace_now_t0(p);
    bool alive = true;
    // (arrivals accumulate over the grid barriers of a launch: the later ones count this one in)
    if (!local_route) {
        // the plan is chosen between arriving at the barrier and waiting on it: the arrival's way to L2 and
        // the wait for the slowest routing CTA hide it
        grid_barrier_arrive(p);
        if (!picked && !ep && p.mode == kModeAuto) {
            pick = model_pick(ma, S, n_sm, w_comp, w_disp, w_comb, cm_ok, cm_bw, cm_tf, cm_bw_n, cm_tf_n);
            picked = true;
        }
        alive = grid_barrier_wait(p, S, (unsigned)n_sm, 1);
    }
    const unsigned long long tk2 = trace_now_t0(p);
    if (tid == 0) {
        trace_ev(p, S, kEvRoute, 0u, tk0, tk1, 0u);
        if (!local_route) trace_ev(p, S, kEvBarrier, 1u, tk1, tk2, 0u);
    }

    // ================= set-up: counts, offsets, plan, segment tables (identical on every CTA)
    int cf[kFine];
    int cnt = 0;
    unsigned ep_xl = 0u, ep_xi = 0u, ep_xu = 0u;
    if (local_route) {
#pragma unroll
        for (int f = 0; f < kFine; ++f) cf[f] = 0;
        for (int bb = 0; bb < p.nblk; ++bb) {
            const int fb = (bb * kFine) / p.nblk;
            const int c = tid >= EE ? 0 : tid < p.E ? __popcll(lmask[bb * (kMaxEE + 1) + tid]) : min(kRouteBlock, p.T - bb * kRouteBlock);
#pragma unroll
            for (int f = 0; f < kFine; ++f) if (f == fb) cf[f] += c;
            cnt += c;
            if (ep) {
                ep_xl += (unsigned)r_cnt[2 * bb]; ep_xi += (unsigned)r_cnt[2 * bb + 1];
                ep_xu += (unsigned)__popcll(lmask[bb * (kMaxEE + 1) + kMaxEE]);
            }
        }
    } else {
#pragma unroll
        for (int f = 0; f < kFine; ++f) {
            cf[f] = (alive && tid < EE) ? (int)__ldcg(p.fcnt + f * kMaxEE + tid) : 0;
            cnt += cf[f];
        }
        // (asked for together with the counts: one L2 round trip instead of two)
        if (alive && ep) { ep_xl = __ldcg(&p.ctl->x_local); ep_xi = __ldcg(&p.ctl->x_in); ep_xu = __ldcg(&p.ctl->x_in_uniq); }
    }
    int total_rows;
    const int off = block_excl_scan(cnt, S, total_rows);
    if (tid < EE) S.offsets[tid] = off;
    if (tid == 0) S.offsets[EE] = total_rows;
    if (blockIdx.x == 0 && tid < EE) {
        p.counts[tid] = cnt;
        p.offsets[tid] = off;
        if (tid == 0) p.offsets[EE] = total_rows;
    }
    if (blockIdx.x == 0 && tid == 0) { p.ctl->ep_x_local = ep_xl; p.ctl->ep_x_in = ep_xi; p.ctl->ep_x_in_uniq = ep_xu; }
    int plan_c, plan_ki, plan_steal = 0, plan_kind = kPlanSplit;
    float plan_t = 0.f;
    if (p.mode == kModeAuto) {
        if (ep) {
            // Eq. 1-3 literally: X_local + X_in pairs are computed here, each unique remote token is
            // pulled once, one result goes back per remote pair
            w_comp = __fmul_rn(__fmul_rn(__fmul_rn((float)(ep_xl + ep_xi), 6.0f), (float)p.H), (float)p.I);
            w_disp = __fmul_rn((float)ep_xu, B);
            w_comb = __fmul_rn((float)ep_xi, B);
            pick = model_pick(ma, S, n_sm, w_comp, w_disp, w_comb, cm_ok, cm_bw, cm_tf, cm_bw_n, cm_tf_n);
        }
        plan_c = pick.c; plan_ki = pick.ki; plan_kind = pick.kind; plan_t = pick.t;
        // the steal quota of Eq. 11-14 belongs to the paper's plan kind; in the other kinds the movement
        // SMs have nothing to wait out (they take GEMM tiles while no combine chunk is ready)
        if (plan_kind == kPlanSplit) {
            const float bw_c = __ldg(p.bw + plan_c), tf_c = __ldg(p.tf + n_sm - plan_c);
            // the pair tiles (256 rows) of the layer at the chosen K (a segment = one expert's rows inside
            // one chunk; its last pair tile may be half empty)
            const int Kc = 1 << plan_ki, sh = 3 - plan_ki;
            int acc = 0;
            for (int j = 0; j < Kc; ++j) {
                int rows = 0;
#pragma unroll
                for (int f = 0; f < kFine; ++f) if ((f >> sh) == j) rows += cf[f];
                acc += (rows + 2 * kBM - 1) / (2 * kBM);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) S.red_i[warp][3] = acc;
            __syncthreads();
            int n_tiles = 0;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) n_tiles += S.red_i[w][3];
            n_tiles *= p.nt0 + p.nt1;
            plan_steal = model_n_steal(n_sm, bw_c, tf_c, w_comp, w_disp, w_comb, n_tiles);      // per CTA pair
        }
    } else if (p.mode == kModeFixed) {
        plan_c = max(2, min((p.fixed_c + 1) & ~1, n_sm - 2));     // whole CTA pairs
        plan_ki = p.fixed_K >= 8 ? 3 : p.fixed_K >= 4 ? 2 : p.fixed_K >= 2 ? 1 : 0;
        while (plan_ki > 0 && (EE << plan_ki) > kMaxSeg) --plan_ki;
        plan_steal = max(0, p.fixed_steal);
    } else {
        plan_c = n_sm;
        plan_ki = 0;
        plan_steal = 0;
        plan_kind = kPlanPhased;
    }
    const int K = 1 << plan_ki;
    if (tid == 0) S.elastic = (p.elastic_steal || plan_kind == kPlanRejoin) ? 1 : 0;
    {
        const int sh = 3 - plan_ki;      // fine chunks per chunk = kFine >> plan_ki
        int run_row = tid < EE ? off : 0;
        int mb_base = 0, pt_base = 0;
        for (int j = 0; j < K; ++j) {
            int rows = 0;
#pragma unroll
            for (int f = 0; f < kFine; ++f) if ((f >> sh) == j) rows += cf[f];
            const int mbs = (rows + kBM - 1) / kBM;
            // m-blocks, pair tiles and unpaired m-blocks of the experts before this one: one packed scan
            unsigned long long tot3;
            const unsigned long long ex3 = block_excl_scan_packed((unsigned long long)mbs | ((unsigned long long)((mbs + 1) >> 1) << 24) |
                                                                      ((unsigned long long)(mbs & 1) << 48), S, tot3);
            const int ex = (int)(ex3 & 0xFFFFFFull), pex = (int)((ex3 >> 24) & 0xFFFFFFull);
            const int tot = (int)(tot3 & 0xFFFFFFull), ptot = (int)((tot3 >> 24) & 0xFFFFFFull), nodd = (int)(tot3 >> 48);
            if (tid < EE) {
                S.seg_mb0[j * EE + tid] = mb_base + ex;
                S.seg_pt0[j * EE + tid] = pt_base + pex;
                S.seg_row0[j * EE + tid] = run_row;
                S.seg_rows[j * EE + tid] = rows;
            }
            if (tid == 0) {
                S.chunk_mb0[j] = mb_base;
                S.chunk_pt0[j] = pt_base;
                S.chunk_tile0[j] = pt_base * (p.nt0 + p.nt1);
                S.chunk_nswap[j] = nodd;
            }
            run_row += rows;
            mb_base += tot;
            pt_base += ptot;
        }
        if (tid == 0) {
            S.seg_mb0[K * EE] = mb_base;
            S.seg_pt0[K * EE] = pt_base;
            S.chunk_mb0[K] = mb_base;
            S.chunk_pt0[K] = pt_base;
            S.chunk_tile0[K] = pt_base * (p.nt0 + p.nt1);
            S.c = plan_c; S.K = K; S.steal = plan_steal;
            S.nmb = mb_base;
            S.n_gemm = pt_base * (p.nt0 + p.nt1);
            // a small batch is cut into smaller combine tiles (powers of two, so that a tile never
            // straddles two chunks) until every SM has one: its final combine is a latency chain
            // per tile, not a bandwidth problem  (ceil(T / ct) < N  <=>  T <= (N - 1) * ct)
            int ct = kCombTile;
            while (ct > 1 && p.T <= (n_sm - 1) * ct) ct >>= 1;
            S.comb_tok = ct;
            S.n_comb = (p.T + ct - 1) / ct;
            if (blockIdx.x == 0) {
                p.ctl->plan_c = plan_c; p.ctl->plan_K = K; p.ctl->plan_steal = plan_steal; p.ctl->plan_t = plan_t;
                p.ctl->plan_nmb = mb_base; p.ctl->plan_ngemm = pt_base * (p.nt0 + p.nt1);
                p.ctl->plan_kind = plan_kind;
            }
        }
    }
    __syncthreads();

    const unsigned long long tk3 = trace_now_t0(p);
    if (tid == 0) trace_ev(p, S, kEvSetup, 0u, tk2, tk3, 0u);
    // ================= permutation fix-up: in-block rank + rows of earlier blocks + expert offset
    if (alive) {
        int fixed = 0;
        const bool from_smem = p.nblk <= n_sm;      // this CTA's block is still in its shared memory
        for (int b = blockIdx.x; b < p.nblk; b += n_sm) {
            const int slot = local_route ? b : 0;
            const unsigned long long *r_mask = lmask + slot * (kMaxEE + 1);
            const int *idx_b = r_idx + slot * kRouteBlock * kMaxTopK;
            if (tid < EE) {
                int base = off;
                if (local_route) {
                    for (int bb = 0; bb < b; ++bb) base += __popcll(lmask[bb * (kMaxEE + 1) + tid]);
                } else {
                    const int f = (b * kFine) / p.nblk;
                    const int bstart = (f * p.nblk + kFine - 1) / kFine;
#pragma unroll
                    for (int ff = 0; ff < kFine; ++ff) if (ff < f) base += cf[ff];
                    for (int bb = bstart; bb < b; ++bb) base += __ldcg(p.hist + (size_t)bb * kMaxEE + tid);
                }
                r_base[tid] = base;
            }
            __syncthreads();
            for (int pi = tid; pi < kRouteBlock * p.k; pi += kThreads) {
                const int tl = pi / p.k, j = pi - tl * p.k;
                const int t = b * kRouteBlock + tl;
                if (t < p.T) {
                    const int e = from_smem ? idx_b[tl * kMaxTopK + j] : __ldcg(p.topk_idx + (size_t)t * p.k + j);
                    const int rk = from_smem ? (e >= 0 ? __popcll(r_mask[e] & ((1ull << tl) - 1ull)) : -1)
                                             : __ldcg(p.row_of + (size_t)t * p.k + j);
                    if (rk >= 0) {
                        const int r = rk + r_base[e];
                        p.row_of[(size_t)t * p.k + j] = r;
                        p.token_of[r] = t;
                    } else if (from_smem) {
                        p.row_of[(size_t)t * p.k + j] = -1;
                    }
                }
            }
            for (int pi = tid; pi < kRouteBlock * p.S; pi += kThreads) {
                const int tl = pi / p.S, s = pi - tl * p.S;
                const int t = b * kRouteBlock + tl;
                if (t < p.T) p.token_of[S.offsets[p.E + s] + t] = t;
            }
            __syncthreads();
            ++fixed;
        }
        if (tid == 0 && fixed) {
            __threadfence();
            red_release_add_u32(&p.ctl->fix_done, (unsigned)fixed);
        }
    }

    if (tid == 0) trace_ev(p, S, kEvFixup, 0u, tk3, trace_now(p), 0u);
    // ================= main phases
    PipeState ps;
    if (alive) {
        // The serial schedule is the phased plan with a grid barrier between the phases (one copy of each
        // phase's code serves both).
        const bool serial = p.mode == kModeSerial;
        const unsigned bar0 = p.nblk <= kLocalBlocks ? 0u : (unsigned)n_sm;      // no routing barrier in a small batch
        const bool mover = (int)blockIdx.x < plan_c;      // role from c* and the block index
        // movement CTAs work through the dispatch queue; every GEMM CTA first dispatches one
        // m-block too, so that the first wave of GEMM tiles does not wait for a handful of movers
        // (the mirror image of the final combine on all SMs); the forced "no temporal
        // scheduling" ablation keeps the two groups apart
        // (plan kinds beyond the paper's: every CTA works through the dispatch queue first; in the
        // phased plan every CTA is a "mover" without a steal limit)
        const bool two_roles = plan_kind == kPlanSplit || plan_kind == kPlanRejoin;
        const int dmax = (mover || !two_roles) ? 0x7fffffff : (S.elastic ? 1 : 0);
        const int n_disp = (!two_roles || S.elastic) ? n_sm : plan_c;       // who dispatches at all
        if (dmax > 0) dispatch_phase(p, S, stages, dmax, n_disp, p.nblk <= kLocalBlocks);
        if (serial) alive = grid_barrier(p, S, bar0 + (unsigned)n_sm, 2);
        const int budget = (mover && plan_kind != kPlanPhased) ? plan_steal : 0x7fffffff;
        if (alive && (budget > 0 || S.elastic)) gemm_phase(p, S, stages, tmem_base, &tm, budget, ps);
        if (serial) alive = alive && grid_barrier(p, S, bar0 + 2u * (unsigned)n_sm, 3);
        if (alive) combine_phase(p, S, stages);
    }

    // ================= leave: free TMEM; the last CTA out re-zeroes the control words
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    cluster_sync_all();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (tid == 0) {
        if (p.trace)     // last record of the CTA's slice: how many events were written
            p.trace[(size_t)blockIdx.x * p.trace_cap + p.trace_cap - 1] =
                make_uint4(min(S.trace_n, (unsigned)p.trace_cap - 1u), 0u, 0u, 0u);
        __threadfence();
        S.bcast[0] = atom_acqrel_add_u32(&p.ctl->exit_count, 1u) == (unsigned)(n_sm - 1) ? 1 : 0;
    }
    __syncthreads();
    if (S.bcast[0]) {
        if (p.nblk > kLocalBlocks)      // (a batch that every CTA routed for itself left the counts untouched)
            for (int i = tid; i < kFine * kMaxEE; i += kThreads) p.fcnt[i] = 0u;
        for (int i = tid; i < p.nmb_max; i += kThreads) { p.xe_ready[i] = 0u; p.h_ready[i] = 0u; }
        unsigned *z = reinterpret_cast<unsigned *>(p.ctl);
        if (tid < kCtlZeroWords) z[tid] = 0u;
    }
}

}  // namespace weave
