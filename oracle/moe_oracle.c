/*
 * CPU oracle of one Mixture-of-Experts layer.  TEST INFRASTRUCTURE ONLY.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
 * this file; the product path never calls it and shares no code with it.
 *
 * What it computes is the plain definition of the layer the paper's Section 2.1
 * describes (five stages: dispatch, GEMM0 = up+gate projection, activation =
 * SiLU followed by element-wise multiplication, GEMM1 = down projection,
 * combine = weighted summation of the per-expert results; Figure 3 names them
 * gemm0 (UP+GATE), silu_mul, gemm1 (DOWN)).  Eq. 1 counts 6*H*I FLOPs per
 * token-expert pair, i.e. three H x I projections: gate, up and down.
 *
 * The paper leaves the router outside its kernel, so the routing rule is this
 * build's stated reading:
 *   - the k experts with the largest fp32 logits, ties to the lowest index,
 *     listed in descending-logit order;
 *   - gates = softmax over those k logits only;
 *   - rows of an expert are its tokens in ascending token order (stable);
 *   - S optional shared experts process every token with weight 1.
 *
 * Arithmetic: fp32 on the bf16 inputs, nothing rounded in between; acc_double=1
 * switches every accumulation to fp64 (a cross-check only; the fp32 path is what the GPU is compared with).
 * Parity pins: tests/test_oracle_*.py (brute force, closed forms, library
 * routines, invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline float bf16_to_f32(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* ------------------------------------------------------------------ routing */

/* Stage "select" + "gates" for one token.  logit: [E].  Returns 0, or -1 if a
 * logit is not finite (the rule is only defined for finite logits). */
static int route_token(const float *logit, int E, int k, int32_t *idx, float *gate)
{
    for (int e = 0; e < E; ++e)
        if (!isfinite(logit[e])) return -1;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
            int taken = 0;
            for (int q = 0; q < j; ++q) taken |= (idx[q] == e);
            if (taken) continue;
            /* strict '>' keeps the lowest index among equal logits (-0 == +0) */
            if (best < 0 || logit[e] > logit[best]) best = e;
        }
        idx[j] = best;
    }
    float m = logit[idx[0]];
    float p[64];
    float sum = 0.0f;
    for (int j = 0; j < k; ++j) {
        p[j] = expf(logit[idx[j]] - m);
        sum += p[j];
    }
    for (int j = 0; j < k; ++j) gate[j] = p[j] / sum;
    return 0;
}

/* logits [T][E] -> idx [T][k], gates [T][k].  k <= 64. */
int oracle_route(const float *logits, int T, int E, int k, int32_t *idx, float *gates)
{
    if (k < 1 || k > E || k > 64) return -2;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int t = 0; t < T; ++t)
        if (route_token(logits + (size_t)t * E, E, k, idx + (size_t)t * k, gates + (size_t)t * k))
            bad |= 1;
    return bad ? -1 : 0;
}

/*
 * counts / offsets / permutation.
 *   counts[e]  = number of (t,j) with idx[t][j] == e            (e <  E)
 *              = T                                              (E <= e < E+S)
 *   offsets    = exclusive prefix sum of counts, offsets[E+S] = T*(k+S)
 *   row_of[t][j], j<k : offsets[e] + #{t' < t : e in idx[t']}
 *   row_of[t][k+s]    : offsets[E+s] + t
 *   token_of[row]     : inverse (the token the row belongs to)
 */
int oracle_permute(const int32_t *idx, int T, int E, int k, int S,
                   int32_t *counts, int32_t *offsets, int32_t *row_of, int32_t *token_of)
{
    int EE = E + S, ks = k + S;
    for (int e = 0; e < EE; ++e) counts[e] = 0;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = idx[(size_t)t * k + j];
            if (e < 0 || e >= E) return -1;
            counts[e] += 1;
        }
    for (int s = 0; s < S; ++s) counts[E + s] = T;
    offsets[0] = 0;
    for (int e = 0; e < EE; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)(EE > 0 ? EE : 1));
    if (!cursor) return -3;
    for (int e = 0; e < EE; ++e) cursor[e] = offsets[e];
    for (int t = 0; t < T; ++t) {            /* ascending token order => stable */
        for (int j = 0; j < k; ++j) {
            int e = idx[(size_t)t * k + j];
            int r = cursor[e]++;
            row_of[(size_t)t * ks + j] = r;
            token_of[r] = t;
        }
        for (int s = 0; s < S; ++s) {
            int r = cursor[E + s]++;
            row_of[(size_t)t * ks + k + s] = r;
            token_of[r] = t;
        }
    }
    free(cursor);
    return 0;
}

/* ------------------------------------------------------------------ expert FFN */

static inline float silu_f(float z) { return z / (1.0f + expf(-z)); }

/* one projection row: sum_h w[h]*v[h], w bf16, v fp32 */
static inline float dot_bf16_f32(const uint16_t *w, const float *v, int n, int acc_double)
{
    if (acc_double) {
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int h = 0; h < n; ++h) acc += (double)bf16_to_f32(w[h]) * (double)v[h];
        return (float)acc;
    }
    float acc = 0.0f;
#pragma omp simd reduction(+ : acc)
    for (int h = 0; h < n; ++h) acc += bf16_to_f32(w[h]) * v[h];
    return acc;
}

/*
 * y = W_down * ( silu(W_gate x) (.) (W_up x) )  for one row.
 *   xrow   [H] fp32 (the bf16 input widened)
 *   gu     [2I][H] bf16: rows [0,I) are the gate projection (SiLU applied),
 *                         rows [I,2I) the up projection
 *   dn     [H][I] bf16
 *   hbuf   [I] scratch, receives the activation output
 *   y      [H]
 * par=1 spreads the output rows over OpenMP threads.
 */
static void expert_ffn_row(const float *xrow, const uint16_t *gu, const uint16_t *dn,
                           int H, int I, int acc_double, int par, float *hbuf, float *y)
{
#pragma omp parallel for schedule(static) if (par)
    for (int i = 0; i < I; ++i) {
        float g = dot_bf16_f32(gu + (size_t)i * H, xrow, H, acc_double);
        float u = dot_bf16_f32(gu + (size_t)(I + i) * H, xrow, H, acc_double);
        hbuf[i] = silu_f(g) * u;
    }
#pragma omp parallel for schedule(static) if (par)
    for (int o = 0; o < H; ++o) y[o] = dot_bf16_f32(dn + (size_t)o * I, hbuf, I, acc_double);
}

/* exported single-row FFN (used by the pins that compare with library matmuls) */
void oracle_expert_ffn(const uint16_t *x_bf16, const uint16_t *gu, const uint16_t *dn,
                       int H, int I, int acc_double, float *h_out, float *y_out)
{
    float *xr = (float *)malloc(sizeof(float) * (size_t)H);
    for (int h = 0; h < H; ++h) xr[h] = bf16_to_f32(x_bf16[h]);
    expert_ffn_row(xr, gu, dn, H, I, acc_double, 1, h_out, y_out);
    free(xr);
}

/* ------------------------------------------------------------------ whole layer, staged */

/*
 * The five stages with every intermediate materialised, in the paper's order:
 *   dispatch : Xe[row]  = x[token_of[row]]
 *   gemm0 + silu_mul : Hbuf[row] = silu(Wg[e] Xe[row]) (.) (Wu[e] Xe[row])
 *   gemm1    : Y[row]   = Wd[e] Hbuf[row]
 *   combine  : out[t]   = sum_{j<k} gate[t][j] * Y[row_of[t][j]]  +  sum_s Y[row_of[t][k+s]]
 * (slot order, then the shared experts).  out is fp32 [T][H].
 * Optional outputs (may be NULL): xe_out [P][H] fp32, h_out [P][I], y_out [P][H].
 */
int oracle_moe_layer(const uint16_t *x, const float *logits, const uint16_t *gate_up,
                     const uint16_t *down, int T, int H, int I, int E, int k, int S,
                     int acc_double, int32_t *idx, float *gates, int32_t *counts,
                     int32_t *offsets, int32_t *row_of, int32_t *token_of, float *out,
                     float *xe_out, float *h_out, float *y_out)
{
    int EE = E + S, ks = k + S;
    size_t P = (size_t)T * ks;
    int rc = oracle_route(logits, T, E, k, idx, gates);
    if (rc) return rc;
    rc = oracle_permute(idx, T, E, k, S, counts, offsets, row_of, token_of);
    if (rc) return rc;

    float *Xe = (float *)malloc(sizeof(float) * (P * H + 1));
    float *Hb = (float *)malloc(sizeof(float) * (P * I + 1));
    float *Y = (float *)malloc(sizeof(float) * (P * H + 1));
    if (!Xe || !Hb || !Y) { free(Xe); free(Hb); free(Y); return -3; }

    /* dispatch */
    for (size_t r = 0; r < P; ++r)
        for (int h = 0; h < H; ++h) Xe[r * H + h] = bf16_to_f32(x[(size_t)token_of[r] * H + h]);

    /* gemm0 + silu_mul, gemm1: rows [offsets[e], offsets[e+1]) belong to expert e */
    for (int e = 0; e < EE; ++e) {
        const uint16_t *gu = gate_up + (size_t)e * 2 * I * H;
        const uint16_t *dn = down + (size_t)e * H * I;
#pragma omp parallel for schedule(dynamic, 1)
        for (int r = offsets[e]; r < offsets[e + 1]; ++r)
            expert_ffn_row(Xe + (size_t)r * H, gu, dn, H, I, acc_double, 0,
                           Hb + (size_t)r * I, Y + (size_t)r * H);
    }

    /* combine */
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < H; ++h) {
            if (acc_double) {
                double acc = 0.0;
                for (int j = 0; j < k; ++j)
                    acc += (double)gates[(size_t)t * k + j] * (double)Y[(size_t)row_of[(size_t)t * ks + j] * H + h];
                for (int s = 0; s < S; ++s) acc += (double)Y[(size_t)row_of[(size_t)t * ks + k + s] * H + h];
                out[(size_t)t * H + h] = (float)acc;
            } else {
                float acc = 0.0f;
                for (int j = 0; j < k; ++j)
                    acc += gates[(size_t)t * k + j] * Y[(size_t)row_of[(size_t)t * ks + j] * H + h];
                for (int s = 0; s < S; ++s) acc += Y[(size_t)row_of[(size_t)t * ks + k + s] * H + h];
                out[(size_t)t * H + h] = acc;
            }
        }
    }
    if (xe_out) memcpy(xe_out, Xe, sizeof(float) * P * H);
    if (h_out) memcpy(h_out, Hb, sizeof(float) * P * I);
    if (y_out) memcpy(y_out, Y, sizeof(float) * P * H);
    free(Xe); free(Hb); free(Y);
    return 0;
}

/* ------------------------------------------------------------------ selected tokens, no permutation */

/*
 * out[i] for the n listed tokens, computed token by token straight from the
 * definition: route the token, run each selected (then each shared) expert on
 * x[t] as a dense mat-vec, add with the gate weights in slot order.  No
 * dispatch, no permutation, no intermediate buffers shared between tokens.
 * Used (a) as brute force against the staged pipeline and (b) to check sampled
 * tokens of layers far too large for a CPU to evaluate in full.
 */
int oracle_moe_tokens(const uint16_t *x, const float *logits, const uint16_t *gate_up,
                      const uint16_t *down, int H, int I, int E, int k, int S, int acc_double,
                      const int32_t *tokens, int n, float *out)
{
    if (k < 1 || k > E || k > 64) return -2;
    float *xr = (float *)malloc(sizeof(float) * (size_t)H);
    float *hb = (float *)malloc(sizeof(float) * (size_t)I);
    float *y = (float *)malloc(sizeof(float) * (size_t)H * (size_t)(k + S));
    if (!xr || !hb || !y) { free(xr); free(hb); free(y); return -3; }
    int rc = 0;
    for (int i = 0; i < n && !rc; ++i) {
        int t = tokens[i];
        int32_t idx[64];
        float gate[64];
        if (route_token(logits + (size_t)t * E, E, k, idx, gate)) { rc = -1; break; }
        for (int h = 0; h < H; ++h) xr[h] = bf16_to_f32(x[(size_t)t * H + h]);
        for (int j = 0; j < k + S; ++j) {
            int e = j < k ? idx[j] : E + (j - k);
            expert_ffn_row(xr, gate_up + (size_t)e * 2 * I * H, down + (size_t)e * H * I, H, I,
                           acc_double, 1, hb, y + (size_t)j * H);
        }
        for (int h = 0; h < H; ++h) {
            if (acc_double) {
                double acc = 0.0;
                for (int j = 0; j < k; ++j) acc += (double)gate[j] * (double)y[(size_t)j * H + h];
                for (int s = 0; s < S; ++s) acc += (double)y[(size_t)(k + s) * H + h];
                out[(size_t)i * H + h] = (float)acc;
            } else {
                float acc = 0.0f;
                for (int j = 0; j < k; ++j) acc += gate[j] * y[(size_t)j * H + h];
                for (int s = 0; s < S; ++s) acc += y[(size_t)(k + s) * H + h];
                out[(size_t)i * H + h] = acc;
            }
        }
    }
    free(xr); free(hb); free(y);
    return rc;
}

/* ------------------------------------------------------------------ one expert-parallel rank's share */

/*
 * Expert parallelism (the paper's Section 2.1 / 3.1 setting) as seen by one rank r of R: the rank
 * hosts experts [r*E/R, (r+1)*E/R) and owns the tokens of shard r, where shard s = tokens
 * [s*Ts, min(T,(s+1)*Ts)), Ts = ceil(T/R).  Routing is global (all E experts, gates normalised
 * over all k selected experts).  The rank computes, for every token, the partial sum over the
 * token's experts that live on this rank (the per-pair results a real system would send back to
 * the token's owner); tokens without a local expert get zeros.  Summing the partial outputs of all
 * R ranks gives the full layer.
 *
 * Workload descriptors of Section 3.1:
 *   x_local      pairs (token, local expert) whose token is in the rank's own shard
 *   x_in         pairs whose token belongs to another rank ("remote tokens routed to local experts")
 *   x_in_uniq    distinct remote tokens with at least one local expert (each is transferred once)
 */
int oracle_ep_descriptors(const int32_t *idx, int T, int E, int k, int ep_rank, int ep_size,
                          int64_t *x_local, int64_t *x_in, int64_t *x_in_uniq)
{
    if (ep_size < 1 || ep_rank < 0 || ep_rank >= ep_size || E % ep_size) return -2;
    const int el = ep_rank * (E / ep_size), eh = el + E / ep_size;
    const int Ts = (T + ep_size - 1) / ep_size;
    int64_t xl = 0, xi = 0, xu = 0;
    for (int t = 0; t < T; ++t) {
        const int own = (t / Ts) == ep_rank;
        int n = 0;
        for (int j = 0; j < k; ++j) {
            int e = idx[(size_t)t * k + j];
            if (e >= el && e < eh) ++n;
        }
        if (own) xl += n; else { xi += n; if (n) ++xu; }
    }
    *x_local = xl; *x_in = xi; *x_in_uniq = xu;
    return 0;
}

/* counts / offsets / permutation restricted to the rank's experts: other experts have count 0,
 * slots that point to them get row -1; rows of a local expert are its tokens in ascending order. */
int oracle_permute_ep(const int32_t *idx, int T, int E, int k, int ep_rank, int ep_size,
                      int32_t *counts, int32_t *offsets, int32_t *row_of, int32_t *token_of)
{
    if (ep_size < 1 || ep_rank < 0 || ep_rank >= ep_size || E % ep_size) return -2;
    const int el = ep_rank * (E / ep_size), eh = el + E / ep_size;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = idx[(size_t)t * k + j];
            if (e < 0 || e >= E) return -1;
            if (e >= el && e < eh) counts[e] += 1;
        }
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    if (!cursor) return -3;
    for (int e = 0; e < E; ++e) cursor[e] = offsets[e];
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = idx[(size_t)t * k + j];
            if (e >= el && e < eh) {
                int r = cursor[e]++;
                row_of[(size_t)t * k + j] = r;
                token_of[r] = t;
            } else {
                row_of[(size_t)t * k + j] = -1;
            }
        }
    free(cursor);
    return 0;
}

/* partial output rows of the listed tokens for rank ep_rank (see above); out [n][H] fp32 */
int oracle_moe_tokens_ep(const uint16_t *x, const float *logits, const uint16_t *gate_up,
                         const uint16_t *down, int H, int I, int E, int k, int ep_rank, int ep_size,
                         int acc_double, const int32_t *tokens, int n, float *out)
{
    if (k < 1 || k > E || k > 64) return -2;
    if (ep_size < 1 || ep_rank < 0 || ep_rank >= ep_size || E % ep_size) return -2;
    const int el = ep_rank * (E / ep_size), eh = el + E / ep_size;
    float *xr = (float *)malloc(sizeof(float) * (size_t)H);
    float *hb = (float *)malloc(sizeof(float) * (size_t)I);
    float *y = (float *)malloc(sizeof(float) * (size_t)H);
    if (!xr || !hb || !y) { free(xr); free(hb); free(y); return -3; }
    int rc = 0;
    for (int i = 0; i < n && !rc; ++i) {
        int t = tokens[i];
        int32_t idx[64];
        float gate[64];
        if (route_token(logits + (size_t)t * E, E, k, idx, gate)) { rc = -1; break; }
        for (int h = 0; h < H; ++h) xr[h] = bf16_to_f32(x[(size_t)t * H + h]);
        for (int h = 0; h < H; ++h) out[(size_t)i * H + h] = 0.0f;
        for (int j = 0; j < k; ++j) {                 /* slot order, local experts only */
            int e = idx[j];
            if (e < el || e >= eh) continue;
            expert_ffn_row(xr, gate_up + (size_t)e * 2 * I * H, down + (size_t)e * H * I, H, I,
                           acc_double, 1, hb, y);
            for (int h = 0; h < H; ++h) out[(size_t)i * H + h] += gate[j] * y[h];
        }
    }
    free(xr); free(hb); free(y);
    return rc;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
