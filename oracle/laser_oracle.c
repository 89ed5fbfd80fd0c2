/*
 * LASER routing oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-purpose CPU statement of what the routing path computes:
 * gate logits, softmax, the top-k mass test, the thresholded candidate pool, the
 * k least-loaded candidates, the load update, and the expert dispatch.  It shares
 * no code with the CUDA library and is only ever called from tests, the smoke
 * check and the CPU-baseline leg of the benchmark.
 *
 * Every function names the passage of the paper it follows (LASER: Load- and
 * Score-based Expert Routing).  Where the paper is silent on floating point the
 * arithmetic is fixed here in fp32 so that an integer decision (which expert, which
 * branch) is taken in the same precision as on the GPU:
 *   - every fp32 operation is a single IEEE round-to-nearest-even operation
 *     (compile with -ffp-contract=off, no fast-math),
 *   - fmaf() is the correctly rounded fused multiply-add.
 *
 * Parity unpinned by anything the paper prints (pinned by argument and by constructed
 * cases only): the combine weights (the paper never mentions them), the granularity of
 * the load update (no printed number depends on it), the RANDOM trimming convention
 * (the paper names no generator or sampling procedure).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- bf16 bits -> exact double ------------------------------------------------ */
static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Gate logits  x[t,e] = sum_j h[t,j] * W[e,j]  (+ b[e])   -- the "lightweight gating
 * network" of the Introduction; "computes router logits" in Evaluation/Integration.
 * Definition written out: fp64 accumulation over the exact bf16 values in index order,
 * one rounding to fp32, then one fp32 add of the bias.
 * h: [T, ldh] bf16 bits, W: [E, ldw] bf16 bits, bias: [E] or NULL, x: [T, E].
 */
void lo_logits(const uint16_t* h, int64_t ldh, const uint16_t* W, int64_t ldw,
               const float* bias, int32_t T, int32_t d, int32_t E, float* x) {
#pragma omp parallel for schedule(static)
    for (int32_t t = 0; t < T; ++t) {
        for (int32_t e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int32_t j = 0; j < d; ++j)
                acc += bf16_to_double(h[(int64_t)t * ldh + j]) * bf16_to_double(W[(int64_t)e * ldw + j]);
            float v = (float)acc;
            if (bias) v = v + bias[e];
            x[(int64_t)t * E + e] = v;
        }
    }
}

/*
 * EXP32(y), y <= 0: the fp32 exponential used by the softmax (Problem formulation:
 * scores s_i >= 0 with sum 1).  Fixed recipe, every step one rounded fp32 operation:
 *   y < -80            -> 0
 *   n  = rint(y * LOG2E)                     (round half to even)
 *   r  = fma(n, -LN2_HI, y); r = fma(n, -LN2_LO, r)
 *   p  = degree-7 Taylor polynomial of e^r in Horner form with fma
 *   result = p * 2^n                          (exact scaling, n in [-116, 0])
 * EXP32(0) is exactly 1.
 */
static float bits_to_float(uint32_t u) { float f; memcpy(&f, &u, sizeof f); return f; }

float lo_exp32(float y) {
    if (y < -80.0f) return 0.0f;
    const float LOG2E  = bits_to_float(0x3FB8AA3Bu); /* 1.44269502 */
    const float LN2_HI = bits_to_float(0x3F317200u); /* 0.693145752 */
    const float LN2_LO = bits_to_float(0x35BFBE8Eu); /* 1.42860677e-06 */
    float n = rintf(y * LOG2E);
    float r = fmaf(n, -LN2_HI, y);
    r = fmaf(n, -LN2_LO, r);
    float p = bits_to_float(0x39500D01u);            /* 1/5040 */
    p = fmaf(p, r, bits_to_float(0x3AB60B61u));      /* 1/720  */
    p = fmaf(p, r, bits_to_float(0x3C088889u));      /* 1/120  */
    p = fmaf(p, r, bits_to_float(0x3D2AAAABu));      /* 1/24   */
    p = fmaf(p, r, bits_to_float(0x3E2AAAABu));      /* 1/6    */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    return ldexpf(p, (int)n);
}

/* Ranking pi: experts by (logit descending, index ascending). */
typedef struct { float x; int32_t e; } ranked_t;
static int rank_cmp(const void* a, const void* b) {
    const ranked_t* p = (const ranked_t*)a;
    const ranked_t* q = (const ranked_t*)b;
    if (p->x > q->x) return -1;
    if (p->x < q->x) return 1;
    return (p->e > q->e) - (p->e < q->e);
}

/*
 * Softmax of one token's logits (Problem formulation / Algorithm 1 precondition:
 * s_i >= 0, sum_i s_i = 1), over all E experts.
 *   e_i = EXP32(x_i - x_max);
 *   Z   = eight interleaved running sums  a_j = sum_{i = j mod 8, i ascending} e_i,
 *         combined as ((a0+a1)+(a2+a3)) + ((a4+a5)+(a6+a7));
 *   s_i = e_i / Z.
 */
void lo_softmax(const float* x, int32_t E, float* s) {
    float xmax = x[0];
    for (int32_t i = 1; i < E; ++i) if (x[i] > xmax) xmax = x[i];
    float a[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int32_t i = 0; i < E; ++i) {
        s[i] = lo_exp32(x[i] - xmax);
        a[i & 7] = a[i & 7] + s[i];
    }
    float Z = ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
    for (int32_t i = 0; i < E; ++i) s[i] = s[i] / Z;
}

/*
 * LASER routing of T tokens in row order (Algorithm 1, "per token, per layer"; prose in
 * The Method: Expansion rule, Final assignment).  Loads are integer assignment counts
 * (Problem formulation: "current load L_e"); they are read by the token being routed and
 * incremented by one for each of its k experts before the next token is routed, on both
 * branches.  The k picks of one token are one sort under the loads seen on entry.
 *
 * For each token, with pi the ranking by (logit descending, index ascending):
 *   M_k = s_pi(0) + ... + s_pi(k-1)                    (left to right, fp32)
 *   M_k >= eps_high      -> A = (pi(0..k-1))            top-k, score order
 *   else  thr = t_fix * s_pi(0)
 *         m'  = #{ j < c : s_pi(j) >= thr }            pool restricted to the c best
 *         c*  = max(k, m')                              = min(c, |pool united with top-k|)
 *         Cand = pi(0..c*-1); sort by (load ascending, score rank ascending); A = first k.
 *   w_j = s[A_j], divided by their left-to-right sum when renormalize != 0.
 *
 * x: [T,E] fp32 logits.  loads: [E] in/out.  ids: [T,k].  weights: [T,k].
 * cstar: [T] or NULL; 0 for a token that took the top-k branch, else c*.
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int32_t lo_route(const float* x, int32_t T, int32_t E, int32_t k, int32_t c,
                 float eps_high, float t_fix, int32_t renormalize,
                 int32_t* loads, int32_t* ids, float* weights, int32_t* cstar) {
    if (T < 0 || E < 1 || k < 1 || k > c || c > E) return -1;
    float* s = (float*)malloc(sizeof(float) * (size_t)E);
    ranked_t* pi = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)E);
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)E); /* rank positions */
    if (!s || !pi || !cand) { free(s); free(pi); free(cand); return -1; }

    for (int32_t t = 0; t < T; ++t) {
        const float* xt = x + (int64_t)t * E;
        lo_softmax(xt, E, s);
        for (int32_t e = 0; e < E; ++e) { pi[e].x = xt[e]; pi[e].e = e; }
        qsort(pi, (size_t)E, sizeof(ranked_t), rank_cmp);

        float Mk = s[pi[0].e];
        for (int32_t j = 1; j < k; ++j) Mk = Mk + s[pi[j].e];

        int32_t* A = ids + (int64_t)t * k;
        if (Mk >= eps_high) {
            for (int32_t j = 0; j < k; ++j) A[j] = pi[j].e;
            if (cstar) cstar[t] = 0;
        } else {
            float thr = t_fix * s[pi[0].e];
            int32_t mprime = 0;
            for (int32_t j = 0; j < c; ++j) if (s[pi[j].e] >= thr) ++mprime;
            int32_t cs = mprime > k ? mprime : k;
            /* insertion sort of rank positions 0..cs-1 by (load, rank) */
            for (int32_t j = 0; j < cs; ++j) {
                int32_t pos = j;
                while (pos > 0 && loads[pi[cand[pos - 1]].e] > loads[pi[j].e]) {
                    cand[pos] = cand[pos - 1];
                    --pos;
                }
                cand[pos] = j;
            }
            for (int32_t j = 0; j < k; ++j) A[j] = pi[cand[j]].e;
            if (cstar) cstar[t] = cs;
        }

        float* w = weights + (int64_t)t * k;
        for (int32_t j = 0; j < k; ++j) w[j] = s[A[j]];
        if (renormalize) {
            float sum = w[0];
            for (int32_t j = 1; j < k; ++j) sum = sum + w[j];
            for (int32_t j = 0; j < k; ++j) w[j] = w[j] / sum;
        }
        for (int32_t j = 0; j < k; ++j) loads[A[j]] += 1;
    }
    free(s); free(pi); free(cand);
    return 0;
}

/*
 * RELAXED variant of the load update -- not the method's rule, kept apart from lo_route and
 * only ever reported beside it.  The text says loads are tracked "per token and per batch";
 * the reading taken for the method is "after every token" (lo_route).  Here the loads that a
 * token SEES are refreshed only every G tokens: tokens are cut into chunks of G consecutive
 * rows, and every token of a chunk ranks its candidates by the loads as they stood when the
 * chunk began (G = 0: one chunk per call, i.e. a per-call snapshot).  The counters themselves
 * still grow by one per assignment.  G = 1 is lo_route.  Everything else (softmax, top-k
 * mass test, pool, trimming, tie-breaks, weights) is as in lo_route.
 */
int32_t lo_route_relaxed(const float* x, int32_t T, int32_t E, int32_t k, int32_t c,
                         float eps_high, float t_fix, int32_t renormalize, int32_t G,
                         int32_t* loads, int32_t* ids, float* weights, int32_t* cstar) {
    if (T < 0 || E < 1 || k < 1 || k > c || c > E || G < 0) return -1;
    float* s = (float*)malloc(sizeof(float) * (size_t)E);
    ranked_t* pi = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)E);
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);
    int32_t* seen = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);   /* loads at chunk start */
    if (!s || !pi || !cand || !seen) { free(s); free(pi); free(cand); free(seen); return -1; }

    for (int32_t t = 0; t < T; ++t) {
        if (G == 0 ? t == 0 : t % G == 0) memcpy(seen, loads, sizeof(int32_t) * (size_t)E);
        const float* xt = x + (int64_t)t * E;
        lo_softmax(xt, E, s);
        for (int32_t e = 0; e < E; ++e) { pi[e].x = xt[e]; pi[e].e = e; }
        qsort(pi, (size_t)E, sizeof(ranked_t), rank_cmp);

        float Mk = s[pi[0].e];
        for (int32_t j = 1; j < k; ++j) Mk = Mk + s[pi[j].e];

        int32_t* A = ids + (int64_t)t * k;
        if (Mk >= eps_high) {
            for (int32_t j = 0; j < k; ++j) A[j] = pi[j].e;
            if (cstar) cstar[t] = 0;
        } else {
            float thr = t_fix * s[pi[0].e];
            int32_t mprime = 0;
            for (int32_t j = 0; j < c; ++j) if (s[pi[j].e] >= thr) ++mprime;
            int32_t cs = mprime > k ? mprime : k;
            for (int32_t j = 0; j < cs; ++j) {   /* insertion sort by (load seen, rank) */
                int32_t pos = j;
                while (pos > 0 && seen[pi[cand[pos - 1]].e] > seen[pi[j].e]) {
                    cand[pos] = cand[pos - 1];
                    --pos;
                }
                cand[pos] = j;
            }
            for (int32_t j = 0; j < k; ++j) A[j] = pi[cand[j]].e;
            if (cstar) cstar[t] = cs;
        }

        float* w = weights + (int64_t)t * k;
        for (int32_t j = 0; j < k; ++j) w[j] = s[A[j]];
        if (renormalize) {
            float sum = w[0];
            for (int32_t j = 1; j < k; ++j) sum = sum + w[j];
            for (int32_t j = 0; j < k; ++j) w[j] = w[j] / sum;
        }
        for (int32_t j = 0; j < k; ++j) loads[A[j]] += 1;
    }
    free(s); free(pi); free(cand); free(seen);
    return 0;
}

/*
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
 * SC 2011): a counter-based generator, out = f(counter[4], key[2]).  Ten rounds of
 *   hi0:lo0 = M0 * c0, hi1:lo1 = M1 * c2;  (c0,c1,c2,c3) <- (hi1^c1^k0, lo1, hi0^c3^k1, lo0)
 * with the key bumped by the Weyl constants between rounds.
 */
void lo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * LASER routing with RANDOM trimming (Algorithm 1, mode RANDOM: "sample c* indices uniformly
 * from T", without replacement; Final assignment in The Method).  The paper fixes neither a
 * generator nor a sampling procedure; this library's convention:
 *   pool    P = (pi(0), ..., pi(m-1)),  m = max(k, #{i : s_i >= t_fix * s_pi(0)})  -- the
 *           thresholded set united with the top-k is a prefix of the score ranking
 *   c*      = min(c, m);  if c* == m nothing is drawn and Cand = P
 *   draws   u_0, u_1, ...: 32-bit words of Philox4x32-10 with key = (seed low, seed high) and
 *           counter = (token index, layer, block, 0); draw i is word i % 4 of block i / 4
 *   sample  partial Fisher-Yates: for i = 0 .. c*-1:  j = i + u_i mod (m - i);  swap P[i], P[j]
 *   Cand    = {P[0..c*-1]}, listed in score-rank order; then, as in lo_route, the k
 *           candidates with the smallest (load, score rank), loads updated after every token.
 * Unlike TOP trimming the k best need not survive the sampling.  cstar[t] = 0 on the top-k
 * branch, else c*.  cand_out, if not NULL, receives the c* sampled experts of every token in
 * score-rank order ([T, c], unused entries -1).
 */
int32_t lo_route_random(const float* x, int32_t T, int32_t E, int32_t k, int32_t c,
                        float eps_high, float t_fix, int32_t renormalize, uint64_t seed,
                        int32_t layer, int32_t* loads, int32_t* ids, float* weights,
                        int32_t* cstar, int32_t* cand_out) {
    if (T < 0 || E < 1 || k < 1 || k > c || c > E) return -1;
    float* s = (float*)malloc(sizeof(float) * (size_t)E);
    ranked_t* pi = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)E);
    int32_t* P = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);     /* rank positions */
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);
    if (!s || !pi || !P || !cand) { free(s); free(pi); free(P); free(cand); return -1; }
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};

    for (int32_t t = 0; t < T; ++t) {
        const float* xt = x + (int64_t)t * E;
        lo_softmax(xt, E, s);
        for (int32_t e = 0; e < E; ++e) { pi[e].x = xt[e]; pi[e].e = e; }
        qsort(pi, (size_t)E, sizeof(ranked_t), rank_cmp);
        float Mk = s[pi[0].e];
        for (int32_t j = 1; j < k; ++j) Mk = Mk + s[pi[j].e];
        int32_t* A = ids + (int64_t)t * k;
        if (cand_out) for (int32_t j = 0; j < c; ++j) cand_out[(int64_t)t * c + j] = -1;
        if (Mk >= eps_high) {
            for (int32_t j = 0; j < k; ++j) A[j] = pi[j].e;
            if (cstar) cstar[t] = 0;
        } else {
            float thr = t_fix * s[pi[0].e];
            int32_t m = 0;
            for (int32_t e = 0; e < E; ++e) if (s[e] >= thr) ++m;
            if (m < k) m = k;
            int32_t cs = c < m ? c : m;
            for (int32_t i = 0; i < m; ++i) P[i] = i;
            if (cs < m) {
                uint32_t blk[4];
                for (int32_t i = 0; i < cs; ++i) {
                    if ((i & 3) == 0) {
                        const uint32_t ctr[4] = {(uint32_t)t, (uint32_t)layer, (uint32_t)(i >> 2), 0u};
                        lo_philox4x32_10(ctr, key, blk);
                    }
                    int32_t j = i + (int32_t)(blk[i & 3] % (uint32_t)(m - i));
                    int32_t tmp = P[i]; P[i] = P[j]; P[j] = tmp;
                }
            }
            /* the sample in score-rank order */
            for (int32_t i = 1; i < cs; ++i) {
                int32_t v = P[i], pos = i;
                while (pos > 0 && P[pos - 1] > v) { P[pos] = P[pos - 1]; --pos; }
                P[pos] = v;
            }
            if (cand_out) for (int32_t j = 0; j < cs; ++j) cand_out[(int64_t)t * c + j] = pi[P[j]].e;
            /* by (load, position in the sample), first k */
            for (int32_t j = 0; j < cs; ++j) {
                int32_t pos = j;
                while (pos > 0 && loads[pi[P[cand[pos - 1]]].e] > loads[pi[P[j]].e]) {
                    cand[pos] = cand[pos - 1];
                    --pos;
                }
                cand[pos] = j;
            }
            for (int32_t j = 0; j < k; ++j) A[j] = pi[P[cand[j]]].e;
            if (cstar) cstar[t] = cs;
        }
        float* w = weights + (int64_t)t * k;
        for (int32_t j = 0; j < k; ++j) w[j] = s[A[j]];
        if (renormalize) {
            float sum = w[0];
            for (int32_t j = 1; j < k; ++j) sum = sum + w[j];
            for (int32_t j = 0; j < k; ++j) w[j] = w[j] / sum;
        }
        for (int32_t j = 0; j < k; ++j) loads[A[j]] += 1;
    }
    free(s); free(pi); free(P); free(cand);
    return 0;
}

/*
 * Vanilla top-k routing (Introduction: "selects the k experts with the highest scores";
 * the Baselines paragraph).  Written independently of lo_route: k rounds of argmax over
 * the logits with already-taken experts masked out; ties go to the lower index.
 */
void lo_topk(const float* x, int32_t T, int32_t E, int32_t k, int32_t* ids) {
    unsigned char* taken = (unsigned char*)malloc((size_t)E);
    for (int32_t t = 0; t < T; ++t) {
        memset(taken, 0, (size_t)E);
        for (int32_t j = 0; j < k; ++j) {
            int32_t best = -1;
            for (int32_t e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || x[(int64_t)t * E + e] > x[(int64_t)t * E + best]) best = e;
            }
            taken[best] = 1;
            ids[(int64_t)t * k + j] = best;
        }
    }
    free(taken);
}

/*
 * Dispatch: per-call counts N_e (the per-batch, per-layer counts of the imbalance
 * definition in Motivation), exclusive offsets, and the pair ids t*k+j stably grouped by
 * expert.  Counting sort.  offsets: [E+1], perm: [T*k].
 */
void lo_dispatch(const int32_t* ids, int32_t T, int32_t k, int32_t E,
                 int32_t* offsets, int32_t* perm) {
    int64_t n = (int64_t)T * k;
    for (int32_t e = 0; e <= E; ++e) offsets[e] = 0;
    for (int64_t p = 0; p < n; ++p) offsets[ids[p] + 1] += 1;
    for (int32_t e = 0; e < E; ++e) offsets[e + 1] += offsets[e];
    int32_t* cursor = (int32_t*)malloc(sizeof(int32_t) * (size_t)E);
    for (int32_t e = 0; e < E; ++e) cursor[e] = offsets[e];
    for (int64_t p = 0; p < n; ++p) perm[cursor[ids[p]]++] = (int32_t)p;
    free(cursor);
}

/*
 * Device-bin load accounting: N_g = sum_e A[g,e] N_e with a pure placement A in {0,1}
 * given as expert_to_bin (Motivation, placement matrix and induced GPU load).
 * bin_loads: [n_bins] in/out, counts: [E].
 */
void lo_bins(const int32_t* counts, const int32_t* expert_to_bin, int32_t E, int32_t* bin_loads) {
    for (int32_t e = 0; e < E; ++e) bin_loads[expert_to_bin[e]] += counts[e];
}
