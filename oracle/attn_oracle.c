/*
 * CPU oracle for BF16 flash attention (forward, delta, backward).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, by-eye-checkable
 * restatement of the paper's definitions and algorithms.  It shares no code
 * with the CUDA path and is only ever called from tests, from the smoke
 * check and from the CPU-baseline leg of the benchmark.
 *
 * Two references live here:
 *
 *   (i)  orc_ref_*  : fp64, the plain definition of attention
 *                     O = softmax(alpha Q K^T) V  (Sec. 2.2) and its closed-form
 *                     gradients (Algorithm 2 with the tiling removed; the
 *                     alpha on dS is the equation dS = alpha P o (dP - delta),
 *                     Sec. 3.3.1 / App. E.2).
 *
 *   (ii) orc_emu_*  : the tiled algorithms step by step, Algorithm 1
 *                     (standard), Algorithm 3 (stabilised: Algorithm 1 plus three added steps)
 *                     and Algorithm 2 (backward), in emulated FP32 with the
 *                     BF16 rounding points the paper's analysis fixes:
 *                     P-bar is a BF16 value (Sec. 4 relies on entries of P-bar
 *                     that equal 1 exactly), the P-bar V dot product accumulates in FP32
 *                     and its final result is rounded to BF16 (Sec. 3.3.2,
 *                     the (.)_lp definition), then O = O-bar / rowsum(P-bar)
 *                     is rounded to BF16 again.
 *
 * Pins (tests/test_oracle_*.py): BF16 rounding and the FP32-accumulate-then-
 * round model are pinned to the worked example of Sec. 3.3.2; the fp64
 * forward to softmax identities and closed forms; the fp64 backward to
 * central finite differences, to delta = rowsum(dO o O) = rowsum(dP o P)
 * (Sec. 3.2) and to Eq. 1; orc_ref_delta_dp (the second form as a function
 * of its own) to rowsum(dO o O) of the fp64 forward, which it must equal; the tiled emulation to the fp64 reference, to
 * tile-size independence in mode 0, to the shift invariance of Sec. 4 and
 * to hand-made rows for the tie rule.
 *   parity unpinned: the magnitude of the rounding-bias statistic (only its
 *   sign and the biased/unbiased contrast are fixed by the paper), and the
 *   rounding points of the emulated backward (the paper gives Algorithm 2
 *   only in exact arithmetic).
 *
 * Layout: every tensor is row-major [B][H][N][d]; BF16 tensors are passed
 * as uint16_t bit patterns; L and delta are [B][H][N].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* BF16: 1 sign, 8 exponent, 7 fraction bits (Sec. 2.1, App. B).       */
/* ------------------------------------------------------------------ */

float orc_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* Round-to-nearest, ties-to-even (App. B step 4): keep the top 16 bits of
 * the FP32 pattern; the 16 discarded bits decide.  More than half an LSB:
 * up.  Exactly half: to the even neighbour.  A carry out of the fraction
 * walks into the exponent, which is the re-normalisation of App. B step 3. */
uint16_t orc_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u)          /* NaN stays NaN */
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t keep = u >> 16;
    uint32_t rest = u & 0xffffu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u)))
        keep += 1u;
    return (uint16_t)keep;
}

static inline float round_bf16(float f)
{
    return orc_bf16_to_f32(orc_f32_to_bf16(f));
}

/* Round an FP32 value to an 8-bit floating-point format with `ebits` exponent bits and `mbits` fraction bits
 * (1 + ebits + mbits = 8), round to nearest even, gradual underflow, saturating at the largest finite value:
 *   ebits = 4, mbits = 3  "E4M3": bias 7, largest finite value 448 (the all-ones exponent holds numbers, only the
 *                         all-ones fraction with it is NaN), smallest subnormal 2^-9
 *   ebits = 5, mbits = 2  "E5M2": bias 15, IEEE-like (all-ones exponent is inf / NaN), largest finite 57344, smallest
 *                         subnormal 2^-16
 * Used only by the FP8 study of the forward pass (the paper names FP8 as future work). */
float orc_round_fp8(float x, int ebits, int mbits)
{
    if (x != x) return x;
    const int bias = (1 << (ebits - 1)) - 1;
    const int emin = 1 - bias;                                  /* exponent of the smallest normal */
    const double maxv = (ebits == 4) ? 448.0 : 57344.0;
    const double ax = fabs((double)x);
    if (ax == 0.0) return x;
    int e;
    frexp(ax, &e);                                              /* ax = f * 2^e, f in [0.5, 1) */
    int ex = e - 1;                                             /* ax in [2^ex, 2^(ex+1)) */
    if (ex < emin) ex = emin;                                   /* subnormal range: fixed spacing */
    const double ulp = ldexp(1.0, ex - mbits);
    double r = nearbyint(ax / ulp) * ulp;                       /* round half to even (default rounding mode) */
    if (r > maxv) r = maxv;
    return (float)(x < 0 ? -r : r);
}

/* FP32 exp / log: the correctly rounded FP32 value of the real function
 * (double evaluation, one rounding to float). */
static inline float exp_f32(float x) { return (float)exp((double)x); }
static inline float log_f32(float x) { return (float)log((double)x); }

/* ------------------------------------------------------------------ */
/* (i) fp64 reference: the definition, Sec. 2.2.                        */
/* ------------------------------------------------------------------ */

/* O = softmax(alpha Q K^T) V and L = logsumexp(alpha Q K^T) per row.
 * Inputs are doubles (BF16 tensors are widened exactly by the caller; the
 * finite-difference pins pass perturbed reals).  causal != 0 masks key
 * t > query T.  P (optional, may be NULL) receives the full N x N
 * probability matrix per head; only sensible for small N. */
void orc_ref_fwd(const double *q, const double *k, const double *v,
                 int B, int H, int N, int d, int causal, double alpha,
                 double *O, double *L, double *P)
{
    const long heads = (long)B * H;
    /* every query row is an independent problem */
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (long bh = 0; bh < heads; ++bh) {
        for (int T = 0; T < N; ++T) {
            const double *qh = q + bh * (long)N * d;
            const double *kh = k + bh * (long)N * d;
            const double *vh = v + bh * (long)N * d;
            double *s = (double *)malloc(sizeof(double) * (size_t)N);
            const int nk = causal ? T + 1 : N;
            double m = -INFINITY;
            for (int t = 0; t < nk; ++t) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c)
                    acc += qh[(long)T * d + c] * kh[(long)t * d + c];
                s[t] = alpha * acc;
                if (s[t] > m) m = s[t];
            }
            double l = 0.0;
            for (int t = 0; t < nk; ++t) {
                s[t] = exp(s[t] - m);
                l += s[t];
            }
            double *o = O + (bh * N + T) * (long)d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int t = 0; t < nk; ++t) {
                const double p = s[t] / l;
                if (P) P[(bh * N + T) * (long)N + t] = p;
                for (int c = 0; c < d; ++c)
                    o[c] += p * vh[(long)t * d + c];
            }
            if (P)
                for (int t = nk; t < N; ++t) P[(bh * N + T) * (long)N + t] = 0.0;
            L[bh * N + T] = m + log(l);
            free(s);
        }
    }
}

/* Closed-form gradients (Algorithm 2 without tiles):
 *   P = exp(S - L), dV = P^T dO, dP = dO V^T, delta = rowsum(dO o O),
 *   dS = P o (dP - delta), dQ = alpha dS K, dK = alpha dS^T Q.
 * O and L come from orc_ref_fwd.  delta_override (may be NULL) replaces the
 * delta computed here; delta_out (may be NULL) receives the delta used. */
void orc_ref_bwd(const double *q, const double *k, const double *v,
                 const double *dO, const double *O, const double *L,
                 int B, int H, int N, int d, int causal, double alpha,
                 const double *delta_override,
                 double *dQ, double *dK, double *dV, double *delta_out)
{
    const long heads = (long)B * H;
    double *delta = (double *)malloc(sizeof(double) * (size_t)(heads * N));
    /* delta, one value per query row */
#pragma omp parallel for
    for (long r = 0; r < heads * N; ++r) {
        double del = 0.0;
        for (int c = 0; c < d; ++c) del += dO[r * d + c] * O[r * d + c];
        if (delta_override) del = delta_override[r];
        delta[r] = del;
        if (delta_out) delta_out[r] = del;
    }
    /* dQ: one independent sum per query row T;  dK, dV: one per key row t */
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (long bh = 0; bh < heads; ++bh) {
        for (int T = 0; T < N; ++T) {
            const long off = bh * (long)N * d;
            const double *qh = q + off, *kh = k + off, *vh = v + off, *gh = dO + off;
            double *dq = dQ + off + (long)T * d;
            for (int c = 0; c < d; ++c) dq[c] = 0.0;
            const int nk = causal ? T + 1 : N;
            for (int t = 0; t < nk; ++t) {
                double acc = 0.0, dp = 0.0;
                for (int c = 0; c < d; ++c) {
                    acc += qh[(long)T * d + c] * kh[(long)t * d + c];
                    dp += gh[(long)T * d + c] * vh[(long)t * d + c];
                }
                const double p = exp(alpha * acc - L[bh * N + T]);
                const double ds = p * (dp - delta[bh * N + T]);
                for (int c = 0; c < d; ++c) dq[c] += alpha * ds * kh[(long)t * d + c];
            }
        }
    }
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (long bh = 0; bh < heads; ++bh) {
        for (int t = 0; t < N; ++t) {
            const long off = bh * (long)N * d;
            const double *qh = q + off, *kh = k + off, *vh = v + off, *gh = dO + off;
            double *dk = dK + off + (long)t * d, *dv = dV + off + (long)t * d;
            for (int c = 0; c < d; ++c) dk[c] = dv[c] = 0.0;
            for (int T = causal ? t : 0; T < N; ++T) {
                double acc = 0.0, dp = 0.0;
                for (int c = 0; c < d; ++c) {
                    acc += qh[(long)T * d + c] * kh[(long)t * d + c];
                    dp += gh[(long)T * d + c] * vh[(long)t * d + c];
                }
                const double p = exp(alpha * acc - L[bh * N + T]);
                const double ds = p * (dp - delta[bh * N + T]);
                for (int c = 0; c < d; ++c) {
                    dv[c] += p * gh[(long)T * d + c];
                    dk[c] += alpha * ds * qh[(long)T * d + c];
                }
            }
        }
    }
    free(delta);
}

/* delta by the alternative formulation of Sec. 3.2: delta = rowsum(dP o P) with dP = dO V^T and
 * P = exp(alpha Q K^T - L), which never touches O (in exact arithmetic it equals rowsum(dO o O)).
 * L is the log-sum-exp the backward pass is given. */
void orc_ref_delta_dp(const double *q, const double *k, const double *v, const double *dO, const double *L,
                      int B, int H, int N, int d, int causal, double alpha, double *delta)
{
    const long heads = (long)B * H;
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (long bh = 0; bh < heads; ++bh) {
        for (int T = 0; T < N; ++T) {
            const long off = bh * (long)N * d;
            const double *qh = q + off, *kh = k + off, *vh = v + off, *gh = dO + off;
            const int nk = causal ? T + 1 : N;
            double del = 0.0;
            for (int t = 0; t < nk; ++t) {
                double acc = 0.0, dp = 0.0;
                for (int c = 0; c < d; ++c) {
                    acc += qh[(long)T * d + c] * kh[(long)t * d + c];
                    dp += gh[(long)T * d + c] * vh[(long)t * d + c];
                }
                del += exp(alpha * acc - L[bh * N + T]) * dp;
            }
            delta[bh * N + T] = del;
        }
    }
}

/* ------------------------------------------------------------------ */
/* (ii) emulated tiled algorithms.                                      */
/* ------------------------------------------------------------------ */

/* The tie rule of Sec. 4 / Algorithm 3 for one row of one key block: given the n scaled scores of the
 * block (masked entries are -inf), r_m = rowmax, r_s = #{r_m - s <= eps} (the maximum itself counts; for a
 * masked entry r_m - (-inf) = inf is not counted), and the returned m' is
 *   beta r_m if r_m > 0 and r_s > 1;   0 if r_m < 0 and r_s > 1;   r_m otherwise.
 * This is the only copy of the rule: orc_emu_fwd calls it for every row and block, and the hand-made rows of
 * the tests drive it both directly and through orc_emu_fwd. */
float orc_tie_rule(const float *s, int n, float beta, float eps, int *r_s_out)
{
    float r_m = -INFINITY;
    for (int t = 0; t < n; ++t) if (s[t] > r_m) r_m = s[t];
    int r_s = 0;
    for (int t = 0; t < n; ++t) if (r_m - s[t] <= eps) r_s += 1;
    float mp = r_m;
    if (r_m > 0.0f && r_s > 1) mp = beta * r_m;
    if (r_m < 0.0f && r_s > 1) mp = 0.0f;
    if (r_s_out) *r_s_out = r_s;
    return mp;
}

/*
 * Forward, Algorithm 1 (mode 0) / Algorithm 3 (mode 1).
 *
 * Per query block i and key block j (blocks entirely above the causal
 * diagonal are skipped, which is the same as all their scores being -inf):
 *   S      = fl32(alpha * fl32dot(Q_i, K_j))              [FP32, not rounded to BF16]
 *   mode 1 : r_m = rowmax(S), r_s = #{r_m - S <= eps},
 *            m' = beta r_m if (r_m > 0 and r_s > 1), 0 if (r_m < 0 and r_s > 1), else r_m
 *            (guard_cap > 0: the guarded variant described at the rule below; not the paper's)
 *   mode 0 : m' = rowmax(S)
 *   m      = max(m_prev, m'),  a = exp(m_prev - m)  (a = 0 on the first block)
 *   P-bar  = bf16(exp(S - m))
 *   l      = a l + rowsum(P-bar)                            [FP32, of the BF16 values]
 *   O-bar  = a O-bar + P-bar V_j                            [FP32 accumulate]
 * After the last block:
 *   O-bar <- bf16(O-bar)  (if round_obar),  O = bf16(O-bar / l),  L = m + log l.
 *
 * Optional per-row diagnostics (each may be NULL):
 *   obar_f32   [B][H][N][d]  O-bar before its rounding
 *   l_out, m_out [B][H][N]   final l and m
 *   pmax_out   [B][H][N]     largest P-bar value produced for the row
 *   nones_out  [B][H][N]     number of P-bar entries equal to exactly 1
 */
void orc_emu_fwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                 int B, int H, int N, int d, int causal, float alpha,
                 int mode, float beta, float eps, int Br, int Bc, int round_obar, float guard_cap, int pbar_fmt,
                 uint16_t *O, float *L,
                 float *obar_f32, float *l_out, float *m_out,
                 float *pmax_out, int32_t *nones_out)
{
    const long heads = (long)B * H;
    const int Tr = (N + Br - 1) / Br, Tc = (N + Bc - 1) / Bc;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (long bh = 0; bh < heads; ++bh) {
        for (int i = 0; i < Tr; ++i) {
            const long off = bh * (long)N * d;
            const uint16_t *qh = q + off, *kh = k + off, *vh = v + off;
            float *s = (float *)malloc(sizeof(float) * (size_t)Bc);
            float *pb = (float *)malloc(sizeof(float) * (size_t)Bc);
            float *ob = (float *)malloc(sizeof(float) * (size_t)d);
            const int r_end = (i + 1) * Br < N ? (i + 1) * Br : N;
            /* rows of a block are independent; handle them one at a time */
            for (int T = i * Br; T < r_end; ++T) {
                float m = -INFINITY, l = 0.0f, pmax = 0.0f;
                float r_run = -INFINITY;                       /* guarded variant: largest r_m of the earlier blocks */
                int32_t nones = 0;
                for (int c = 0; c < d; ++c) ob[c] = 0.0f;
                for (int j = 0; j < Tc; ++j) {
                    const int t0 = j * Bc;
                    const int t1 = (j + 1) * Bc < N ? (j + 1) * Bc : N;
                    if (causal && t0 > r_end - 1) continue;   /* block fully masked for the whole Q block */
                    float r_m = -INFINITY;
                    for (int t = t0; t < t1; ++t) {
                        float acc = 0.0f;
                        for (int c = 0; c < d; ++c)
                            acc += orc_bf16_to_f32(qh[(long)T * d + c]) *
                                   orc_bf16_to_f32(kh[(long)t * d + c]);
                        float sc = alpha * acc;
                        if (causal && t > T) sc = -INFINITY;
                        s[t - t0] = sc;
                        if (sc > r_m) r_m = sc;
                    }
                    float mp = r_m;
                    if (mode == 1) {
                        int r_s = 0;
                        const float mp_rule = orc_tie_rule(s, t1 - t0, beta, eps, &r_s);   /* Algorithm 3's three added steps */
                        if (guard_cap > 0.0f) {
                            /* Guarded variant (an extension, not in the paper): the maximum also counts as repeated
                             * when it equals, within eps, the largest row maximum of the earlier blocks (a tie split
                             * across blocks), and the upward shift of m is limited to guard_cap, so that the
                             * block's own maximum keeps an exponent >= -guard_cap and l cannot underflow to 0. */
                            int repeated = r_s > 1;
                            if (r_run != -INFINITY && r_m != -INFINITY && fabsf(r_m - r_run) <= eps) repeated = 1;
                            if (r_m > r_run) r_run = r_m;
                            /* the paper's m' unless it lies more than guard_cap above r_m */
                            if (repeated && r_m > 0.0f) mp = ((beta - 1.0f) * r_m <= guard_cap) ? beta * r_m : r_m + guard_cap;
                            if (repeated && r_m < 0.0f) mp = (-r_m <= guard_cap) ? 0.0f : r_m + guard_cap;
                        } else {
                            mp = mp_rule;
                        }
                    }
                    const float m_new = (m > mp) ? m : mp;
                    if (m_new == -INFINITY) continue;          /* row sees no key in this block and none before */
                    const float a = (m == -INFINITY) ? 0.0f : exp_f32(m - m_new);
                    float rowsum = 0.0f;
                    for (int t = t0; t < t1; ++t) {
                        const float sc = s[t - t0];
                        const float p32 = (sc == -INFINITY) ? 0.0f : exp_f32(sc - m_new);
                        /* pbar_fmt: 0 = BF16 (the paper's setting); 1 = E4M3, 2 = E5M2 (FP8 study only) */
                        const float p = pbar_fmt == 1 ? orc_round_fp8(p32, 4, 3)
                                      : pbar_fmt == 2 ? orc_round_fp8(p32, 5, 2) : round_bf16(p32);
                        pb[t - t0] = p;
                        rowsum += p;
                        if (p > pmax) pmax = p;
                        if (p == 1.0f) nones += 1;
                    }
                    l = a * l + rowsum;
                    for (int c = 0; c < d; ++c) ob[c] = a * ob[c];
                    for (int t = t0; t < t1; ++t) {
                        const float p = pb[t - t0];
                        for (int c = 0; c < d; ++c)
                            ob[c] += p * orc_bf16_to_f32(vh[(long)t * d + c]);
                    }
                    m = m_new;
                }
                const long row = bh * N + T;
                for (int c = 0; c < d; ++c) {
                    if (obar_f32) obar_f32[row * d + c] = ob[c];
                    const float obr = round_obar ? round_bf16(ob[c]) : ob[c];
                    O[row * d + c] = orc_f32_to_bf16(obr / l);
                }
                L[row] = m + log_f32(l);
                if (l_out) l_out[row] = l;
                if (m_out) m_out[row] = m;
                if (pmax_out) pmax_out[row] = pmax;
                if (nones_out) nones_out[row] = nones;
            }
            free(s); free(pb); free(ob);
        }
    }
}

/* delta = rowsum(dO o O), Algorithm 2 preprocessing step, FP32 accumulation
 * of the exact products of the BF16 O and dO. */
void orc_emu_delta(const uint16_t *o, const uint16_t *dO,
                   int B, int H, int N, int d, float *delta)
{
    const long rows = (long)B * H * N;
#pragma omp parallel for
    for (long r = 0; r < rows; ++r) {
        float acc = 0.0f;
        for (int c = 0; c < d; ++c)
            acc += orc_bf16_to_f32(dO[r * d + c]) * orc_bf16_to_f32(o[r * d + c]);
        delta[r] = acc;
    }
}

/*
 * Backward, Algorithm 2, with the usual mixed-precision convention:
 *   S as in the forward; p32 = exp(S - L); P = bf16(p32) feeds dV;
 *   dP = dO V^T in FP32; dS = bf16(p32 * (dP - delta)) feeds dQ and dK;
 *   dV, dK, dQ accumulate in FP32 over all blocks; dQ and dK are multiplied
 *   by alpha in FP32; all three are rounded to BF16 once at the end.
 * Loop order is the algorithm's: key blocks outside, query blocks inside.
 */
void orc_emu_bwd(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                 const uint16_t *dO, const float *L, const float *delta,
                 int B, int H, int Hkv, int N, int d, int causal, float alpha,
                 int Br, int Bc,
                 uint16_t *dQ, uint16_t *dK, uint16_t *dV)
{
    /* Grouped-query attention: H query heads share Hkv key/value heads, query head h uses key/value head
     * h / (H / Hkv); k, v, dK, dV are [B][Hkv][N][d].  dK and dV of a key/value head accumulate, in FP32, the
     * contributions of the H / Hkv query heads of its group (in head order) before the single rounding.
     * Hkv == H is ordinary multi-head attention. */
    const int group = H / Hkv;
    const long kvheads = (long)B * Hkv;
    const int Tr = (N + Br - 1) / Br, Tc = (N + Bc - 1) / Bc;
    /* dK_j, dV_j: for each key block j, query blocks i in order (the algorithm's loops). */
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (long kvh = 0; kvh < kvheads; ++kvh) {
        for (int j = 0; j < Tc; ++j) {
            const long koff = kvh * (long)N * d;
            const uint16_t *kh = k + koff, *vh = v + koff;
            const int t0 = j * Bc, t1 = (j + 1) * Bc < N ? (j + 1) * Bc : N;
            float *dk = (float *)calloc((size_t)(t1 - t0) * d, sizeof(float));
            float *dv = (float *)calloc((size_t)(t1 - t0) * d, sizeof(float));
            for (int g = 0; g < group; ++g) {
                const long bh = kvh * group + g;                 /* [B][H] index of the query head */
                const long off = bh * (long)N * d;
                const uint16_t *qh = q + off, *gh = dO + off;
                for (int i = 0; i < Tr; ++i) {
                    const int r0 = i * Br, r1 = (i + 1) * Br < N ? (i + 1) * Br : N;
                    if (causal && t0 > r1 - 1) continue;
                    for (int T = r0; T < r1; ++T) {
                        const float Lr = L[bh * N + T], del = delta[bh * N + T];
                        for (int t = t0; t < t1; ++t) {
                            if (causal && t > T) continue;          /* P = 0 there */
                            float acc = 0.0f, dp = 0.0f;
                            for (int c = 0; c < d; ++c)
                                acc += orc_bf16_to_f32(qh[(long)T * d + c]) *
                                       orc_bf16_to_f32(kh[(long)t * d + c]);
                            for (int c = 0; c < d; ++c)
                                dp += orc_bf16_to_f32(gh[(long)T * d + c]) *
                                      orc_bf16_to_f32(vh[(long)t * d + c]);
                            const float sc = alpha * acc;
                            const float p32 = exp_f32(sc - Lr);
                            const float p = round_bf16(p32);
                            const float ds = round_bf16(p32 * (dp - del));
                            for (int c = 0; c < d; ++c) {
                                dv[(long)(t - t0) * d + c] += p * orc_bf16_to_f32(gh[(long)T * d + c]);
                                dk[(long)(t - t0) * d + c] += ds * orc_bf16_to_f32(qh[(long)T * d + c]);
                            }
                        }
                    }
                }
            }
            for (long e = 0; e < (long)(t1 - t0) * d; ++e) {
                dK[koff + (long)t0 * d + e] = orc_f32_to_bf16(alpha * dk[e]);
                dV[koff + (long)t0 * d + e] = orc_f32_to_bf16(dv[e]);
            }
            free(dk); free(dv);
        }
    }
    const long heads = (long)B * H;
    /* dQ_i: accumulated over the key blocks j in order; the same P and dS are recomputed
     * so that the query blocks can be handled independently. */
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (long bh = 0; bh < heads; ++bh) {
        for (int i = 0; i < Tr; ++i) {
            const long off = bh * (long)N * d, koff = (bh / group) * (long)N * d;
            const uint16_t *qh = q + off, *kh = k + koff, *vh = v + koff, *gh = dO + off;
            const int r0 = i * Br, r1 = (i + 1) * Br < N ? (i + 1) * Br : N;
            float *dq = (float *)calloc((size_t)(r1 - r0) * d, sizeof(float));
            for (int j = 0; j < Tc; ++j) {
                const int t0 = j * Bc, t1 = (j + 1) * Bc < N ? (j + 1) * Bc : N;
                if (causal && t0 > r1 - 1) continue;
                for (int T = r0; T < r1; ++T) {
                    const float Lr = L[bh * N + T], del = delta[bh * N + T];
                    for (int t = t0; t < t1; ++t) {
                        if (causal && t > T) continue;
                        float acc = 0.0f, dp = 0.0f;
                        for (int c = 0; c < d; ++c)
                            acc += orc_bf16_to_f32(qh[(long)T * d + c]) *
                                   orc_bf16_to_f32(kh[(long)t * d + c]);
                        for (int c = 0; c < d; ++c)
                            dp += orc_bf16_to_f32(gh[(long)T * d + c]) *
                                  orc_bf16_to_f32(vh[(long)t * d + c]);
                        const float p32 = exp_f32(alpha * acc - Lr);
                        const float ds = round_bf16(p32 * (dp - del));
                        for (int c = 0; c < d; ++c)
                            dq[(long)(T - r0) * d + c] += ds * orc_bf16_to_f32(kh[(long)t * d + c]);
                    }
                }
            }
            for (long e = 0; e < (long)(r1 - r0) * d; ++e)
                dQ[off + (long)r0 * d + e] = orc_f32_to_bf16(alpha * dq[e]);
            free(dq);
        }
    }
}

/* Prefix trace of Sec. 3.3.2: for one row of BF16 weights p[0..n) and one
 * BF16 value column v[0..n), out_lp[t] = bf16(FP32 prefix sum up to t) and
 * out_hp[t] = the FP32 prefix sum itself (the paper's hp is FP32). */
void orc_prefix_trace(const uint16_t *p, const uint16_t *v, int n,
                      float *out_lp, float *out_hp)
{
    float acc = 0.0f;
    for (int t = 0; t < n; ++t) {
        acc += orc_bf16_to_f32(p[t]) * orc_bf16_to_f32(v[t]);
        out_hp[t] = acc;
        out_lp[t] = round_bf16(acc);
    }
}

int orc_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
