/*
 * EARS verification step -- CPU oracle (TEST INFRASTRUCTURE, not product code).
 *
 * A plain, slow, scalar fp64 statement of what one speculative-decoding
 * verification step computes under the EARS acceptance rule.  It exists so that
 * the CUDA library can be checked against something written independently from
 * the paper; it shares no source, table, constant generator or helper with the
 * CUDA path and must never be called from it.  Only tests, the smoke check and
 * the benchmark's CPU-baseline leg load this file.
 *
 * What is computed (paper section in brackets):
 *   - temperature softmax of every target and draft row            [Sec. 3.1, 4.3]
 *   - R_i = P_t(x_i) / max(P_d(x_i), eps), eps = 1e-10              [Sec. 3.2 step 2, Sec. 3.3 item 2]
 *   - Uncertainty_i = 1 - max_v P_t(v), Tolerance_i = beta * it     [Sec. 3.2, tolerance equation]
 *     or, on request, Uncertainty_i = H(P_t) / ln V with H = -sum_v P_t(v) ln P_t(v): the paper
 *     names "distribution entropy" as a more refined measure [Sec. 5, future work item 1] and gives
 *     no formula; dividing by ln V (the entropy of the flat distribution over the V entries) is
 *     this library's reading, chosen so that the measure runs over [0, 1] like the printed one
 *   - accept iff R_i >= max(U_i - Tolerance_i, 0)                   [Sec. 3.2 acceptance condition, Sec. 3.3 item 2]
 *   - direct / pardon / reject classification                       [Sec. 3.2 step 5]
 *   - first rejection ends the accepted prefix                      [Sec. 3.1]
 *   - token at the first rejected position: inverse-CDF draw from
 *     normalize(max(0, P_t - P_d)); if nothing was rejected, a bonus
 *     token drawn from P_t of the extra target row.  The paper only says that
 *     the target model continues from the rejected position [Sec. 3.1]; this is
 *     the standard speculative-sampling completion of its refs. [1], [2].
 *   - uniforms: Philox4x32-10 (Salmon et al., SC'11), key = seed, counter =
 *     (offset, sequence index, slot).  Not in the paper; fixed by this library's
 *     interface so that both sides draw identical numbers.
 *
 * Parity pins for every function here live in tests/test_oracle_*.py
 * (published Philox known answers, closed-form acceptance probabilities,
 * brute-force output laws on tiny vocabularies, library softmax / searchsorted,
 * total-variation identity, monotonicity in beta and temperature).
 * End-to-end numbers of the paper (throughput, accuracy) need its models and
 * datasets: parity unpinned for those, and nothing here tries to reproduce them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define EARS_ORACLE_EPS 1e-10 /* division guard, Sec. 3.3 item 2 */

/* ------------------------------------------------------------------------- */
/* Philox4x32-10, written from the published definition (Salmon, Moraes,      */
/* Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11).          */
/* ------------------------------------------------------------------------- */
void ears_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; /* golden-ratio Weyl increment */
        k1 += 0xBB67AE85u; /* sqrt(3)-1 Weyl increment */
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static void draw_words(uint64_t seed, uint64_t offset, uint32_t b, uint32_t slot, uint32_t w[4])
{
    uint32_t ctr[4] = { (uint32_t)offset, (uint32_t)(offset >> 32), b, slot };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    ears_oracle_philox4x32_10(ctr, key, w);
}

/* Accept uniform U(b,k) in [0,1): top 24 bits of word 0.  [Sec. 3.2 step 3] */
double ears_oracle_uniform_accept(uint64_t seed, uint64_t offset, int64_t b, int k)
{
    uint32_t w[4];
    draw_words(seed, offset, (uint32_t)b, (uint32_t)k, w);
    return (double)(w[0] >> 8) * (1.0 / 16777216.0);
}

/* Final-token uniform u(b) in [0,1): top 53 bits of words 0,1; slot = K. */
double ears_oracle_uniform_final(uint64_t seed, uint64_t offset, int64_t b, int K)
{
    uint32_t w[4];
    draw_words(seed, offset, (uint32_t)b, (uint32_t)K, w);
    uint64_t bits = (((uint64_t)w[0] << 32) | (uint64_t)w[1]) >> 11;
    return (double)bits * (1.0 / 9007199254740992.0);
}

/* ------------------------------------------------------------------------- */
/* Row access: logits are fp32 (dtype 0), bf16 bit patterns (dtype 1) or IEEE  */
/* binary16 bit patterns (dtype 2).  All widen to double without rounding.    */
/* ------------------------------------------------------------------------- */

/* IEEE 754 binary16: 1 sign bit, 5 exponent bits (bias 15), 10 fraction bits. */
double ears_oracle_half_to_double(uint16_t h)
{
    const int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 31) v = f ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)f, -24);               /* subnormal: f * 2^-10 * 2^-14 */
    else v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

static double logit_at(const void* base, int dtype, int64_t index)
{
    if (dtype == 0) return (double)((const float*)base)[index];
    if (dtype == 2) return ears_oracle_half_to_double(((const uint16_t*)base)[index]);
    uint32_t bits = (uint32_t)((const uint16_t*)base)[index] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/*
 * Temperature softmax of one row [Sec. 3.1; temperature as in Sec. 4.3]:
 * p_v = exp((l_v - m)/T) / Z, m = max_v l_v, Z = sum_v exp((l_v - m)/T),
 * summed left to right.  Returns 0, or -1 when the row has a NaN, a +inf or
 * no finite entry (such a row has no softmax).  -inf entries get p = 0.
 */
int ears_oracle_softmax(const double* logits, int V, double T, double* p, double* m_out, double* Z_out)
{
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (isnan(logits[v]) || logits[v] == INFINITY) return -1;
        if (logits[v] > m) m = logits[v];
    }
    if (m == -INFINITY) return -1;
    double Z = 0.0;
    for (int v = 0; v < V; ++v) {
        p[v] = exp((logits[v] - m) / T);
        Z += p[v];
    }
    for (int v = 0; v < V; ++v) p[v] /= Z;
    if (m_out) *m_out = m;
    if (Z_out) *Z_out = Z;
    return 0;
}

/*
 * Shannon entropy (nats) of a distribution p[0..V): H = -sum_v p_v ln p_v, with 0 ln 0 = 0
 * [Sec. 5 item 1 names it as an uncertainty measure; the definition is the textbook one].
 */
double ears_oracle_entropy(const double* p, int V)
{
    double H = 0.0;
    for (int v = 0; v < V; ++v)
        if (p[v] > 0.0) H -= p[v] * log(p[v]);
    return H;
}

/* Uncertainty in [0, 1] from the entropy: H / ln V (0 when V = 1: one entry leaves no doubt). */
double ears_oracle_entropy_uncertainty(double H, int V)
{
    return V > 1 ? H / log((double)V) : 0.0;
}

/*
 * Inverse-CDF draw from unnormalised masses r[0..V) at uniform u in [0,1):
 * S = sum r, C_j = sum_{v<=j} r_v; the token is the smallest j with u*S < C_j.
 * Zero-mass entries are therefore never chosen.  If rounding leaves u*S >= C_{V-1}
 * the last entry with positive mass is taken.  Returns -1 when S is not positive.
 * Optional outputs: S; lo/hi = the CDF interval [C_{j-1}/S, C_j/S) of the token;
 * band_lo/band_hi = first and last positive-mass tokens whose interval comes
 * within `band` of u (the tokens another rounding order could legitimately pick).
 */
int ears_oracle_inverse_cdf(const double* r, int V, double u, double band,
                            double* S_out, double* lo_out, double* hi_out,
                            int* band_lo_out, int* band_hi_out)
{
    double S = 0.0;
    for (int v = 0; v < V; ++v) S += r[v];
    if (S_out) *S_out = S;
    if (!(S > 0.0)) return -1;
    double target = u * S;
    double C = 0.0;
    int token = -1, last_pos = -1;
    double lo = 0.0, hi = 0.0;
    int band_lo = -1, band_hi = -1;
    for (int v = 0; v < V; ++v) {
        double before = C;
        C += r[v];
        if (r[v] > 0.0) {
            last_pos = v;
            if (token < 0 && target < C) { token = v; lo = before / S; hi = C / S; }
            /* interval [before/S, C/S) comes within band of u */
            if (C / S > u - band && before / S < u + band) {
                if (band_lo < 0) band_lo = v;
                band_hi = v;
            }
        }
    }
    if (token < 0) { token = last_pos; lo = hi = 1.0; }
    if (band_lo < 0) band_lo = band_hi = token;
    if (lo_out) *lo_out = lo;
    if (hi_out) *hi_out = hi;
    if (band_lo_out) *band_lo_out = band_lo;
    if (band_hi_out) *band_hi_out = band_hi;
    return token;
}

/* ------------------------------------------------------------------------- */
/* One sequence.                                                              */
/* ------------------------------------------------------------------------- */
typedef struct {
    double* pt_tok;      /* [B,K]  P_t(x_k)                               */
    double* pd_tok;      /* [B,K]  P_d(x_k)                               */
    double* max_pt;      /* [B,K]  max_v P_t(v) on target row k           */
    double* margin;      /* [B,K]  R - max(U - Tol, 0) (signed)           */
    uint8_t* cls;        /* [B,K]  0 reject, 1 direct accept, 2 pardon    */
    double* resid_mass;  /* [B]    S of the row the final token came from */
    double* cdf_margin;  /* [B]    distance of u to the chosen interval's nearer end */
    int32_t* band_lo;    /* [B]    see ears_oracle_inverse_cdf            */
    int32_t* band_hi;    /* [B]                                           */
    double* entropy;     /* [B,K]  H(P_t) of target row k, in nats        */
} ears_oracle_diag;

static void mark_invalid(int b, int K, int32_t* out_accept_len, int32_t* out_tokens)
{
    out_accept_len[b] = -1;
    for (int j = 0; j <= K; ++j) out_tokens[(int64_t)b * (K + 1) + j] = -1;
}

static void verify_one(const void* tl, const void* dl, int dtype, const int32_t* x,
                       int b, int K, int V, double T, double beta, int stop_at_first_reject, int uncertainty,
                       uint64_t seed, uint64_t offset, int64_t b_first, double band,
                       int32_t* out_accept_len, int32_t* out_tokens,
                       const ears_oracle_diag* dg,
                       double* row, double* pt, double* pd)
{
    int64_t gb = b_first + b; /* global sequence index used in the random counter */
    int n = K;                /* accepted prefix length, Sec. 3.1 */
    int valid = 1;

    for (int k = 0; k < K && valid; ++k) {
        int tok = x[(int64_t)b * K + k];
        if (tok < 0 || tok >= V) { valid = 0; break; }
        double Zt, Zd;
        for (int v = 0; v < V; ++v) row[v] = logit_at(tl, dtype, ((int64_t)b * (K + 1) + k) * V + v);
        if (ears_oracle_softmax(row, V, T, pt, NULL, &Zt)) { valid = 0; break; }
        for (int v = 0; v < V; ++v) row[v] = logit_at(dl, dtype, ((int64_t)b * K + k) * V + v);
        if (ears_oracle_softmax(row, V, T, pd, NULL, &Zd)) { valid = 0; break; }

        double maxp = 0.0;                                   /* Sec. 3.2: max_v P_t(v) */
        for (int v = 0; v < V; ++v) if (pt[v] > maxp) maxp = pt[v];
        double pd_safe = pd[tok] > EARS_ORACLE_EPS ? pd[tok] : EARS_ORACLE_EPS; /* Sec. 3.3 item 2 */
        double R = pt[tok] / pd_safe;                        /* Sec. 3.2 step 2 */
        double H = 0.0;
        if (uncertainty == 1 || (dg && dg->entropy)) H = ears_oracle_entropy(pt, V);
        double unc = uncertainty == 1 ? ears_oracle_entropy_uncertainty(H, V)   /* Sec. 5 item 1 */
                                      : 1.0 - maxp;                             /* Sec. 3.2 */
        double tol = beta * unc;                             /* tolerance equation */
        double U = ears_oracle_uniform_accept(seed, offset, gb, k);
        double thr = U - tol > 0.0 ? U - tol : 0.0;          /* Sec. 3.3 item 2, clamp */
        int accept = R >= thr;                               /* acceptance condition */
        int cls = R >= U ? 1 : (accept ? 2 : 0);             /* Sec. 3.2 step 5 */
        if (dg) {
            int64_t i = (int64_t)b * K + k;
            if (dg->pt_tok) dg->pt_tok[i] = pt[tok];
            if (dg->pd_tok) dg->pd_tok[i] = pd[tok];
            if (dg->max_pt) dg->max_pt[i] = maxp;
            if (dg->margin) dg->margin[i] = R - thr;
            if (dg->cls) dg->cls[i] = (uint8_t)cls;
            if (dg->entropy) dg->entropy[i] = H;
        }
        if (!accept && n == K) n = k; /* first rejection; later positions are diagnostics only */
        /* Sec. 3.1: a rejection discards every later draft token, so a caller may ask that their
         * rows are not read at all (then they are neither validated nor reported) */
        if (!accept && stop_at_first_reject) break;
    }
    /* the bonus row is part of the step's input: validate it even when unused
     * (unless the caller asked to stop at the first rejection and there was one) */
    if (valid && !(stop_at_first_reject && n < K)) {
        for (int v = 0; v < V; ++v) row[v] = logit_at(tl, dtype, ((int64_t)b * (K + 1) + K) * V + v);
        if (ears_oracle_softmax(row, V, T, pt, NULL, NULL)) valid = 0;
    }
    if (!valid) { mark_invalid(b, K, out_accept_len, out_tokens); return; }

    /* final token */
    double u = ears_oracle_uniform_final(seed, offset, gb, K);
    double S = 0.0, lo = 0.0, hi = 0.0;
    int blo = -1, bhi = -1, token;
    if (n < K) {
        for (int v = 0; v < V; ++v) row[v] = logit_at(tl, dtype, ((int64_t)b * (K + 1) + n) * V + v);
        ears_oracle_softmax(row, V, T, pt, NULL, NULL);
        for (int v = 0; v < V; ++v) row[v] = logit_at(dl, dtype, ((int64_t)b * K + n) * V + v);
        ears_oracle_softmax(row, V, T, pd, NULL, NULL);
        for (int v = 0; v < V; ++v) row[v] = pt[v] > pd[v] ? pt[v] - pd[v] : 0.0; /* residual */
        double S_res = 0.0;
        for (int v = 0; v < V; ++v) S_res += row[v];
        if (S_res < 1e-300) { /* cannot follow a rejection (R<1 implies mass); defensive: use P_t */
            for (int v = 0; v < V; ++v) row[v] = pt[v];
        }
        token = ears_oracle_inverse_cdf(row, V, u, band, &S, &lo, &hi, &blo, &bhi);
    } else {
        /* pt already holds the softmax of the bonus row */
        token = ears_oracle_inverse_cdf(pt, V, u, band, &S, &lo, &hi, &blo, &bhi);
    }
    out_accept_len[b] = n;
    for (int j = 0; j < n; ++j) out_tokens[(int64_t)b * (K + 1) + j] = x[(int64_t)b * K + j];
    out_tokens[(int64_t)b * (K + 1) + n] = token;
    for (int j = n + 1; j <= K; ++j) out_tokens[(int64_t)b * (K + 1) + j] = -1;
    if (dg) {
        if (dg->resid_mass) dg->resid_mass[b] = S;
        if (dg->cdf_margin) { double a = u - lo, c = hi - u; dg->cdf_margin[b] = a < c ? a : c; }
        if (dg->band_lo) dg->band_lo[b] = blo;
        if (dg->band_hi) dg->band_hi[b] = bhi;
    }
}

/*
 * One verification step over B independent sequences [Sec. 3.3 item 3 batches
 * "all active sequences"].  All pointers are host memory.
 *   target_logits [B,K+1,V], draft_logits [B,K,V] (dtype 0 fp32, 1 bf16 bits, 2 fp16 bits),
 *   draft_tokens [B,K]; b_first = global index of local sequence 0 (batch shards);
 *   band = half-width, in probability, used for the near-boundary token range.
 * Outputs: out_accept_len [B] (n in [0,K], or -1 for an invalid sequence),
 *   out_tokens [B,K+1] (n accepted draft tokens, then the resampled or bonus
 *   token, then -1).  Any diagnostic pointer may be NULL.
 * nthreads > 1 spreads sequences over OpenMP threads; results do not depend on it.
 * seq_temperature, seq_beta: optional [B] arrays that replace the scalars per sequence.
 * stop_at_first_reject != 0: rows and tokens after a sequence's first rejected position (and the
 *   extra target row, unless everything was accepted) are not read: not validated, no diagnostics.
 * uncertainty: 0 = 1 - max P_t [Sec. 3.2], 1 = H(P_t) / ln V [Sec. 5 item 1, see the header];
 *   entropy: optional [B,K] output of H(P_t) of every target row that was looked at.
 * Returns 0, -1 on bad arguments, -2 when out of memory.
 */
int ears_oracle_verify_unc(const void* target_logits, const void* draft_logits, int dtype,
                           const int32_t* draft_tokens, int B, int K, int V,
                           float temperature, float beta,
                           const float* seq_temperature, const float* seq_beta,
                           int stop_at_first_reject, int uncertainty,
                           uint64_t seed, uint64_t offset,
                           int64_t b_first, double band,
                           int32_t* out_accept_len, int32_t* out_tokens,
                           double* pt_tok, double* pd_tok, double* max_pt, double* margin,
                           uint8_t* cls, double* resid_mass, double* cdf_margin,
                           int32_t* band_lo, int32_t* band_hi, double* entropy, int nthreads)
{
    if (!target_logits || !draft_logits || !draft_tokens || !out_accept_len || !out_tokens) return -1;
    if (B < 1 || K < 1 || V < 1 || (dtype < 0 || dtype > 2)) return -1;
    if (!seq_temperature && (!(temperature > 0.0f) || !isfinite(temperature))) return -1;
    if (!seq_beta && (!(beta >= 0.0f) || !isfinite(beta))) return -1;
    if (uncertainty != 0 && uncertainty != 1) return -1;
    ears_oracle_diag dg = { pt_tok, pd_tok, max_pt, margin, cls, resid_mass, cdf_margin, band_lo, band_hi, entropy };
    if (nthreads < 1) nthreads = 1;
    int failed = 0;
#ifdef _OPENMP
#pragma omp parallel num_threads(nthreads)
#endif
    {
        double* row = (double*)malloc(sizeof(double) * (size_t)V);
        double* pt = (double*)malloc(sizeof(double) * (size_t)V);
        double* pd = (double*)malloc(sizeof(double) * (size_t)V);
        if (!row || !pt || !pd) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        }
#ifdef _OPENMP
#pragma omp barrier
#pragma omp for schedule(dynamic, 1)
#endif
        for (int b = 0; b < B; ++b) {
            if (failed) continue;
            /* Every sequence is verified on its own [Sec. 3.3 item 3], so each may carry its own
             * temperature [Sec. 4.3] and base tolerance beta [Sec. 3.2]; a value that the scalar
             * form would refuse makes that one sequence invalid. */
            float Tb = seq_temperature ? seq_temperature[b] : temperature;
            float bb = seq_beta ? seq_beta[b] : beta;
            if (!(Tb > 0.0f) || !isfinite(Tb) || !(bb >= 0.0f) || !isfinite(bb)) {
                mark_invalid(b, K, out_accept_len, out_tokens);
                continue;
            }
            verify_one(target_logits, draft_logits, dtype, draft_tokens, b, K, V, (double)Tb, (double)bb,
                       stop_at_first_reject, uncertainty, seed, offset, b_first, band, out_accept_len, out_tokens, &dg,
                       row, pt, pd);
        }
        free(row); free(pt); free(pd);
    }
    return failed ? -2 : 0;
}

/* The step with the uncertainty measure the paper prints (1 - max P_t). */
int ears_oracle_verify_var(const void* target_logits, const void* draft_logits, int dtype,
                           const int32_t* draft_tokens, int B, int K, int V,
                           float temperature, float beta,
                           const float* seq_temperature, const float* seq_beta,
                           int stop_at_first_reject,
                           uint64_t seed, uint64_t offset,
                           int64_t b_first, double band,
                           int32_t* out_accept_len, int32_t* out_tokens,
                           double* pt_tok, double* pd_tok, double* max_pt, double* margin,
                           uint8_t* cls, double* resid_mass, double* cdf_margin,
                           int32_t* band_lo, int32_t* band_hi, int nthreads)
{
    return ears_oracle_verify_unc(target_logits, draft_logits, dtype, draft_tokens, B, K, V, temperature, beta,
                                  seq_temperature, seq_beta, stop_at_first_reject, 0, seed, offset, b_first, band,
                                  out_accept_len, out_tokens, pt_tok, pd_tok, max_pt, margin, cls, resid_mass,
                                  cdf_margin, band_lo, band_hi, NULL, nthreads);
}

/* The same with one temperature and one beta for the whole batch. */
int ears_oracle_verify(const void* target_logits, const void* draft_logits, int dtype,
                       const int32_t* draft_tokens, int B, int K, int V,
                       float temperature, float beta, uint64_t seed, uint64_t offset,
                       int64_t b_first, double band,
                       int32_t* out_accept_len, int32_t* out_tokens,
                       double* pt_tok, double* pd_tok, double* max_pt, double* margin,
                       uint8_t* cls, double* resid_mass, double* cdf_margin,
                       int32_t* band_lo, int32_t* band_hi, int nthreads)
{
    return ears_oracle_verify_var(target_logits, draft_logits, dtype, draft_tokens, B, K, V, temperature, beta,
                                  NULL, NULL, 0, seed, offset, b_first, band, out_accept_len, out_tokens,
                                  pt_tok, pd_tok, max_pt, margin, cls, resid_mass, cdf_margin,
                                  band_lo, band_hi, nthreads);
}

/*
 * The temperature -> 0 limit of the step (the deterministic regime of Sec. 1): every softmax
 * becomes one-hot at its row's largest logit (the smallest index among equal ones), so
 * max_v P_t = 1, the tolerance beta (1 - max P_t) vanishes [Sec. 3.2], and for a draft token
 * drawn greedily (P_d(x_k) = 1) the ratio R_k is 1 if x_k is the target's top token and 0
 * otherwise: x_k is accepted iff it equals argmax of target row k.  The token at the first
 * rejected position n is argmax of target row n (the residual of two different one-hot
 * distributions is the target's), the bonus token argmax of row K.  No random numbers, no draft
 * logits.  Rows are validated like everywhere else (NaN, +inf, no finite entry: the sequence is
 * marked invalid); a draft token outside [0, V) is invalid too.
 */
int ears_oracle_verify_greedy(const void* target_logits, int dtype, const int32_t* draft_tokens,
                              int B, int K, int V, int32_t* out_accept_len, int32_t* out_tokens,
                              int32_t* argmax_out /* [B,K+1] or NULL */)
{
    if (!target_logits || !draft_tokens || !out_accept_len || !out_tokens) return -1;
    if (B < 1 || K < 1 || V < 1 || (dtype < 0 || dtype > 2)) return -1;
    for (int b = 0; b < B; ++b) {
        int valid = 1, n = K;
        for (int k = 0; k <= K; ++k) {
            int best = -1;
            double top = -INFINITY;
            for (int v = 0; v < V; ++v) {
                double l = logit_at(target_logits, dtype, ((int64_t)b * (K + 1) + k) * V + v);
                if (isnan(l) || l == INFINITY) valid = 0;
                if (l > top) { top = l; best = v; }   /* strict: the first of equal entries stays */
            }
            if (best < 0) valid = 0;                  /* nothing finite */
            if (argmax_out) argmax_out[(int64_t)b * (K + 1) + k] = best;
            if (k < K) {
                int tok = draft_tokens[(int64_t)b * K + k];
                if (tok < 0 || tok >= V) valid = 0;
                if (tok != best && n == K) n = k;     /* first rejection [Sec. 3.1] */
            }
        }
        if (!valid) { mark_invalid(b, K, out_accept_len, out_tokens); continue; }
        out_accept_len[b] = n;
        for (int j = 0; j <= K; ++j) {
            int64_t o = (int64_t)b * (K + 1) + j;
            out_tokens[o] = j < n ? draft_tokens[(int64_t)b * K + j] : -1;
        }
    }
    /* second sweep for the emitted token keeps the first one simple to read */
    for (int b = 0; b < B; ++b) {
        int n = out_accept_len[b];
        if (n < 0) continue;
        int best = -1;
        double top = -INFINITY;
        for (int v = 0; v < V; ++v) {
            double l = logit_at(target_logits, dtype, ((int64_t)b * (K + 1) + n) * V + v);
            if (l > top) { top = l; best = v; }
        }
        out_tokens[(int64_t)b * (K + 1) + n] = best;
    }
    return 0;
}

/* Softmax of one stored row, for tests that need the full distribution. */
int ears_oracle_row_softmax(const void* logits, int dtype, int64_t row_index, int V,
                            float temperature, double* p_out)
{
    double* row = (double*)malloc(sizeof(double) * (size_t)V);
    if (!row) return -2;
    for (int v = 0; v < V; ++v) row[v] = logit_at(logits, dtype, row_index * V + v);
    int rc = ears_oracle_softmax(row, V, (double)temperature, p_out, NULL, NULL);
    free(row);
    return rc;
}

int ears_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
