/*
 * CPU oracle for the WISV edge-side verifier.  TEST INFRASTRUCTURE ONLY: it is
 * the slow, plain statement of what the verifier computes, used by the tests,
 * the smoke check and the CPU-baseline leg of the benchmark.  The library
 * itself never calls it, and it shares no code with the CUDA path.
 *
 * Every function is the paper's definition written out with scalar loops and
 * double accumulation; OpenMP is applied only across independent outputs
 * (rows, vocabulary entries, positions), never inside a sum.
 *
 * Numeric convention (the paper fixes none beyond 16-bit uploaded hidden
 * states, Section IV-A, b_h = 16): hidden states are rounded to bf16 (nearest even)
 * before any matrix product, weights are bf16, products and sums are exact /
 * double here.
 *
 * Pins (tests/test_oracle_pins.py): torch float64 matmul/logsumexp/argmax,
 * closed forms (uniform logits, shift invariance, softmax sums to one), a
 * hand-worked decision-head example, exhaustive enumeration of the first-reject
 * rule for K <= 4 and the invariants of Algorithm 1.  The end-to-end figures of
 * Table I need trained weights and a dataset: parity unpinned, out of scope.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_bits_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* fp32 -> nearest-even bf16, returned as a double holding that bf16 value. */
static inline double round_to_bf16(float x)
{
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) {      /* NaN stays NaN */
        return (double)x;
    }
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int wisv_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * LM-head rows (Algorithm 1, Verify: the logits L of the target model; Section
 * IV-B notes they serve mismatch localisation and correction).
 *
 *   L[r][v] = sum_h bf16(Ht[r][h]) * W[v][h]
 *   argmax[r]   = lowest v attaining max_v L[r][v]
 *   lse[r]      = log sum_v exp(L[r][v])
 *   tok_logit[r]= L[r][row_token[r]]           (row_token[r] < 0: not requested -> NaN)
 *   top2_gap[r] = max - (largest logit at any other index)
 *
 * W: bf16 bit patterns [V][H] row-major; Ht: fp32 [R][H]; outputs have R entries.
 * logits_out, if not NULL, receives the full double logits [R][V] (tiny cases only).
 */
int wisv_oracle_lm_head(const uint16_t* W, const float* Ht, int64_t R, int32_t H, int32_t V,
                        const int32_t* row_token, int32_t* argmax, double* lse,
                        double* tok_logit, double* top2_gap, double* logits_out)
{
    if (R < 0 || H <= 0 || V <= 0) return -1;
    enum { ROW_BLOCK = 8 };
    double* x = (double*)malloc(sizeof(double) * (size_t)ROW_BLOCK * (size_t)H);
    double* L = (double*)malloc(sizeof(double) * (size_t)ROW_BLOCK * (size_t)V);
    if (!x || !L) { free(x); free(L); return -2; }

    for (int64_t r0 = 0; r0 < R; r0 += ROW_BLOCK) {
        int nb = (int)((R - r0) < ROW_BLOCK ? (R - r0) : ROW_BLOCK);
        /* x is stored [h][row-in-block] so the rows of a block share one pass over W[v] */
        for (int32_t h = 0; h < H; ++h)
            for (int i = 0; i < ROW_BLOCK; ++i)
                x[(size_t)h * ROW_BLOCK + i] =
                    i < nb ? round_to_bf16(Ht[(size_t)(r0 + i) * H + h]) : 0.0;

        /* every logit is an independent sum over h, taken in index order */
        #pragma omp parallel for schedule(static)
        for (int32_t v = 0; v < V; ++v) {
            const uint16_t* w = W + (size_t)v * H;
            double acc[ROW_BLOCK];
            for (int i = 0; i < ROW_BLOCK; ++i) acc[i] = 0.0;
            for (int32_t h = 0; h < H; ++h) {
                const double wv = bf16_bits_to_double(w[h]);
                const double* xh = x + (size_t)h * ROW_BLOCK;
                for (int i = 0; i < ROW_BLOCK; ++i) acc[i] += xh[i] * wv;
            }
            for (int i = 0; i < nb; ++i) L[(size_t)i * V + v] = acc[i];
        }

        for (int i = 0; i < nb; ++i) {
            const double* Li = L + (size_t)i * V;
            int64_t r = r0 + i;
            double best = Li[0], second = -INFINITY;
            int32_t arg = 0;
            for (int32_t v = 1; v < V; ++v) {
                if (Li[v] > best) { second = best; best = Li[v]; arg = v; }
                else if (Li[v] > second) { second = Li[v]; }
            }
            double sum = 0.0;
            for (int32_t v = 0; v < V; ++v) sum += exp(Li[v] - best);
            argmax[r] = arg;
            lse[r] = best + log(sum);
            if (top2_gap) top2_gap[r] = best - second;
            if (tok_logit) {
                int32_t t = row_token ? row_token[r] : -1;
                tok_logit[r] = (t >= 0 && t < V) ? Li[t] : NAN;
            }
            if (logits_out) memcpy(logits_out + (size_t)r * V, Li, sizeof(double) * (size_t)V);
        }
    }
    free(x); free(L);
    return 0;
}

static inline double act_relu(double x) { return x > 0.0 ? x : 0.0; }
static inline double act_gelu(double x) { return 0.5 * x * (1.0 + erf(x * 0.70710678118654752440)); }

/*
 * Decision head (Eqs. 23-25), dropout being the identity at
 * inference:
 *   z_p = [ bf16(hD[p]) ; bf16(Ht[tgt_row[p]]) ; csi[req[p]] ]
 *   s_p = w2 . act(W1 z_p + b1) + b2,   prob_p = 1 / (1 + exp(-s_p))
 *
 * W1: bf16 bits [d_J][H_d + H + d_c], columns ordered [h^D | h^T | c].
 * act: 0 = ReLU (the paper's), 1 = exact-erf GELU.
 * hD: fp32 [P][H_d]; Ht: fp32 [*][H]; csi: fp32 [*][d_c] consumed unrounded.
 */
int wisv_oracle_head(const uint16_t* W1, const float* b1, const float* w2, double b2,
                     int32_t H, int32_t H_d, int32_t d_c, int32_t d_J, int32_t act,
                     const float* hD, const float* Ht, const float* csi,
                     const int32_t* tgt_row, const int32_t* req, int64_t P,
                     double* logit_out, double* prob_out)
{
    if (P < 0 || H <= 0 || H_d < 0 || d_c < 0 || d_J <= 0) return -1;
    if (act != 0 && act != 1) return -1;
    const int32_t d_in = H_d + H + d_c;
    int fail = 0;
    #pragma omp parallel for schedule(dynamic)
    for (int64_t p = 0; p < P; ++p) {
        double* z = (double*)malloc(sizeof(double) * (size_t)d_in);
        if (!z) { fail = 1; continue; }
        for (int32_t k = 0; k < H_d; ++k) z[k] = round_to_bf16(hD[(size_t)p * H_d + k]);
        for (int32_t k = 0; k < H; ++k)   z[H_d + k] = round_to_bf16(Ht[(size_t)tgt_row[p] * H + k]);
        for (int32_t k = 0; k < d_c; ++k) z[H_d + H + k] = (double)csi[(size_t)req[p] * d_c + k];
        double s = 0.0;
        for (int32_t j = 0; j < d_J; ++j) {
            const uint16_t* w = W1 + (size_t)j * d_in;
            double pre = 0.0;
            for (int32_t k = 0; k < d_in; ++k) pre += bf16_bits_to_double(w[k]) * z[k];
            pre += (double)b1[j];
            s += (double)w2[j] * (act == 0 ? act_relu(pre) : act_gelu(pre));
        }
        s += b2;
        if (logit_out) logit_out[p] = s;
        prob_out[p] = 1.0 / (1.0 + exp(-s));
        free(z);
    }
    return fail ? -2 : 0;
}

/*
 * First-reject scan and emission (Algorithm 1: the min over S of positions whose
 * rejection probability reaches tau, then full accept or commit-and-correct;
 * Eq. 27 for the >= test).
 *
 * For request b with window length K_b = k_off[b+1]-k_off[b]; t = k_off[b]+i:
 *   rej_i = cand[t] && ( !has_prob[t] || prob[t] >= tau )
 *   accept_len[b] = min{ i : rej_i }, or K_b if none
 *   correction[b] = argmax[ row_off(b) + accept_len[b] ],  row_off(b) = k_off[b] + b
 * A candidate without an uploaded hidden state falls back to plain greedy
 * rejection (the tau = 0 behaviour of Section VI-B).
 */
int wisv_oracle_scan(int32_t B, const int32_t* k_off, const uint8_t* cand,
                     const uint8_t* has_prob, const double* prob, double tau,
                     const int32_t* argmax, int32_t* accept_len, int32_t* correction)
{
    if (B < 0) return -1;
    for (int32_t b = 0; b < B; ++b) {
        int32_t K = k_off[b + 1] - k_off[b];
        int32_t A = K;
        for (int32_t i = 0; i < K; ++i) {
            int64_t t = (int64_t)k_off[b] + i;
            int rej = cand[t] && (!has_prob[t] || prob[t] >= tau);
            if (rej) { A = i; break; }
        }
        accept_len[b] = A;
        correction[b] = argmax[(int64_t)k_off[b] + b + A];
    }
    return 0;
}
