/*
 * EntropyCache hot path -- CPU oracle, fp64.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, direct statement of what one cached denoising layer-step and
 * the entropy gate compute, written from the paper's definitions.  It is used
 * by the tests, by the smoke check and by the benchmark's CPU-baseline leg and
 * by nothing else: the product path never calls it.  It shares no code, header,
 * table or helper with the CUDA library.
 *
 * Inputs arrive in their storage encoding (dtype 0: IEEE fp32; dtype 1: bf16
 * bit patterns in uint16) and are widened exactly to double before any
 * arithmetic.  All arithmetic is double.  There is no tiling, no online
 * softmax, no fusion: every function is the definition written out.  The only
 * concession to run time is an OpenMP "parallel for" over independent outputs.
 *
 * Passages followed:
 *   refresh  -- Section 4.2 (last sentence of the tau_R paragraph): on a partial
 *               step only the mask tokens and the selected recent tokens get new
 *               K,V; every other position keeps its cached K,V.  Appendix A,
 *               partial branch: K,V of rows M u R are the fresh projections.
 *   attend   -- Appendix A, partial branch: TransformerBlock(Q[M u R], K[I], V[I]):
 *               queries are the active rows only, keys/values are all positions,
 *               attention is bidirectional (Sections 1 and 2.1: no causal mask).
 *               The full branch is the same with the active rows = all rows.
 *   gate     -- Eq. 1 and the paragraph after it; Algorithm 1 (entropy, then
 *               "E <= tau: reuse cache, else full recompute").
 *
 * Readings where the paper is silent (all listed in the design notes):
 *   natural logarithm (nats); E == tau skips (strict ">" recomputes); argmax
 *   ties go to the smallest index; -inf logits carry probability 0 and add 0 to
 *   the entropy; an empty decoded set gives E = -inf and the decision "skip";
 *   softmax scale 1/sqrt(head_dim) unless given; GQA maps query head h to kv
 *   head h / (n_q_heads / n_kv_heads); refresh happens before attending.
 *
 * Pins (tests/test_oracle_pins.py): closed-form entropies (uniform, one-hot,
 * two-way tie, m-spike rows), shift invariance, bounds, scipy/torch fp64
 * library routines, brute-force matrix attention, constant-V / constant-K /
 * dominant-key special cases, permutation invariance, GQA = repeated-head MHA,
 * byte-level refresh checks, gate flip at tau.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double widen(const void *base, int64_t i, int dtype)
{
    if (dtype == 0) {
        return (double)((const float *)base)[i];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* -------------------------------------------------------------------------
 * Refresh: Kc[b, h, idx[b,i], :] <- k_new[b, i, h, :] (same for V), bytes
 * copied verbatim.  active_idx == NULL means idx[b,i] = i (recompute step).
 * Returns 0, or 1 if an index is out of range (nothing is written then).
 * ------------------------------------------------------------------------- */
int oracle_kv_refresh(int batch, int ctx_len, int n_kv_heads, int head_dim, int elem_bytes,
                      void *k_cache, void *v_cache, const void *k_new, const void *v_new,
                      const int32_t *active_idx, int n_active)
{
    const size_t row = (size_t)head_dim * (size_t)elem_bytes;
    if (active_idx) {
        for (int64_t t = 0; t < (int64_t)batch * n_active; ++t)
            if (active_idx[t] < 0 || active_idx[t] >= ctx_len) return 1;
    } else if (n_active > ctx_len) {
        return 1;
    }
    for (int b = 0; b < batch; ++b)
        for (int i = 0; i < n_active; ++i) {
            const int pos = active_idx ? active_idx[(int64_t)b * n_active + i] : i;
            for (int h = 0; h < n_kv_heads; ++h) {
                const size_t src = (((size_t)b * n_active + i) * n_kv_heads + h) * row;
                const size_t dst = (((size_t)b * n_kv_heads + h) * ctx_len + pos) * row;
                memcpy((char *)k_cache + dst, (const char *)k_new + src, row);
                memcpy((char *)v_cache + dst, (const char *)v_new + src, row);
            }
        }
    return 0;
}

/* -------------------------------------------------------------------------
 * Attend: for every selected active row i, query head hq:
 *     s_j = scale * sum_d Q[b,i,hq,d] * K[b,hq/g,j,d]      for all j in [0, L)
 *     p_j = exp(s_j - max_j s_j) / sum_j exp(s_j - max_j s_j)
 *     O[d] = sum_j p_j * V[b,hq/g,j,d]
 * The caches are read as they are (i.e. after any refresh).  row_sel (indices
 * into 0..n_active-1, shared by all sequences) picks which query rows are
 * computed; NULL computes all of them.  out is double
 * [batch, n_sel, n_q_heads, head_dim].
 * ------------------------------------------------------------------------- */
int oracle_attend(int batch, int ctx_len, int n_q_heads, int n_kv_heads, int head_dim, int dtype,
                  double scale, const void *q, const void *k_cache, const void *v_cache,
                  int n_active, const int32_t *row_sel, int n_sel, double *out)
{
    if (n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0) return 1;
    const int g = n_q_heads / n_kv_heads;
    const int rows = row_sel ? n_sel : n_active;
    if (scale == 0.0) scale = 1.0 / sqrt((double)head_dim);
    const int64_t n_jobs = (int64_t)batch * rows * n_q_heads;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t job = 0; job < n_jobs; ++job) {
        const int hq = (int)(job % n_q_heads);
        const int r = (int)((job / n_q_heads) % rows);
        const int b = (int)(job / ((int64_t)n_q_heads * rows));
        const int i = row_sel ? row_sel[r] : r;
        if (i < 0 || i >= n_active) {
#pragma omp atomic write
            err = 1;
            continue;
        }
        const int hk = hq / g;
        const int64_t qoff = (((int64_t)b * n_active + i) * n_q_heads + hq) * head_dim;
        const int64_t coff = ((int64_t)b * n_kv_heads + hk) * ctx_len * (int64_t)head_dim;
        double *s = (double *)malloc(sizeof(double) * (size_t)ctx_len);
        double m = -INFINITY;
        for (int j = 0; j < ctx_len; ++j) {
            double acc = 0.0;
            for (int d = 0; d < head_dim; ++d)
                acc += widen(q, qoff + d, dtype) * widen(k_cache, coff + (int64_t)j * head_dim + d, dtype);
            s[j] = acc * scale;
            if (s[j] > m) m = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j < ctx_len; ++j) {
            s[j] = exp(s[j] - m);
            denom += s[j];
        }
        double *o = out + (((int64_t)b * rows + r) * n_q_heads + hq) * head_dim;
        for (int d = 0; d < head_dim; ++d) {
            double acc = 0.0;
            for (int j = 0; j < ctx_len; ++j)
                acc += (s[j] / denom) * widen(v_cache, coff + (int64_t)j * head_dim + d, dtype);
            o[d] = acc;
        }
        free(s);
    }
    return err;
}

/* -------------------------------------------------------------------------
 * Gate (Eq. 1): for each logits row r
 *     p_j    = softmax(x)_j
 *     argmax = smallest j with x_j == max x ;  conf = p_argmax
 *     H_r    = - sum_{j : p_j > 0} p_j ln p_j
 * then per sequence b (rows_per_seq consecutive rows):
 *     E_b = max over rows with flag != 0 of H_r   (-inf if none)
 *     decision_b = 1 (recompute) if E_b > tau else 0 (skip)
 * probs_out (nullable) receives the full softmax, double [n_rows, vocab].
 * ------------------------------------------------------------------------- */
int oracle_entropy_gate(const void *logits, int dtype, int n_rows, int vocab, int64_t row_stride,
                        int rows_per_seq, const uint8_t *decoded_flags, float tau,
                        int32_t *argmax_out, double *conf_out, double *entropy_out,
                        double *max_entropy_out, int32_t *decision_out, double *probs_out)
{
    if (rows_per_seq <= 0 || n_rows % rows_per_seq != 0) return 1;
    double *H = (double *)malloc(sizeof(double) * (size_t)(n_rows > 0 ? n_rows : 1));
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int64_t off = (int64_t)r * row_stride;
        double m = -INFINITY;
        int am = 0;
        for (int j = 0; j < vocab; ++j) {
            const double x = widen(logits, off + j, dtype);
            if (x > m) { m = x; am = j; }
        }
        double S = 0.0;
        for (int j = 0; j < vocab; ++j)
            S += exp(widen(logits, off + j, dtype) - m);
        double h = 0.0;
        for (int j = 0; j < vocab; ++j) {
            const double p = exp(widen(logits, off + j, dtype) - m) / S;
            if (probs_out) probs_out[(int64_t)r * vocab + j] = p;
            if (p > 0.0) h -= p * log(p);
        }
        H[r] = h;
        if (argmax_out) argmax_out[r] = am;
        if (conf_out) conf_out[r] = exp(widen(logits, off + am, dtype) - m) / S;
        if (entropy_out) entropy_out[r] = h;
    }
    const int n_seq = n_rows / rows_per_seq;
    for (int b = 0; b < n_seq; ++b) {
        double E = -INFINITY;
        for (int r = b * rows_per_seq; r < (b + 1) * rows_per_seq; ++r)
            if (decoded_flags[r] && H[r] > E) E = H[r];
        if (max_entropy_out) max_entropy_out[b] = E;
        if (decision_out) decision_out[b] = (E > (double)tau) ? 1 : 0;
    }
    free(H);
    return 0;
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
