/*
 * svip_oracle.c -- plain fp64 CPU oracle for the SVIP speculative-decoding epilogues.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, scalar, one-row-at-a-time
 * definition that the CUDA library is checked against.  It shares no code,
 * header, table or helper with the CUDA path, and nothing in the product
 * (the CUDA library or its Python binding) may include, link or call it.
 *
 * What it follows (paper: "SVIP: Towards Training-free Dynamic Draft Length
 * Policy for Speculative Decoding", arXiv 2411.18462):
 *   - draft sampling and entropy stop test: Algorithm 1 (inner loop), Eq. 7
 *   - acceptance test:   Algorithm 2 (sampling), Algorithm 3 (greedy)
 *   - correction token:  Algorithm 4 (sampling), Algorithm 5 (greedy)
 *   - verify loop, bonus token: Algorithm 1 (outer loop body) / Algorithm 6
 *   - several candidates per position (tree verification, the EAGLE-2 setting
 *     of Section 3.3): not defined by the paper; the published recursive
 *     rejection rule, see svip_oracle_verify_tree
 *   - expected acceptance beta, TVD, KL: Eq. 1 - Eq. 4
 *   - top-k / nucleus truncation (end of this file): not defined by the paper;
 *     the published definitions, ties kept by threshold, pinned by hand-made
 *     rows, a brute-force construction and the law of the emitted token
 *
 * Readings of the paper that this file fixes (each is pinned by a CPU test):
 *   - Algorithm 4 prints the residual with draft minus target.  Only
 *     max(0, p - q) (target minus draft) makes the emitted token follow the
 *     target distribution, which is the premise of speculative decoding, so
 *     that sign is used.
 *   - entropy is in nats (Pinsker's inequality in Eq. 3 is stated for nats).
 *   - the stop test is exactly sqrt(H) > h, strict.
 *   - the accept test is exactly r < p(x)/q(x), strict, r in [0,1).
 *   - T > 0: every distribution is softmax(logits / T), and H is taken on it.
 *     T == 0 (greedy): tokens are lowest-index argmax of the raw logits and
 *     H is the entropy of softmax(logits) at temperature 1.
 *   - argmax ties: lowest index among the maxima of the raw logits.
 *   - inverse CDF: running sum in index order; the first index whose
 *     cumulative weight EXCEEDS u * total; if rounding leaves none, the last
 *     index with positive weight.
 *
 * Every function is pinned (closed forms, brute force on tiny vocabularies,
 * chi-square tests of the emitted-token law); none is "parity unpinned".
 *
 * Logit rows come as raw memory: dtype 0 = IEEE fp32, dtype 1 = bfloat16 bits
 * (uint16).  Both convert exactly to fp64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { SVIP_ORACLE_F32 = 0, SVIP_ORACLE_BF16 = 1 };

static double logit_at(const void *row, int dtype, long i)
{
    if (dtype == SVIP_ORACLE_F32)
        return (double)((const float *)row)[i];
    uint32_t bits = (uint32_t)((const uint16_t *)row)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Lowest index among the maxima of the raw logits. */
long svip_oracle_argmax(const void *row, int dtype, long V)
{
    long best = 0;
    double bv = logit_at(row, dtype, 0);
    for (long i = 1; i < V; ++i) {
        double v = logit_at(row, dtype, i);
        if (v > bv) { bv = v; best = i; }
    }
    return best;
}

/* prob[i] = exp(l_i/T - M) / sum_j exp(l_j/T - M),  M = max_j l_j/T.  T > 0. */
void svip_oracle_softmax(const void *row, int dtype, long V, double T, double *prob)
{
    double M = -INFINITY;
    for (long i = 0; i < V; ++i) {
        double s = logit_at(row, dtype, i) / T;
        if (s > M) M = s;
    }
    double Z = 0.0;
    for (long i = 0; i < V; ++i) {
        double s = logit_at(row, dtype, i) / T;
        double e = (s == -INFINITY) ? 0.0 : exp(s - M);
        prob[i] = e;
        Z += e;
    }
    for (long i = 0; i < V; ++i)
        prob[i] /= Z;
}

/* H(p) = -sum p_i ln p_i, with 0 ln 0 = 0 (nats). */
double svip_oracle_entropy(const double *prob, long V)
{
    double H = 0.0;
    for (long i = 0; i < V; ++i)
        if (prob[i] > 0.0)
            H -= prob[i] * log(prob[i]);
    return H;
}

/* First index whose cumulative weight exceeds u * total (index order). */
long svip_oracle_invcdf(const double *w, long V, double u)
{
    double total = 0.0;
    for (long i = 0; i < V; ++i)
        total += w[i];
    double target = u * total;
    double c = 0.0;
    long last_pos = -1;
    for (long i = 0; i < V; ++i) {
        c += w[i];
        if (w[i] > 0.0) last_pos = i;
        if (c > target) return i;
    }
    return last_pos;
}

/*
 * One draft token (Algorithm 1, inner loop; Eq. 7).
 *   T > 0 : q = softmax(l/T); token ~ q by inverse CDF at u; H = H(q)
 *   T == 0: token = argmax l;  H = H(softmax(l))
 *   stop  = sqrt(H) > h
 * Returns 0, or -1 if scratch memory could not be obtained.
 */
int svip_oracle_draft_step(const void *row, int dtype, long V, double T, double h,
                           double u, long *token, double *entropy, int *stop)
{
    double *q = (double *)malloc((size_t)V * sizeof(double));
    if (!q) return -1;
    if (T > 0.0) {
        svip_oracle_softmax(row, dtype, V, T, q);
        *token = svip_oracle_invcdf(q, V, u);
    } else {
        svip_oracle_softmax(row, dtype, V, 1.0, q);
        *token = svip_oracle_argmax(row, dtype, V);
    }
    double H = svip_oracle_entropy(q, V);
    *entropy = H;
    *stop = sqrt(H) > h ? 1 : 0;
    free(q);
    return 0;
}

/* Acceptance probability min(1, p(x)/q(x)) of Algorithm 2; q(x) == 0 accepts iff p(x) > 0. */
static double accept_probability(const double *p, const double *q, long x)
{
    if (q[x] > 0.0) {
        double ratio = p[x] / q[x];
        return ratio < 1.0 ? ratio : 1.0;
    }
    return p[x] > 0.0 ? 1.0 : 0.0;
}

/*
 * One verification round of one sequence (Algorithm 1 outer-loop body with
 * Algorithms 2-5).
 *   K               draft length of this sequence (>= 1)
 *   draft_tokens    K draft tokens x_0..x_{K-1}
 *   q_rows          draft logits; row j starts q_stride elements after row j-1
 *   t_rows          K+1 target logit rows, same convention with t_stride
 *   r               K+1 uniforms in [0,1): r[0..K-1] accept draws, r[K] the
 *                   draw for the correction or the bonus token
 *   accept_prob     optional, K entries: min(1, p/q) at every position
 *                   (filled for all K positions, also past the rejection)
 * Outputs n_accepted in [0,K] and next_token (correction at position
 * n_accepted when n_accepted < K, else the bonus token from row K).
 * T == 0 selects the greedy variants; r is then unused and accept_prob is
 * filled with 1.0 / 0.0.
 */
int svip_oracle_verify(long K, const int32_t *draft_tokens,
                       const void *q_rows, long q_stride,
                       const void *t_rows, long t_stride,
                       int dtype, long V, double T, const double *r,
                       long *n_accepted, long *next_token, double *accept_prob)
{
    size_t esz = dtype == SVIP_ORACLE_F32 ? 4 : 2;
    const char *qb = (const char *)q_rows;
    const char *tb = (const char *)t_rows;

    if (!(T > 0.0)) {
        long n_acc = K;
        for (long j = 0; j < K; ++j) {
            long am = svip_oracle_argmax(tb + (size_t)j * t_stride * esz, dtype, V);
            int ok = am == (long)draft_tokens[j];
            if (accept_prob) accept_prob[j] = ok ? 1.0 : 0.0;
            if (!ok && n_acc == K) n_acc = j;
        }
        *n_accepted = n_acc;
        *next_token = svip_oracle_argmax(tb + (size_t)n_acc * t_stride * esz, dtype, V);
        return 0;
    }

    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *q = (double *)malloc((size_t)V * sizeof(double));
    if (!p || !q) { free(p); free(q); return -1; }

    long n_acc = K;
    long next = -1;
    for (long j = 0; j < K; ++j) {
        if (n_acc < K && !accept_prob) break;
        svip_oracle_softmax(tb + (size_t)j * t_stride * esz, dtype, V, T, p);
        svip_oracle_softmax(qb + (size_t)j * q_stride * esz, dtype, V, T, q);
        double a = accept_probability(p, q, (long)draft_tokens[j]);
        if (accept_prob) accept_prob[j] = a;
        if (n_acc < K) continue;           /* already rejected: only recording a_j */
        if (!(r[j] < a)) {
            n_acc = j;
            double S = 0.0;
            for (long i = 0; i < V; ++i) {
                double w = p[i] - q[i];
                q[i] = w > 0.0 ? w : 0.0;  /* q now holds the residual weights */
                S += q[i];
            }
            next = S > 0.0 ? svip_oracle_invcdf(q, V, r[K])
                           : svip_oracle_invcdf(p, V, r[K]);
        }
    }
    if (n_acc == K) {
        svip_oracle_softmax(tb + (size_t)K * t_stride * esz, dtype, V, T, p);
        next = svip_oracle_invcdf(p, V, r[K]);
    }
    *n_accepted = n_acc;
    *next_token = next;
    free(p);
    free(q);
    return 0;
}

/*
 * Verification of a TREE of draft candidates for one sequence (several
 * candidates per position, as in the EAGLE-2 setting of Section 3.3).  The
 * paper names that setting but states no accept rule for it; the rule here is
 * the published multi-candidate generalisation of Algorithms 2 and 4
 * (recursive rejection sampling), which keeps the paper's premise that every
 * emitted token follows the target distribution when the candidates of a node
 * are drawn independently from the draft distribution q of that node:
 *
 *   at a node with target distribution p and draft distribution q, and
 *   candidates x_1..x_m (its children, in index order):
 *     p_1 = p
 *     for i = 1..m:  accept x_i if r_i < min(1, p_i(x_i) / q(x_i));
 *                    else p_{i+1} = max(0, p_i - q) / sum max(0, p_i - q)
 *     a child accepted: descend into it; none accepted (or no child):
 *     the next token is drawn from p_{m+1} (from p itself at a leaf) and the
 *     walk ends.
 *   With one child per node this is exactly svip_oracle_verify.
 *
 * Layout: nodes 0..N-1, parent[i] = -1 for a child of the root, else an index
 * below i; token[i] the candidate token.  Row k of q_rows / t_rows belongs to
 * the root for k = 0 and to node k-1 otherwise (N+1 rows each, strides in
 * elements); q rows of leaves are not read.  r[i] is the accept draw of node
 * i, r[N] the draw for the final token.
 * Outputs: *n_accepted, path[0..n_accepted) (the accepted nodes, root to
 * leaf), *next_token, and, if accept_prob is given (N entries), min(1, p_i/q)
 * of every candidate that was tried (-1 for the others), and, if final_w is
 * given (V entries, sampling only), the unnormalised weights the next token was
 * drawn from.
 * T == 0: a child is accepted iff its token is the argmax of the node's
 * target row (first such child); the next token is that argmax otherwise.
 * A residual without mass (cannot happen after a rejection in exact
 * arithmetic) leaves the distribution as it was, as in svip_oracle_verify.
 */
int svip_oracle_verify_tree(long N, const int32_t *parent, const int32_t *token,
                            const void *q_rows, long q_stride,
                            const void *t_rows, long t_stride,
                            int dtype, long V, double T, const double *r,
                            long *n_accepted, int32_t *path, long *next_token,
                            double *accept_prob, double *final_w)
{
    size_t esz = dtype == SVIP_ORACLE_F32 ? 4 : 2;
    const char *qb = (const char *)q_rows;
    const char *tb = (const char *)t_rows;
    long n = 0, cur = -1;
    if (accept_prob)
        for (long i = 0; i < N; ++i) accept_prob[i] = -1.0;

    if (!(T > 0.0)) {
        for (;;) {
            long am = svip_oracle_argmax(tb + (size_t)(cur + 1) * t_stride * esz, dtype, V);
            long taken = -1;
            for (long i = 0; i < N && taken < 0; ++i) {
                if (parent[i] != cur) continue;
                int ok = am == (long)token[i];
                if (accept_prob) accept_prob[i] = ok ? 1.0 : 0.0;
                if (ok) taken = i;
            }
            if (taken < 0) { *next_token = am; break; }
            path[n++] = (int32_t)taken;
            cur = taken;
        }
        *n_accepted = n;
        return 0;
    }

    double *w = (double *)malloc((size_t)V * sizeof(double));   /* weights of the current p_i */
    double *q = (double *)malloc((size_t)V * sizeof(double));
    if (!w || !q) { free(w); free(q); return -1; }
    for (;;) {
        svip_oracle_softmax(tb + (size_t)(cur + 1) * t_stride * esz, dtype, V, T, w);
        double tot = 1.0;                                       /* p_i = w / tot; p_1 = p */
        int have_q = 0;
        long taken = -1;
        for (long i = 0; i < N && taken < 0; ++i) {
            if (parent[i] != cur) continue;
            if (!have_q) {
                svip_oracle_softmax(qb + (size_t)(cur + 1) * q_stride * esz, dtype, V, T, q);
                have_q = 1;
            }
            long x = (long)token[i];
            double px = w[x] / tot, a;
            if (q[x] > 0.0) { a = px / q[x]; if (a > 1.0) a = 1.0; }
            else a = px > 0.0 ? 1.0 : 0.0;
            if (accept_prob) accept_prob[i] = a;
            if (r[i] < a) { taken = i; break; }
            /* rejected: p_{i+1} = max(0, p_i - q), renormalised */
            double S = 0.0;
            for (long v = 0; v < V; ++v) {
                double d = w[v] / tot - q[v];
                S += d > 0.0 ? d : 0.0;
            }
            if (S > 0.0) {
                for (long v = 0; v < V; ++v) {
                    double d = w[v] / tot - q[v];
                    w[v] = d > 0.0 ? d : 0.0;
                }
                tot = S;
            }
        }
        if (taken < 0) {
            *next_token = svip_oracle_invcdf(w, V, r[N]);
            if (final_w) memcpy(final_w, w, (size_t)V * sizeof(double));
            break;
        }
        path[n++] = (int32_t)taken;
        cur = taken;
    }
    *n_accepted = n;
    free(w);
    free(q);
    return 0;
}

/* Eq. 1: beta = sum_x min(p(x), q(x)). */
double svip_oracle_beta(const double *p, const double *q, long V)
{
    double b = 0.0;
    for (long i = 0; i < V; ++i)
        b += p[i] < q[i] ? p[i] : q[i];
    return b;
}

/* Total variation distance, (1/2) sum |p - q| (Eq. 2). */
double svip_oracle_tvd(const double *p, const double *q, long V)
{
    double s = 0.0;
    for (long i = 0; i < V; ++i)
        s += fabs(p[i] - q[i]);
    return 0.5 * s;
}

/* Cross entropy H_{q,p} = -sum q ln p (Eq. 4); +inf if q > 0 where p == 0. */
double svip_oracle_cross_entropy(const double *q, const double *p, long V)
{
    double s = 0.0;
    for (long i = 0; i < V; ++i)
        if (q[i] > 0.0)
            s -= q[i] * log(p[i]);
    return s;
}

/* Residual weights max(0, p - q) of Algorithm 4 (sign as fixed above); returns their sum. */
double svip_oracle_residual(const double *p, const double *q, long V, double *w)
{
    double S = 0.0;
    for (long i = 0; i < V; ++i) {
        double d = p[i] - q[i];
        w[i] = d > 0.0 ? d : 0.0;
        S += w[i];
    }
    return S;
}

/*
 * The quantities of the paper's analysis for one (target row, draft row) pair, all in nats:
 *   out[0] beta   = sum_x min(p, q)                                   (Eq. 1)
 *   out[1] H_q    = entropy of the draft distribution                 (Eq. 4)
 *   out[2] H_qp   = cross entropy -sum q ln p                         (Eq. 4)
 *   out[3] KL     = KL(q || p) = H_qp - H_q                           (Eq. 3 / Eq. 4)
 *   out[4] gamma  = H_qp / H_q = 1 + KL / H_q                         (Section 2.2);
 *                   for a one-hot draft row (H_q = 0): +inf if KL > 0, 1 if KL = 0
 *                   (gamma - 1 = KL / H_q is 0 for KL = 0 whatever H_q)
 *   out[5] 1 - sqrt(KL / 2)                 Pinsker "oracle bound"    (Eq. 3)
 *   out[6] 1 - sqrt(1 - exp(-KL))           Bretagnolle-Huber bound   (Appendix B)
 *   out[7] 1 - sqrt(c * H_q)                approximation bound       (Eq. 6)
 * p = softmax(target row / T), q = softmax(draft row / T), T > 0.
 */
int svip_oracle_pair_stats(const void *t_row, const void *q_row, int dtype, long V, double T,
                           double c_bound, double *out)
{
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *q = (double *)malloc((size_t)V * sizeof(double));
    if (!p || !q) { free(p); free(q); return -1; }
    svip_oracle_softmax(t_row, dtype, V, T, p);
    svip_oracle_softmax(q_row, dtype, V, T, q);
    double beta = svip_oracle_beta(p, q, V);
    double Hq = svip_oracle_entropy(q, V);
    double Hqp = svip_oracle_cross_entropy(q, p, V);
    double KL = Hqp - Hq;
    out[0] = beta;
    out[1] = Hq;
    out[2] = Hqp;
    out[3] = KL;
    out[4] = Hq > 0.0 ? Hqp / Hq : (KL > 0.0 ? INFINITY : 1.0);
    out[5] = 1.0 - sqrt(0.5 * (KL > 0.0 ? KL : 0.0));
    out[6] = 1.0 - sqrt(1.0 - exp(-(KL > 0.0 ? KL : 0.0)));
    out[7] = 1.0 - sqrt(c_bound * Hq);
    free(p);
    free(q);
    return 0;
}

/* ------------------------------------------------------------------------
 * Top-k / nucleus (top-p) truncation of a distribution.
 *
 * The paper applies its length policy on top of systems that sample from
 * truncated distributions but does not define the truncation itself; the
 * definitions here are the published ones (top-k: keep the k most likely
 * tokens; nucleus: keep the smallest set of most likely tokens whose mass
 * reaches top_p), made order-independent by a threshold reading of ties:
 *
 *   tau_k  = the k-th largest raw logit (1 <= k < V), else the smallest logit
 *   Z_k    = sum of exp(l_i/T - M) over {l_i >= tau_k},  M = max_i l_i/T
 *   tau_p  = the largest logit value v with  sum over {l_i >= v} >= top_p*Z_k
 *            (top_p < 1), else tau_k
 *   tau    = tau_p (which is >= tau_k); the kept set is {i : l_i >= tau}:
 *            every token tied with the last kept one is kept too.
 *
 * The truncated distribution is softmax(l/T) restricted to the kept set and
 * renormalised; everything else (sampling, entropy, acceptance, residual) is
 * the plain definition applied to rows whose dropped logits are -inf.
 * Sums run over the logits sorted in descending order.
 * Returns 0, or -1 if scratch memory could not be obtained.
 */
static int cmp_desc(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

int svip_oracle_threshold(const void *row, int dtype, long V, double T, long top_k, double top_p,
                          double *tau, double *Z_topk, double *Z_kept, long *n_kept)
{
    double *v = (double *)malloc((size_t)V * sizeof(double));
    if (!v) return -1;
    for (long i = 0; i < V; ++i)
        v[i] = logit_at(row, dtype, i);
    qsort(v, (size_t)V, sizeof(double), cmp_desc);
    const double tau_k = (top_k >= 1 && top_k < V) ? v[top_k - 1] : v[V - 1];
    const double M = v[0] / T;
    double Zk = 0.0;
    for (long i = 0; i < V && v[i] >= tau_k; ++i)
        Zk += (v[i] == -INFINITY) ? 0.0 : exp(v[i] / T - M);
    double t = tau_k;
    if (top_p < 1.0) {
        double c = 0.0;
        long i = 0;
        while (i < V && v[i] >= tau_k) {
            const double val = v[i];
            while (i < V && v[i] == val) {          /* the whole group of tied logits */
                c += (val == -INFINITY) ? 0.0 : exp(val / T - M);
                ++i;
            }
            if (c >= top_p * Zk) { t = val; break; }
        }
    }
    double Zt = 0.0;
    long n = 0;
    for (long i = 0; i < V && v[i] >= t; ++i) {
        Zt += (v[i] == -INFINITY) ? 0.0 : exp(v[i] / T - M);
        ++n;
    }
    *tau = t; *Z_topk = Zk; *Z_kept = Zt; *n_kept = n;
    free(v);
    return 0;
}
