/*
 * mars_oracle.c -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-pass-per-row CPU statement of margin-aware speculative
 * verification (MARS), written from the paper's text:
 *   - top-2 tokens of a logits row and the logit ratio r = z(2)/z(1)   (Sec. 3.3, Eq. 4)
 *   - three-way rule: exact match / adaptive relaxation / rejection     (Sec. 3.4)
 *   - chain verification loop with stop at the first failure            (Algorithm 1)
 *   - bonus token when every draft is accepted                          (Table 1 caption)
 *   - token-tree form of the same rule                                  (Sec. 2.3)
 *   - logits from the output projection z = W_o h + b_o                 (Eq. 2; logits
 *     are produced by the Python wrapper with an fp64 matmul, the rule below then
 *     runs on double rows)
 *   - stochastic (T > 0) verification: Eq. 1 acceptance, residual draw     (Sec. 2.2, Eq. 3;
 *     its composition with the relaxation is a reading of this repository, PARITY
 *     UNPINNED by the paper -- see the block comment above that function)
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this file.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * Precision: the paper never states one.  Decisions on stored logits are taken in
 * fp32: bf16 widens exactly to fp32, every comparison is an IEEE fp32 comparison and
 * the ratio is one round-to-nearest fp32 division.  Build with
 *   gcc -O2 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 * The "_f64" entry points take the same decisions in fp64 on double logits.
 *
 * Readings where the paper is silent (each is a convention of this repository):
 *   - threshold is strict: r == theta rejects (the paper writes r > theta throughout);
 *   - sign guard: relaxation needs z(1) > 0 unless MARS_ORACLE_SIGN_LITERAL is set;
 *     with the guard, r > theta agrees with the paper's equivalent margin form
 *     Delta < (1-theta) z(1) (Eq. 6) for every sign when theta < 1;
 *   - total order on a row: larger value first, lower token id first among equal
 *     values (IEEE ==, so -0 == +0); NaN counts as -inf;
 *   - tree: node i>0 is accepted iff its parent is accepted and tok[i] passes the
 *     three-way rule on the parent's row; the result is the deepest accepted node,
 *     lowest node index among equally deep ones; the emitted next token is the top-1
 *     of that node's row.
 *   Pinned by tests against: a sort-based top-2, the paper's Fig. 2 worked example,
 *   planted ratios one ulp around theta (in fp32 and, for the "_f64" rule, in fp64, directly
 *   and through a one-hot output projection), strict-greedy equivalence for theta >= 1,
 *   brute-force path enumeration on all small trees, closed-form acceptance rates.
 *   Parity unpinned by the paper (conventions only): the sign guard, NaN handling,
 *   the tie rules (equal logits; equally deep accepted paths).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define MARS_ORACLE_SIGN_LITERAL 1u
#define MARS_ORACLE_SHARED_PARENT 2u
#define MARS_ORACLE_RULE_MARGIN 8u
#define MARS_ORACLE_RULE_PROB_RATIO 16u

enum { ORACLE_BF16 = 0, ORACLE_FP32 = 1, ORACLE_FP64 = 2 };

int mars_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Host threads for the loop over rows (the container may see more cores than it may use). */
void mars_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* bf16 is the upper half of an fp32 word: widening is exact. */
static float bf16_to_f32(uint16_t h)
{
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return f;
}

/* ---- total order on (value, token id): Sec. 3.3 names z(1) >= z(2); ties by id ---- */
static int beats_f32(float ax, int64_t aj, float bx, int64_t bj)
{
    return (ax > bx) || (ax == bx && aj < bj);
}
static int beats_f64(double ax, int64_t aj, double bx, int64_t bj)
{
    return (ax > bx) || (ax == bx && aj < bj);
}

/*
 * Top-2 of one row (Algorithm 1, "identify top-2 tokens"; Sec. 3.3).
 * get(j) is the j-th logit widened to the decision type, NaN mapped to -inf.
 */
#define DEFINE_TOP2(NAME, T, BEATS, NEG_INF)                                            \
    static void NAME(const void *row, int dtype, int64_t V, T *val2, int32_t *id2)      \
    {                                                                                   \
        T bx = 0, sx = 0;                                                               \
        int64_t bj = -1, sj = -1;                                                       \
        for (int64_t j = 0; j < V; ++j) {                                               \
            T x;                                                                        \
            if (dtype == ORACLE_BF16) x = (T)bf16_to_f32(((const uint16_t *)row)[j]);   \
            else if (dtype == ORACLE_FP32) x = (T)((const float *)row)[j];              \
            else x = (T)((const double *)row)[j];                                       \
            if (x != x) x = NEG_INF;                                                    \
            if (bj < 0 || BEATS(x, j, bx, bj)) {                                        \
                sx = bx; sj = bj;                                                       \
                bx = x;  bj = j;                                                        \
            } else if (sj < 0 || BEATS(x, j, sx, sj)) {                                 \
                sx = x;  sj = j;                                                        \
            }                                                                           \
        }                                                                               \
        val2[0] = bx + (T)0; val2[1] = sx + (T)0; /* -0 -> +0 */                        \
        id2[0] = (int32_t)bj; id2[1] = (int32_t)sj;                                     \
    }

DEFINE_TOP2(top2_row_f32, float, beats_f32, -INFINITY)
DEFINE_TOP2(top2_row_f64, double, beats_f64, -INFINITY)

/* Eq. 4 and the "Adaptive Relaxation" condition r > theta, one IEEE division.
 * Variants (Sec. 3.3 names both as the alternatives to the logit ratio):
 *   RULE_MARGIN      Delta = z(1) - z(2) < theta, the fixed-margin indicator (Delta as in Eq. 5);
 *   RULE_PROB_RATIO  p2/p1 = exp(z(2) - z(1)) > theta, taken as Delta < (T)(-ln theta) with the
 *                    logarithm in double; theta <= 0 always relaxes. */
int mars_oracle_relax_f32(float z1, float z2, float theta, uint32_t flags)
{
    if (flags & MARS_ORACLE_RULE_PROB_RATIO) {
        double t = (double)theta;
        volatile float c = t > 0.0 ? (float)(-log(t)) : INFINITY;
        volatile float d = z1 - z2;
        return d < c;
    }
    if (flags & MARS_ORACLE_RULE_MARGIN) {
        volatile float d = z1 - z2;
        return d < theta;
    }
    int guard = (flags & MARS_ORACLE_SIGN_LITERAL) ? 1 : (z1 > 0.0f);
    volatile float r = z2 / z1;
    return guard && (r > theta);
}
int mars_oracle_relax_f64(double z1, double z2, double theta, uint32_t flags)
{
    if (flags & MARS_ORACLE_RULE_PROB_RATIO) {
        /* theta arrives as the fp32 threshold widened; the margin is rounded to fp32 as on the device */
        double c = theta > 0.0 ? (double)(float)(-log(theta)) : INFINITY;
        return (z1 - z2) < c;
    }
    if (flags & MARS_ORACLE_RULE_MARGIN) return (z1 - z2) < theta;
    int guard = (flags & MARS_ORACLE_SIGN_LITERAL) ? 1 : (z1 > 0.0);
    volatile double r = z2 / z1;
    return guard && (r > theta);
}

/* The three-way rule for one draft token against one row's top-2 (Sec. 3.4).
 * Returns 1 exact match, 2 relaxed accept, 0 reject. */
static int rule(int32_t t, const int32_t *id2, int relax)
{
    if (t < 0) return 0;
    if (t == id2[0]) return 1;
    if (t == id2[1] && relax) return 2;
    return 0;
}

/*
 * Top-2 of R rows.  Rows are independent; the loop over rows may run on several
 * host threads, the scan of a row is always the sequential one above.
 *   logits : [R, ld] of dtype (0 bf16, 1 fp32, 2 fp64); only the first V of a row are read
 *   val    : [R,2] float (dtype 0/1) or double (dtype 2);  id : [R,2]
 */
void mars_oracle_top2(const void *logits, int dtype, int64_t ld, int64_t R, int64_t V,
                      void *val, int32_t *id)
{
    size_t e = dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < R; ++r) {
        const char *row = (const char *)logits + (size_t)r * (size_t)ld * e;
        if (dtype == ORACLE_FP64) top2_row_f64(row, dtype, V, (double *)val + 2 * r, id + 2 * r);
        else top2_row_f32(row, dtype, V, (float *)val + 2 * r, id + 2 * r);
    }
}

static void fill(int32_t *p, int n, int32_t v)
{
    if (!p) return;
    for (int i = 0; i < n; ++i) p[i] = v;
}

/*
 * Tree resolve for ONE sequence from per-row top-2 records (Sec. 2.3 names the tree,
 * Sec. 3.4 / Algorithm 1 give the per-token decision and the stop at the first failure).
 *   relax[i]   : adaptive-relaxation bit of row i
 *   tok[i]     : draft token at node i (tok[0] ignored); parent[i] < i, parent[0] = -1
 *   outputs    : accept_len, out_tokens[Dcap+1], path_nodes[Dcap+1] (may be NULL),
 *                out_len, status, node_flags[N] (may be NULL)
 */
static void resolve_tree(const int32_t *id /*[N,2]*/, const uint8_t *relax, const int32_t *tok,
                         const int32_t *parent, int N, int Dcap, int32_t *accept_len,
                         int32_t *out_tokens, int32_t *path_nodes, int32_t *out_len,
                         int32_t *status, uint8_t *node_flags, int32_t *depth /*scratch[N]*/,
                         uint8_t *acc /*scratch[N]*/)
{
    int st = 0;
    if (parent[0] != -1) st = 1;
    for (int i = 1; i < N && !st; ++i)
        if (parent[i] >= i || parent[i] < -1) st = 1;

    int best = 0;
    if (!st) {
        acc[0] = 1; depth[0] = 0;
        if (node_flags) node_flags[0] = 4;
        for (int i = 1; i < N; ++i) {
            int p = parent[i];
            int how = 0;
            if (p >= 0) how = rule(tok[i], id + 2 * p, relax[p]);
            acc[i] = (uint8_t)(p >= 0 && acc[p] && how != 0);
            depth[i] = p >= 0 ? depth[p] + 1 : 0;
            if (node_flags) node_flags[i] = (uint8_t)((how == 1 ? 1 : 0) | (how == 2 ? 2 : 0) | (acc[i] ? 4 : 0));
            /* deepest accepted node; strict > keeps the lowest index among equals */
            if (acc[i] && depth[i] > depth[best]) best = i;
        }
        if (depth[best] > Dcap) st = 2;
    }
    fill(out_tokens, Dcap + 1, -1);
    fill(path_nodes, Dcap + 1, -1);
    if (st) {
        if (node_flags) { memset(node_flags, 0, (size_t)N); node_flags[0] = 4 | 8; }
        *accept_len = 0; *out_len = 1;
        out_tokens[0] = id[0];
        if (path_nodes) path_nodes[0] = 0;
        if (status) *status = st;
        return;
    }
    int a = depth[best];
    for (int n = best, d = a; d >= 0; --d, n = parent[n]) {
        if (d > 0) out_tokens[d - 1] = tok[n];
        if (path_nodes) path_nodes[d] = n;
        if (node_flags) node_flags[n] |= 8;
    }
    out_tokens[a] = id[2 * best]; /* correction token, or the bonus token at a leaf */
    *accept_len = a; *out_len = a + 1;
    if (status) *status = 0;
}

/*
 * Whole path, tree form.  logits [B*N, ld]; tok [B,N]; parent [B,N] (or [N] with
 * MARS_ORACLE_SHARED_PARENT); outputs as resolve_tree, per sequence.
 * dbg_val [B*N,2] / dbg_id [B*N,2] / node_flags [B,N] may be NULL.
 * dtype 2 (double logits) takes every decision in fp64.
 * scratch: caller-provided, B*N*(8+8+8) bytes is ample.
 */
void mars_oracle_verify_tree(const void *logits, int dtype, int64_t ld, const int32_t *tok,
                             const int32_t *parent, int B, int N, int64_t V, double theta,
                             uint32_t flags, int Dcap, int32_t *accept_len, int32_t *out_tokens,
                             int32_t *path_nodes, int32_t *out_len, int32_t *status,
                             void *dbg_val, int32_t *dbg_id, uint8_t *node_flags, void *val_buf,
                             int32_t *id_buf, uint8_t *relax_buf, int32_t *depth_buf,
                             uint8_t *acc_buf)
{
    int64_t R = (int64_t)B * N;
    mars_oracle_top2(logits, dtype, ld, R, V, val_buf, id_buf);
    for (int64_t r = 0; r < R; ++r) {
        if (dtype == ORACLE_FP64) {
            const double *v = (const double *)val_buf + 2 * r;
            relax_buf[r] = (uint8_t)mars_oracle_relax_f64(v[0], v[1], theta, flags);
            if (dbg_val) { ((double *)dbg_val)[2 * r] = v[0]; ((double *)dbg_val)[2 * r + 1] = v[1]; }
        } else {
            const float *v = (const float *)val_buf + 2 * r;
            relax_buf[r] = (uint8_t)mars_oracle_relax_f32(v[0], v[1], (float)theta, flags);
            if (dbg_val) { ((float *)dbg_val)[2 * r] = v[0]; ((float *)dbg_val)[2 * r + 1] = v[1]; }
        }
        if (dbg_id) { dbg_id[2 * r] = id_buf[2 * r]; dbg_id[2 * r + 1] = id_buf[2 * r + 1]; }
    }
    for (int b = 0; b < B; ++b) {
        const int32_t *par = (flags & MARS_ORACLE_SHARED_PARENT) ? parent : parent + (size_t)b * N;
        resolve_tree(id_buf + 2 * (size_t)b * N, relax_buf + (size_t)b * N, tok + (size_t)b * N, par,
                     N, Dcap, accept_len + b, out_tokens + (size_t)b * (Dcap + 1),
                     path_nodes ? path_nodes + (size_t)b * (Dcap + 1) : NULL, out_len + b,
                     status ? status + b : NULL, node_flags ? node_flags + (size_t)b * N : NULL,
                     depth_buf, acc_buf);
    }
}

/*
 * Whole path, chain form (the rule of Sec. 3.4 applied along a chain, as Algorithm 1 / Sec. 3.4
 * define it): K rows, K-1 drafts; row i is the target's distribution that judges draft i.
 * Stated as a definition rather than as a loop with early exit:
 *   keep[i]    = draft i, taken alone, passes the three-way rule on row i
 *   accept_len = a = the number of leading positions with keep[i] set (the first failure ends
 *                the accepted prefix, whatever comes after it)
 *   output     = draft[0..a) followed by the top-1 of row a -- the target's own choice at the
 *                first failed position, or, when a = K-1, the extra token that the last row
 *                supplies (Table 1 caption), so out_len = a + 1 <= K.
 *   draft [B,K-1]; out_tokens [B,K] padded with -1.
 */
void mars_oracle_verify_chain(const void *logits, int dtype, int64_t ld, const int32_t *draft,
                              int B, int K, int64_t V, double theta, uint32_t flags,
                              int32_t *accept_len, int32_t *out_tokens, int32_t *out_len,
                              void *dbg_val, int32_t *dbg_id, void *val_buf, int32_t *id_buf)
{
    int64_t R = (int64_t)B * K;
    mars_oracle_top2(logits, dtype, ld, R, V, val_buf, id_buf);
    if (dbg_id) memcpy(dbg_id, id_buf, (size_t)R * 2 * sizeof(int32_t));
    if (dbg_val) memcpy(dbg_val, val_buf, (size_t)R * 2 * (dtype == ORACLE_FP64 ? 8 : 4));
    for (int b = 0; b < B; ++b) {
        const int32_t *d = draft + (size_t)b * (K - 1);
        const int32_t *ids = id_buf + 2 * (size_t)b * K;
        uint8_t keep[K];                       /* K >= 1 */
        for (int i = 0; i < K - 1; ++i) {
            int64_t r = (int64_t)b * K + i;
            int relax = dtype == ORACLE_FP64
                ? mars_oracle_relax_f64(((const double *)val_buf)[2 * r], ((const double *)val_buf)[2 * r + 1], theta, flags)
                : mars_oracle_relax_f32(((const float *)val_buf)[2 * r], ((const float *)val_buf)[2 * r + 1], (float)theta, flags);
            keep[i] = (uint8_t)(rule(d[i], ids + 2 * i, relax) != 0);
        }
        int a = 0;
        while (a < K - 1 && keep[a]) ++a;
        int32_t *out = out_tokens + (size_t)b * K;
        fill(out, K, -1);
        memcpy(out, d, (size_t)a * sizeof(int32_t));
        out[a] = ids[2 * a];
        accept_len[b] = a;
        out_len[b] = a + 1;
    }
}

/*
 * Histograms of the top-2 statistics plotted in the paper's Fig. 3 (top-1 logit, logit ratio
 * z2/z1, probability ratio p2/p1 = exp(z2 - z1) by Eq. 3), from [rows, 2] fp32 top-2 values.
 * Bin rules (all fp32, one operation at a time):
 *   z1:     [lo, hi) in nbins equal bins, bin = floor((z1 - lo) * (nbins / (hi - lo)));
 *   ratio:  rows with z1 > 0 and 0 <= r <= 1, bin = min(nbins-1, floor(r * nbins));
 *   p2/p1:  bin k holds k/nbins <= p2/p1 < (k+1)/nbins, decided in the logit-difference domain:
 *           bin = #{k in 1..nbins-1 : z1 - z2 <= (float)(-ln(k/nbins))}.
 * Rows outside a histogram's range are counted in outliers[which].
 */
void mars_oracle_histograms(const float *val, int64_t rows, float lo, float hi, int nbins,
                            uint32_t *hist, uint32_t *outliers)
{
    memset(hist, 0, sizeof(uint32_t) * 3 * (size_t)nbins);
    memset(outliers, 0, sizeof(uint32_t) * 3);
    volatile float inv_w = (float)nbins / (hi - lo);
    for (int64_t r = 0; r < rows; ++r) {
        float z1 = val[2 * r], z2 = val[2 * r + 1];
        if (z1 >= lo && z1 < hi) {
            volatile float d = z1 - lo;
            volatile float t = d * inv_w;
            int b = (int)floorf(t);
            if (b < 0) b = 0;
            if (b > nbins - 1) b = nbins - 1;
            hist[b]++;
        } else outliers[0]++;
        volatile float ratio = z2 / z1;
        if (z1 > 0.0f && ratio >= 0.0f && ratio <= 1.0f) {
            volatile float t = ratio * (float)nbins;
            int b = (int)floorf(t);
            if (b > nbins - 1) b = nbins - 1;
            hist[nbins + b]++;
        } else outliers[1]++;
        volatile float delta = z1 - z2;
        if (delta >= 0.0f) {
            int b = 0;
            for (int k = 1; k < nbins; ++k) {
                float e = (float)(-log((double)k / (double)nbins));
                if (delta <= e) b++;
            }
            hist[2 * nbins + b]++;
        } else outliers[2]++;
    }
}

/*
 * Exact top-k of each row under the total order (value descending, token id ascending, NaN as
 * -inf): one sequential pass per row keeping a sorted list of the k best so far.  Used for the
 * draft-tree expansion with the k best continuations (the paper's setup: top-k = 10, Sec. 4.1).
 *   val [R,k] (float for dtype 0/1, double for 2), id [R,k], best first.
 */
void mars_oracle_topk(const void *logits, int dtype, int64_t ld, int64_t R, int64_t V, int k,
                      void *val, int32_t *id)
{
    size_t e = dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < R; ++r) {
        const char *row = (const char *)logits + (size_t)r * (size_t)ld * e;
        double bx[64];
        int64_t bj[64];
        int n = 0;
        for (int64_t j = 0; j < V; ++j) {
            double x;
            if (dtype == ORACLE_BF16) x = (double)bf16_to_f32(((const uint16_t *)row)[j]);
            else if (dtype == ORACLE_FP32) x = (double)((const float *)row)[j];
            else x = ((const double *)row)[j];
            if (x != x) x = -INFINITY;
            /* position of (x, j) in the sorted list: behind everything that beats it */
            int pos = n;
            while (pos > 0 && beats_f64(x, j, bx[pos - 1], bj[pos - 1])) --pos;
            if (pos >= k) continue;
            int last = n < k ? n : k - 1;
            for (int t = last; t > pos; --t) { bx[t] = bx[t - 1]; bj[t] = bj[t - 1]; }
            bx[pos] = x; bj[pos] = j;
            if (n < k) ++n;
        }
        for (int t = 0; t < k; ++t) {
            if (dtype == ORACLE_FP64) ((double *)val)[r * k + t] = bx[t] + 0.0;
            else ((float *)val)[r * k + t] = (float)bx[t] + 0.0f;
            id[r * k + t] = (int32_t)bj[t];
        }
    }
}

/* ======================================================================================
 * Stochastic (temperature T > 0) verification.
 *
 * What the paper fixes (Sec. 2.2): in stochastic decoding a drafted token is accepted with
 * probability min(1, P_target / P_draft) (Eq. 1); on rejection the corrected token is drawn
 * from a residual distribution that compensates for the draft; tree-based methods extend the
 * same logic to a token tree; the target probabilities are the softmax of the logits (Eq. 3).
 * Sec. 2.2 also says that MARS changes only the accept/reject decision and applies on top of
 * sampling-based verification, and Sec. 4.1 that draft trees are built from the drafter's k
 * best continuations.  HOW the relaxation composes with Eq. 1 is not stated anywhere.
 *
 * Reading taken here (a convention of this repository; the composition is PARITY UNPINNED by
 * the paper, the pieces are pinned, see below):
 *   - P(v) = exp(z_v / T) / sum_u exp(z_u / T) per row, evaluated in fp64 as
 *     exp((z_v - m) / T) with m the row maximum (the same number); NaN logits count as -inf.
 *   - Candidates are deterministic (a top-k expansion), so the draft distribution at a node is
 *     a point mass on the candidate and Eq. 1 reads "accept x with probability P(x)".  The
 *     children of the current node are tried in node order.  When child x is rejected, the
 *     target distribution is replaced by its residual, which for a point-mass draft is P with
 *     x removed and renormalised; the next sibling is judged against that residual, i.e. it
 *     is accepted iff u * rem < e_x, where e_x is x's unnormalised mass, rem the mass that is
 *     left, and u the node's uniform in [0, 1).  If no child is accepted the walk stops
 *     and the next token is drawn from the residual by inverting its CDF in token-id order with
 *     the sequence's uniform uniform[b, 0]: the smallest id j with sum_{k <= j} w_k > u * W.
 *     At a leaf nothing was removed and the draw is from P itself (the bonus token).
 *   - Composition with MARS (flags): by default a child that passes the three-way rule of
 *     Sec. 3.4 on the current row (exact match, or runner-up with r > theta) is accepted
 *     outright, and only the others take the Eq. 1 test; STOCH_RELAX_ONLY keeps Eq. 1 for the
 *     top-1 as well and adds only the relaxed runner-up; STOCH_PLAIN is Eq. 1 alone (standard
 *     speculative sampling, which preserves the target distribution exactly).
 *   - A row whose maximum is not finite, or a residual without mass, has no distribution to
 *     draw from: the walk stops there, the row's top-1 is emitted and the status is 4.
 *   Pinned by tests: softmax against a library routine; CDF inversion against cumsum +
 *   searchsorted; exact preservation of the target distribution for the first and second
 *   emitted token in STOCH_PLAIN (the theorem behind Eq. 1); T -> 0 equals strict greedy;
 *   u -> 1 in the default mode equals Algorithm 1 on chains; invariance under scaling logits
 *   and T by a power of two.
 * ==================================================================================== */
#define MARS_ORACLE_STOCH_PLAIN 32u
#define MARS_ORACLE_STOCH_RELAX_ONLY 64u

static double row_get(const void *row, int dtype, int64_t j)
{
    double x;
    if (dtype == ORACLE_BF16) x = (double)bf16_to_f32(((const uint16_t *)row)[j]);
    else if (dtype == ORACLE_FP32) x = (double)((const float *)row)[j];
    else x = ((const double *)row)[j];
    return (x != x) ? -INFINITY : x;
}

/* Row maximum and softmax denominator sum_j exp((z_j - m)/T) (Eq. 3 with temperature). */
static void row_softmax_stats(const void *row, int dtype, int64_t V, double T, double *m_out,
                              double *S_out)
{
    double m = -INFINITY;
    for (int64_t j = 0; j < V; ++j) { double x = row_get(row, dtype, j); if (x > m) m = x; }
    double S = 0.0;
    if (isfinite(m))
        for (int64_t j = 0; j < V; ++j) S += exp((row_get(row, dtype, j) - m) / T);
    *m_out = m;
    *S_out = S;
}

/*
 *   uniform   float [B,N]: uniform[b,i] (i > 0) judges node i; uniform[b,0] draws the final token
 *   node_prob double [B,N] or NULL: P(tok[i]) under the PARENT's row (plain softmax, nothing removed);
 *             0 for the root, padding nodes and ids outside [0,V)
 *   node_how  uint8 [B,N] or NULL: 0 not visited, 1 exact match, 2 relaxed runner-up, 3 accepted by
 *             Eq. 1, 4 rejected
 *   margin    double [B,2] or NULL: [0] the smallest |e_x - u*rem| / S over the Eq. 1 tests taken,
 *             [1] the distance of u*W from the nearer edge of the drawn token's CDF interval, / W
 *             (how close each decision was to flipping; +inf where no such decision was taken)
 */
void mars_oracle_verify_tree_stochastic(const void *logits, int dtype, int64_t ld, const int32_t *tok,
                                        const int32_t *parent, const float *uniform, int B, int N,
                                        int64_t V, double theta, double temperature, uint32_t flags,
                                        int Dcap, int32_t *accept_len, int32_t *out_tokens,
                                        int32_t *path_nodes, int32_t *out_len, int32_t *status,
                                        double *node_prob, uint8_t *node_how, double *margin)
{
    size_t e = dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8;
    const double T = temperature;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int32_t *par = (flags & MARS_ORACLE_SHARED_PARENT) ? parent : parent + (size_t)b * N;
        const int32_t *tk = tok + (size_t)b * N;
        const float *u = uniform + (size_t)b * N;
        int32_t *otok = out_tokens + (size_t)b * (Dcap + 1);
        int32_t *opath = path_nodes ? path_nodes + (size_t)b * (Dcap + 1) : NULL;
        double *nprob = node_prob ? node_prob + (size_t)b * N : NULL;
        uint8_t *nhow = node_how ? node_how + (size_t)b * N : NULL;
        double mg_test = INFINITY, mg_draw = INFINITY;
        fill(otok, Dcap + 1, -1);
        fill(opath, Dcap + 1, -1);
        if (nhow) memset(nhow, 0, (size_t)N);
        if (nprob) for (int i = 0; i < N; ++i) nprob[i] = 0.0;

        int st = 0;
        if (par[0] != -1) st = 1;
        for (int i = 1; i < N && !st; ++i)
            if (par[i] >= i || par[i] < -1) st = 1;

        /* plain softmax probability of every node's token under its parent's row */
        if (nprob && !st) {
            for (int i = 1; i < N; ++i) {
                int p = par[i];
                if (p < 0 || tk[i] < 0 || tk[i] >= V) continue;
                const char *row = (const char *)logits + ((size_t)b * N + p) * (size_t)ld * e;
                double m, S;
                row_softmax_stats(row, dtype, V, T, &m, &S);
                if (isfinite(m) && S > 0.0) nprob[i] = exp((row_get(row, dtype, tk[i]) - m) / T) / S;
            }
        }

        int cur = 0, a = 0, bad_dist = 0;
        int32_t removed[1024];
        int nrem = 0;
        float v2[2];
        int32_t id2[2] = {0, 1};
        double m = 0, S = 0;
        const char *row = NULL;
        if (opath) opath[0] = 0;
        while (!st) {
            row = (const char *)logits + ((size_t)b * N + cur) * (size_t)ld * e;
            top2_row_f32(row, dtype, V, v2, id2);
            int relax = mars_oracle_relax_f32(v2[0], v2[1], (float)theta, flags);
            row_softmax_stats(row, dtype, V, T, &m, &S);
            nrem = 0;
            if (!isfinite(m) || !(S > 0.0)) { bad_dist = 1; break; }
            double rem = S;
            int next = -1;
            for (int i = cur + 1; i < N && next < 0; ++i) {
                if (par[i] != cur || tk[i] < 0) continue;
                int32_t x = tk[i];
                int gone = 0;
                for (int k = 0; k < nrem; ++k) if (removed[k] == x) gone = 1;
                double ex = (x < V && !gone) ? exp((row_get(row, dtype, x) - m) / T) : 0.0;
                int how = (flags & MARS_ORACLE_STOCH_PLAIN) ? 0 : rule(x, id2, relax);
                if ((flags & MARS_ORACLE_STOCH_RELAX_ONLY) && how == 1) how = 0;
                if (how == 0) {
                    double lhs = (double)u[i] * rem;          /* Eq. 1 on the running residual */
                    double d = fabs(ex - lhs) / S;
                    if (d < mg_test) mg_test = d;
                    how = (lhs < ex) ? 3 : 4;
                }
                if (nhow) nhow[i] = (uint8_t)how;
                if (how == 4) {
                    if (ex > 0.0 && nrem < 1024) {
                        rem -= ex; if (rem < 0.0) rem = 0.0;
                        removed[nrem++] = x;
                    }
                } else next = i;
            }
            if (next < 0) break;
            cur = next; ++a;
            if (a <= Dcap) { otok[a - 1] = tk[cur]; if (opath) opath[a] = cur; }
        }
        if (!st && a > Dcap) st = 2;
        if (st) {   /* malformed tree or path deeper than the outputs: accept nothing, emit the root's top-1 */
            fill(otok, Dcap + 1, -1);
            fill(opath, Dcap + 1, -1);
            if (nhow) memset(nhow, 0, (size_t)N);
            row = (const char *)logits + ((size_t)b * N) * (size_t)ld * e;
            top2_row_f32(row, dtype, V, v2, id2);
            accept_len[b] = 0; out_len[b] = 1; otok[0] = id2[0];
            if (opath) opath[0] = 0;
            if (status) status[b] = st;
            if (margin) { margin[2 * b] = INFINITY; margin[2 * b + 1] = INFINITY; }
            continue;
        }
        /* the next token: a draw from the residual of row `cur` (nothing removed at a leaf) */
        int32_t drawn = id2[0];
        if (!bad_dist) {
            double W = 0.0;
            for (int64_t j = 0; j < V; ++j) {
                int gone = 0;
                for (int k = 0; k < nrem; ++k) if (removed[k] == j) gone = 1;
                if (!gone) W += exp((row_get(row, dtype, j) - m) / T);
            }
            if (!(W > 0.0)) bad_dist = 1;
            else {
                double target = (double)u[0] * W, c = 0.0, lo = 0.0;
                int64_t pick = -1, last = -1;
                for (int64_t j = 0; j < V && pick < 0; ++j) {
                    int gone = 0;
                    for (int k = 0; k < nrem; ++k) if (removed[k] == j) gone = 1;
                    double w = gone ? 0.0 : exp((row_get(row, dtype, j) - m) / T);
                    if (w > 0.0) last = j;
                    lo = c;
                    c += w;
                    if (c > target) pick = j;
                }
                if (pick < 0) { pick = last; }
                drawn = (int32_t)pick;
                double d0 = (target - lo) / W, d1 = (c - target) / W;
                mg_draw = d0 < d1 ? d0 : d1;
            }
        }
        otok[a] = drawn;
        accept_len[b] = a; out_len[b] = a + 1;
        if (status) status[b] = bad_dist ? 4 : 0;
        if (margin) { margin[2 * b] = mg_test; margin[2 * b + 1] = mg_draw; }
    }
}

/* ======================================================================================
 * Stochastic verification of chains whose drafts were SAMPLED from a drafter's distribution:
 * Eq. 1 in its general form (Sec. 2.2).  Draft i was drawn from Q_i = softmax(zq_i / Tq) with
 * probability qx_i = Q_i(draft_i), supplied by the caller.  It is accepted with probability
 * min(1, P_i(x) / Q_i(x)), i.e. iff u_i * Q_i(x) < P_i(x) for the position's uniform u_i (for a
 * ratio of one or more this always holds since u_i < 1).  The first rejected position emits a
 * token drawn from the residual distribution, which "compensates for the draft's approximation
 * error": norm(max(0, P_i - Q_i)), by CDF inversion in token-id order with uniform[b, 0].  If
 * every draft is accepted the bonus token is drawn from P of the last row.  The composition with
 * the relaxation follows the same three modes as the tree form above (a reading of this
 * repository; PARITY UNPINNED by the paper).  With STOCH_PLAIN this is standard speculative
 * sampling, which leaves the target distribution unchanged -- the pin for this function.
 *   logits  [B*K, ld]   target rows;  qlogits [B*(K-1), ldq] drafter rows (dtype_q);
 *   draft   [B, K-1] (a negative id ends the chain: no draft there, the token is drawn from P);
 *   qx      [B, K-1] float: probability with which the drafter drew the token;
 *   uniform [B, K]:     [b, i+1] judges draft i, [b, 0] draws the emitted token;
 *   node_how [B, K] as in the tree form (index i+1 for draft i); margin [B, 2] as there, with the
 *   draw margin in units of total probability (not of the residual's mass).
 *   Status 4: a row on the way has no softmax (target or drafter), or the residual has no mass.
 * ==================================================================================== */
void mars_oracle_verify_chain_sampled(const void *logits, int dtype, int64_t ld, const void *qlogits,
                                      int dtype_q, int64_t ldq, const int32_t *draft, const float *qx,
                                      const float *uniform, int B, int K, int64_t V, double theta,
                                      double temperature, double draft_temperature, uint32_t flags,
                                      int32_t *accept_len, int32_t *out_tokens, int32_t *out_len,
                                      int32_t *status, double *node_prob, uint8_t *node_how, double *margin)
{
    size_t e = dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8;
    size_t eq = dtype_q == ORACLE_BF16 ? 2 : dtype_q == ORACLE_FP32 ? 4 : 8;
    const double T = temperature, Tq = draft_temperature;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const float *u = uniform + (size_t)b * K;
        int32_t *otok = out_tokens + (size_t)b * K;
        uint8_t *nhow = node_how ? node_how + (size_t)b * K : NULL;
        double *nprob = node_prob ? node_prob + (size_t)b * K : NULL;
        double mg_test = INFINITY, mg_draw = INFINITY;
        fill(otok, K, -1);
        for (int i = 0; i < K; ++i) { if (nhow) nhow[i] = 0; if (nprob) nprob[i] = 0.0; }
        int a = 0, st = 0, rejected_at = -1;
        float v2[2];
        int32_t id2[2] = {0, 1};
        double m = 0, S = 0;
        const char *row = NULL;
        /* plain softmax probability of every draft under its row (reported, not part of the walk) */
        for (int i = 0; nprob && i < K - 1; ++i) {
            int32_t x = draft[(size_t)b * (K - 1) + i];
            row = (const char *)logits + ((size_t)b * K + i) * (size_t)ld * e;
            row_softmax_stats(row, dtype, V, T, &m, &S);
            if (x >= 0 && x < V && isfinite(m) && S > 0.0) nprob[i + 1] = exp((row_get(row, dtype, x) - m) / T) / S;
        }
        for (int i = 0; i < K; ++i) {       /* row i judges draft i; row K-1 only supplies the bonus */
            row = (const char *)logits + ((size_t)b * K + i) * (size_t)ld * e;
            top2_row_f32(row, dtype, V, v2, id2);
            row_softmax_stats(row, dtype, V, T, &m, &S);
            if (!isfinite(m) || !(S > 0.0)) { st = 4; break; }
            if (i == K - 1) break;
            int32_t x = draft[(size_t)b * (K - 1) + i];
            if (x < 0) break;                /* no draft here (padding): the chain ends, draw from P_i */
            double px = (x < V) ? exp((row_get(row, dtype, x) - m) / T) / S : 0.0;
            int relax = mars_oracle_relax_f32(v2[0], v2[1], (float)theta, flags);
            int how = (flags & MARS_ORACLE_STOCH_PLAIN) ? 0 : rule(x, id2, relax);
            if ((flags & MARS_ORACLE_STOCH_RELAX_ONLY) && how == 1) how = 0;
            if (how == 0) {
                double lhs = (double)u[i + 1] * (double)qx[(size_t)b * (K - 1) + i];   /* Eq. 1 */
                double d = fabs(px - lhs);
                if (d < mg_test) mg_test = d;
                how = (lhs < px) ? 3 : 4;
            }
            if (nhow) nhow[i + 1] = (uint8_t)how;
            if (how == 4) { rejected_at = i; break; }
            otok[a++] = x;
        }
        int32_t drawn = id2[0];
        if (st == 0) {
            /* weights of the distribution to draw from, in token-id order */
            const char *qrow = NULL;
            double mq = 0, Sq = 0;
            if (rejected_at >= 0) {
                qrow = (const char *)qlogits + ((size_t)b * (K - 1) + rejected_at) * (size_t)ldq * eq;
                row_softmax_stats(qrow, dtype_q, V, Tq, &mq, &Sq);
                if (!isfinite(mq) || !(Sq > 0.0)) st = 4;
            }
            if (st == 0) {
                double W = 0.0;
                for (int64_t j = 0; j < V; ++j) {
                    double w = exp((row_get(row, dtype, j) - m) / T) / S;
                    if (qrow) { w -= exp((row_get(qrow, dtype_q, j) - mq) / Tq) / Sq; if (w < 0.0) w = 0.0; }
                    W += w;
                }
                if (!(W > 0.0)) st = 4;
                else {
                    double target = (double)u[0] * W, c = 0.0, lo = 0.0;
                    int64_t pick = -1, last = -1;
                    for (int64_t j = 0; j < V && pick < 0; ++j) {
                        double w = exp((row_get(row, dtype, j) - m) / T) / S;
                        if (qrow) { w -= exp((row_get(qrow, dtype_q, j) - mq) / Tq) / Sq; if (w < 0.0) w = 0.0; }
                        if (w > 0.0) last = j;
                        lo = c;
                        c += w;
                        if (c > target) pick = j;
                    }
                    if (pick < 0) pick = last;
                    drawn = (int32_t)pick;
                    double d0 = target - lo, d1 = c - target;
                    mg_draw = d0 < d1 ? d0 : d1;
                }
            }
        }
        otok[a] = drawn;
        accept_len[b] = a; out_len[b] = a + 1;
        if (status) status[b] = st;
        if (margin) { margin[2 * b] = mg_test; margin[2 * b + 1] = mg_draw; }
    }
}
