/*
 * Plain C, fp64 oracle of RADAR's stochastic tree acceptance and of the
 * acceptance-length distribution.  TEST INFRASTRUCTURE ONLY: the product path
 * never links or calls this file.
 *
 * Written from the paper's definitions:
 *   - single-draft acceptance probability min(1, p/q)           (Sec. 3, Eq. 1)
 *   - rectified distribution norm(max(0, p - q)) after a reject (Sec. 3, Eq. 2)
 *   - bonus token from the target distribution when a path ends (Sec. 3)
 *   - siblings are tried one after the other; "all children rejected" has
 *     probability 1 - sum_j P_acc(l_j | v_1)                    (Sec. 4.3, Eq. 13)
 *   - P_stop(v_1) = P_acc(v_0) P_acc(v_1|v_0) P_rej(l|v_1), p_i = sum over
 *     depth-i nodes of P_stop                                    (Sec. 4.3, Eq. 11-12)
 *
 * Tree layout: node 0 is the root; parent[i] < i; the children of a node are
 * tried in ascending node index.  Logits are float32 rows; everything else is
 * double.  No blocking, no fusion: each step is the formula written out.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* p <- softmax(z / T) in fp64 */
static void softmax_row(const float* z, int V, double T, double* p) {
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) { double x = (double)z[v] / T; if (x > m) m = x; }
    double s = 0.0;
    for (int v = 0; v < V; ++v) { p[v] = exp((double)z[v] / T - m); s += p[v]; }
    for (int v = 0; v < V; ++v) p[v] /= s;
}

/* inverse-CDF draw in vocabulary order: smallest v with sum_{v'<=v} w > u * sum w.
 * margin = distance (relative to the total) of u*total from the nearest CDF step edge. */
static int sample_cdf(const double* w, int V, double u, double* margin) {
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += w[v];
    double target = u * total, run = 0.0, prev = 0.0;
    int last_pos = -1;
    for (int v = 0; v < V; ++v) {
        prev = run;
        run += w[v];
        if (w[v] > 0.0) last_pos = v;
        if (run > target) {
            if (margin) { double a = run - target, b = target - prev; *margin = (a < b ? a : b) / total; }
            return v;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/* Eq. 2: p <- norm(max(0, p - q)); returns the un-normalised residual mass.
 * If the mass is zero (p <= q everywhere) p is left as it is. */
static double rectify(double* p, const double* q, int V) {
    double s = 0.0;
    for (int v = 0; v < V; ++v) { double r = p[v] - q[v]; s += r > 0.0 ? r : 0.0; }
    if (s > 0.0)
        for (int v = 0; v < V; ++v) { double r = p[v] - q[v]; p[v] = (r > 0.0 ? r : 0.0) / s; }
    return s;
}

/* remove token x from q and renormalise; returns the remaining mass before renormalising */
static double remove_token(double* q, int V, int x) {
    q[x] = 0.0;
    double s = 0.0;
    for (int v = 0; v < V; ++v) s += q[v];
    if (s > 0.0) for (int v = 0; v < V; ++v) q[v] /= s;
    return s;
}

/*
 * One sequence.  target_logits [n_nodes][V], draft_logits [R][V],
 * node_to_draft_row[i] = row of draft_logits whose distribution produced i's children
 * (unused for nodes without children), u_accept[i] = uniform used when node i is tried,
 * u_sample = uniform for the final draw.  Outputs: accept_len (accepted draft nodes),
 * path_nodes/path_tokens [t_max+1] (-1 padded, entry 0 = root), next_token.
 * accept_margin = min over tests of |u - p/q| (inf when the ratio is >= 1 or q = 0),
 * sample_margin as in sample_cdf.  Returns 0, or -1 on bad arguments / allocation failure.
 */
int radar_oracle_accept_stochastic(int V, int n_nodes, int t_max,
                                   const int* tok, const int* parent,
                                   const float* target_logits, const float* draft_logits,
                                   const int* node_to_draft_row,
                                   const float* u_accept, float u_sample, double temperature,
                                   int* accept_len, int* path_nodes, int* path_tokens, int* next_token,
                                   double* accept_margin, double* sample_margin) {
    if (V <= 0 || n_nodes <= 0 || temperature <= 0.0) return -1;
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    if (!p || !q) { free(p); free(q); return -1; }
    for (int d = 0; d <= t_max; ++d) { path_nodes[d] = -1; path_tokens[d] = -1; }
    int cur = 0, len = 0;
    path_nodes[0] = 0; path_tokens[0] = tok[0];
    double amargin = INFINITY;
    for (;;) {
        softmax_row(target_logits + (size_t)cur * V, V, temperature, p);
        int nchild = 0;
        for (int j = cur + 1; j < n_nodes; ++j) if (parent[j] == cur) ++nchild;
        if (nchild == 0 || len >= t_max) break;            /* bonus token from the target distribution */
        softmax_row(draft_logits + (size_t)node_to_draft_row[cur] * V, V, temperature, q);
        int accepted = -1;
        for (int j = cur + 1; j < n_nodes; ++j) {
            if (parent[j] != cur) continue;
            int x = tok[j];
            int acc;
            if (q[x] <= 0.0) {
                acc = p[x] > 0.0;                            /* ratio is +inf */
            } else {
                double ratio = p[x] / q[x];                  /* Eq. 1 */
                double a = ratio < 1.0 ? ratio : 1.0;
                acc = (double)u_accept[j] < a;
                if (ratio < 1.0) { double g = fabs((double)u_accept[j] - ratio); if (g < amargin) amargin = g; }
            }
            if (acc) { accepted = j; break; }
            rectify(p, q, V);                                /* Eq. 2 */
            if (remove_token(q, V, x) <= 0.0) break;         /* nothing left to propose */
        }
        if (accepted < 0) break;                             /* every child rejected: sample the residual */
        cur = accepted; ++len;
        path_nodes[len] = cur; path_tokens[len] = tok[cur];
    }
    *next_token = sample_cdf(p, V, (double)u_sample, sample_margin);
    *accept_len = len;
    if (accept_margin) *accept_margin = amargin;
    free(p); free(q);
    return 0;
}

/*
 * Acceptance-length distribution of a verified tree (Sec. 4.3, Eq. 11-13).
 * For node c with children l_1..l_n tried in order, P_acc(l_j | c) is the probability
 * that the first j-1 are rejected and l_j accepted; P_rej = 1 - sum_j P_acc(l_j | c);
 * P_acc(node) is the product along its path; P_stop(c) = P_acc(c) * P_rej(c).
 * dist[0..t_max] receives p_i; p_acc_node [n_nodes] (optional) receives P_acc of each node.
 */
int radar_oracle_accept_length_distribution(int V, int n_nodes, int t_max,
                                            const int* tok, const int* parent, const int* depth,
                                            const float* target_logits, const float* draft_logits,
                                            const int* node_to_draft_row, double temperature,
                                            double* dist, double* p_acc_node) {
    if (V <= 0 || n_nodes <= 0 || temperature <= 0.0) return -1;
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    double* pacc = (double*)malloc(sizeof(double) * (size_t)n_nodes);
    if (!p || !q || !pacc) { free(p); free(q); free(pacc); return -1; }
    for (int d = 0; d <= t_max; ++d) dist[d] = 0.0;
    pacc[0] = 1.0;
    for (int c = 0; c < n_nodes; ++c) {                      /* parents precede children */
        int nchild = 0;
        for (int j = c + 1; j < n_nodes; ++j) if (parent[j] == c) ++nchild;
        double sum_acc = 0.0;
        if (nchild > 0) {
            softmax_row(target_logits + (size_t)c * V, V, temperature, p);
            softmax_row(draft_logits + (size_t)node_to_draft_row[c] * V, V, temperature, q);
            double reach = 1.0;                              /* probability that every earlier sibling was rejected */
            int exhausted = 0;
            for (int j = c + 1; j < n_nodes; ++j) {
                if (parent[j] != c) continue;
                if (exhausted) { pacc[j] = 0.0; continue; }
                int x = tok[j];
                double a;
                if (q[x] <= 0.0) a = p[x] > 0.0 ? 1.0 : 0.0;
                else { a = p[x] / q[x]; if (a > 1.0) a = 1.0; }
                double pj = reach * a;                       /* P_acc(l_j | c) */
                pacc[j] = pacc[c] * pj;
                sum_acc += pj;
                reach *= (1.0 - a);
                rectify(p, q, V);
                if (remove_token(q, V, x) <= 0.0) exhausted = 1;
            }
        }
        dist[depth[c]] += pacc[c] * (1.0 - sum_acc);         /* P_stop(c) */
    }
    if (p_acc_node) memcpy(p_acc_node, pacc, sizeof(double) * (size_t)n_nodes);
    free(p); free(q); free(pacc);
    return 0;
}
