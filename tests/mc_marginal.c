/*
 * Monte-Carlo driver for the oracle's stochastic acceptance (test code, CPU only).
 *
 * For each draw it builds a fresh one- or two-level tree whose children are sampled
 * WITHOUT replacement from the draft distribution of their parent (for such drafts
 * sibling-sequential rejection sampling reproduces the target distribution exactly),
 * runs the oracle's accept routine with fresh uniforms, and histograms
 *   hist1[v]       first emitted token,
 *   hist2[j][v]    second emitted token given that depth-1 slot j was accepted,
 *   hist_len[l]    acceptance length.
 * The caller compares them with softmax(target / T) computed independently.
 *
 * Rows: target_logits[1 + n1][V] (row 0 = root, row j = depth-1 slot j; deeper nodes reuse row 0),
 *       draft_logits [1 + n1][V] (row 0 proposes the root's children, row j those of slot j).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

int radar_oracle_accept_stochastic(int V, int n_nodes, int t_max, const int* tok, const int* parent,
                                   const float* target_logits, const float* draft_logits,
                                   const int* node_to_draft_row, const float* u_accept, float u_sample,
                                   double temperature, int* accept_len, int* path_nodes, int* path_tokens,
                                   int* next_token, double* accept_margin, double* sample_margin);

static uint64_t splitmix(uint64_t* s) {
    uint64_t z = (*s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static float uni(uint64_t* s) { return (float)(splitmix(s) >> 40) * (1.0f / 16777216.0f); }

/* n distinct tokens drawn one after the other from softmax(z/T), each removed after it is drawn */
static void draw_without_replacement(const float* z, int V, double T, int n, int* out, uint64_t* s) {
    double w[64];
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) if (z[v] / T > m) m = z[v] / T;
    for (int v = 0; v < V; ++v) w[v] = exp(z[v] / T - m);
    for (int i = 0; i < n; ++i) {
        double tot = 0.0;
        for (int v = 0; v < V; ++v) tot += w[v];
        double u = (double)uni(s) * tot, run = 0.0;
        int pick = -1;
        for (int v = 0; v < V; ++v) { run += w[v]; if (w[v] > 0.0 && run > u) { pick = v; break; } }
        if (pick < 0) for (int v = V - 1; v >= 0; --v) if (w[v] > 0.0) { pick = v; break; }
        out[i] = pick;
        w[pick] = 0.0;
    }
}

int mc_marginal(int V, int n1, int n2, double T, long draws, uint64_t seed,
                const float* target_rows, const float* draft_rows,
                long* hist1, long* hist2, long* hist_len) {
    if (V > 64 || n1 > 8 || n2 > 8) return -1;
    uint64_t s = seed;
    int n_nodes = 1 + n1 + n1 * n2;
    int tok[1 + 8 + 64], parent[1 + 8 + 64], drow[1 + 8 + 64];
    float uacc[1 + 8 + 64];
    float* tl = (float*)malloc(sizeof(float) * (size_t)n_nodes * V);
    if (!tl) return -1;
    for (int i = 0; i < n_nodes; ++i)                       /* node i's target row */
        memcpy(tl + (size_t)i * V, target_rows + (size_t)(i <= n1 ? i : 0) * V, sizeof(float) * V);
    memset(hist1, 0, sizeof(long) * V);
    memset(hist2, 0, sizeof(long) * n1 * V);
    memset(hist_len, 0, sizeof(long) * 3);
    for (long it = 0; it < draws; ++it) {
        tok[0] = 0; parent[0] = -1; drow[0] = 0;
        draw_without_replacement(draft_rows, V, T, n1, tok + 1, &s);
        for (int j = 1; j <= n1; ++j) { parent[j] = 0; drow[j] = n2 > 0 ? j : -1; }
        for (int j = 1; j <= n1; ++j) {
            int base = 1 + n1 + (j - 1) * n2;
            draw_without_replacement(draft_rows + (size_t)j * V, V, T, n2, tok + base, &s);
            for (int c = 0; c < n2; ++c) { parent[base + c] = j; drow[base + c] = -1; }
        }
        for (int i = 0; i < n_nodes; ++i) uacc[i] = uni(&s);
        float us = uni(&s);
        int alen, nxt, pn[3], pt[3];
        if (radar_oracle_accept_stochastic(V, n_nodes, 2, tok, parent, tl, draft_rows, drow, uacc, us, T,
                                           &alen, pn, pt, &nxt, 0, 0) != 0) { free(tl); return -2; }
        hist_len[alen]++;
        int first = alen >= 1 ? pt[1] : nxt;
        hist1[first]++;
        if (alen >= 1) {
            int slot = pn[1] - 1;
            int second = alen >= 2 ? pt[2] : nxt;
            hist2[(size_t)slot * V + second]++;
        }
    }
    free(tl);
    return 0;
}

/* Fixed tree, fresh uniforms per draw: histogram of the acceptance length (for Eq. 11-13). */
int mc_fixed_tree(int V, int n_nodes, int t_max, const int* tok, const int* parent, const int* drow,
                  const float* target_logits, const float* draft_logits, double T, long draws, uint64_t seed,
                  long* hist_len) {
    if (n_nodes > 64 || t_max > 15) return -1;
    uint64_t s = seed;
    float uacc[64];
    int pn[16], pt[16], alen, nxt;
    memset(hist_len, 0, sizeof(long) * (size_t)(t_max + 1));
    for (long it = 0; it < draws; ++it) {
        for (int i = 0; i < n_nodes; ++i) uacc[i] = uni(&s);
        float us = uni(&s);
        if (radar_oracle_accept_stochastic(V, n_nodes, t_max, tok, parent, target_logits, draft_logits, drow,
                                           uacc, us, T, &alen, pn, pt, &nxt, 0, 0) != 0) return -2;
        hist_len[alen]++;
    }
    return 0;
}
