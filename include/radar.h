/*
 * radar.h - C ABI of the B200 (sm_100a) hot path of one RADAR speculative step.
 *
 * The four calls are the data-parallel stages of one speculative step as the paper
 * states it (Sec. 4.1 "Inference Pipeline" and the appendix walkthrough): draft-tree
 * expansion with the continue/stop prediction model, rerank + serialisation of the tree,
 * tree-masked verification attention, and acceptance.
 *
 * Conventions for every call
 *   - Returns an int status (0 = RADAR_OK, negative = error).  Host-detectable errors
 *     (NULL pointers, unsupported sizes, workspace too small) are returned at once and
 *     nothing is launched.  Errors only the device can see (NaN logits, a pool that is not
 *     ancestor-closed, a wait that ran out) are recorded in a sticky device status word
 *     that radar_read_device_status() returns; kernels never trap.
 *   - Every pointer in an argument struct is a DEVICE pointer owned by the caller unless
 *     its comment says "host".  The library keeps no reference after the call returns.
 *   - Calls are asynchronous on the given CUDA stream (passed as void*, 0 = default stream),
 *     perform no host synchronisation and allocate nothing; scratch memory is the caller's
 *     `workspace` (size from the matching *_workspace_bytes function, 256-byte aligned).
 *   - Outputs are fully overwritten for every processed sequence; padding entries are
 *     written as documented.  Inputs are never modified except the documented in/out state.
 *   - Tree rows: row 0 is the root (the last committed token), rows 1..n_nodes-1 the kept
 *     draft nodes; at most RADAR_MAX_NODES rows so that an ancestor set is one 64-bit word.
 */
#ifndef RADAR_H
#define RADAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RADAR_MAX_NODES 64      /* tree rows incl. root */
#define RADAR_GATE_HIDDEN 128   /* LSTM / MLP hidden size of the prediction model (App. "Implementation Details") */
#define RADAR_MAX_K 32          /* branching factor limit */
#define RADAR_MAX_POOL 8192     /* pool capacity limit for radar_rerank_build_tree */

enum {
    RADAR_OK = 0,
    RADAR_ERR_INVALID_ARG = -1,
    RADAR_ERR_UNSUPPORTED = -2,
    RADAR_ERR_WORKSPACE = -3,
    RADAR_ERR_CUDA = -4,
    RADAR_ERR_TIMEOUT = -5,
    RADAR_ERR_NUMERIC = -6,
    RADAR_ERR_TREE = -7
};

enum { RADAR_F32 = 0, RADAR_BF16 = 1 };
enum { RADAR_GREEDY = 0, RADAR_STOCHASTIC = 1 };

typedef struct radar_ctx radar_ctx;

/* Context: remembers the device, its SM count and owns the 4-byte device status word
 * (the only allocation the library ever makes).  `out` is a host pointer.  A context belongs to one
 * device and is used by one host thread at a time; make one per device. */
int radar_create(radar_ctx** out, int device);
int radar_destroy(radar_ctx* ctx);
const char* radar_status_string(int status);
/* Synchronises `stream`, returns the sticky device status (RADAR_OK or the first device-side
 * error recorded since the last read) and clears it. */
int radar_read_device_status(radar_ctx* ctx, void* stream);

/* Measurement helpers (no counterpart in the paper): host-side launch counts per kernel and,
 * between radar_profile_begin and radar_profile_end, a CUDA-event pair around every kernel the
 * library launches (on the launching stream).  radar_profile_begin creates 2 * max_records events;
 * radar_profile_end synchronises the device, accumulates the durations and destroys the events.
 * Do not profile inside a stream capture.  radar_kernel_stats: all out-pointers are host, optional. */
int radar_profile_begin(radar_ctx* ctx, int max_records);
int radar_profile_end(radar_ctx* ctx);
int radar_kernel_count(void);
const char* radar_kernel_name(int id);
int radar_kernel_stats(const radar_ctx* ctx, int id, long long* launches, double* timed_ms, long long* timed_launches);
int radar_reset_launch_counts(radar_ctx* ctx);

/* ------------------------------------------------------------------------------------------
 * radar_expand_step - one draft call's worth of tree expansion for every active sequence.
 * (Appendix walkthrough: each frontier token yields its k most probable tokens with their
 * confidence scores; the k best candidates over all parents are kept; the prediction model
 * of Sec. 4.2 then emits continue/stop.  State s_t of the MDP = those k confidence scores.)
 *
 * For sequence b with active[b] != 0, and each of its F frontier rows f:
 *   log-softmax over the V logits, top-k by (logit desc, token id asc);
 *   candidate score = parent_score[b,f] + log-prob; all F*k candidates are appended to the
 *   pool in (f, j) order at pool_len[b]; the k best by (score desc, flat index asc) become the
 *   frontier outputs.  If t < t_max the prediction model runs on x = exp(frontier_score):
 *   single-layer LSTM (gate blocks i,f,g,o; state h,c) then Linear(H+k,H)-ReLU-Linear(H,2) on
 *   [h';x]; cont = logit[1] > logit[0].  At t == t_max the model is skipped, cont = 0 and
 *   gate_logits = 0.  If force_calls is given, cont = (t < force_calls[b]) instead.
 *   active[b] <- cont[b].  For t > 1, sequences with active[b] == 0 are skipped: nothing of
 *   theirs is touched, except cont[b] <- 0.  Call t == 1 starts a new speculative step for every
 *   sequence: the incoming active, h, c and pool_len are ignored (taken as 1, 0, 0 and 0), so a
 *   step needs no separate reset.
 * A NaN logit records RADAR_ERR_NUMERIC (outputs of that sequence unspecified).
 * Limits: 1 <= k <= RADAR_MAX_K, 1 <= F <= 32, V >= k, pool_len[b] + F*k <= pool_capacity;
 * w_ih, w_hh and w1 16-byte aligned.  The gate's weights must not be written between call 1 of a step and
 * its last call: calls t >= 2 may fetch them before the work queued ahead of them on the stream has finished.
 *
 * `policy` selects the policy networks of the paper's ablation (Table 3):
 *   RADAR_POLICY_LSTM_SCORES  the model above (the default, value 0);
 *   RADAR_POLICY_MLP_SCORES   memoryless: Linear(k,H)-ReLU-Linear(H,2) on x; w1 is [H][k]; w_ih, w_hh,
 *                             b_ih, b_hh may be NULL; h and c are neither read nor written;
 *   RADAR_POLICY_LSTM_HIDDEN  the same LSTM + head fed with `features`[b] (the draft model's hidden
 *                             state of this call, feat_dim floats) in place of x: w_ih is
 *                             [4H][feat_dim], w1 is [H][H+feat_dim]; feat_dim a multiple of 4 in
 *                             [4, 16384], features 16-byte aligned.
 * Everything else of the call (candidates, pool, frontier) is the same for the three.
 */
enum { RADAR_POLICY_LSTM_SCORES = 0, RADAR_POLICY_MLP_SCORES = 1, RADAR_POLICY_LSTM_HIDDEN = 2 };
/* `phase` lets a caller overlap the two halves of consecutive draft calls (the bandwidth-bound vocabulary pass of
 * call t+1 next to the latency-bound select + gate block of call t, on two streams):
 *   RADAR_EXPAND_ALL     both halves, back to back on the given stream (the default, value 0);
 *   RADAR_EXPAND_VOCAB   only the vocabulary pass (and the input-side products of the hidden-state policy) into
 *                        `workspace`.  `active` is only READ here, as the mask of sequences whose rows are worth
 *                        reading: it may be an older mask than the one the select half will see (a sequence that has
 *                        stopped since is read in vain, nothing else), or NULL for "all";
 *   RADAR_EXPAND_SELECT  only the select + gate half, on the records a RADAR_EXPAND_VOCAB call with the same
 *                        arguments left in the same `workspace`.  The caller orders it after that call and after the
 *                        previous draft call's select half.
 * Results are identical in the three forms. */
enum { RADAR_EXPAND_ALL = 0, RADAR_EXPAND_VOCAB = 1, RADAR_EXPAND_SELECT = 2 };

typedef struct {
    int B, F, V, k;
    int t, t_max;                       /* 1-based index of this draft call, and the maximum */
    const void* logits;                 /* [B][F][V] draft logits; element type logits_dtype */
    int logits_dtype;                   /* RADAR_F32 or RADAR_BF16 */
    int64_t logits_row_stride;          /* elements between consecutive rows f   (>= V)      */
    int64_t logits_seq_stride;          /* elements between consecutive sequences b          */
    const float* parent_score;          /* [B][F] cumulative log-prob of each frontier row   */
    const int32_t* parent_pool_idx;     /* [B][F] pool index of each frontier row, -1 = root */
    uint8_t* active;                    /* [B] in/out (out only at t = 1)                    */
    const int32_t* force_calls;         /* [B] or NULL                                       */
    const float *w_ih, *w_hh, *b_ih, *b_hh;   /* LSTM: [4H][k], [4H][H], [4H], [4H]          */
    const float *w1, *b1, *w2, *b2;           /* MLP : [H][H+k], [H], [2][H], [2]            */
    float* h;                           /* [B][H] in/out (out only at t = 1)                 */
    float* c;                           /* [B][H] in/out                                     */
    int pool_capacity;                  /* C                                                 */
    int32_t *pool_tok, *pool_parent, *pool_depth, *pool_draft_row;   /* [B][C] in/out        */
    float* pool_score;                  /* [B][C] in/out                                     */
    int32_t* pool_len;                  /* [B] in/out                                        */
    int32_t* frontier_tok;              /* [B][k] out */
    float* frontier_score;              /* [B][k] out (also the next call's parent_score)    */
    int32_t* frontier_pool_idx;         /* [B][k] out (also the next call's parent_pool_idx) */
    int32_t* frontier_src_row;          /* [B][k] out: which row f produced the survivor     */
    int32_t* topk_tok;                  /* [B][F][k] out */
    float* topk_logp;                   /* [B][F][k] out */
    float* gate_logits;                 /* [B][2] out */
    uint8_t* cont;                      /* [B] out */
    void* workspace;
    size_t workspace_bytes;
    int policy;                         /* RADAR_POLICY_*                                    */
    int feat_dim;                       /* RADAR_POLICY_LSTM_HIDDEN: length of a feature row */
    const float* features;              /* RADAR_POLICY_LSTM_HIDDEN: [B][feat_dim], device   */
    int phase;                          /* RADAR_EXPAND_*                                    */
} radar_expand_args;

size_t radar_expand_workspace_bytes(const radar_ctx* ctx, int B, int F, int V, int k);
int radar_expand_step(radar_ctx* ctx, const radar_expand_args* args, void* stream);

/* ------------------------------------------------------------------------------------------
 * radar_rerank_build_tree - top-N rerank of the pool and serialisation for one masked pass.
 * (Sec. 1: the candidates form a tree that is serialised and verified via masked attention
 * in a single pass; Sec. 2.3: nodes are reordered and pruned by confidence.)
 *
 * Keeps the n = min(N_b, pool_len[b], 63) best pool entries by (score desc, pool index asc),
 * N_b = n_keep[b] if given else N; lays them out after the root in ascending pool index;
 * writes per tree row: token, parent row, depth, position id = prefix_len[b] + depth, pool
 * index, score, draft row (row of the draft logits that produced the node's children, -1 if
 * it has none), ancestor mask (bit j of mask[i] <=> row j is i or an ancestor of i).
 * Rows >= n_nodes[b]: tok/parent/pool_idx/draft_row = -1, depth/pos = 0, score = 0, mask = 0.
 * retrieve[b][l][0..depth] = rows from the root to the l-th leaf (leaves in ascending row
 * order), -1 padded; rows l >= n_leaves[b] are all -1.
 * A kept entry whose parent was not kept records RADAR_ERR_TREE.
 * Limits: pool_capacity <= RADAR_MAX_POOL, 1 <= N < RADAR_MAX_NODES, t_max < 64.
 */
typedef struct {
    int B, N, t_max, pool_capacity;
    const int32_t *pool_tok, *pool_parent, *pool_depth, *pool_draft_row;   /* [B][C] */
    const float* pool_score;            /* [B][C] */
    const int32_t* pool_len;            /* [B] */
    const int32_t* n_keep;              /* [B] or NULL */
    const int32_t* root_tok;            /* [B] */
    const int32_t* prefix_len;          /* [B] */
    int32_t *tree_tok, *tree_parent, *tree_depth, *tree_pos, *tree_pool_idx, *tree_draft_row;  /* [B][64] out */
    float* tree_score;                  /* [B][64] out */
    uint64_t* tree_mask;                /* [B][64] out */
    int32_t* n_nodes;                   /* [B] out */
    int32_t* retrieve;                  /* [B][N][t_max+1] out */
    int32_t* n_leaves;                  /* [B] out */
} radar_tree_args;

int radar_rerank_build_tree(radar_ctx* ctx, const radar_tree_args* args, void* stream);

/* ------------------------------------------------------------------------------------------
 * radar_tree_attention - tree-masked verification attention of one layer, GQA.
 * (Sec. 3: the target model scores the whole draft in one parallel pass; Sec. 1: the
 * serialised tree is verified via masked attention.)
 *
 * For sequence b, query head h (KV head h / (Hq/Hkv)) and tree row i < n_nodes[b]:
 *   O[b,i,h,:] = sum_j softmax_j(scale * q.k_j) v_j over j in prefix[0, prefix_len[b]) and
 *   tree rows t with bit t of mask[b,i] set.  Rows i >= n_nodes[b] of O are left untouched.
 * Layouts: Q, O [B][64][Hq][d]; Kt, Vt [B][64][Hkv][d]; prefix cache Kc, Vc token-major
 * [token][Hkv][d] where sequence b's tokens start at row kv_start[b] (dense caches:
 * kv_start[b] = b * Pmax; packed: the cumulative lengths).  dtype applies to Q, K, V and O;
 * accumulation is fp32.  lse (optional) [B][Hq][64] receives log sum_j exp(scale * q.k_j).
 * max_prefix_len (host) bounds prefix_len[] and sizes the launch; cache_rows (host) is the number
 * of token rows allocated in Kc / Vc and bounds every read of them.  A sequence whose device-side
 * prefix_len is negative or larger than max_prefix_len, or whose kv_start + prefix_len exceeds
 * cache_rows, records RADAR_ERR_INVALID_ARG on the device status word and is skipped.
 * Q, Kc, Vc, Kt, Vt and O must be 16-byte aligned (both kernels move them in 16-byte pieces); a misaligned
 * tensor is refused on the host with RADAR_ERR_INVALID_ARG.
 * bf16 with Hq / Hkv a power of two (<= 128) runs on the tensor cores (TMA-staged K/V tiles, tcgen05 MMA for
 * QK^T and PV); every other case, and all of fp32, runs on an fp32 FMA kernel.  radar_tree_attention_path()
 * tells which of the two a given argument struct will take, so that a caller (or a benchmark) is never
 * switched to the other kernel unawares.
 * Paged prefix cache (block_table != NULL): prefix token j of sequence b is cache row
 *   block_table[b * max_pages + j / page_size] * page_size + j % page_size
 * and kv_start is not read (it may be NULL).  page_size is 16, 32, 64 or a multiple of 128; a
 * sequence needs ceil(prefix_len / page_size) <= max_pages entries; entries past that are not read.
 * A page index whose page does not lie inside [0, cache_rows) records RADAR_ERR_INVALID_ARG on the
 * device status word (the read goes to page 0).  The paper has no paged cache; this is the layout
 * serving systems keep their KV in, so that verification can read it in place.
 * Multi-layer form (n_layers > 1; Sec. 3: the target model's one parallel pass runs every layer over the same
 * tree): the same attention for n_layers sets of Q / K / V / O that share the tree, its masks and the prefix
 * lengths - the verification pass of a whole model issues its layers' attention in one call.  On the
 * tensor-core path all layers run in ONE persistent launch (the tile space of a layer is repeated per layer and
 * cut into equal ranges as before); the FMA path launches layer by layer.  The workspace of one layer suffices.
 * Limits: d in {64, 128}; Hq a multiple of Hkv; cache_rows < 2^31.
 */
typedef struct {
    int B, Hq, Hkv, d;
    int dtype;                          /* RADAR_F32 or RADAR_BF16 */
    const void* Q;
    const void *Kc, *Vc;
    const int64_t* kv_start;            /* [B] */
    const int32_t* prefix_len;          /* [B] */
    int max_prefix_len;                 /* host value */
    int64_t cache_rows;                 /* host value: token rows in Kc / Vc */
    const void *Kt, *Vt;
    const uint64_t* mask;               /* [B][64] */
    const int32_t* n_nodes;             /* [B] */
    float scale;                        /* <= 0 selects 1/sqrt(d) */
    void* O;
    float* lse;                         /* or NULL */
    void* workspace;
    size_t workspace_bytes;
    const int32_t* block_table;         /* [B][max_pages] page indices, or NULL for the contiguous layout */
    int page_size;                      /* tokens per page                                               */
    int max_pages;                      /* entries per sequence in block_table                           */
    /* Several layers in one call (0 or 1: one layer, the strides are ignored).  Layer l uses Q, Kc / Vc, Kt / Vt, O
     * and lse at l times the given stride (in ELEMENTS of the tensor's type; multiples of 8 elements); the tree
     * (mask, n_nodes), prefix_len, kv_start, block_table, scale and the workspace are the same for all layers. */
    int n_layers;
    int64_t q_layer_stride;             /* also the stride of O                                          */
    int64_t cache_layer_stride;         /* Kc and Vc                                                     */
    int64_t tree_kv_layer_stride;       /* Kt and Vt                                                     */
    int64_t o_layer_stride;
    int64_t lse_layer_stride;
} radar_attn_args;

enum { RADAR_ATTN_PATH_FMA = 0, RADAR_ATTN_PATH_TENSOR_CORE = 1 };

size_t radar_attn_workspace_bytes(const radar_ctx* ctx, int B, int Hq, int Hkv, int d, int dtype, int max_prefix_len);
int radar_tree_attention(radar_ctx* ctx, const radar_attn_args* args, void* stream);
/* Which kernel radar_tree_attention runs for these arguments (host pointer): RADAR_ATTN_PATH_TENSOR_CORE or
 * RADAR_ATTN_PATH_FMA; negative status if args is NULL.  Reads only the host fields of the struct. */
int radar_tree_attention_path(const radar_attn_args* args);

/* ------------------------------------------------------------------------------------------
 * radar_verify_accept - acceptance of the verified tree.
 * Greedy (temperature-0 rows of the paper's temperature study): a_i = argmax of the target
 *   logits at row i (lowest token id on ties); from the root move to the child whose token is
 *   a_cur, else stop; next_token = a at the last accepted row.
 * Stochastic (Sec. 3, Eq. 1-2, applied sibling by sibling as Sec. 4.3, Eq. 13 assumes):
 *   p = softmax(target[cur]/T), q = softmax(draft[tree_draft_row[cur]]/T); children in
 *   ascending row order; child x accepted iff u_accept[row] < min(1, p(x)/q(x)) (q(x) = 0:
 *   accepted iff p(x) > 0); on reject p <- norm(max(0, p - q)), q(x) <- 0, q <- q / sum q;
 *   when every child is rejected next_token is drawn from the current p, when the path
 *   reaches a row without children it is drawn from softmax(target[row]/T); draws use the
 *   inverse CDF in token order with u_sample[b].  Probabilities are evaluated in fp64.
 * Outputs: accept_len[b] = accepted draft rows (root excluded); path_nodes/path_tokens
 * [B][t_max+1] (entry 0 = root, -1 padded); next_token[b]; best_retrieve_row[b] = lowest
 * retrieve row that contains the accepted path (-1 if the tree has no leaves).
 * target_logits [B][64][V] (rows >= n_nodes[b] are not read); draft_logits [B][R][V].
 */
typedef struct {
    int B, V, t_max, N, mode;
    float temperature;                  /* stochastic only, > 0 */
    const void* target_logits;
    int logits_dtype;                   /* RADAR_F32 or RADAR_BF16 (both logits tensors) */
    const int32_t *tree_tok, *tree_parent, *tree_draft_row;   /* [B][64] */
    const int32_t* n_nodes;             /* [B] */
    const int32_t* retrieve;            /* [B][N][t_max+1] */
    const int32_t* n_leaves;            /* [B] */
    const void* draft_logits;           /* stochastic: [B][R][V] */
    int R;
    const float* u_accept;              /* stochastic: [B][64] */
    const float* u_sample;              /* stochastic: [B] */
    int32_t *accept_len, *path_nodes, *path_tokens, *next_token, *best_retrieve_row;
    void* workspace;
    size_t workspace_bytes;
} radar_accept_args;

size_t radar_accept_workspace_bytes(const radar_ctx* ctx, int B, int V, int mode);
int radar_verify_accept(radar_ctx* ctx, const radar_accept_args* args, void* stream);

/* ------------------------------------------------------------------------------------------
 * radar_accept_length_distribution - acceptance-length distribution of a verified tree.
 * (Sec. 4.3, Eq. 11-13: for node v with children l_1..l_n tried in order, P_acc(l_j | v) is the
 * probability that l_1..l_{j-1} are rejected and l_j accepted under the sibling-sequential scheme of
 * radar_verify_accept; P_rej(l | v) = 1 - sum_j P_acc(l_j | v); P_acc(v) is the product along v's
 * path; P_stop(v) = P_acc(v) P_rej(l | v); p_i = sum of P_stop over the rows of depth i.)
 *
 * Inputs as for stochastic radar_verify_accept (target / draft logits, temperature, tree arrays)
 * plus tree_depth; no uniforms: every internal row is evaluated, not only one sampled path.
 * Outputs, fp64: dist[b][0..t_max] = p_0..p_tmax (sums to 1); p_acc_node[b][row] = P_acc(row)
 * (rows >= n_nodes[b]: 0).  Probabilities are evaluated in fp64.
 * Workspace: radar_acclen_workspace_bytes (two fp64 vocabulary rows per resident block).
 */
typedef struct {
    int B, V, t_max;
    float temperature;                  /* > 0 */
    const void* target_logits;          /* [B][64][V] */
    int logits_dtype;                   /* RADAR_F32 or RADAR_BF16 (both logits tensors) */
    const int32_t *tree_tok, *tree_parent, *tree_depth, *tree_draft_row;   /* [B][64] */
    const int32_t* n_nodes;             /* [B] */
    const void* draft_logits;           /* [B][R][V] */
    int R;
    double* dist;                       /* [B][t_max+1] out */
    double* p_acc_node;                 /* [B][64] out */
    void* workspace;
    size_t workspace_bytes;
} radar_acclen_args;

size_t radar_acclen_workspace_bytes(const radar_ctx* ctx, int B, int V);
int radar_accept_length_distribution(radar_ctx* ctx, const radar_acclen_args* args, void* stream);

/* ------------------------------------------------------------------------------------------
 * radar_verify_accept_greedy_noalloc - greedy acceptance that needs no workspace from the caller.
 * (The paper has no counterpart: this is a deployment variant of radar_verify_accept in greedy
 * mode, with the same inputs, outputs and results.)
 *
 * For hosts that cannot allocate when they reach this call - an inference server that has handed
 * all free device memory to its own cache pool at start-up, or a decode loop that must not take
 * the device-wide synchronisation of cudaMalloc / cudaFree - and that have no spare buffer to pass
 * as `workspace`.  The scratch is a fixed array of radar_noalloc_scratch_bytes() = 1 MiB inside
 * the library image.  The driver materialises it (and the kernels' code) on a GPU when the image is
 * first used there; radar_create does that for its device, so create the context before the host
 * freezes device memory - the array then stays until the process exits.
 * `workspace` / `workspace_bytes` of the argument struct are ignored; `mode` must be RADAR_GREEDY.
 *   - Sizes whose chunk records (about 16 bytes x B x 64 x chunks-per-row) exceed the array, and
 *     stochastic mode, return RADAR_ERR_UNSUPPORTED and launch nothing.
 *   - The call makes no cudaMalloc / cudaFree and calls no allocating routine; after radar_create on the
 *     same device it leaves the amount of free device memory unchanged.
 *   - Every call on a device uses the same array, which still holds the previous call's records;
 *     nothing needs to be cleared because each record is written before it is read within a call.
 *     Calls that may overlap on the GPU (two streams, concurrent graph replays) race: serialise them.
 *   - ctx's device must be the current device (otherwise RADAR_ERR_INVALID_ARG).  radar_create has
 *     resolved the array's device address; should a call find none cached it resolves it itself, so make
 *     the first call outside stream capture. */
size_t radar_noalloc_scratch_bytes(void);
int radar_verify_accept_greedy_noalloc(radar_ctx* ctx, const radar_accept_args* args, void* stream);

/* ------------------------------------------------------------------------------------------
 * radar_policy_train_step - one REINFORCE step of the prediction model on a batch of data points {S, D}.
 * (Sec. 4.2: the MDP of Eq. 3-9 and the loss of Eq. 10; Sec. 4.3: the data point x = {S, D}, the acceptance
 * length drawn from d_T; App. "Implementation Details": the network, learning rate 1e-4, batches of 256.  The
 * optimiser is not named there: Adam is used.)
 *
 * For data point j: the prediction model of radar_expand_step (LSTM + MLP, the RADAR_POLICY_LSTM_SCORES
 * network) is rolled out over the states s_t = exp(log_states[t-1][j][:]), t = 1, 2, ...; after draft call t
 * it CONTINUES iff u_action[j][t-1] < pi(continue | s_1..s_t) (softmax of the two logits), else stops: T = t.
 * A trajectory that reaches t_max ends there without a decision (T = t_max, t_max - 1 decisions).  The
 * acceptance length l_acc is the smallest i with p_0 + .. + p_i > u_length[j] * total over d_T =
 * dists[T-1][j][:] (the last i with mass if none).  Rewards (Eq. 6): r_t = -alpha for t < T,
 * r_T = l_acc / T_gen(T), T_gen(t) = T_o + T_d t + T_p (t + 1 if t < t_max else t) (Eq. 7-8).  The decision
 * after call t collects G_t = sum_{t' = t..T} gamma^(t' - t) r_t' (Eq. 9-10).  Loss = mean over j of
 * - sum_t G_t log pi(a_t | .); its gradient by backpropagation through time (actions and l_acc are constants
 * of the gradient); no baseline, no dropout.  With step >= 1 the parameters then take one Adam update
 * (bias-corrected, no weight decay): m, v and theta are updated in place; step == 0 leaves them alone.
 *
 * Layouts (all device): log_states [t_max][n][k] fp32 = the frontier_score buffers of t_max draft calls;
 * dists [t_max][n][t_max+1] fp64, slice i-1 = what radar_accept_length_distribution wrote for the trees of
 * i draft calls; theta / adam_m / adam_v / grad [radar_policy_param_count(k)] fp32 in the order
 * w_ih [4H][k] | w_hh [4H][H] | b_ih [4H] | b_hh [4H] | w1 [H][H+k] | b1 [H] | w2 [2][H] | b2 [2]
 * (every tensor starts 16-byte aligned when theta is, so radar_expand_step can be pointed into it).
 * Outputs: grad, loss [1], calls [n] (T), l_acc [n], actions [n][t_max] (0 / 1, 255 where no decision was taken).
 * Limits: 1 <= k <= RADAR_MAX_K, 2 <= t_max <= 16, n >= 1; theta and the workspace 16-byte aligned.
 * Workspace: radar_train_workspace_bytes. */
typedef struct {
    int n, k, t_max;
    const float* log_states;
    const double* dists;
    const float* u_action;              /* [n][t_max] uniforms in [0,1) */
    const float* u_length;              /* [n] */
    float alpha, gamma, T_o, T_d, T_p;
    float lr, beta1, beta2, eps;
    int step;                           /* Adam step counted from 1; 0: loss and gradient only */
    float* theta;
    float* adam_m;
    float* adam_v;
    float* grad;
    float* loss;
    int32_t* calls;
    int32_t* l_acc;
    uint8_t* actions;
    void* workspace;
    size_t workspace_bytes;
} radar_train_args;

size_t radar_policy_param_count(int k);
size_t radar_train_workspace_bytes(const radar_ctx* ctx, int n, int k, int t_max);
int radar_policy_train_step(radar_ctx* ctx, const radar_train_args* args, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RADAR_H */
