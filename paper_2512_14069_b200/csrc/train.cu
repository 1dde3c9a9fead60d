// One REINFORCE step of the prediction model (Sec. 4.2, Eq. 3-10; data points {S, D} of Sec. 4.3).
//
// Three kernels:
//   train_rollout_kernel   one block per data point: rolls the LSTM + MLP out over the states with sampled
//                          actions, draws the acceptance length from d_T, forms the returns, and runs
//                          backpropagation through time.  What the parameter gradients need - the deltas of
//                          every layer and the activations they multiply - goes to a record per (data point,
//                          decision) in the workspace.
//   train_outer_kernel     the parameter gradients: sums over all records of delta (x) activation, one output
//                          tile and one slice of the records per block, each slice in a fixed order into its own
//                          partial buffer (no atomics: the result does not depend on scheduling).
//   train_adam_kernel      adds the slices up (fixed order), batch loss (fixed-order sum) and the Adam update.
// The network is the one expand.cu runs at inference; the forward arithmetic is fp32 like there.
#include "common.cuh"

namespace radar {
namespace {

constexpr int H = kHidden;            // 128
constexpr int kTrainThreads = 4 * H;  // one thread per LSTM gate row
constexpr int kMaxSteps = 16;
constexpr int kXPad = 32;             // room for the k scores behind h in the head's input
constexpr int kSlices = 8;            // the records are summed in this many slices, one block each per output tile

// record of one decision (floats)
constexpr int R_DPRE = 0;                       // [4H] delta of the LSTM pre-activations
constexpr int R_DPRE1 = R_DPRE + 4 * H;         // [H]  delta of the head's hidden pre-activations
constexpr int R_DY = R_DPRE1 + H;               // [2]  delta of the logits (+2 padding)
constexpr int R_HPREV = R_DY + 4;               // [H]  h before the step
constexpr int R_CAT = R_HPREV + H;              // [H + kXPad]  h after the step, then the k scores
constexpr int R_HID = R_CAT + H + kXPad;        // [H]  relu output
constexpr int R_GATES = R_HID + H;              // [4H] i, f, g, o after their non-linearities
constexpr int R_C = R_GATES + 4 * H;            // [H]  c after the step
constexpr int R_CPREV = R_C + H;                // [H]
constexpr int R_STRIDE = R_CPREV + H;

struct Theta {
    float *w_ih, *w_hh, *b_ih, *b_hh, *w1, *b1, *w2, *b2;
};
__host__ __device__ inline Theta carve_theta(float* t, int k) {
    Theta o;
    o.w_ih = t;
    o.w_hh = o.w_ih + (size_t)4 * H * k;
    o.b_ih = o.w_hh + (size_t)4 * H * H;
    o.b_hh = o.b_ih + 4 * H;
    o.w1 = o.b_hh + 4 * H;
    o.b1 = o.w1 + (size_t)H * (H + k);
    o.w2 = o.b1 + H;
    o.b2 = o.w2 + 2 * H;
    return o;
}
__host__ __device__ inline size_t param_count(int k) { return (size_t)4 * H * k + 4 * H * H + 8 * H + (size_t)H * (H + k) + H + 2 * H + 2; }

struct TrainParams {
    radar_train_args a;
    float* rec;          // [n][t_max - 1][R_STRIDE]
    int* ndec;           // [n] decisions taken
    float* point_loss;   // [n]
    float* part;         // [kSlices][parameters] partial gradient sums
};

__device__ __forceinline__ float sigmoidf(float v) { return 1.f / (1.f + __expf(-v)); }
__device__ __forceinline__ float softplusf(float v) { return v > 0.f ? v + log1pf(expf(-v)) : log1pf(expf(v)); }

__global__ void __launch_bounds__(kTrainThreads, 1) train_rollout_kernel(const TrainParams P) {
    chain_wait();
    const radar_train_args& a = P.a;
    const int j = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k = a.k, t_max = a.t_max, n = a.n;
    const Theta W = carve_theta(a.theta, k);
    __shared__ __align__(16) float sh[H], sc[H], sx[kXPad], sg[4 * H], shid[H], sd1[H], sdp[4 * H], sdh[H], sdc[H], spart[4][H];
    __shared__ float sy[2], spi1[kMaxSteps], sG[kMaxSteps];
    __shared__ int sact[kMaxSteps];
    if (tid < H) { sh[tid] = 0.f; sc[tid] = 0.f; }
    __syncthreads();
    float* rec0 = P.rec + (size_t)j * (t_max - 1) * R_STRIDE;

    // ---- rollout ----
    int T = t_max, ndec = 0;
    for (int t = 1; t < t_max; ++t) {
        float* rec = rec0 + (size_t)(t - 1) * R_STRIDE;
        if (tid < kXPad) sx[tid] = tid < k ? __expf(a.log_states[((size_t)(t - 1) * n + j) * k + tid]) : 0.f;
        if (tid < H) { rec[R_HPREV + tid] = sh[tid]; rec[R_CPREV + tid] = sc[tid]; }
        __syncthreads();
        // LSTM pre-activations: warp w owns rows 32 w .. 32 w + 31, the lanes share each row's dot products
        float mine = 0.f;
        for (int rr = 0; rr < 32; ++rr) {
            const int row = warp * 32 + rr;
            const float4 wv = *reinterpret_cast<const float4*>(W.w_hh + (size_t)row * H + 4 * lane);
            const float4 hv = *reinterpret_cast<const float4*>(sh + 4 * lane);
            float p = wv.x * hv.x + wv.y * hv.y + wv.z * hv.z + wv.w * hv.w;
            if (lane < k) p += W.w_ih[(size_t)row * k + lane] * sx[lane];
            p = warp_sum(p);
            if (lane == rr) mine = p;
        }
        {
            const float pre = mine + W.b_ih[tid] + W.b_hh[tid];
            sg[tid] = (tid >= 2 * H && tid < 3 * H) ? tanhf(pre) : sigmoidf(pre);
            rec[R_GATES + tid] = sg[tid];
        }
        __syncthreads();
        if (tid < H) {
            const float cn = sg[H + tid] * sc[tid] + sg[tid] * sg[2 * H + tid];
            const float hn = sg[3 * H + tid] * tanhf(cn);
            sc[tid] = cn;
            sh[tid] = hn;
            rec[R_C + tid] = cn;
            rec[R_CAT + tid] = hn;
        } else if (tid < H + kXPad) {
            rec[R_CAT + tid] = sx[tid - H];
        }
        __syncthreads();
        // head: warp w owns hidden rows 8 w .. 8 w + 7
        for (int rr = 0; rr < 8; ++rr) {
            const int row = warp * 8 + rr;
            const float* wr = W.w1 + (size_t)row * (H + k);
            float p = 0.f;
            for (int c = lane; c < H + k; c += 32) p += wr[c] * (c < H ? sh[c] : sx[c - H]);
            p = warp_sum(p);
            if (lane == 0) {
                const float hv = fmaxf(p + W.b1[row], 0.f);
                shid[row] = hv;
                rec[R_HID + row] = hv;
            }
        }
        __syncthreads();
        if (warp < 2) {
            float p = 0.f;
            for (int c = lane; c < H; c += 32) p += W.w2[warp * H + c] * shid[c];
            p = warp_sum(p);
            if (lane == 0) sy[warp] = p + W.b2[warp];
        }
        __syncthreads();
        const float d = sy[1] - sy[0];
        const float pi1 = 1.f / (1.f + expf(-d));
        const int act = a.u_action[(size_t)j * t_max + (t - 1)] < pi1 ? 1 : 0;
        if (tid == 0) {
            spi1[t - 1] = pi1;
            sact[t - 1] = act;
            sG[t - 1] = act ? -softplusf(-d) : -softplusf(d);       // log pi(a_t) for now
        }
        ndec = t;
        if (!act) { T = t; break; }                                   // the same in every thread
    }
    __syncthreads();

    // ---- acceptance length, reward, returns, loss (one thread, fp64) ----
    if (tid == 0) {
        const double* drow = a.dists + ((size_t)(T - 1) * n + j) * (t_max + 1);
        double total = 0.0;
        for (int i = 0; i <= t_max; ++i) total += drow[i];
        const double target = (double)a.u_length[j] * total;
        double run = 0.0;
        int len = -1, last_pos = -1;
        for (int i = 0; i <= t_max; ++i) {
            run += drow[i];
            if (drow[i] > 0.0) last_pos = i;
            if (run > target) { len = i; break; }
        }
        if (len < 0) len = last_pos;
        const double t_pred = (double)a.T_p * (T < t_max ? T + 1 : T);
        const double reward_T = (double)len / ((double)a.T_o + (double)a.T_d * T + t_pred);
        // G_t = r_t + gamma G_{t+1}, backwards from the last call
        double g = reward_T, loss = 0.0;
        for (int t = T; t >= 1; --t) {
            if (t < T) g = -(double)a.alpha + (double)a.gamma * g;
            if (t <= ndec) {
                loss -= g * (double)sG[t - 1];
                sG[t - 1] = (float)g;
            }
        }
        P.point_loss[j] = (float)loss;
        P.ndec[j] = ndec;
        a.calls[j] = T;
        a.l_acc[j] = len;
        for (int t = 1; t <= t_max; ++t) a.actions[(size_t)j * t_max + (t - 1)] = t <= ndec ? (uint8_t)sact[t - 1] : (uint8_t)255;
    }
    if (tid < H) { sdh[tid] = 0.f; sdc[tid] = 0.f; }
    __syncthreads();

    // ---- backpropagation through time ----
    const int q = tid >> 7, col = tid & (H - 1);
    for (int s = ndec - 1; s >= 0; --s) {
        float* rec = rec0 + (size_t)s * R_STRIDE;
        const float G = sG[s], pi1 = spi1[s];
        const int act = sact[s];
        const float dy0 = -G * ((act == 0 ? 1.f : 0.f) - (1.f - pi1));
        const float dy1 = -G * ((act == 1 ? 1.f : 0.f) - pi1);
        if (tid == 0) { rec[R_DY] = dy0; rec[R_DY + 1] = dy1; }
        if (tid < H) {
            const float v = rec[R_HID + tid] > 0.f ? W.w2[tid] * dy0 + W.w2[H + tid] * dy1 : 0.f;
            sd1[tid] = v;
            rec[R_DPRE1 + tid] = v;
        }
        __syncthreads();
        {   // dh = W1[:, :H]^T dpre1 + dh from the next step: thread (q, col) sums 32 rows
            float p = 0.f;
            for (int r = q * 32; r < q * 32 + 32; ++r) p += W.w1[(size_t)r * (H + k) + col] * sd1[r];
            spart[q][col] = p;
        }
        __syncthreads();
        if (tid < H) {
            const float dh = spart[0][tid] + spart[1][tid] + spart[2][tid] + spart[3][tid] + sdh[tid];
            const float gi = rec[R_GATES + tid], gf = rec[R_GATES + H + tid], gg = rec[R_GATES + 2 * H + tid], go = rec[R_GATES + 3 * H + tid];
            const float tc = tanhf(rec[R_C + tid]);
            const float dc = dh * go * (1.f - tc * tc) + sdc[tid];
            const float di = dc * gg * gi * (1.f - gi), df = dc * rec[R_CPREV + tid] * gf * (1.f - gf);
            const float dg = dc * gi * (1.f - gg * gg), dob = dh * tc * go * (1.f - go);
            sdp[tid] = di; sdp[H + tid] = df; sdp[2 * H + tid] = dg; sdp[3 * H + tid] = dob;
            rec[R_DPRE + tid] = di; rec[R_DPRE + H + tid] = df; rec[R_DPRE + 2 * H + tid] = dg; rec[R_DPRE + 3 * H + tid] = dob;
            sdc[tid] = dc * gf;
        }
        __syncthreads();
        {   // dh for the step before: W_hh^T dpre, thread (q, col) sums 128 rows
            float p = 0.f;
            for (int r = q * H; r < q * H + H; ++r) p += W.w_hh[(size_t)r * H + col] * sdp[r];
            spart[q][col] = p;
        }
        __syncthreads();
        if (tid < H) sdh[tid] = spart[0][tid] + spart[1][tid] + spart[2][tid] + spart[3][tid];
        __syncthreads();
    }
}

// out[m][c] = scale * sum over valid records of A[rec][m] * B[rec][c]   (B absent: a column of ones)
struct OuterJob {
    int a_off, M, b_off, N;     // offsets into a record; b_off < 0: ones
    int ld_out;                 // row stride of the output (N for matrices, 1 for vectors)
    long long out_off, out_off2;   // offsets into grad (out_off2 >= 0: a second copy, for the two LSTM biases)
};
struct OuterParams {
    OuterJob job[8];
    const float* rec;
    const int* ndec;
    float* part;                // [kSlices][count]
    long long count;
    int n, steps;               // records per data point = t_max - 1
};

__global__ void __launch_bounds__(256) train_outer_kernel(const OuterParams P) {
    chain_wait();
    const OuterJob J = P.job[blockIdx.z % 7];
    const int slice = blockIdx.z / 7;
    const int m0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    if (m0 >= J.M || c0 >= J.N) return;
    __shared__ float As[32][33], Bs[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;     // 32 x 8
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const int K = P.n * P.steps;
    const int per = ((K + kSlices - 1) / kSlices + 31) / 32 * 32;
    const int r_end = min(K, (slice + 1) * per);
    for (int r0 = slice * per; r0 < r_end; r0 += 32) {
        // stage 32 records x 32 columns of each operand (invalid records and columns past the edge: zero)
        for (int e = ty; e < 32; e += 8) {
            const int r = r0 + e;
            const bool live = r < r_end && (r % P.steps) < P.ndec[r / P.steps];
            const float* rec = P.rec + (size_t)r * R_STRIDE;
            As[e][tx] = live && m0 + tx < J.M ? rec[J.a_off + m0 + tx] : 0.f;
            Bs[e][tx] = live && c0 + tx < J.N ? (J.b_off < 0 ? 1.f : rec[J.b_off + c0 + tx]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int e = 0; e < 32; ++e) {
            const float b = Bs[e][tx];
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] += As[e][ty + 8 * i] * b;
        }
        __syncthreads();
    }
    if (c0 + tx < J.N) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + ty + 8 * i;
            if (m < J.M) {
                float* out = P.part + (long long)slice * P.count;
                out[J.out_off + (long long)m * J.ld_out + c0 + tx] = acc[i];
                if (J.out_off2 >= 0) out[J.out_off2 + (long long)m * J.ld_out + c0 + tx] = acc[i];
            }
        }
    }
}

__global__ void __launch_bounds__(256) train_adam_kernel(const TrainParams P, size_t count) {
    chain_wait();
    const radar_train_args& a = P.a;
    if (blockIdx.x == 0) {
        // batch loss: fixed-order sum
        __shared__ double part[256];
        double s = 0.0;
        for (int j = threadIdx.x; j < a.n; j += 256) s += (double)P.point_loss[j];
        part[threadIdx.x] = s;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) a.loss[0] = (float)(part[0] / a.n);
    }
    const float c1 = 1.f - powf(a.beta1, (float)max(a.step, 1)), c2 = 1.f - powf(a.beta2, (float)max(a.step, 1));
    const float scale = 1.f / (float)a.n;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < count; i += (size_t)gridDim.x * 256) {
        float g = 0.f;
#pragma unroll
        for (int sl = 0; sl < kSlices; ++sl) g += P.part[(size_t)sl * count + i];
        g *= scale;
        a.grad[i] = g;
        if (a.step < 1) continue;
        const float m = a.beta1 * a.adam_m[i] + (1.f - a.beta1) * g;
        const float v = a.beta2 * a.adam_v[i] + (1.f - a.beta2) * g * g;
        a.adam_m[i] = m;
        a.adam_v[i] = v;
        a.theta[i] -= a.lr * (m / c1) / (sqrtf(v / c2) + a.eps);
    }
}

}  // namespace
}  // namespace radar

using namespace radar;

extern "C" size_t radar_policy_param_count(int k) { return k >= 1 && k <= RADAR_MAX_K ? param_count(k) : 0; }

extern "C" size_t radar_train_workspace_bytes(const radar_ctx*, int n, int k, int t_max) {
    if (n < 1 || k < 1 || t_max < 2) return 0;
    return align_up((size_t)n * (t_max - 1) * R_STRIDE * sizeof(float), 256) + align_up((size_t)n * sizeof(int), 256) +
           align_up((size_t)n * sizeof(float), 256) + align_up((size_t)kSlices * param_count(k) * sizeof(float), 256);
}

extern "C" int radar_policy_train_step(radar_ctx* ctx, const radar_train_args* a, void* stream_) {
    if (!ctx || !a) return RADAR_ERR_INVALID_ARG;
    if (a->n < 1 || a->k < 1 || a->k > RADAR_MAX_K || a->t_max < 2 || a->t_max > kMaxSteps) return RADAR_ERR_INVALID_ARG;
    if (!a->log_states || !a->dists || !a->u_action || !a->u_length || !a->theta || !a->grad || !a->loss || !a->calls ||
        !a->l_acc || !a->actions || !a->workspace)
        return RADAR_ERR_INVALID_ARG;
    if (a->step < 0 || (a->step >= 1 && (!a->adam_m || !a->adam_v))) return RADAR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(a->theta) & 15) || (reinterpret_cast<uintptr_t>(a->workspace) & 15)) return RADAR_ERR_INVALID_ARG;
    if (a->workspace_bytes < radar_train_workspace_bytes(ctx, a->n, a->k, a->t_max)) return RADAR_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    TrainParams P;
    P.a = *a;
    unsigned char* w = static_cast<unsigned char*>(a->workspace);
    P.rec = reinterpret_cast<float*>(w);
    w += align_up((size_t)a->n * (a->t_max - 1) * R_STRIDE * sizeof(float), 256);
    P.ndec = reinterpret_cast<int*>(w);
    w += align_up((size_t)a->n * sizeof(int), 256);
    P.point_loss = reinterpret_cast<float*>(w);
    w += align_up((size_t)a->n * sizeof(float), 256);
    P.part = reinterpret_cast<float*>(w);
    const int k = a->k;
    {
        radar_launch_scope scope(ctx, RADAR_K_TRAIN_ROLLOUT, stream);
        RADAR_CUDA_CHECK(launch_chained(train_rollout_kernel, dim3((unsigned)a->n), dim3(kTrainThreads), 0, stream, P));
    }
    {
        // offsets of the tensors inside theta / grad
        const long long o_w_ih = 0, o_w_hh = o_w_ih + 4LL * H * k, o_b_ih = o_w_hh + 4LL * H * H, o_b_hh = o_b_ih + 4 * H;
        const long long o_w1 = o_b_hh + 4 * H, o_b1 = o_w1 + (long long)H * (H + k), o_w2 = o_b1 + H, o_b2 = o_w2 + 2 * H;
        OuterParams O = {};
        O.rec = P.rec; O.ndec = P.ndec; O.part = P.part; O.count = (long long)param_count(k); O.n = a->n; O.steps = a->t_max - 1;
        O.job[0] = {R_DPRE, 4 * H, R_CAT + H, k, k, o_w_ih, -1};            // w_ih: dpre (x) x
        O.job[1] = {R_DPRE, 4 * H, R_HPREV, H, H, o_w_hh, -1};              // w_hh: dpre (x) h before the step
        O.job[2] = {R_DPRE, 4 * H, -1, 1, 1, o_b_ih, o_b_hh};         // both LSTM biases
        O.job[3] = {R_DPRE1, H, R_CAT, H + k, H + k, o_w1, -1};             // w1: dpre1 (x) [h; x]
        O.job[4] = {R_DPRE1, H, -1, 1, 1, o_b1, -1};
        O.job[5] = {R_DY, 2, R_HID, H, H, o_w2, -1};                        // w2: dy (x) relu output
        O.job[6] = {R_DY, 2, -1, 1, 1, o_b2, -1};
        radar_launch_scope scope(ctx, RADAR_K_TRAIN_OUTER, stream);
        RADAR_CUDA_CHECK(launch_chained(train_outer_kernel, dim3((unsigned)((H + k + 31) / 32), (unsigned)(4 * H / 32), 7 * kSlices), dim3(256), 0,
                                        stream, O));
    }
    {
        const size_t count = param_count(k);
        radar_launch_scope scope(ctx, RADAR_K_TRAIN_ADAM, stream);
        RADAR_CUDA_CHECK(launch_chained(train_adam_kernel, dim3((unsigned)ctx->sm_count), dim3(256), 0, stream, P, count));
    }
    return RADAR_OK;
}
