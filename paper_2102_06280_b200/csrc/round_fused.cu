// One iteration of Algorithm 1 in ONE launch, for networks so small that the round is bound by launch
// latency (a handful of workers with an fp32 model: 6 to 14 launches of 3-30 microseconds each otherwise).
//
// A cooperative grid of persistent blocks walks the steps of the round with a grid-wide barrier between
// dependent steps:
//   gather the mini-batches  ||  fastest-neighbour selection, weights, times (one block)      (Eq. 2; Section 2.2)
//   forward, layer by layer                                                                  (Eq. 2)
//   softmax cross-entropy, loss, last layer's bias gradient
//   backward, layer by layer: dW_l, db_l, dZ_l
//   masked mix + SGD step over column panels                                                 (Eqs. 4-5 / Eq. 3)
// Every step runs the device function the stand-alone kernel of that step runs (round_dev.cuh), so the
// result is bit-identical to the multi-launch path: each output element is produced by the same sequence of
// floating-point operations, only the assignment of tiles to blocks differs.  Data produced inside the
// launch is read with plain (coherent) loads after the grid barrier, never through the non-coherent path.
// The launch is cooperative, so all blocks are resident and the barrier cannot deadlock.
#include <cooperative_groups.h>

#include <algorithm>

#include "common.cuh"
#include "round_dev.cuh"

namespace dbw {

namespace {

namespace cg = cooperative_groups;
using namespace dev;

constexpr int kThreads = 256;
constexpr int kMixGS = 32;                       // 128-column panels
constexpr int kMaxWorkers = 64;                  // N * kMixGS * 16 bytes of panel <= 32 KiB
constexpr int kSmemBytes = 2 * 128 * 36 * 4;     // the largest GEMM staging (32 x 32 tiles, 128-deep steps): 36,864 bytes
constexpr int kBlocksPerSM = 1;                  // registers are spent on deep k-steps (a step costs one memory round trip)
constexpr long long kAutoMaxMacs = 64ll << 20;   // multiply-adds of the forward pass up to which the launch is used unasked

// GEMM tile variants (R, TK) the kernel instantiates; which one a GEMM uses is chosen on the host.
enum { V_2_16 = 0, V_2_64 = 1, V_4_16 = 2, V_4_64 = 3, V_2_128 = 4, kVariants = 5 };

struct FusedArgs {
    int N, B, S, L, C;
    int dims[DBW_MAX_LAYERS + 1];
    long long w_off[DBW_MAX_LAYERS], b_off[DBW_MAX_LAYERS];
    long long ld;
    const float* X;
    float* Xout;
    float* G;
    const float* feat;
    const int32_t* labels;
    const int32_t* batch_idx;
    float* act[DBW_MAX_LAYERS + 1];
    float* dz[DBW_MAX_LAYERS + 1];
    int32_t* ylab;
    const int32_t* rowptr;
    const int32_t* col;
    const double* t;
    const double* t_edge;
    const int32_t* b;
    uint8_t* kept;
    double* T_nbr_ws;
    double* T_nbr;
    double* T_worker;
    double* T_round;
    uint32_t* waited;
    uint32_t* status;
    MixPlan plan;
    int uniform, mix_then_correct;
    float lr;
    const float* lr_pw;
    float* loss;
    signed char fwd_var[DBW_MAX_LAYERS], dw_var[DBW_MAX_LAYERS], da_var[DBW_MAX_LAYERS];
    int head;  // the last layer takes the small-output steps (at most 32 classes)
};

template <int R, int TK>
__device__ __forceinline__ void gemm_tiles(const GemmArgs& g, int workers, float* smem) {
    constexpr int T = 16 * R;
    float(*As)[T + 4] = reinterpret_cast<float(*)[T + 4]>(smem);
    float(*Bs)[T + 4] = reinterpret_cast<float(*)[T + 4]>(smem + TK * (T + 4));
    const int tiles_n = (g.N + T - 1) / T, tiles_m = (g.M + T - 1) / T;
    const int items = tiles_n * tiles_m * workers;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int z = item / (tiles_n * tiles_m), rem = item % (tiles_n * tiles_m);
        gemm_tile<R, TK, false>(g, z, (rem / tiles_n) * T, (rem % tiles_n) * T, As, Bs);
    }
}

__device__ __forceinline__ void gemm_any(int variant, const GemmArgs& g, int workers, float* smem) {
    switch (variant) {
        case V_2_16: gemm_tiles<2, 16>(g, workers, smem); break;
        case V_2_64: gemm_tiles<2, 64>(g, workers, smem); break;
        case V_4_16: gemm_tiles<4, 16>(g, workers, smem); break;
        case V_4_64: gemm_tiles<4, 64>(g, workers, smem); break;
        default: gemm_tiles<2, 128>(g, workers, smem); break;  // a handful of tiles with a long reduction
    }
}

__global__ void __launch_bounds__(kThreads, kBlocksPerSM) round_fused_kernel(FusedArgs a) {
    extern __shared__ __align__(16) float smem[];
    __shared__ float sl[8];
    __shared__ double red[kThreads / 32];
    cg::grid_group grid = cg::this_grid();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.B, N = a.N, L = a.L;

    // Last layer of at most 32 classes: forward + loss by a warp per sample, backward by a block per worker and
    // 128 features, instead of three GEMMs and the loss step.
    const int Lg = a.head ? L - 1 : L;  // layers that run as GEMMs
    HeadRows rows{};
    if (L > 1) {
        rows.act = a.act[L - 1]; rows.ylab = a.ylab;
    } else {
        rows.feat = a.feat; rows.labels = a.labels; rows.batch_idx = a.batch_idx; rows.S = a.S;
    }
    float* loss_s = a.act[L];
    auto head_forward = [&](int first, int step) {
        for (int item = first * (kThreads / 32) + warp; item < N * B; item += step * (kThreads / 32)) {
            const int i = item / B;
            const float* Xi = a.X + (size_t)i * a.ld;
            if (a.C <= 16)
                head_forward_sample<16, false>(i, item % B, B, a.dims[L - 1], a.C, rows, Xi + a.w_off[L - 1], Xi + a.b_off[L - 1], a.dz[L], loss_s, a.status);
            else
                head_forward_sample<32, false>(i, item % B, B, a.dims[L - 1], a.C, rows, Xi + a.w_off[L - 1], Xi + a.b_off[L - 1], a.dz[L], loss_s, a.status);
        }
    };

    // ---- mini-batch gather (a one-layer model with the small-output last layer: its forward pass and loss
    //      straight from the data set); the last block does the selection, the weights and the times instead ----
    if (blockIdx.x == gridDim.x - 1) {
        for (int i = warp; i < N; i += kThreads / 32)
            select_worker(i, lane, a.rowptr, a.col, a.t, a.t_edge, a.b, a.kept, a.T_nbr_ws, a.waited, a.status, a.plan, 1, a.uniform);
        __threadfence();
        __syncthreads();
        double tr = round_times_part(N, a.rowptr, a.t, a.b, a.T_nbr_ws, a.T_nbr, a.T_worker, a.waited, a.status);
        tr = warp_max(tr);
        if (lane == 0) red[warp] = tr;
        __syncthreads();
        if (tid == 0) {
            for (int k = 1; k < kThreads / 32; ++k) tr = fmax(tr, red[k]);
            if (a.T_round) *a.T_round = tr;
        }
    } else if (Lg > 0 || !a.head) {  // the grid has at least two blocks
        for (int item = blockIdx.x; item < N * B; item += gridDim.x - 1)
            gather_row(item % B, item / B, B, a.S, a.dims[0], a.C, a.feat, a.labels, a.batch_idx, a.act[0], a.ylab, a.status);
    } else {
        head_forward(blockIdx.x, gridDim.x - 1);
    }
    grid.sync();

    // ---- forward: Z_l = A_{l-1} W_l^T + b_l, A_l = ReLU(Z_l), logits for the last layer ----
    for (int l = 0; l < Lg; ++l) {
        const int in = a.dims[l], out = a.dims[l + 1];
        GemmArgs g{};
        g.A = a.act[l]; g.sAz = (long long)B * in; g.sAm = in; g.sAk = 1;
        g.B = a.X + a.w_off[l]; g.sBz = a.ld; g.sBn = in; g.sBk = 1;
        g.C = a.act[l + 1]; g.sCz = (long long)B * out; g.sCm = out;
        g.bias = a.X + a.b_off[l]; g.sBiasz = a.ld;
        g.M = B; g.N = out; g.K = in; g.relu = l < L - 1;
        gemm_any(a.fwd_var[l], g, N, smem);
        grid.sync();
    }

    if (a.head) {
        if (Lg > 0) {
            head_forward(blockIdx.x, gridDim.x);
            grid.sync();
        }
        // ---- last layer backward: dW_L, db_L, the loss, dZ_{L-1} ----
        const int in = a.dims[L - 1], in4 = in >> 2;
        const int chunks = (in4 + kHeadChunk4 - 1) / kHeadChunk4;
        for (int item = blockIdx.x; item < N * chunks; item += gridDim.x) {
            const int i = item / chunks, k_lo = (item % chunks) * kHeadChunk4;
            const int k_hi = min(in4, k_lo + kHeadChunk4);
            const float* Xi = a.X + (size_t)i * a.ld;
            float* Gi = a.G + (size_t)i * a.ld;
            float* dz_prev = L > 1 ? a.dz[L - 1] : nullptr;
            if (a.C <= 16)
                head_backward_part<16, false>(i, k_lo, k_hi, B, in, a.C, rows, a.dz[L], loss_s, Xi + a.w_off[L - 1], Gi + a.w_off[L - 1],
                                              Gi + a.b_off[L - 1], a.loss, dz_prev, Gi + (L > 1 ? a.b_off[L - 2] : 0), smem, a.status);
            else
                head_backward_part<32, false>(i, k_lo, k_hi, B, in, a.C, rows, a.dz[L], loss_s, Xi + a.w_off[L - 1], Gi + a.w_off[L - 1],
                                              Gi + a.b_off[L - 1], a.loss, dz_prev, Gi + (L > 1 ? a.b_off[L - 2] : 0), smem, a.status);
        }
        grid.sync();
    } else {
        // ---- loss, dZ_L, last layer's bias gradient ----
        for (int i = blockIdx.x; i < N; i += gridDim.x) {
            softmax_ce_worker(i, B, a.C, a.act[L], a.ylab, a.dz[L], a.loss, a.G, a.ld, a.b_off[L - 1], sl);
            __syncthreads();
        }
        grid.sync();
    }

    // ---- backward ----
    for (int l = Lg - 1; l >= 0; --l) {
        const int in = a.dims[l], out = a.dims[l + 1];
        GemmArgs g{};  // dW_l[o][k] = sum_m dZ[m][o] A_l[m][k]
        g.A = a.dz[l + 1]; g.sAz = (long long)B * out; g.sAm = 1; g.sAk = out;
        g.B = a.act[l]; g.sBz = (long long)B * in; g.sBn = 1; g.sBk = in;
        g.C = a.G + a.w_off[l]; g.sCz = a.ld; g.sCm = in;
        g.M = out; g.N = in; g.K = B;
        gemm_any(a.dw_var[l], g, N, smem);
        if (l < L - 1 && !(a.head && l == L - 2))  // the last layer's bias gradient came out of the loss step, the one before's out of the last layer's backward step
            for (int e = blockIdx.x * kThreads + tid; e < N * out; e += gridDim.x * kThreads)
                bias_grad_col(e / out, e % out, B, out, a.dz[l + 1], a.G, a.ld, a.b_off[l]);
        if (l > 0) {  // dZ_l[m][k] = (sum_o dZ_{l+1}[m][o] W_l[o][k]) * [A_l[m][k] > 0]
            GemmArgs d{};
            d.A = a.dz[l + 1]; d.sAz = (long long)B * out; d.sAm = out; d.sAk = 1;
            d.B = a.X + a.w_off[l]; d.sBz = a.ld; d.sBn = 1; d.sBk = in;
            d.C = a.dz[l]; d.sCz = (long long)B * in; d.sCm = in;
            d.mask = a.act[l]; d.sMz = (long long)B * in; d.sMm = in;
            d.M = B; d.N = in; d.K = out;
            gemm_any(a.da_var[l], d, N, smem);
        }
        grid.sync();
    }

    // ---- masked mix + SGD step ----
    const int n_panels = (int)((a.ld + 4 * kMixGS - 1) / (4 * kMixGS));
    for (int panel = blockIdx.x; panel < n_panels; panel += gridDim.x) {
        mix_panel_body<kMixGS, kThreads, false>(panel, reinterpret_cast<float4*>(smem), N, a.ld, a.X, a.G, a.lr, a.lr_pw, a.Xout, nullptr,
                                               a.plan, a.mix_then_correct);
        __syncthreads();
    }
}

// Which tile variant a GEMM of `workers` problems M x N x K should take on a grid of `grid` blocks: the
// one with the fewest waves x k-steps, a k-step costing a global-memory round trip plus its multiply-adds.
int pick_variant(int M, int Nn, int K, int workers, int grid) {
    const int Rs[kVariants] = {2, 2, 4, 4, 2}, TKs[kVariants] = {16, 64, 16, 64, 128};
    int best = 0;
    double best_cost = 1e300;
    for (int v = 0; v < kVariants; ++v) {
        const int T = 16 * Rs[v];
        const long long tiles = (long long)((M + T - 1) / T) * ((Nn + T - 1) / T) * workers;
        const long long waves = (tiles + grid - 1) / grid;
        const int steps = (K + TKs[v] - 1) / TKs[v];
        const double cost = (double)waves * steps * (700.0 + 2.5 * TKs[v] * Rs[v] * Rs[v]);
        if (cost < best_cost) {
            best_cost = cost;
            best = v;
        }
    }
    return best;
}

}  // namespace

struct FusedState {
    bool usable = false;
    bool auto_on = false;
    int max_blocks = 0;
};

void round_fused_free(dbw_handle* h) {
    delete h->fused;
    h->fused = nullptr;
}

// Set-up at dbw_init (the handle's device current): can the device launch cooperatively, and how many
// blocks of the kernel are resident at once.
void round_fused_prepare(dbw_handle* h) {
    if (h->fused || !h->has_model || (h->flags & DBW_GEMM_BF16) || h->N > kMaxWorkers) return;
    FusedState* st = new (std::nothrow) FusedState();
    if (!st) return;
    h->fused = st;
    int coop = 0, per_sm = 0;
    if (!cuda_ok(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, h->device)) || !coop) return;
    if (!cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, round_fused_kernel, kThreads, kSmemBytes)) || per_sm < 1) return;
    st->max_blocks = h->sm_count * std::min(per_sm, kBlocksPerSM);
    long long macs = 0;
    for (int l = 0; l < h->model.n_layers; ++l) macs += (long long)h->N * h->model.batch * h->model.dims[l] * h->model.dims[l + 1];
    st->auto_on = macs <= kAutoMaxMacs;
    st->usable = true;
}

// Used when asked for, or, left to itself, for networks so small that launch latency is most of the round
// (measured: above roughly 1e8 multiply-adds per round the per-step kernels, which fill the SMs with more
// blocks than a cooperative grid can hold, are faster).
bool round_fused_usable(const dbw_handle* h) {
    if (!h->fused || !h->fused->usable || !h->feat || h->fused_mode == 0) return false;
    return h->fused_mode > 0 || h->fused->auto_on;
}

int launch_round_fused(dbw_handle* h, const float* X, const double* t, const int32_t* b, const int32_t* batch_idx, float lr,
                       const float* lr_pw, float* X_out, uint8_t* kept, double* T_worker, double* T_nbr, double* T_round,
                       float* loss, cudaStream_t s) {
    const dbw_model_desc& m = h->model;
    FusedArgs a{};
    a.N = h->N; a.B = m.batch; a.S = h->S; a.L = m.n_layers; a.C = m.dims[m.n_layers];
    for (int l = 0; l <= m.n_layers; ++l) {
        a.dims[l] = m.dims[l];
        a.act[l] = h->d_act[l];
        a.dz[l] = h->d_dz[l];
    }
    for (int l = 0; l < m.n_layers; ++l) {
        a.w_off[l] = m.w_off[l];
        a.b_off[l] = m.b_off[l];
    }
    a.ld = h->ld;
    a.X = X; a.Xout = X_out; a.G = h->d_G;
    a.feat = h->feat; a.labels = h->labels; a.batch_idx = batch_idx; a.ylab = h->d_ylab;
    a.rowptr = h->d_rowptr; a.col = h->d_col; a.t = t; a.t_edge = h->t_edge; a.b = b; a.kept = kept;
    a.T_nbr_ws = h->d_Tnbr_ws; a.T_nbr = T_nbr; a.T_worker = T_worker; a.T_round = T_round;
    a.waited = h->d_waited; a.status = h->d_status;
    a.plan = h->plan;
    a.uniform = (h->flags & DBW_WEIGHT_UNIFORM) ? 1 : 0;
    a.mix_then_correct = (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0;
    a.lr = lr; a.lr_pw = lr_pw; a.loss = loss;
    a.head = (fp32_head_usable(h) && (((uintptr_t)X | (uintptr_t)h->d_G) & 15) == 0) ? 1 : 0;
    // grid: as many blocks as the widest step has work items, at most one per SM
    const int B = m.batch, N = h->N;
    long long widest = (long long)N * B;  // gather rows
    for (int l = 0; l < m.n_layers; ++l) {
        widest = std::max(widest, (long long)((B + 31) / 32) * ((m.dims[l + 1] + 31) / 32) * N);
        widest = std::max(widest, (long long)((m.dims[l + 1] + 31) / 32) * ((m.dims[l] + 31) / 32) * N);
    }
    widest = std::max<long long>(widest, (h->ld + 4 * kMixGS - 1) / (4 * kMixGS));
    widest = std::max<long long>(widest, ((long long)N * B + kThreads / 32 - 1) / (kThreads / 32));  // last layer: a warp per sample
    widest = std::max<long long>(widest, (long long)N * (((m.dims[m.n_layers - 1] >> 2) + kHeadChunk4 - 1) / kHeadChunk4));
    const int grid = (int)std::min<long long>(h->fused->max_blocks, std::max<long long>(widest + 1, 2));
    for (int l = 0; l < m.n_layers; ++l) {
        a.fwd_var[l] = (signed char)pick_variant(B, m.dims[l + 1], m.dims[l], N, grid);
        a.dw_var[l] = (signed char)pick_variant(m.dims[l + 1], m.dims[l], B, N, grid);
        a.da_var[l] = (signed char)pick_variant(B, m.dims[l], m.dims[l + 1], N, grid);
    }
    void* params[] = {&a};
    DBW_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(round_fused_kernel), dim3(grid), dim3(kThreads), params, kSmemBytes, s));
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
