// Mini-batch stochastic gradient (Eq. 2) of the ReLU MLP with softmax cross-entropy, fp32 on the
// CUDA cores, for all workers at once: every kernel is batched over workers (blockIdx.z), whose
// weights are slices of their rows of X.
#include "common.cuh"
#include "round_dev.cuh"

namespace dbw {

namespace {

using namespace dev;

// ------------------------------------------------------------------ kernels (bodies in round_dev.cuh)
__global__ void gather_batch_kernel(int B, int S, int in_dim, int C, const float* __restrict__ feat,
                                    const int32_t* __restrict__ labels, const int32_t* __restrict__ batch_idx,
                                    float* __restrict__ A0, int32_t* __restrict__ ylab, uint32_t* status) {
    gather_row(blockIdx.x, blockIdx.y, B, S, in_dim, C, feat, labels, batch_idx, A0, ylab, status);
}

template <int R, int TK>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
    constexpr int T = 16 * R;
    __shared__ __align__(16) float As[TK][T + 4];
    __shared__ __align__(16) float Bs[TK][T + 4];
    gemm_tile<R, TK>(g, blockIdx.z, blockIdx.y * T, blockIdx.x * T, As, Bs);
}

__global__ void __launch_bounds__(256)
softmax_ce_kernel(int B, int C, const float* __restrict__ logits, const int32_t* __restrict__ ylab,
                  float* dz, float* __restrict__ loss, float* __restrict__ G, long long ld, long long b_off) {
    __shared__ float sl[8];
    softmax_ce_worker(blockIdx.x, B, C, logits, ylab, dz, loss, G, ld, b_off, sl);
}

__global__ void bias_grad_kernel(int B, int out_dim, const float* __restrict__ dz, float* __restrict__ G,
                                 long long ld, long long b_off) {
    bias_grad_col(blockIdx.y, blockIdx.x * blockDim.x + threadIdx.x, B, out_dim, dz, G, ld, b_off);
}

int run_gemm(const GemmArgs& g, int batch, int sm_count, cudaStream_t s) {
    const long long big = (long long)((g.N + 63) / 64) * ((g.M + 63) / 64) * batch;
    if (big >= 4LL * sm_count) {
        dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, batch);
        gemm_simt_kernel<4, 16><<<grid, 256, 0, s>>>(g);
    } else {
        dim3 grid((g.N + 31) / 32, (g.M + 31) / 32, batch);
        const long long ctas = (long long)grid.x * grid.y * grid.z;
        if (g.K >= 128 && ctas < 2LL * sm_count)  // few CTAs, long reduction
            gemm_simt_kernel<2, 64><<<grid, 256, 0, s>>>(g);
        else
            gemm_simt_kernel<2, 16><<<grid, 256, 0, s>>>(g);
    }
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace

int grad_fp32_alloc(dbw_handle* h) {
    const dbw_model_desc& m = h->model;
    const size_t NB = (size_t)h->N * m.batch;
    for (int l = 0; l <= m.n_layers; ++l) {
        DBW_CUDA(cudaMalloc(&h->d_act[l], NB * m.dims[l] * sizeof(float)));
        if (l >= 1) DBW_CUDA(cudaMalloc(&h->d_dz[l], NB * m.dims[l] * sizeof(float)));
    }
    DBW_CUDA(cudaMalloc(&h->d_ylab, NB * sizeof(int32_t)));
    return DBW_OK;
}

void grad_fp32_free(dbw_handle* h) {
    for (int l = 0; l <= DBW_MAX_LAYERS; ++l) {
        if (h->d_act[l]) cudaFree(h->d_act[l]);
        if (h->d_dz[l]) cudaFree(h->d_dz[l]);
        h->d_act[l] = h->d_dz[l] = nullptr;
    }
    if (h->d_ylab) cudaFree(h->d_ylab);
    h->d_ylab = nullptr;
}

int launch_grad_fp32(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss,
                     cudaStream_t s) {
    const dbw_model_desc& m = h->model;
    const int B = m.batch, L = m.n_layers, N = h->N;
    gather_batch_kernel<<<dim3(B, N), 128, 0, s>>>(B, h->S, m.dims[0], m.dims[L], h->feat, h->labels, batch_idx,
                                                   h->d_act[0], h->d_ylab, h->d_status);
    DBW_LAUNCHED();
    int rc;
    // forward: Z_l = A_{l-1} W_l^T + b_l, A_l = ReLU(Z_l), logits for the last layer
    for (int l = 0; l < L; ++l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        GemmArgs g{};
        g.A = h->d_act[l]; g.sAz = (long long)B * in; g.sAm = in; g.sAk = 1;
        g.B = X + m.w_off[l]; g.sBz = h->ld; g.sBn = in; g.sBk = 1;
        g.C = h->d_act[l + 1]; g.sCz = (long long)B * out; g.sCm = out;
        g.bias = X + m.b_off[l]; g.sBiasz = h->ld;
        g.M = B; g.N = out; g.K = in; g.relu = l < L - 1;
        if ((rc = run_gemm(g, N, h->sm_count, s)) != DBW_OK) return rc;
    }
    softmax_ce_kernel<<<N, 256, 0, s>>>(B, m.dims[L], h->d_act[L], h->d_ylab, h->d_dz[L], loss, G, h->ld, m.b_off[L - 1]);
    DBW_LAUNCHED();
    // backward
    for (int l = L - 1; l >= 0; --l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        GemmArgs g{};  // dW_l[o][k] = sum_m dZ[m][o] A_{l}[m][k]
        g.A = h->d_dz[l + 1]; g.sAz = (long long)B * out; g.sAm = 1; g.sAk = out;
        g.B = h->d_act[l]; g.sBz = (long long)B * in; g.sBn = 1; g.sBk = in;
        g.C = G + m.w_off[l]; g.sCz = h->ld; g.sCm = in;
        g.M = out; g.N = in; g.K = B;
        if ((rc = run_gemm(g, N, h->sm_count, s)) != DBW_OK) return rc;
        if (l < L - 1) {  // the last layer's bias gradient came out of the loss kernel
            bias_grad_kernel<<<dim3((out + 127) / 128, N), 128, 0, s>>>(B, out, h->d_dz[l + 1], G, h->ld, m.b_off[l]);
            DBW_LAUNCHED();
        }
        if (l > 0) {  // dZ_{l}[m][k] = (sum_o dZ_{l+1}[m][o] W_l[o][k]) * [A_l[m][k] > 0]
            GemmArgs a{};
            a.A = h->d_dz[l + 1]; a.sAz = (long long)B * out; a.sAm = out; a.sAk = 1;
            a.B = X + m.w_off[l]; a.sBz = h->ld; a.sBn = 1; a.sBk = in;
            a.C = h->d_dz[l]; a.sCz = (long long)B * in; a.sCm = in;
            a.mask = h->d_act[l]; a.sMz = (long long)B * in; a.sMm = in;
            a.M = B; a.N = in; a.K = out;
            if ((rc = run_gemm(a, N, h->sm_count, s)) != DBW_OK) return rc;
        }
    }
    return DBW_OK;
}

}  // namespace dbw
