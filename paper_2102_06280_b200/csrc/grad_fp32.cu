// Mini-batch stochastic gradient (Eq. 2) of the ReLU MLP with softmax cross-entropy, fp32 on the
// CUDA cores, for all workers at once: every kernel is batched over workers (blockIdx.z), whose
// weights are slices of their rows of X.
#include "common.cuh"

namespace dbw {

namespace {

// ------------------------------------------------------------------ batch gather
// A sample index outside [0, S) or a label outside [0, C) is clamped and reported in the status word.
__global__ void gather_batch_kernel(int B, int S, int in_dim, int C, const float* __restrict__ feat,
                                    const int32_t* __restrict__ labels, const int32_t* __restrict__ batch_idx,
                                    float* __restrict__ A0, int32_t* __restrict__ ylab, uint32_t* status) {
    const int s = blockIdx.x, i = blockIdx.y;
    int src = batch_idx[(size_t)i * B + s];
    if (src < 0 || src >= S) {
        if (threadIdx.x == 0) atomicOr(status, DBW_STATUS_BAD_INDEX);
        src = src < 0 ? 0 : S - 1;
    }
    const float* from = feat + ((size_t)i * S + src) * in_dim;
    float* to = A0 + ((size_t)i * B + s) * in_dim;
    if ((in_dim & 3) == 0) {
        for (int k = threadIdx.x; k < in_dim / 4; k += blockDim.x)
            reinterpret_cast<float4*>(to)[k] = __ldg(reinterpret_cast<const float4*>(from) + k);
    } else {
        for (int k = threadIdx.x; k < in_dim; k += blockDim.x) to[k] = from[k];
    }
    if (threadIdx.x == 0) {
        int y = labels[(size_t)i * S + src];
        if (y < 0 || y >= C) {
            atomicOr(status, DBW_STATUS_BAD_INDEX);
            y = y < 0 ? 0 : C - 1;
        }
        ylab[(size_t)i * B + s] = y;
    }
}

// ------------------------------------------------------------------ batched strided GEMM
// C[z][m][n] = epilogue( sum_k A[z](m,k) * B[z](k,n) ), operands addressed through strides so
// that the same kernel serves Z = A W^T, dW = dZ^T A and dA = dZ W.
struct GemmArgs {
    const float* A;
    long long sAz, sAm, sAk;
    const float* B;
    long long sBz, sBn, sBk;
    float* C;
    long long sCz, sCm;
    const float* bias;  // indexed by n, nullable
    long long sBiasz;
    const float* mask;  // same shape as C, nullable: C *= (mask > 0)
    long long sMz, sMm;
    int M, N, K;
    int relu;
};


// 256 threads, each an R x R micro-tile: tiles of 64 x 64 (R = 4) for large outputs, 32 x 32 (R = 2)
// when the larger tile would leave most SMs idle.  TK = depth of one k-step: 16, or 64 for the few-CTA
// case with a long reduction, where a step costs one global-memory round trip whatever its depth
// (the order of the additions is the same).
template <int R, int TK>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
    constexpr int T = 16 * R;        // tile edge
    constexpr int PER = T * TK / 256;  // elements of each operand tile a thread stages
    __shared__ __align__(16) float As[TK][T + 4];
    __shared__ __align__(16) float Bs[TK][T + 4];
    const int z = blockIdx.z;
    const int m0 = blockIdx.y * T, n0 = blockIdx.x * T;
    const float* A = g.A + (size_t)z * g.sAz;
    const float* B = g.B + (size_t)z * g.sBz;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const bool a_k_fast = g.sAk == 1;
    const bool b_k_fast = g.sBk == 1;
    float acc[R][R] = {};
    float pa[PER], pb[PER];  // next k-step's operand elements, in flight while this one is multiplied
    auto fetch = [&](int k0) {
#pragma unroll
        for (int r = 0; r < PER; ++r) {
            const int e = tid + r * 256;
            const int ka = a_k_fast ? (e % TK) : (e / T);
            const int ma = a_k_fast ? (e / TK) : (e % T);
            pa[r] = (m0 + ma < g.M && k0 + ka < g.K) ? __ldg(A + (size_t)(m0 + ma) * g.sAm + (size_t)(k0 + ka) * g.sAk) : 0.f;
            const int kb = b_k_fast ? (e % TK) : (e / T);
            const int nb = b_k_fast ? (e / TK) : (e % T);
            pb[r] = (n0 + nb < g.N && k0 + kb < g.K) ? __ldg(B + (size_t)(n0 + nb) * g.sBn + (size_t)(k0 + kb) * g.sBk) : 0.f;
        }
    };
    fetch(0);
    for (int k0 = 0; k0 < g.K; k0 += TK) {
#pragma unroll
        for (int r = 0; r < PER; ++r) {
            const int e = tid + r * 256;
            As[a_k_fast ? (e % TK) : (e / T)][a_k_fast ? (e / TK) : (e % T)] = pa[r];
            Bs[b_k_fast ? (e % TK) : (e / T)][b_k_fast ? (e / TK) : (e % T)] = pb[r];
        }
        __syncthreads();
        fetch(k0 + TK);  // all zero past the end
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float av[R], bv[R];
            if constexpr (R == 4) {  // one 128-bit shared load per operand (rows are 16-byte aligned: T + 4 = 68 floats)
                const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
                const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
                av[0] = a4.x; av[1] = a4.y; av[2] = a4.z; av[3] = a4.w;
                bv[0] = b4.x; bv[1] = b4.y; bv[2] = b4.z; bv[3] = b4.w;
            } else {
                const float2 a2 = *reinterpret_cast<const float2*>(&As[kk][ty * 2]);
                const float2 b2 = *reinterpret_cast<const float2*>(&Bs[kk][tx * 2]);
                av[0] = a2.x; av[1] = a2.y;
                bv[0] = b2.x; bv[1] = b2.y;
            }
#pragma unroll
            for (int i = 0; i < R; ++i)
#pragma unroll
                for (int j = 0; j < R; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* C = g.C + (size_t)z * g.sCz;
    const float* bias = g.bias ? g.bias + (size_t)z * g.sBiasz : nullptr;
    const float* mask = g.mask ? g.mask + (size_t)z * g.sMz : nullptr;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        const int m = m0 + ty * R + i;
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int n = n0 + tx * R + j;
            if (n >= g.N) continue;
            float v = acc[i][j];
            if (bias) v += bias[n];
            if (g.relu) v = fmaxf(v, 0.f);
            if (mask && !(mask[(size_t)m * g.sMm + n] > 0.f)) v = 0.f;
            C[(size_t)m * g.sCm + n] = v;
        }
    }
}

// ------------------------------------------------------------------ softmax cross-entropy
// One CTA per worker, one warp per sample at a time.  dZ = (softmax(z) - onehot(y)) / B;
// loss = mean over the batch of (logsumexp(z) - z_y), summed in a fixed order.  The CTA then also sums
// its worker's dZ over the batch: the bias gradient of the last layer (one launch less per round).
__global__ void __launch_bounds__(256)
softmax_ce_kernel(int B, int C, const float* __restrict__ logits, const int32_t* __restrict__ ylab,
                  float* dz, float* __restrict__ loss, float* __restrict__ G, long long ld, long long b_off) {
    const int i = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float invB = 1.0f / (float)B;
    float wloss = 0.f;
    for (int s = warp; s < B; s += 8) {
        const float* z = logits + ((size_t)i * B + s) * C;
        float* o = dz + ((size_t)i * B + s) * C;
        const int y = ylab[(size_t)i * B + s];
        float mx = -INFINITY;
        for (int c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
#pragma unroll
        for (int k = 16; k > 0; k >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, k));
        float sum = 0.f;
        for (int c = lane; c < C; c += 32) sum += expf(z[c] - mx);
#pragma unroll
        for (int k = 16; k > 0; k >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, k);
        const float inv = 1.0f / sum;
        for (int c = lane; c < C; c += 32) o[c] = (expf(z[c] - mx) * inv - (c == y ? 1.f : 0.f)) * invB;
        wloss += (mx + logf(sum)) - z[y];
    }
    __shared__ float sl[8];
    if (lane == 0) sl[warp] = wloss;
    __syncthreads();
    if (threadIdx.x == 0 && loss) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += sl[w];
        loss[i] = t * invB;
    }
    // db[c] = sum over the samples of dZ[s][c], in sample order (the barrier above ordered the dZ stores)
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const float* p = dz + (size_t)i * B * C + c;
        float t = 0.f;
        for (int s = 0; s < B; ++s) t += p[(size_t)s * C];
        G[(size_t)i * ld + b_off + c] = t;
    }
}

// db[z][o] = sum_m dZ[z][m][o]
__global__ void bias_grad_kernel(int B, int out_dim, const float* __restrict__ dz, float* __restrict__ G,
                                 long long ld, long long b_off) {
    const int i = blockIdx.y;
    const int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= out_dim) return;
    const float* p = dz + (size_t)i * B * out_dim + o;
    float s = 0.f;
    for (int m = 0; m < B; ++m) s += p[(size_t)m * out_dim];
    G[(size_t)i * ld + b_off + o] = s;
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
