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

// The GEMM for operands whose unit-stride dimension allows 128-bit accesses (every layer whose width and
// batch are multiples of four).  A CTA of WM warps owns a tile of 2 RM WM x 64 outputs; a warp owns 2 RM rows x 64
// columns of it as RM x 4 per thread (RM = 8 or 4; lane / 16 picks the row half, lane mod 16 the columns), so that per
// k a warp reads RM + 4 floats through 128-bit shared-memory loads of which the row loads are broadcasts:
// with RM = 8, 32 multiply-adds per thread for about four shared-memory wavefronts per warp, where the
// 4 x 4 layout of gemm_simt_kernel needs the same four wavefronts for 16.  Global loads and stores are
// 128-bit along the operand's unit-stride dimension.  Every output element is summed over k in ascending
// order, exactly as in gemm_simt_kernel: the two give the same bits.
template <int WM, int RM>
__global__ void __launch_bounds__(32 * WM) gemm_vec_kernel(GemmArgs g) {
    constexpr int BM = 2 * RM * WM, BN = 64, TK = 16, THREADS = 32 * WM;
    constexpr int PA = BM * TK / 4 / THREADS, PB = BN * TK / 4 / THREADS;  // float4 per thread and k-step
    __shared__ __align__(16) float As[TK][BM + 4];
    __shared__ __align__(16) float Bs[TK][BN + 4];
    const int z = blockIdx.z, m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const float* __restrict__ A = g.A + (size_t)z * g.sAz;
    const float* __restrict__ B = g.B + (size_t)z * g.sBz;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int mw = warp * 2 * RM + (lane >> 4) * RM, nw = (lane & 15) * 4;
    const bool a_k_fast = g.sAk == 1, b_k_fast = g.sBk == 1;
    float acc[RM][4] = {};
    float4 pa[PA], pb[PB];
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    auto fetch = [&](int k0) {
#pragma unroll
        for (int r = 0; r < PA; ++r) {
            const int e = tid + r * THREADS;
            if (a_k_fast) {  // four consecutive k of row e / 4
                const int m = m0 + (e >> 2), k = k0 + 4 * (e & 3);
                pa[r] = (m < g.M && k < g.K) ? __ldg(reinterpret_cast<const float4*>(A + (size_t)m * g.sAm + k)) : zero4;
            } else {         // four consecutive rows at k = e / (BM / 4)
                const int m = m0 + 4 * (e % (BM / 4)), k = k0 + e / (BM / 4);
                pa[r] = (m < g.M && k < g.K) ? __ldg(reinterpret_cast<const float4*>(A + (size_t)k * g.sAk + m)) : zero4;
            }
        }
#pragma unroll
        for (int r = 0; r < PB; ++r) {
            const int e = tid + r * THREADS;
            if (b_k_fast) {
                const int n = n0 + (e >> 2), k = k0 + 4 * (e & 3);
                pb[r] = (n < g.N && k < g.K) ? __ldg(reinterpret_cast<const float4*>(B + (size_t)n * g.sBn + k)) : zero4;
            } else {
                const int n = n0 + 4 * (e % (BN / 4)), k = k0 + e / (BN / 4);
                pb[r] = (n < g.N && k < g.K) ? __ldg(reinterpret_cast<const float4*>(B + (size_t)k * g.sBk + n)) : zero4;
            }
        }
    };
    fetch(0);
    for (int k0 = 0; k0 < g.K; k0 += TK) {
#pragma unroll
        for (int r = 0; r < PA; ++r) {
            const int e = tid + r * THREADS;
            if (a_k_fast) {
                const int m = e >> 2, k = 4 * (e & 3);
                As[k][m] = pa[r].x; As[k + 1][m] = pa[r].y; As[k + 2][m] = pa[r].z; As[k + 3][m] = pa[r].w;
            } else {
                *reinterpret_cast<float4*>(&As[e / (BM / 4)][4 * (e % (BM / 4))]) = pa[r];
            }
        }
#pragma unroll
        for (int r = 0; r < PB; ++r) {
            const int e = tid + r * THREADS;
            if (b_k_fast) {
                const int n = e >> 2, k = 4 * (e & 3);
                Bs[k][n] = pb[r].x; Bs[k + 1][n] = pb[r].y; Bs[k + 2][n] = pb[r].z; Bs[k + 3][n] = pb[r].w;
            } else {
                *reinterpret_cast<float4*>(&Bs[e / (BN / 4)][4 * (e % (BN / 4))]) = pb[r];
            }
        }
        __syncthreads();
        fetch(k0 + TK);  // all zero past the end
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float av[RM];
#pragma unroll
            for (int i = 0; i < RM; i += 4) {
                const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][mw + i]);
                av[i] = a4.x; av[i + 1] = a4.y; av[i + 2] = a4.z; av[i + 3] = a4.w;
            }
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][nw]);
            const float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < RM; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* C = g.C + (size_t)z * g.sCz;
    const float* bias = g.bias ? g.bias + (size_t)z * g.sBiasz : nullptr;
    const float* mask = g.mask ? g.mask + (size_t)z * g.sMz : nullptr;
    const int n = n0 + nw;
    if (n >= g.N) return;  // N is a multiple of four: the thread's four columns are inside or outside together
    float bb[4] = {0.f, 0.f, 0.f, 0.f};
    if (bias) {
#pragma unroll
        for (int j = 0; j < 4; ++j) bb[j] = __ldg(bias + n + j);
    }
#pragma unroll
    for (int i = 0; i < RM; ++i) {
        const int m = m0 + mw + i;
        if (m >= g.M) break;
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            v[j] = acc[i][j];
            if (bias) v[j] += bb[j];
            if (g.relu) v[j] = fmaxf(v[j], 0.f);
        }
        if (mask) {
            const float4 mk = __ldg(reinterpret_cast<const float4*>(mask + (size_t)m * g.sMm + n));
            if (!(mk.x > 0.f)) v[0] = 0.f;
            if (!(mk.y > 0.f)) v[1] = 0.f;
            if (!(mk.z > 0.f)) v[2] = 0.f;
            if (!(mk.w > 0.f)) v[3] = 0.f;
        }
        *reinterpret_cast<float4*>(C + (size_t)m * g.sCm + n) = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// 128-bit accesses are possible: unit stride along k or along the output dimension, everything else a multiple of four floats
bool gemm_vec_ok(const GemmArgs& g) {
    auto al = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
    const bool a_ok = (g.sAk == 1 && g.K % 4 == 0 && g.sAm % 4 == 0) || (g.sAm == 1 && g.M % 4 == 0 && g.sAk % 4 == 0);
    const bool b_ok = (g.sBk == 1 && g.K % 4 == 0 && g.sBn % 4 == 0) || (g.sBn == 1 && g.N % 4 == 0 && g.sBk % 4 == 0);
    const bool c_ok = g.N % 4 == 0 && g.sCm % 4 == 0 && g.sCz % 4 == 0 && al(g.C);
    const bool m_ok = !g.mask || (g.sMm % 4 == 0 && g.sMz % 4 == 0 && al(g.mask));
    return a_ok && b_ok && c_ok && m_ok && g.sAz % 4 == 0 && g.sBz % 4 == 0 && al(g.A) && al(g.B);
}

// Last layer with at most 32 classes: forward + loss by a warp per sample, backward by a block per worker
// and 128 features (bodies in round_dev.cuh).
template <int CP>
__global__ void __launch_bounds__(256)
last_layer_forward_kernel(int N, int B, int in, int C, HeadRows rows, const float* __restrict__ X, long long ld, long long w_off,
                          long long b_off, float* __restrict__ dz, float* __restrict__ loss_s, uint32_t* status) {
    const int item = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (item >= N * B) return;
    const int i = item / B;
    head_forward_sample<CP, true>(i, item % B, B, in, C, rows, X + (size_t)i * ld + w_off, X + (size_t)i * ld + b_off, dz, loss_s, status);
}

template <int CP>
__global__ void __launch_bounds__(256)
last_layer_backward_kernel(int B, int in, int C, HeadRows rows, const float* __restrict__ dz, const float* __restrict__ loss_s,
                           const float* __restrict__ X, float* __restrict__ G, long long ld, long long w_off, long long b_off,
                           float* __restrict__ loss, float* __restrict__ dz_prev, long long b_off_prev, uint32_t* status) {
    extern __shared__ __align__(16) float head_smem[];
    const int i = blockIdx.y, k_lo = blockIdx.x * kHeadChunk4;
    const int k_hi = min(in >> 2, k_lo + kHeadChunk4);
    head_backward_part<CP, true>(i, k_lo, k_hi, B, in, C, rows, dz, loss_s, X + (size_t)i * ld + w_off, G + (size_t)i * ld + w_off,
                                 G + (size_t)i * ld + b_off, loss, dz_prev, G + (size_t)i * ld + b_off_prev, head_smem, status);
}

int run_gemm(const GemmArgs& g, int batch, int sm_count, cudaStream_t s) {
    if (gemm_vec_ok(g)) {
        // 8 x 4 outputs per thread where that still gives every SM several warps, else 4 x 4 (twice the warps
        // for the same tile), on tiles of 64, 32 or 16 rows
        const long long t64 = (long long)((g.N + 63) / 64) * ((g.M + 63) / 64) * batch;
        const long long t32 = (long long)((g.N + 63) / 64) * ((g.M + 31) / 32) * batch;
        if (t64 >= 2LL * sm_count)
            gemm_vec_kernel<4, 8><<<dim3((g.N + 63) / 64, (g.M + 63) / 64, batch), 128, 0, s>>>(g);
        else if (t32 >= sm_count)
            gemm_vec_kernel<4, 4><<<dim3((g.N + 63) / 64, (g.M + 31) / 32, batch), 128, 0, s>>>(g);
        else
            gemm_vec_kernel<2, 4><<<dim3((g.N + 63) / 64, (g.M + 15) / 16, batch), 64, 0, s>>>(g);
        DBW_LAUNCHED();
        return DBW_OK;
    }
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
    // A last layer of at most 32 classes runs as two kernels of its own instead of a GEMM, the loss kernel and
    // two more GEMMs; a one-layer model then needs no gathered copy of the mini-batch either.
    const bool head = fp32_head_usable(h) && (((uintptr_t)X | (uintptr_t)G) & 15) == 0;
    const int Lg = head ? L - 1 : L;  // layers that run as GEMMs
    if (Lg > 0 || !head) {
        gather_batch_kernel<<<dim3(B, N), 128, 0, s>>>(B, h->S, m.dims[0], m.dims[L], h->feat, h->labels, batch_idx,
                                                       h->d_act[0], h->d_ylab, h->d_status);
        DBW_LAUNCHED();
    }
    int rc;
    // forward: Z_l = A_{l-1} W_l^T + b_l, A_l = ReLU(Z_l), logits for the last layer
    for (int l = 0; l < Lg; ++l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        GemmArgs g{};
        g.A = h->d_act[l]; g.sAz = (long long)B * in; g.sAm = in; g.sAk = 1;
        g.B = X + m.w_off[l]; g.sBz = h->ld; g.sBn = in; g.sBk = 1;
        g.C = h->d_act[l + 1]; g.sCz = (long long)B * out; g.sCm = out;
        g.bias = X + m.b_off[l]; g.sBiasz = h->ld;
        g.M = B; g.N = out; g.K = in; g.relu = l < L - 1;
        if ((rc = run_gemm(g, N, h->sm_count, s)) != DBW_OK) return rc;
    }
    if (head) {
        const int in = m.dims[L - 1], C = m.dims[L];
        HeadRows rows{};
        if (L > 1) {
            rows.act = h->d_act[L - 1]; rows.ylab = h->d_ylab;
        } else {
            rows.feat = h->feat; rows.labels = h->labels; rows.batch_idx = batch_idx; rows.S = h->S;
        }
        float* loss_s = h->d_act[L];  // [N][B] of the logits' buffer: the logits themselves are never stored
        float* dz_prev = L > 1 ? h->d_dz[L - 1] : nullptr;
        const dim3 bgrid(((in >> 2) + kHeadChunk4 - 1) / kHeadChunk4, N);
        const size_t smem = fp32_head_smem_bytes(B, C);
        if (C <= 16) {
            last_layer_forward_kernel<16><<<(N * B + 7) / 8, 256, 0, s>>>(N, B, in, C, rows, X, h->ld, m.w_off[L - 1], m.b_off[L - 1],
                                                                          h->d_dz[L], loss_s, h->d_status);
            DBW_LAUNCHED();
            last_layer_backward_kernel<16><<<bgrid, 256, smem, s>>>(B, in, C, rows, h->d_dz[L], loss_s, X, G, h->ld, m.w_off[L - 1],
                                                                    m.b_off[L - 1], loss, dz_prev, L > 1 ? m.b_off[L - 2] : 0, h->d_status);
        } else {
            last_layer_forward_kernel<32><<<(N * B + 7) / 8, 256, 0, s>>>(N, B, in, C, rows, X, h->ld, m.w_off[L - 1], m.b_off[L - 1],
                                                                          h->d_dz[L], loss_s, h->d_status);
            DBW_LAUNCHED();
            last_layer_backward_kernel<32><<<bgrid, 256, smem, s>>>(B, in, C, rows, h->d_dz[L], loss_s, X, G, h->ld, m.w_off[L - 1],
                                                                    m.b_off[L - 1], loss, dz_prev, L > 1 ? m.b_off[L - 2] : 0, h->d_status);
        }
        DBW_LAUNCHED();
    } else {
        softmax_ce_kernel<<<N, 256, 0, s>>>(B, m.dims[L], h->d_act[L], h->d_ylab, h->d_dz[L], loss, G, h->ld, m.b_off[L - 1]);
        DBW_LAUNCHED();
    }
    // backward
    for (int l = Lg - 1; l >= 0; --l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        GemmArgs g{};  // dW_l[o][k] = sum_m dZ[m][o] A_{l}[m][k]
        g.A = h->d_dz[l + 1]; g.sAz = (long long)B * out; g.sAm = 1; g.sAk = out;
        g.B = h->d_act[l]; g.sBz = (long long)B * in; g.sBn = 1; g.sBk = in;
        g.C = G + m.w_off[l]; g.sCz = h->ld; g.sCm = in;
        g.M = out; g.N = in; g.K = B;
        if ((rc = run_gemm(g, N, h->sm_count, s)) != DBW_OK) return rc;
        if (l < L - 1 && !(head && l == L - 2)) {  // the last layer's bias gradient came out of the loss kernel, the one before's out of the last layer's backward kernel
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
