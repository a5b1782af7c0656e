// Device-side bodies of the round's CUDA-core kernels, shared by the stand-alone kernels (one launch per
// step) and the single-launch round for small networks (round_fused.cu).  Every function computes exactly
// what the kernel of the same name computed, in the same order of floating-point operations, so the two
// paths give the same bits.  Device code only; each translation unit that includes this instantiates its own.
#pragma once

#include "common.cuh"

namespace dbw {
namespace dev {

// ------------------------------------------------------------------ batch gather (Eq. 2: the mini-batch C_j(k))
// Row s of worker i's mini-batch: features copied to A0, label to ylab.  A sample index outside [0, S)
// or a label outside [0, C) is clamped and reported in the status word.  Called by all threads of a block.
__device__ __forceinline__ void gather_row(int s, int i, int B, int S, int in_dim, int C, const float* __restrict__ feat,
                                           const int32_t* __restrict__ labels, const int32_t* __restrict__ batch_idx,
                                           float* __restrict__ A0, int32_t* __restrict__ ylab, uint32_t* status) {
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
// One tile (z, m0, n0) by a block of 256 threads; As / Bs are the block's staging tiles.  Ends with a
// block barrier, so tiles may follow each other in a loop.  Every output element is summed over k in
// ascending order whatever R and TK are.
// NC = true reads the operands through the non-coherent path (they are constant while the kernel runs);
// NC = false with plain loads, for operands written earlier in the same launch.
template <bool NC, typename T>
__device__ __forceinline__ T load_g(const T* p) {
    if constexpr (NC) return __ldg(p);
    else return *p;
}

template <int R, int TK, bool NC = true>
__device__ __forceinline__ void gemm_tile(const GemmArgs& g, int z, int m0, int n0, float (*As)[16 * R + 4], float (*Bs)[16 * R + 4]) {
    constexpr int T = 16 * R;        // tile edge
    constexpr int PER = T * TK / 256;  // elements of each operand tile a thread stages
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
            pa[r] = (m0 + ma < g.M && k0 + ka < g.K) ? load_g<NC>(A + (size_t)(m0 + ma) * g.sAm + (size_t)(k0 + ka) * g.sAk) : 0.f;
            const int kb = b_k_fast ? (e % TK) : (e / T);
            const int nb = b_k_fast ? (e / TK) : (e % T);
            pb[r] = (n0 + nb < g.N && k0 + kb < g.K) ? load_g<NC>(B + (size_t)(n0 + nb) * g.sBn + (size_t)(k0 + kb) * g.sBk) : 0.f;
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
// Worker i by a block of 256 threads; sl = eight floats of shared memory (free again after a block barrier).
// (No __restrict__ on data another step of the same launch may have produced: the compiler must not route
// those loads through the non-coherent path.)
__device__ __forceinline__ void softmax_ce_worker(int i, int B, int C, const float* logits, const int32_t* ylab,
                                                  float* dz, float* loss, float* G, long long ld, long long b_off,
                                                  float* sl) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float invB = 1.0f / (float)B;
    float wloss = 0.f;
    if (C <= 32) {
        // at most one class per lane: four samples of this warp per pass, their loads issued together (the
        // arithmetic of each sample and the order in which the losses are added are those of the loop below)
        for (int s0 = warp; s0 < B; s0 += 32) {
            float zv[4];
            int yv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int s = s0 + 8 * u;
                zv[u] = (s < B && lane < C) ? logits[((size_t)i * B + s) * C + lane] : -INFINITY;
                yv[u] = s < B ? ylab[(size_t)i * B + s] : 0;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int s = s0 + 8 * u;
                if (s >= B) break;  // warp-uniform
                float mx = zv[u];
#pragma unroll
                for (int k = 16; k > 0; k >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, k));
                const float ez = lane < C ? expf(zv[u] - mx) : 0.f;
                float sum = ez;
#pragma unroll
                for (int k = 16; k > 0; k >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, k);
                const float inv = 1.0f / sum;
                if (lane < C) dz[((size_t)i * B + s) * C + lane] = (ez * inv - (lane == yv[u] ? 1.f : 0.f)) * invB;
                wloss += (mx + logf(sum)) - __shfl_sync(0xffffffffu, zv[u], yv[u] & 31);
            }
        }
    } else {
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
    }
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
#pragma unroll 8
        for (int s = 0; s < B; ++s) t += p[(size_t)s * C];
        G[(size_t)i * ld + b_off + c] = t;
    }
}

// db[i][o] = sum over the batch of dZ[i][m][o], in sample order
__device__ __forceinline__ void bias_grad_col(int i, int o, int B, int out_dim, const float* dz, float* G,
                                              long long ld, long long b_off) {
    if (o >= out_dim) return;
    const float* p = dz + (size_t)i * B * out_dim + o;
    float s = 0.f;
#pragma unroll 8
    for (int m = 0; m < B; ++m) s += p[(size_t)m * out_dim];
    G[(size_t)i * ld + b_off + o] = s;
}


// ------------------------------------------------------------------ last layer with at most 32 classes (Eq. 2)
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// A layer with a handful of outputs is a poor GEMM (one 32-wide tile, mostly padding, and a reduction as
// long as the layer is wide), so the last layer's forward pass, the loss and its backward pass run as two
// steps of their own: a warp per sample forward (every lane a slice of the features, all classes at once),
// and eight lanes per four features backward (the worker's dZ out of shared memory).
// For a one-layer model the rows are read straight from the data set through the batch indices.
struct HeadRows {
    const float* act;            // [N][B][in] output of the layer before, or null
    const int32_t* ylab;         // [N][B] gathered labels (with act)
    const float* feat;           // else: the data set, [N][S][in] ...
    const int32_t* labels;       // ... [N][S]
    const int32_t* batch_idx;    // ... and the round's sample indices [N][B]
    int S;
};

// Row s of worker i and its label; a sample index or label out of range is clamped and reported.
template <bool NC>
__device__ __forceinline__ const float* head_row(const HeadRows& r, int i, int s, int B, int in, int C, uint32_t* status, int* y) {
    if (r.act) {
        if (y) *y = r.ylab[(size_t)i * B + s];
        return r.act + ((size_t)i * B + s) * in;
    }
    int src = load_g<NC>(r.batch_idx + (size_t)i * B + s);
    if (src < 0 || src >= r.S) {
        atomicOr(status, DBW_STATUS_BAD_INDEX);
        src = src < 0 ? 0 : r.S - 1;
    }
    if (y) {
        int lab = __ldg(r.labels + (size_t)i * r.S + src);
        if (lab < 0 || lab >= C) {
            atomicOr(status, DBW_STATUS_BAD_INDEX);
            lab = lab < 0 ? 0 : C - 1;
        }
        *y = lab;
    }
    return r.feat + ((size_t)i * r.S + src) * in;
}

// Sample s of worker i by one warp: z = W a + b, dZ = (softmax(z) - onehot(y)) / B, the sample's loss
// logsumexp(z) - z_y into loss_s[i][s].  CP = compile-time bound on the classes (16 or 32); in is a multiple of 4.
// A lane adds its features in ascending order, the lanes are then added by a butterfly.
template <int CP, bool NC>
__device__ __forceinline__ void head_forward_sample(int i, int s, int B, int in, int C, const HeadRows& rows, const float* W,
                                                    const float* bias, float* dz, float* loss_s, uint32_t* status) {
    const int lane = threadIdx.x & 31;
    int y;
    const float4* arow = reinterpret_cast<const float4*>(head_row<NC>(rows, i, s, B, in, C, status, &y));
    const float4* w4 = reinterpret_cast<const float4*>(W);
    const int in4 = in >> 2;
    float acc[CP];
#pragma unroll
    for (int c = 0; c < CP; ++c) acc[c] = 0.f;
    for (int k0 = lane; k0 < in4; k0 += 64) {  // two float4 per lane and pass: twice the loads in flight
        const int k1 = k0 + 32;
        const bool two = k1 < in4;
        const float4 a0 = arow[k0];
        const float4 a1 = two ? arow[k1] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int c0 = 0; c0 < CP; c0 += 8) {  // eight classes at a time: sixteen weight loads in flight per lane
            if (c0 >= C) break;
            float4 w0[8], w1[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u;
                w0[u] = c < C ? load_g<NC>(w4 + (size_t)c * in4 + k0) : make_float4(0.f, 0.f, 0.f, 0.f);
                w1[u] = (c < C && two) ? load_g<NC>(w4 + (size_t)c * in4 + k1) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float t = acc[c0 + u];
                t = fmaf(a0.x, w0[u].x, t); t = fmaf(a0.y, w0[u].y, t); t = fmaf(a0.z, w0[u].z, t); t = fmaf(a0.w, w0[u].w, t);
                t = fmaf(a1.x, w1[u].x, t); t = fmaf(a1.y, w1[u].y, t); t = fmaf(a1.z, w1[u].z, t); t = fmaf(a1.w, w1[u].w, t);
                acc[c0 + u] = t;
            }
        }
    }
    float mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < CP; ++c) {
        if (c < C) {
            acc[c] = warp_sum(acc[c]) + load_g<NC>(bias + c);
            mx = fmaxf(mx, acc[c]);
        }
    }
    float sum = 0.f, zy = 0.f;
#pragma unroll
    for (int c = 0; c < CP; ++c) {
        if (c < C) {
            if (c == y) zy = acc[c];
            acc[c] = expf(acc[c] - mx);
            sum += acc[c];
        }
    }
    const float inv = 1.0f / sum, invB = 1.0f / (float)B;
    float mine = 0.f;
#pragma unroll
    for (int c = 0; c < CP; ++c)
        if (c < C && c == lane) mine = (acc[c] * inv - (c == y ? 1.f : 0.f)) * invB;
    if (lane < C) dz[((size_t)i * B + s) * C + lane] = mine;
    if (lane == 0) loss_s[(size_t)i * B + s] = (mx + logf(sum)) - zy;
}

// Backward of the last layer for worker i, features [4 k_lo, 4 k_hi) (at most kHeadChunk4 groups of four) by a
// block of 256 threads.  A warp owns four feature groups; its lanes split the samples eight ways (lane mod 8):
//   dW[c][f] = sum_s dZ[s][c] a[s][f]: each lane adds its samples in ascending order, a butterfly adds the lanes;
//   with dz_prev also dZ of the layer before, (sum_c dZ[s][c] W[c][f]) [a[s][f] > 0], classes in ascending order,
//   and that layer's bias gradient (the sum of its dZ over the samples) into Gb_prev.
// The block that owns the first features also adds the bias gradient and the worker's mean loss, in sample
// order.  smem: B * C floats + B 64-bit offsets.  Ends with a block barrier (shared memory free again).
constexpr int kHeadChunk4 = 32;
template <int CP, bool NC>
__device__ __forceinline__ void head_backward_part(int i, int k_lo, int k_hi, int B, int in, int C, const HeadRows& rows,
                                                   const float* dz, const float* loss_s, const float* W, float* Gw, float* Gb,
                                                   float* loss, float* dz_prev, float* Gb_prev, float* smem, uint32_t* status) {
    float* dzs = smem;
    long long* rowoff = reinterpret_cast<long long*>(smem + ((B * C + 1) & ~1));
    for (int e = threadIdx.x; e < B * C; e += blockDim.x) dzs[e] = dz[(size_t)i * B * C + e];
    const float* base = rows.act ? rows.act : rows.feat;
    for (int s = threadIdx.x; s < B; s += blockDim.x) rowoff[s] = head_row<NC>(rows, i, s, B, in, C, status, nullptr) - base;
    __syncthreads();
    if (k_lo == 0) {
        if ((int)threadIdx.x < C) {
            float t = 0.f;
            for (int s = 0; s < B; ++s) t += dzs[s * C + threadIdx.x];
            Gb[threadIdx.x] = t;
        }
        if (threadIdx.x == 32 && loss) {
            float t = 0.f;
            for (int s = 0; s < B; ++s) t += loss_s[(size_t)i * B + s];
            loss[i] = t * (1.0f / (float)B);
        }
    }
    const int lane = threadIdx.x & 31, slice = lane & 7;
    const int k = k_lo + (int)(threadIdx.x >> 5) * 4 + (lane >> 3);
    if (k < k_hi) {  // the eight lanes of a feature group stay together
        float4 acc[CP];
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int s = slice; s < B; s += 8) {
            const float4 a = *(reinterpret_cast<const float4*>(base + rowoff[s]) + k);
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                if (c < C) {
                    const float d = dzs[s * C + c];
                    acc[c].x = fmaf(d, a.x, acc[c].x); acc[c].y = fmaf(d, a.y, acc[c].y);
                    acc[c].z = fmaf(d, a.z, acc[c].z); acc[c].w = fmaf(d, a.w, acc[c].w);
                }
            }
        }
        const unsigned grp = 0xffu << (lane & 24);
#pragma unroll
        for (int c = 0; c < CP; ++c) {
            if (c < C) {
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) {
                    acc[c].x += __shfl_xor_sync(grp, acc[c].x, o); acc[c].y += __shfl_xor_sync(grp, acc[c].y, o);
                    acc[c].z += __shfl_xor_sync(grp, acc[c].z, o); acc[c].w += __shfl_xor_sync(grp, acc[c].w, o);
                }
                if ((c & 7) == slice) reinterpret_cast<float4*>(Gw + (size_t)c * in)[k] = acc[c];
            }
        }
        if (dz_prev) {
#pragma unroll
            for (int c = 0; c < CP; ++c)
                if (c < C) acc[c] = load_g<NC>(reinterpret_cast<const float4*>(W + (size_t)c * in) + k);
            float4 db = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
            for (int s = slice; s < B; s += 8) {
                const float4 a = *(reinterpret_cast<const float4*>(base + rowoff[s]) + k);
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int c = 0; c < CP; ++c) {
                    if (c < C) {
                        const float d = dzs[s * C + c];
                        v.x = fmaf(d, acc[c].x, v.x); v.y = fmaf(d, acc[c].y, v.y);
                        v.z = fmaf(d, acc[c].z, v.z); v.w = fmaf(d, acc[c].w, v.w);
                    }
                }
                v.x = a.x > 0.f ? v.x : 0.f; v.y = a.y > 0.f ? v.y : 0.f;
                v.z = a.z > 0.f ? v.z : 0.f; v.w = a.w > 0.f ? v.w : 0.f;
                reinterpret_cast<float4*>(dz_prev + ((size_t)i * B + s) * in)[k] = v;
                db.x += v.x; db.y += v.y; db.z += v.z; db.w += v.w;
            }
            // bias gradient of the layer before: this lane's samples in ascending order, then the eight lanes
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) {
                db.x += __shfl_xor_sync(grp, db.x, o); db.y += __shfl_xor_sync(grp, db.y, o);
                db.z += __shfl_xor_sync(grp, db.z, o); db.w += __shfl_xor_sync(grp, db.w, o);
            }
            if (slice == 0) {
                Gb_prev[4 * k] = db.x; Gb_prev[4 * k + 1] = db.y; Gb_prev[4 * k + 2] = db.z; Gb_prev[4 * k + 3] = db.w;
            }
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------ selection, weights, times
// Arrival time used for ordering: NaN sorts last (as +inf) and is reported in the status word.
__device__ __forceinline__ double order_time(double t, uint32_t* status) {
    if (t != t) {
        atomicOr(status, DBW_STATUS_NAN_TIME);
        return __longlong_as_double(0x7ff0000000000000LL);
    }
    return t;
}

__device__ __forceinline__ int clamped_b(const int32_t* b, int i, int deg, uint32_t* status) {
    int bi = b[i];
    if (bi < 0 || bi > deg) {
        atomicOr(status, DBW_STATUS_BAD_B);
        bi = bi < 0 ? 0 : deg;
    }
    return bi;
}


__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Writes the compacted kept list of worker i (and its weights) given the per-lane keep decision
// of one 32-neighbour chunk.  `running` is the number of entries already written.
__device__ __forceinline__ void plan_append(const MixPlan& plan, int i, int lane, bool keep, int j, float w,
                                            int& running) {
    unsigned m = __ballot_sync(0xffffffffu, keep);
    if (keep) {
        const int pos = checked(running + __popc(m & ((1u << lane) - 1u)), plan.stride, plan.status);
        plan.idx[(size_t)i * plan.stride + pos] = j;
        plan.w[(size_t)i * plan.stride + pos] = w;
    }
    running += __popc(m);
}

__device__ __forceinline__ void plan_finish(const MixPlan& plan, int i, int lane, int cnt, float w_self) {
    for (int k = cnt + lane; k < plan.stride; k += 32) {
        plan.idx[(size_t)i * plan.stride + k] = i;
        plan.w[(size_t)i * plan.stride + k] = 0.f;
    }
    if (lane == 0) {
        plan.cnt[i] = cnt;
        plan.w_self[i] = w_self;
    }
}

__device__ __forceinline__ float edge_weight(bool uniform, int p_i, int p_j) {
    int m = uniform ? p_i : (p_i > p_j ? p_i : p_j);
    return 1.0f / (1.0f + (float)m);
}

// Selection of worker i by one warp (Section 2.2): lane l owns neighbour (base + l); its rank is the number
// of neighbours whose (time, index) key is smaller, counted by shuffling every key past every lane; a
// neighbour is kept when its rank is below p_i.  Also the worker's part of the mixing plan (weights of
// Assumption 1 or uniform), the flags of the workers it waits for, and T_nbr.
__device__ __forceinline__ void select_worker(int i, int lane, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                              const double* __restrict__ t, const double* __restrict__ t_edge,
                                              const int32_t* __restrict__ b, uint8_t* __restrict__ kept, double* __restrict__ T_nbr_ws,
                                              uint32_t* waited, uint32_t* status, const MixPlan& plan, int build_plan, int uniform) {
    const int lo = rowptr[i], hi = rowptr[i + 1], deg = hi - lo;
    const int p = deg - clamped_b(b, i, deg, status);
    double tn = 0.0;
    float wsum = 0.f;
    int running = 0;
    for (int base = 0; base < deg; base += 32) {
        const int e = lo + base + lane;
        const bool valid = e < hi;
        const int j = valid ? checked(col[e], plan.n, status) : 0x7fffffff;
        // arrival of col[e]'s update at worker i: the sender's time, or the link's own time
        const double tj = valid ? order_time(t_edge ? t_edge[e] : t[j], status) : 0.0;
        int rank = 0;
        for (int base2 = 0; base2 < deg; base2 += 32) {
            const int e2 = lo + base2 + lane;
            const int j2 = e2 < hi ? col[e2] : 0x7fffffff;
            const double t2 = e2 < hi ? order_time(t_edge ? t_edge[e2] : t[j2], status) : 0.0;
            const int n2 = min(32, deg - base2);
            for (int s = 0; s < n2; ++s) {
                const double ts = __shfl_sync(0xffffffffu, t2, s);
                const int js = __shfl_sync(0xffffffffu, j2, s);
                rank += (ts < tj) || (ts == tj && js < j);
            }
        }
        const bool keep = valid && rank < p;
        if (valid) kept[e] = keep ? 1 : 0;
        if (keep) {
            waited[j] = 1u;
            tn = fmax(tn, tj);
        }
        if (build_plan) {
            float w = 0.f;
            if (keep) {
                const int dj = rowptr[j + 1] - rowptr[j];
                w = edge_weight(uniform, p, dj - clamped_b(b, j, dj, status));
                wsum += w;
            }
            plan_append(plan, i, lane, keep, j, w, running);
        }
    }
    tn = warp_max(tn);
    if (lane == 0) T_nbr_ws[i] = tn;
    if (build_plan) {
        wsum = warp_sum(wsum);
        plan_finish(plan, i, lane, running, uniform ? 1.0f / (1.0f + (float)p) : 1.0f - wsum);
    }
}

// Per-worker and per-round times (Section 3.2.2) once every worker's selection is visible: the calling
// block's threads share the workers; returns this thread's part of max T_worker over the participants
// (the caller reduces it over the block).  Clears the "waited for" flags for the next round.
__device__ __forceinline__ double round_times_part(int N, const int32_t* __restrict__ rowptr, const double* __restrict__ t,
                                                   const int32_t* __restrict__ b, const double* T_nbr_ws, double* T_nbr_out,
                                                   double* T_worker, uint32_t* waited, uint32_t* status) {
    double tr = 0.0;
    for (int w = threadIdx.x; w < N; w += blockDim.x) {
        const int deg = rowptr[w + 1] - rowptr[w];
        int bw = b[w];
        bw = bw < 0 ? 0 : (bw > deg ? deg : bw);
        const int p = deg - bw;
        const bool part = p >= 1 || __ldcg(&waited[w]) != 0u;
        const double tw = order_time(t[w], status);
        const double tn = __ldcg(&T_nbr_ws[w]);
        if (T_nbr_out) T_nbr_out[w] = tn;
        const double twk = p >= 1 ? fmax(tw, tn) : (part ? tw : 0.0);
        if (T_worker) T_worker[w] = twk;
        if (part) tr = fmax(tr, twk);  // T(k) = max of T_j over the participating workers
        waited[w] = 0u;
    }
    return tr;
}

// ------------------------------------------------------------------ masked mix + SGD, shared-memory panel
__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ float4 fma4(float w, float4 v, float4 a) {
    a.x = fmaf(w, v.x, a.x);
    a.y = fmaf(w, v.y, a.y);
    a.z = fmaf(w, v.z, a.z);
    a.w = fmaf(w, v.w, a.w);
    return a;
}

// One panel of 4*GS columns of all N rows by a block of THREADS threads (Eqs. 4-5, or Eq. 3 over the kept
// set): the panel of X (and G) is staged in shared memory sm [N][GS] as x - lr*g (or x), then every output
// row is the weighted sum of staged rows in plan order (self first, then the kept neighbours in CSR order).
// The caller puts a block barrier after it before the next panel.  G == nullptr: G = 0.
template <int GS, int THREADS, bool NC = true>
__device__ __forceinline__ void mix_panel_body(int panel, float4* sm, int N, long long ld, const float* X, const float* G,
                                               float lr, const float* __restrict__ lr_pw, float* Xout, uint16_t* __restrict__ shadow,
                                               const MixPlan& plan, int mix_then_correct) {
    const int tid = threadIdx.x;
    const int q = tid % GS;
    const int gid = tid / GS;
    constexpr int kGroups = THREADS / GS;
    const int total = N * GS;
    const long long col0 = (long long)panel * (4 * GS);
    // ---- stage the panel: x (Eq. 3 order) or x - lr*g (Eq. 4) ----
#pragma unroll 4
    for (int idx = tid; idx < total; idx += THREADS) {
        const int r = idx / GS;
        const long long c = col0 + 4 * (idx % GS);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < ld) {
            v = ldg4(X + (size_t)r * ld + c);
            if (G && !mix_then_correct) {
                const float4 g = load_g<NC>(reinterpret_cast<const float4*>(G + (size_t)r * ld + c));
                const float nlr = -(lr_pw ? lr_pw[r] : lr);
                v = fma4(nlr, g, v);
            }
        }
        sm[idx] = v;
    }
    __syncthreads();
    // ---- every output row of the panel ----
    const long long c = col0 + 4 * q;
    for (int i = gid; i < N; i += kGroups) {
        const float ws = plan.w_self[i];
        const float4 self = sm[i * GS + q];
        float4 acc = make_float4(ws * self.x, ws * self.y, ws * self.z, ws * self.w);
        const int cnt = plan.cnt[i];
        const int4* pi = reinterpret_cast<const int4*>(plan.idx + (size_t)i * plan.stride);
        const float4* pw = reinterpret_cast<const float4*>(plan.w + (size_t)i * plan.stride);
        for (int k = 0; k < cnt; k += 4) {
            int4 j = load_g<NC>(pi + (k >> 2));
            const float4 w = load_g<NC>(pw + (k >> 2));
            j.x = checked(j.x, N, plan.status); j.y = checked(j.y, N, plan.status);
            j.z = checked(j.z, N, plan.status); j.w = checked(j.w, N, plan.status);
            acc = fma4(w.x, sm[j.x * GS + q], acc);
            acc = fma4(w.y, sm[j.y * GS + q], acc);
            acc = fma4(w.z, sm[j.z * GS + q], acc);
            acc = fma4(w.w, sm[j.w * GS + q], acc);
        }
        if (c < ld) {
            if (G && mix_then_correct) {
                const float4 g = load_g<NC>(reinterpret_cast<const float4*>(G + (size_t)i * ld + c));
                acc = fma4(-(lr_pw ? lr_pw[i] : lr), g, acc);
            }
            *reinterpret_cast<float4*>(Xout + (size_t)i * ld + c) = acc;
            if (shadow) *reinterpret_cast<uint2*>(shadow + (size_t)i * ld + c) = pack_bf16x4_rn(acc.x, acc.y, acc.z, acc.w);
        }
    }
}

}  // namespace dev
}  // namespace dbw
