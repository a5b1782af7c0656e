// Mini-batch stochastic gradient (Eq. 2) with the dense layers on the 5th-generation tensor cores:
// BF16 operands (activations, and weights cast from the fp32 master rows every round), fp32
// accumulation in tensor memory, fp32 gradients.  No operand is ever transposed in memory: the MMA
// reads an operand either K-major (the reduction index contiguous) or MN-major (the row / column
// index contiguous), chosen per GEMM:
//   forward   Z_{l+1} = A_l W_l^T       A: A_l      [B][in]   K-major    B: W_l      [out][in]  K-major
//   dW_l            = dZ_{l+1}^T A_l    A: dZ_{l+1} [B][out]  MN-major   B: A_l      [B][in]    MN-major
//   dA_l            = dZ_{l+1} W_l      A: dZ_{l+1} [B][out]  K-major    B: W_l      [out][in]  MN-major
// Tiles are staged by TMA (3-D maps; 128-byte swizzle; no multicast) through an mbarrier ring, one
// elected thread issues tcgen05.mma into one of two accumulator buffers in tensor memory, and eight
// warps drain the finished buffer with tcgen05.ld into the fused epilogues (bias + ReLU + bf16
// cast, ReLU mask, or fp32 straight into G) while the next tile is already being multiplied.  The
// last layer (a handful of classes) and the loss run on the CUDA cores from the fp32 master weights.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <vector>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace dbw {

namespace {

typedef __nv_bfloat16 bf16;

// ----------------------------------------------------------------------------- PTX wrappers
using namespace ptx;

// Every mbarrier wait is bounded: after kSpinLimit failed polls the status word is flagged, the CTA's abort
// word is set and all later waits of the CTA return at once, so that every role still reaches the end of
// the kernel and tensor memory is released.
constexpr uint32_t kSpinLimit = 1u << 24;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort, uint32_t* status) {
    return mbar_wait_bounded<false>(bar, parity, kSpinLimit, 0, abort, status);
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// MN-major operand tiles of this file are staged in chunks of 64 (MN) x 64 (K rows): chunks 8192 bytes apart
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t smem_addr) { return mnmajor_sw128_desc(smem_addr, 8192); }

// two floats -> packed bf16x2 (low half = first)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ bool bf16_bits_positive(uint32_t bits16) { return (bits16 & 0x8000u) == 0 && (bits16 & 0x7fffu) != 0; }

// ----------------------------------------------------------------------------- tensor-core GEMM
constexpr int BM = 128, BK = 64, UMMA_K = 16;  // tile: 128 rows x BN columns (128 or 256) x 64 deep
constexpr int TILE_BYTES = BM * BK * 2;  // 16 KiB per 128-row operand tile
constexpr int GEMM_THREADS = 320;  // TMA warp, MMA warp, eight epilogue warps (two per accumulator lane quarter)
constexpr int EPI_WARPS = 8;
constexpr size_t gemm_smem(int stages, int bn) {
    return (size_t)stages * (TILE_BYTES + bn * BK * 2) + 8 * 32 * 36 * 4 /*epilogue staging*/ + 1024 /*align slack*/ + 256 /*barriers*/;
}
// kind::f16, D = f32, A = B = bf16, M = 128, N = bn; bits 15 / 16 select MN-major A / B operands
__host__ __device__ constexpr uint32_t idesc_for(int bn, bool a_mn, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(bn >> 3) << 17) |
           ((uint32_t)(BM >> 4) << 24);
}

enum { EPI_FWD = 0, EPI_DA = 1, EPI_DW = 2 };

struct TcArgs {
    int M, N, K, epi;
    bf16* out;  long long out_z;  int out_pitch;    // [M][N] bf16 (EPI_FWD, EPI_DA)
    float* outf; long long outf_z; long long outf_pitch;  // [M][N] fp32 (EPI_DW)
    const float* bias; long long bias_z;            // fp32 [N] (EPI_FWD)
    const bf16* mask; long long mask_z; int mask_pitch;   // bf16 [M][N]: keep where > 0 (EPI_DA)
    uint32_t* status;
};

constexpr int STAGING_FLOATS = EPI_WARPS * 32 * 36;  // per epilogue warp a 32 x 32 fp32 block, rows 36 words apart

// Persistent, warp-specialised GEMM: one CTA per SM walks the tiles (n fastest, then m, then worker).
// Warp 0 streams operand tiles by TMA through a STAGES-deep ring, warp 1 issues the MMAs into one of
// ACC accumulator buffers in tensor memory, warps 2-9 drain a finished buffer through the epilogue
// while the next tile's loads and MMAs are already running.
template <int STAGES, int BN, int ACC, bool AMN, bool BMN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, TcArgs g, int tiles_m,
               int tiles_n, int n_tiles) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int TILE_B_BYTES = BN * BK * 2;
    constexpr uint32_t IDESC = idesc_for(BN, AMN, BMN);
    uint8_t* tilesA = smem;
    uint8_t* tilesB = smem + STAGES * TILE_BYTES;
    float* staging = reinterpret_cast<float*>(smem + STAGES * (TILE_BYTES + TILE_B_BYTES));
    uint64_t* full = reinterpret_cast<uint64_t*>(staging + STAGING_FLOATS);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + ACC;
    uint64_t* drain = acc_empty + ACC;  // shutdown after an expired wait: completion of the MMAs issued so far
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile uint32_t* abort = tmem_slot + 1;  // set by the first wait that runs out; every later wait returns at once

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (g.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        *abort = 0u;
        mbar_init(drain, 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < ACC; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], EPI_WARPS);  // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(ACC * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;  // k-blocks issued so far, over all tiles of this CTA
            bool live = true;
            for (int tile = blockIdx.x; tile < n_tiles && live; tile += gridDim.x) {
                const int n0 = (tile % tiles_n) * BN, m0 = ((tile / tiles_n) % tiles_m) * BM, z = tile / (tiles_n * tiles_m);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (it >= STAGES && !mbar_wait(&empty[s], ((it / STAGES) - 1) & 1, abort, g.status)) {
                        live = false;  // a wait ran out somewhere in this CTA: issue nothing more
                        break;
                    }
                    mbar_expect_tx(&full[s], TILE_BYTES + TILE_B_BYTES);
                    if (!AMN) {
                        tma_load_3d(tilesA + s * TILE_BYTES, &tmA, kb * BK, m0, z, &full[s]);
                    } else {
#pragma unroll
                        for (int c = 0; c < BM / 64; ++c)  // MN-major: 64 x 64 chunks, coordinates (mn, k row, worker)
                            tma_load_3d(tilesA + s * TILE_BYTES + c * 8192, &tmA, m0 + c * 64, kb * BK, z, &full[s]);
                    }
                    if (!BMN) {
                        tma_load_3d(tilesB + s * TILE_B_BYTES, &tmB, kb * BK, n0, z, &full[s]);
                    } else {
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c)
                            tma_load_3d(tilesB + s * TILE_B_BYTES + c * 8192, &tmB, n0 + c * 64, kb * BK, z, &full[s]);
                    }
                }
            }
            // the copies still in flight (the last STAGES at most) have landed before this CTA leaves
            for (int j = it > STAGES ? it - STAGES : 0; j < it; ++j) mbar_wait_quiet<false>(&full[j % STAGES], (j / STAGES) & 1, 1u << 20);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int it = 0, lt = 0;
            bool live = true;
            for (int tile = blockIdx.x; tile < n_tiles && live; tile += gridDim.x, ++lt) {
                const int buf = lt % ACC;
                if (lt >= ACC) {  // the epilogue must have drained this buffer's previous tile
                    if (!mbar_wait(&acc_empty[buf], ((lt / ACC) - 1) & 1, abort, g.status)) break;
                    tc_fence_after();
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(&full[s], (it / STAGES) & 1, abort, g.status)) {
                        live = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tilesA + s * TILE_BYTES), sb = smem_u32(tilesB + s * TILE_B_BYTES);
                    const uint64_t da = AMN ? mnmajor_desc(sa) : kmajor_sw128_desc(sa);
                    const uint64_t db = BMN ? mnmajor_desc(sb) : kmajor_sw128_desc(sb);
                    // 16 further along K: 32 bytes inside the swizzle atom (K-major) or 16 rows of 128 bytes (MN-major)
                    constexpr uint64_t ka = (AMN ? UMMA_K * 128 : UMMA_K * 2) / 16, kbs = (BMN ? UMMA_K * 128 : UMMA_K * 2) / 16;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        tc_mma_bf16(d_tmem, da + (uint64_t)k * ka, db + (uint64_t)k * kbs, IDESC, (kb > 0 || k > 0) ? 1u : 0u);
                    tc_commit(&empty[s]);  // frees the stage once these MMAs have read it
                }
                if (live) tc_commit(&acc_full[buf]);
            }
            if (*abort) {  // shutdown after an expired wait: the MMAs issued so far are complete before tensor memory is freed
                tc_commit(drain);
                mbar_wait_quiet<false>(drain, 0, 1u << 20);
            }
        }
    } else {
        // ---- epilogue: warp w owns accumulator lanes 32*(w%4) .. +31, i.e. those output rows, and
        // one half of the tile's columns (two warps share a lane quarter) ----
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        float* stg = staging + (warp - 2) * (32 * 36);
        int lt = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++lt) {
            const int n0 = (tile % tiles_n) * BN, m0 = ((tile / tiles_n) % tiles_m) * BM, z = tile / (tiles_n * tiles_m);
            const int buf = lt % ACC;
            const bool ready = mbar_wait(&acc_full[buf], (lt / ACC) & 1, abort, g.status);
            if (!__all_sync(0xffffffffu, ready)) break;  // a wait ran out: leave together (the tensor-memory loads below are warp-collective)
            tc_fence_after();
            const int m = m0 + q * 32 + lane;
            const bool m_ok = m < g.M;
            for (int c = half * (BN / 64); c < (half + 1) * (BN / 64); ++c) {
                const int nb = n0 + c * 32;
                if (nb >= g.N) break;  // warp-uniform
                uint32_t r[32];
                tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c * 32), r);
                if (g.epi == EPI_DW) {
                    // Each lane holds one row of a 32 x 32 fp32 block.  It goes through shared memory
                    // (rows 36 words apart keep both 128-bit phases conflict-free) so that a warp
                    // stores four full 128-byte lines per instruction.
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<uint4*>(stg + lane * 36 + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                    __syncwarp();
                    const int f4 = lane & 7;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int row = 4 * i + (lane >> 3);
                        const int mm = m0 + q * 32 + row;
                        const float4 val = *reinterpret_cast<const float4*>(stg + row * 36 + 4 * f4);
                        if (mm < g.M && nb + 4 * f4 < g.N)
                            *reinterpret_cast<float4*>(g.outf + (size_t)z * g.outf_z + (size_t)mm * g.outf_pitch + nb + 4 * f4) = val;
                    }
                    __syncwarp();
                    continue;
                }
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
                if (g.epi == EPI_FWD) {
                    const float* bias = g.bias + (size_t)z * g.bias_z + nb;
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j] + ((nb + j < g.N) ? __ldg(bias + j) : 0.f), 0.f);
                } else if (m_ok) {  // EPI_DA: ReLU'(z) = [a > 0]
                    const bf16* mk = g.mask + (size_t)z * g.mask_z + (size_t)m * g.mask_pitch + nb;
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        if (nb + j < g.N) {
                            const uint4 u = __ldg(reinterpret_cast<const uint4*>(mk + j));
                            const uint32_t wds[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (!bf16_bits_positive((wds[e >> 1] >> (16 * (e & 1))) & 0xffffu)) v[j + e] = 0.f;
                        }
                }
                uint32_t o[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j] = pack_bf16x2(v[2 * j], v[2 * j + 1]);
                if (m_ok) {
                    bf16* dst = g.out + (size_t)z * g.out_z + (size_t)m * g.out_pitch + nb;
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        if (nb + j < g.N)
                            *reinterpret_cast<uint4*>(dst + j) = make_uint4(o[j / 2], o[j / 2 + 1], o[j / 2 + 2], o[j / 2 + 3]);
                }
            }
            // this warp's reads of the buffer are complete (tcgen05.wait::ld): hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(ACC * BN) : "memory");
    }
}

// ----------------------------------------------------------------------------- casts and gathers
// fp32 [rows][cols] (row pitch src_pitch) -> bf16 [rows][cols] (row pitch cols).  Rows may be
// indirect (row_idx: mini-batch gather).  cols % 8 == 0.  Every thread converts 16 consecutive floats
// of one row: four 128-bit loads, two 128-bit stores.
__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
}

__global__ void __launch_bounds__(256)
cast_tile_kernel(int rows, int cols, const float* __restrict__ src, long long src_z, long long src_pitch,
                 const int32_t* __restrict__ row_idx, int idx_z, int idx_limit, bf16* __restrict__ dst, long long dst_z,
                 uint32_t* status) {
    const int z = blockIdx.z;
    const int t = threadIdx.x;
    const int r = blockIdx.y * 64 + (t >> 2);
    const int c0 = blockIdx.x * 64 + (t & 3) * 16;
    if (r >= rows || c0 >= cols) return;
    long long sr = r;
    if (row_idx) {
        int s = row_idx[(size_t)z * idx_z + r];
        if (s < 0 || s >= idx_limit) {
            atomicOr(status, DBW_STATUS_BAD_INDEX);
            s = s < 0 ? 0 : idx_limit - 1;
        }
        sr = s;
    }
    const float* p = src + (size_t)z * src_z + sr * src_pitch + c0;
    bf16* d = dst + (size_t)z * dst_z + (size_t)r * cols + c0;
    float v[16];
#pragma unroll
    for (int e = 0; e < 16; e += 4) {
        float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c0 + e < cols) f = __ldg(reinterpret_cast<const float4*>(p + e));
        v[e] = f.x; v[e + 1] = f.y; v[e + 2] = f.z; v[e + 3] = f.w;
    }
    *reinterpret_cast<uint4*>(d) = pack8(v);
    if (c0 + 8 < cols) *reinterpret_cast<uint4*>(d + 8) = pack8(v + 8);
}

// Labels of the mini-batch; a label outside [0, C) is clamped and reported (the batch index is
// reported by the feature gather).
__global__ void gather_labels_kernel(int B, int S, int C, const int32_t* __restrict__ labels, const int32_t* __restrict__ batch_idx,
                                     int32_t* __restrict__ ylab, uint32_t* status) {
    const int i = blockIdx.x;
    for (int s = threadIdx.x; s < B; s += blockDim.x) {
        int src = batch_idx[(size_t)i * B + s];
        src = src < 0 ? 0 : (src >= S ? S - 1 : src);
        int y = labels[(size_t)i * S + src];
        if (y < 0 || y >= C) {
            atomicOr(status, DBW_STATUS_BAD_INDEX);
            y = y < 0 ? 0 : C - 1;
        }
        ylab[(size_t)i * B + s] = y;
    }
}

// db[o] = sum over the batch of dZ[s][o] (dZ bf16 [B][out], out even).  A block of 256 threads owns 128
// outputs (block bx of worker i): a thread sums two adjacent outputs (one 32-bit load per sample) over every
// fourth sample, and the four partial sums are added through shared memory in a fixed order.
__device__ __forceinline__ void bias_grad_bf16_block(int bx, int i, int out_dim, int B, const bf16* __restrict__ dz, long long dz_z,
                                                     float* __restrict__ G, long long ld, long long b_off, float2 (*part)[64]) {
    const int pair = threadIdx.x & 63, slice = threadIdx.x >> 6;
    const int o = bx * 128 + 2 * pair;
    float2 s = make_float2(0.f, 0.f);
    if (o < out_dim) {
        const bf16* p = dz + (size_t)i * dz_z + o;
#pragma unroll 8
        for (int m = slice; m < B; m += 4) {
            const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(p + (size_t)m * out_dim));
            s.x += __uint_as_float(v << 16);
            s.y += __uint_as_float(v & 0xffff0000u);
        }
    }
    part[slice][pair] = s;
    __syncthreads();
    if (slice == 0 && o < out_dim) {
        const float2 a = part[0][pair], b = part[1][pair], c = part[2][pair], d = part[3][pair];
        G[(size_t)i * ld + b_off + o] = ((a.x + b.x) + c.x) + d.x;
        G[(size_t)i * ld + b_off + o + 1] = ((a.y + b.y) + c.y) + d.y;
    }
}

// ----------------------------------------------------------------------------- last layer on CUDA cores
constexpr int kMaxClasses = 32;
constexpr size_t kHeadStageBytes = 100 * 1024;  // last-layer weights up to this size are staged in shared memory (two CTAs per SM)

// logits = A W^T + b (A bf16 [B][K], W fp32 master [C][K]), then dZ = (softmax - onehot)/B and the
// per-sample loss.  A warp takes HS samples at once: each lane owns 8 consecutive k of every
// 256-wide chunk (one 128-bit load per sample, two per weight row), so a weight row fetched from
// L1/L2 is used for HS samples.
template <int CP, int HS>
__global__ void __launch_bounds__(128)
head_forward_kernel(int B, int K, int C, const bf16* __restrict__ A, const float* __restrict__ X, long long ld, long long w_off,
                    long long b_off, const int32_t* __restrict__ ylab, float* __restrict__ dzL, float* __restrict__ loss_s) {
    const int i = blockIdx.y;
    const int s0 = (blockIdx.x * 4 + (threadIdx.x >> 5)) * HS;
    const int lane = threadIdx.x & 31;
    if (s0 >= B) return;
    const float* W = X + (size_t)i * ld + w_off;
    float acc[HS][CP];
#pragma unroll
    for (int u = 0; u < HS; ++u)
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[u][c] = 0.f;
    auto load_a = [&](int kc, uint4 (&raw)[HS]) {
        const int k = kc + lane * 8;
#pragma unroll
        for (int u = 0; u < HS; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (k < K && s0 + u < B) raw[u] = __ldg(reinterpret_cast<const uint4*>(A + ((size_t)i * B + s0 + u) * K + k));
        }
    };
    uint4 cur[HS], nxt[HS];
    load_a(0, cur);
    for (int kc = 0; kc < K; kc += 256) {
        load_a(kc + 256, nxt);  // next chunk in flight while this one is used (all zero past the end)
        const int k = kc + lane * 8;
        if (k < K) {
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                if (c < C) {
                    const float4 w0 = __ldg(reinterpret_cast<const float4*>(W + (size_t)c * K + k));
                    const float4 w1 = __ldg(reinterpret_cast<const float4*>(W + (size_t)c * K + k + 4));
                    const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                    for (int u = 0; u < HS; ++u) {
                        const uint32_t w4[4] = {cur[u].x, cur[u].y, cur[u].z, cur[u].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {  // bf16 -> fp32 is a 16-bit shift
                            acc[u][c] = fmaf(__uint_as_float(w4[e] << 16), wv[2 * e], acc[u][c]);
                            acc[u][c] = fmaf(__uint_as_float(w4[e] & 0xffff0000u), wv[2 * e + 1], acc[u][c]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < HS; ++u) cur[u] = nxt[u];
    }
#pragma unroll
    for (int u = 0; u < HS; ++u) {
        float z_mine = 0.f;  // lane c ends up holding logit c of sample s0 + u
#pragma unroll
        for (int c = 0; c < CP; ++c) {
            float v = acc[u][c];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == c) z_mine = v;
        }
        const int s = s0 + u;
        if (s >= B) continue;  // warp-uniform
        const float zl = lane < C ? z_mine + X[(size_t)i * ld + b_off + lane] : -INFINITY;
        float mx = zl;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float e = lane < C ? expf(zl - mx) : 0.f;
        float sum = e;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const int y = ylab[(size_t)i * B + s];
        if (lane < C) dzL[((size_t)i * B + s) * C + lane] = (e / sum - (lane == y ? 1.f : 0.f)) / (float)B;
        const float zy = __shfl_sync(0xffffffffu, zl, y & 31);
        if (lane == 0) loss_s[(size_t)i * B + s] = (mx + logf(sum)) - zy;
    }
}

// The same step with the layer's weights in shared memory.  head_forward_kernel fetches every weight row
// again for each pair of samples (L1/L2 latency on every class: 8 % of the fp32 rate on the 1024 -> 10 layer);
// here a CTA of eight warps stages the worker's W (C x K fp32) once and works through a contiguous range of
// (worker, 8 HS samples) items, restaging only when the worker changes; a warp takes HS samples at once, so a
// weight row read from shared memory is used for HS samples.  Same arithmetic and order as head_forward_kernel.
template <int CP, int HS>
__global__ void __launch_bounds__(256, 2)
head_forward_staged_kernel(int N, int B, int K, int C, const bf16* __restrict__ A, const float* __restrict__ X, long long ld,
                           long long w_off, long long b_off, const int32_t* __restrict__ ylab, float* __restrict__ dzL,
                           float* __restrict__ loss_s) {
    extern __shared__ float4 sw4[];  // [C][K]
    const float* sw = reinterpret_cast<const float*>(sw4);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int groups = (B + 8 * HS - 1) / (8 * HS);  // items per worker
    const int items = N * groups;
    const int per = (items + gridDim.x - 1) / gridDim.x;
    const int it0 = blockIdx.x * per, it1 = min(items, it0 + per);
    int staged = -1;
    for (int it = it0; it < it1; ++it) {
        const int i = it / groups, s0 = (it % groups) * 8 * HS + warp * HS;
        if (i != staged) {  // the same for all threads of the CTA
            __syncthreads();
            const float4* src = reinterpret_cast<const float4*>(X + (size_t)i * ld + w_off);
            for (int e = threadIdx.x; e < C * K / 4; e += 256) sw4[e] = __ldg(src + e);
            __syncthreads();
            staged = i;
        }
        if (s0 >= B) continue;  // warp-uniform; the CTA barriers above depend on the item only
        float acc[HS][CP];
#pragma unroll
        for (int u = 0; u < HS; ++u)
#pragma unroll
            for (int c = 0; c < CP; ++c) acc[u][c] = 0.f;
        auto load_a = [&](int kc, uint4 (&raw)[HS]) {
            const int k = kc + lane * 8;
#pragma unroll
            for (int u = 0; u < HS; ++u) {
                raw[u] = make_uint4(0u, 0u, 0u, 0u);
                if (k < K && s0 + u < B) raw[u] = __ldg(reinterpret_cast<const uint4*>(A + ((size_t)i * B + s0 + u) * K + k));
            }
        };
        uint4 cur[HS], nxt[HS];
        load_a(0, cur);
        for (int kc = 0; kc < K; kc += 256) {
            load_a(kc + 256, nxt);  // next chunk in flight while this one is used (all zero past the end)
            const int k = kc + lane * 8;
            if (k < K) {
                float av[HS][8];
#pragma unroll
                for (int u = 0; u < HS; ++u) {
                    const uint32_t w4[4] = {cur[u].x, cur[u].y, cur[u].z, cur[u].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {  // bf16 -> fp32 is a 16-bit shift
                        av[u][2 * e] = __uint_as_float(w4[e] << 16);
                        av[u][2 * e + 1] = __uint_as_float(w4[e] & 0xffff0000u);
                    }
                }
#pragma unroll
                for (int c = 0; c < CP; ++c) {
                    if (c < C) {
                        const float4 w0 = *reinterpret_cast<const float4*>(sw + (size_t)c * K + k);
                        const float4 w1 = *reinterpret_cast<const float4*>(sw + (size_t)c * K + k + 4);
                        const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                        for (int u = 0; u < HS; ++u)
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[u][c] = fmaf(av[u][e], wv[e], acc[u][c]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < HS; ++u) cur[u] = nxt[u];
        }
#pragma unroll
        for (int u = 0; u < HS; ++u) {
            float z_mine = 0.f;  // lane c ends up holding logit c of sample s0 + u
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                if (c < C) {
                    float v = acc[u][c];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (lane == c) z_mine = v;
                }
            }
            const int s = s0 + u;
            if (s >= B) continue;  // warp-uniform
            const float zl = lane < C ? z_mine + __ldg(X + (size_t)i * ld + b_off + lane) : -INFINITY;
            float mx = zl;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float e = lane < C ? expf(zl - mx) : 0.f;
            float sum = e;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const int y = ylab[(size_t)i * B + s];
            if (lane < C) dzL[((size_t)i * B + s) * C + lane] = (e / sum - (lane == y ? 1.f : 0.f)) / (float)B;
            const float zy = __shfl_sync(0xffffffffu, zl, y & 31);
            if (lane == 0) loss_s[(size_t)i * B + s] = (mx + logf(sum)) - zy;
        }
    }
}

// Mean loss of worker i from its per-sample losses, by the first warp of a block (fixed order).
__device__ __forceinline__ void loss_reduce_block(int i, int B, const float* __restrict__ loss_s, float* __restrict__ loss) {
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    float s = 0.f;
    for (int m = lane; m < B; m += 32) s += loss_s[(size_t)i * B + m];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) loss[i] = s / (float)B;
}

// Last layer backward; a thread owns KPT consecutive input features k:
//   dW[c][k] = sum_s dZ[s][c] A[s][k],  db[c] = sum_s dZ[s][c],
//   dZprev[s][k] = [A[s][k] > 0] * sum_c dZ[s][c] W[c][k]   (bf16).
// dZ of the worker sits in shared memory and is read as 128-bit broadcasts.
template <int CP, int KPT>
__global__ void __launch_bounds__(64)
head_backward_kernel(int B, int K, int C, const bf16* __restrict__ A, const float* __restrict__ X, long long ld,
                     long long w_off, const float* __restrict__ dzL, float* __restrict__ G, float* __restrict__ dwp,
                     bf16* __restrict__ dzP) {
    // blockIdx.z splits the batch (in chunks of 8 samples) so that enough blocks are in flight; with
    // more than one part the dW partial sums go to dwp [part][worker][C][K] and grad_tail_kernel
    // adds them in a fixed order.
    extern __shared__ float4 sdz4[];  // [samples of this part][CP] floats
    float* sdz = reinterpret_cast<float*>(sdz4);
    const int i = blockIdx.y;
    const int nch = B / 8;
    const int s_lo = 8 * (int)((long long)blockIdx.z * nch / gridDim.z);
    const int s_hi = 8 * (int)((long long)(blockIdx.z + 1) * nch / gridDim.z);
    for (int e = threadIdx.x; e < (s_hi - s_lo) * CP; e += blockDim.x) {
        const int s = s_lo + e / CP, c = e % CP;
        sdz[e] = c < C ? dzL[((size_t)i * B + s) * C + c] : 0.f;
    }
    __syncthreads();
    const int k = (blockIdx.x * 64 + threadIdx.x) * KPT;
    if (k >= K) return;  // K % 8 == 0, so k + KPT <= K
    float w[CP][KPT], dw[CP][KPT];
#pragma unroll
    for (int c = 0; c < CP; ++c)
#pragma unroll
        for (int q = 0; q < KPT; ++q) {
            w[c][q] = c < C ? X[(size_t)i * ld + w_off + (size_t)c * K + k + q] : 0.f;
            dw[c][q] = 0.f;
        }
    const bf16* a = A + (size_t)i * B * K + k;
    auto load_a = [&](int s0, uint32_t (&raw)[8]) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            raw[u] = 0u;
            if (s0 + u < s_hi) {
                if (KPT == 2)
                    raw[u] = __ldg(reinterpret_cast<const uint32_t*>(a + (size_t)(s0 + u) * K));
                else
                    raw[u] = (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(a + (size_t)(s0 + u) * K)) << 16;
            }
        }
    };
    uint32_t cur[8], nxt[8];
    load_a(s_lo, cur);
    for (int s0 = s_lo; s0 < s_hi; s0 += 8) {  // B % 8 == 0
        load_a(s0 + 8, nxt);  // next eight samples in flight while these are used
        float dav[KPT][8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = s0 + u;
            float av[KPT];
            if (KPT == 2) {
                av[0] = __uint_as_float(cur[u] << 16);
                av[KPT - 1] = __uint_as_float(cur[u] & 0xffff0000u);
            } else {
                av[0] = __uint_as_float(cur[u]);
            }
            float da[KPT];
#pragma unroll
            for (int q = 0; q < KPT; ++q) da[q] = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < CP / 4; ++c4) {
                const float4 d4 = sdz4[(s - s_lo) * (CP / 4) + c4];
                const float dz[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int q = 0; q < KPT; ++q) {
                        dw[4 * c4 + e][q] = fmaf(dz[e], av[q], dw[4 * c4 + e][q]);
                        da[q] = fmaf(dz[e], w[4 * c4 + e][q], da[q]);
                    }
            }
#pragma unroll
            for (int q = 0; q < KPT; ++q) dav[q][u] = av[q] > 0.f ? da[q] : 0.f;
            if (dzP) {
                if (KPT == 2)
                    *reinterpret_cast<uint32_t*>(dzP + ((size_t)i * B + s) * K + k) = pack_bf16x2(dav[0][u], dav[KPT - 1][u]);
                else
                    dzP[((size_t)i * B + s) * K + k] = __float2bfloat16_rn(dav[0][u]);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) cur[u] = nxt[u];
    }
    float* dst = gridDim.z == 1 ? G + (size_t)i * ld + w_off : dwp + ((size_t)blockIdx.z * gridDim.y + i) * C * K;
#pragma unroll
    for (int c = 0; c < CP; ++c)
        if (c < C)
#pragma unroll
            for (int q = 0; q < KPT; ++q) dst[(size_t)c * K + k + q] = dw[c][q];
}

// dW of the last layer = sum of the batch parts' partial sums (fixed order), and db[c] = sum_s dZ[s][c]; block bx of worker i.
__device__ __forceinline__ void head_reduce_block(int bx, int i, int B, int K, int C, int parts, int workers, const float* __restrict__ dwp,
                                                  const float* __restrict__ dzL, float* __restrict__ G, long long ld, long long w_off,
                                                  long long b_off) {
    const int e = bx * 256 + threadIdx.x;
    if (parts > 1 && e < C * K) {
        float t = 0.f;
        for (int z = 0; z < parts; ++z) t += dwp[((size_t)z * workers + i) * C * K + e];
        G[(size_t)i * ld + w_off + e] = t;
    }
    if (e < C) {
        float t = 0.f;
        for (int s = 0; s < B; ++s) t += dzL[((size_t)i * B + s) * C + e];
        G[(size_t)i * ld + b_off + e] = t;
    }
}

// Everything of the gradient that is a reduction over the batch and that only the mix needs, in ONE launch
// after the last GEMM (four launches of 3-19 us each before): the tensor-core layers' bias gradients, the last
// layer's dW and db from its batch parts, and the workers' mean losses.  blockIdx.y = worker; blockIdx.x
// selects the task: [first[t], first[t + 1]) = bias gradient of layer t, then the last layer's reduction,
// then one block for the loss.
struct TailArgs {
    int n_bias;
    int first[DBW_MAX_LAYERS + 2];
    int out_dim[DBW_MAX_LAYERS];
    const bf16* dz[DBW_MAX_LAYERS];
    long long b_off[DBW_MAX_LAYERS];
    int B, K, C, parts, workers;
    const float* dwp;
    const float* dzL;
    const float* loss_s;
    float* loss;  // nullable
    float* G;
    long long ld, w_off_last, b_off_last;
};

__global__ void __launch_bounds__(256) grad_tail_kernel(TailArgs a) {
    __shared__ float2 part[4][64];
    const int bx = blockIdx.x, i = blockIdx.y;
    for (int t = 0; t < a.n_bias; ++t)
        if (bx >= a.first[t] && bx < a.first[t + 1]) {  // the same for all threads of the block
            bias_grad_bf16_block(bx - a.first[t], i, a.out_dim[t], a.B, a.dz[t], (long long)a.B * a.out_dim[t], a.G, a.ld, a.b_off[t], part);
            return;
        }
    if (bx < a.first[a.n_bias + 1]) {
        head_reduce_block(bx - a.first[a.n_bias], i, a.B, a.K, a.C, a.parts, a.workers, a.dwp, a.dzL, a.G, a.ld, a.w_off_last, a.b_off_last);
        return;
    }
    if (a.loss) loss_reduce_block(i, a.B, a.loss_s, a.loss);
}

// ----------------------------------------------------------------------------- host side
// MN-major operand [workers][K rows][MN] bf16 (MN contiguous): box = 64 (MN) x 64 (K rows) x 1.
bool make_operand_map_mn(CUtensorMap* map, const bf16* base, int MN, int Krows, int workers, long long worker_pitch = 0) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if (!worker_pitch) worker_pitch = (long long)MN * Krows;
    cuuint64_t dims[3] = {(cuuint64_t)MN, (cuuint64_t)Krows, (cuuint64_t)workers};
    cuuint64_t strides[2] = {(cuuint64_t)MN * 2, (cuuint64_t)worker_pitch * 2};
    cuuint32_t box[3] = {64, 64, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// K-major operand [workers][rows][K] bf16: box = 64 (K) x 128 (rows) x 1, 128-byte swizzle,
// out-of-range elements read as zero.
bool make_operand_map(CUtensorMap* map, const bf16* base, int K, int rows, int workers, long long worker_pitch = 0,
                      int box_rows = BM) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    if (!worker_pitch) worker_pitch = (long long)K * rows;  // dense blocks unless the operand lives inside a wider row
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)workers};
    cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)worker_pitch * 2};
    cuuint32_t box[3] = {BK, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct BF16State {
    bf16* A[DBW_MAX_LAYERS] = {};    // A_l   [N][B][dims[l]],  l = 0..L-1
    bf16* Wh[DBW_MAX_LAYERS] = {};   // W_l   [out][in] inside the bf16 shadow rows (worker pitch ld), l = 0..L-2
    bf16* dZ[DBW_MAX_LAYERS] = {};   // dZ_l  [N][B][dims[l]],  l = 1..L-1
    float* dzL = nullptr;            // [N][B][C]
    float* dwp = nullptr;            // [4][N][C][K_last] partial dW of the last layer
    float* loss_s = nullptr;         // [N][B]
    int32_t* ylab = nullptr;         // [N][B]
    CUtensorMap fwdA[DBW_MAX_LAYERS], fwdB[DBW_MAX_LAYERS], dwA[DBW_MAX_LAYERS], dwB[DBW_MAX_LAYERS],
        daA[DBW_MAX_LAYERS], daB[DBW_MAX_LAYERS];
    std::vector<void*> owned;
};

namespace {
template <typename T>
bool balloc(BF16State* st, T** p, size_t n) {
    if (!cuda_ok(cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T)))) return false;
    st->owned.push_back(*p);
    return true;
}

// Tile width for an output with N columns: 256 halves the operand re-reads out of L2 per output byte.
// The wide tile only when it still leaves at least one tile per SM (small problems keep more CTAs busy
// with 128-wide tiles).
int tile_bn(int N, int M, int workers, int sm_count) {
    if (N < 256) return 128;
    const long long wide_tiles = (long long)((N + 255) / 256) * ((M + BM - 1) / BM) * workers;
    return wide_tiles >= sm_count ? 256 : 128;
}

template <bool AMN, bool BMN>
int run_tc_major(const dbw_handle* h, const CUtensorMap& a, const CUtensorMap& b, const TcArgs& g, int workers, cudaStream_t s) {
    const int bn = tile_bn(g.N, g.M, workers, h->sm_count);
    const int tiles_n = (g.N + bn - 1) / bn, tiles_m = (g.M + BM - 1) / BM;
    const int n_tiles = tiles_n * tiles_m * workers;
    const int grid = n_tiles < h->sm_count ? n_tiles : h->sm_count;
    static PerDeviceOnce once;
    const int rc = once.run(h->device, []() -> int {
        DBW_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<4, 128, 2, AMN, BMN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(4, 128)));
        DBW_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<3, 256, 2, AMN, BMN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem(3, 256)));
        return DBW_OK;
    });
    if (rc) return rc;
    if (bn == 128)
        gemm_tc_kernel<4, 128, 2, AMN, BMN><<<grid, GEMM_THREADS, gemm_smem(4, 128), s>>>(a, b, g, tiles_m, tiles_n, n_tiles);
    else
        gemm_tc_kernel<3, 256, 2, AMN, BMN><<<grid, GEMM_THREADS, gemm_smem(3, 256), s>>>(a, b, g, tiles_m, tiles_n, n_tiles);
    DBW_LAUNCHED();
    return DBW_OK;
}

// While stage timing is on, every tensor-core GEMM launch sits between a pair of events of its own, so that the
// GEMMs' share of the gradient stage can be read back (dbw_profile_read, ms[3]).
cudaEvent_t gemm_event(dbw_handle* h) {
    if ((int)h->prof_gemm_events.size() <= h->prof_gemm_used) {
        cudaEvent_t e;
        if (!cuda_ok(cudaEventCreate(&e))) return nullptr;
        h->prof_gemm_events.push_back(e);
    }
    return h->prof_gemm_events[h->prof_gemm_used++];
}

int run_tc(dbw_handle* h, const CUtensorMap& a, const CUtensorMap& b, const TcArgs& g, int workers, cudaStream_t s,
           bool a_mn = false, bool b_mn = false) {
    const bool timed = h->profiling && h->prof_gemm_used < 2 * 16 * 4096;
    if (timed) {
        cudaEvent_t e = gemm_event(h);
        if (e) DBW_CUDA(cudaEventRecord(e, s));
    }
    const int rc = (a_mn && b_mn) ? run_tc_major<true, true>(h, a, b, g, workers, s)
                   : b_mn         ? run_tc_major<false, true>(h, a, b, g, workers, s)
                                  : run_tc_major<false, false>(h, a, b, g, workers, s);
    if (timed) {
        cudaEvent_t e = gemm_event(h);
        if (e) DBW_CUDA(cudaEventRecord(e, s));
    }
    return rc;
}
}  // namespace

int grad_bf16_alloc(dbw_handle* h) {
    const dbw_model_desc& m = h->model;
    const int L = m.n_layers, B = m.batch, N = h->N;
    // TMA needs 16-byte row pitches, the transposed stores 16-byte groups of samples
    if (B % 8) return DBW_ERR_BAD_MODEL;
    for (int l = 0; l < L; ++l)
        if (m.dims[l] % 8) return DBW_ERR_BAD_MODEL;
    if (m.dims[L] > kMaxClasses) return DBW_ERR_BAD_MODEL;
    if ((size_t)B * (m.dims[L] <= 16 ? 16 : 32) * 4 > 200 * 1024) return DBW_ERR_BAD_MODEL;
    BF16State* st = new (std::nothrow) BF16State();
    if (!st) return DBW_ERR_CUDA;
    h->bf16 = st;
    bool ok = true;
    const size_t NB = (size_t)N * B;
    for (int l = 0; l < L && ok; ++l) {
        ok = ok && balloc(st, &st->A[l], NB * m.dims[l]);
        if (l >= 1) ok = ok && balloc(st, &st->dZ[l], NB * m.dims[l]);
    }
    bf16* shadow = nullptr;
    ok = ok && balloc(st, &shadow, (size_t)N * h->ld);
    h->d_shadow = reinterpret_cast<uint16_t*>(shadow);
    for (int l = 0; l <= L - 2 && ok; ++l) st->Wh[l] = shadow + m.w_off[l];
    ok = ok && balloc(st, &st->dwp, (size_t)4 * N * m.dims[L] * m.dims[L - 1]);
    ok = ok && balloc(st, &st->dzL, NB * m.dims[L]) && balloc(st, &st->loss_s, NB) && balloc(st, &st->ylab, NB);
    if (!ok) return DBW_ERR_CUDA;
    for (int l = 0; l <= L - 2; ++l) {
        ok = ok && make_operand_map(&st->fwdA[l], st->A[l], m.dims[l], B, N);
        ok = ok && make_operand_map(&st->fwdB[l], st->Wh[l], m.dims[l], m.dims[l + 1], N, h->ld, tile_bn(m.dims[l + 1], B, N, h->sm_count));
        ok = ok && make_operand_map_mn(&st->dwA[l], st->dZ[l + 1], m.dims[l + 1], B, N);
        ok = ok && make_operand_map_mn(&st->dwB[l], st->A[l], m.dims[l], B, N);
        if (l >= 1) {
            ok = ok && make_operand_map(&st->daA[l], st->dZ[l + 1], m.dims[l + 1], B, N);
            ok = ok && make_operand_map_mn(&st->daB[l], st->Wh[l], m.dims[l], m.dims[l + 1], N, h->ld);
        }
    }
    if (!ok) return DBW_ERR_CUDA;
    DBW_CUDA(cudaFuncSetAttribute(head_forward_staged_kernel<12, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHeadStageBytes));
    DBW_CUDA(cudaFuncSetAttribute(head_forward_staged_kernel<16, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHeadStageBytes));
    DBW_CUDA(cudaFuncSetAttribute(head_backward_kernel<12, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    DBW_CUDA(cudaFuncSetAttribute(head_backward_kernel<16, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    DBW_CUDA(cudaFuncSetAttribute(head_backward_kernel<32, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    return DBW_OK;
}

void grad_bf16_free(dbw_handle* h) {
    if (!h->bf16) return;
    h->d_shadow = nullptr;
    for (void* p : h->bf16->owned) cudaFree(p);
    delete h->bf16;
    h->bf16 = nullptr;
}

int launch_grad_bf16(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss, cudaStream_t s) {
    const dbw_model_desc& m = h->model;
    BF16State* st = h->bf16;
    const int L = m.n_layers, B = m.batch, N = h->N, C = m.dims[L];
    int rc;
    // bf16 copies of the weights of the tensor-core layers (inside the shadow rows), unless the
    // previous mix already wrote the shadow of this very X.
    const bool have_shadow = h->track_params && h->shadow_valid && h->shadow_of == X;
    for (int l = 0; l <= L - 2 && !have_shadow; ++l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        cast_tile_kernel<<<dim3((in + 63) / 64, (out + 63) / 64, N), 256, 0, s>>>(
            out, in, X + m.w_off[l], h->ld, in, nullptr, 0, 0, st->Wh[l], h->ld, h->d_status);
        DBW_LAUNCHED();
    }
    // mini-batch gather: A_0 in bf16
    cast_tile_kernel<<<dim3((m.dims[0] + 63) / 64, (B + 63) / 64, N), 256, 0, s>>>(
        B, m.dims[0], h->feat, (long long)h->S * m.dims[0], m.dims[0], batch_idx, B, h->S, st->A[0], (long long)B * m.dims[0],
        h->d_status);
    DBW_LAUNCHED();
    gather_labels_kernel<<<N, 128, 0, s>>>(B, h->S, C, h->labels, batch_idx, st->ylab, h->d_status);
    DBW_LAUNCHED();
    // forward through the tensor-core layers
    for (int l = 0; l <= L - 2; ++l) {
        TcArgs g{};
        g.M = B; g.N = m.dims[l + 1]; g.K = m.dims[l]; g.epi = EPI_FWD;
        g.out = st->A[l + 1]; g.out_z = (long long)B * g.N; g.out_pitch = g.N;
        g.bias = X + m.b_off[l]; g.bias_z = h->ld;
        g.status = h->d_status;
        if ((rc = run_tc(h, st->fwdA[l], st->fwdB[l], g, N, s))) return rc;
    }
    // last layer, loss, and its backward
    const int K = m.dims[L - 1];
    bf16* dzP = L >= 2 ? st->dZ[L - 1] : nullptr;
    const size_t w_bytes = (size_t)C * K * sizeof(float);
    if (C <= 16 && w_bytes <= kHeadStageBytes && (m.w_off[L - 1] & 3) == 0) {  // weights staged in shared memory
        const int items = N * ((B + 31) / 32);
        const int grid = std::min(items, 2 * h->sm_count);
        if (C <= 12)  // ten classes: a quarter fewer accumulators than with the 16-class instance
            head_forward_staged_kernel<12, 4><<<grid, 256, w_bytes, s>>>(N, B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1], m.b_off[L - 1],
                                                                         st->ylab, st->dzL, st->loss_s);
        else
            head_forward_staged_kernel<16, 4><<<grid, 256, w_bytes, s>>>(N, B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1], m.b_off[L - 1],
                                                                         st->ylab, st->dzL, st->loss_s);
    } else if (C <= 16) {
        head_forward_kernel<16, 2><<<dim3((B + 7) / 8, N), 128, 0, s>>>(B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1],
                                                                       m.b_off[L - 1], st->ylab, st->dzL, st->loss_s);
    } else {
        head_forward_kernel<32, 2><<<dim3((B + 7) / 8, N), 128, 0, s>>>(B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1],
                                                                       m.b_off[L - 1], st->ylab, st->dzL, st->loss_s);
    }
    DBW_LAUNCHED();
    const int parts = B >= 64 ? 4 : 1;
    if (C <= 12)  // ten classes: a quarter fewer multiply-adds than with the 16-class instance
        head_backward_kernel<12, 2><<<dim3((K + 127) / 128, N, parts), 64, (size_t)B * 12 * 4, s>>>(
            B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1], st->dzL, G, st->dwp, dzP);
    else if (C <= 16)
        head_backward_kernel<16, 2><<<dim3((K + 127) / 128, N, parts), 64, (size_t)B * 16 * 4, s>>>(
            B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1], st->dzL, G, st->dwp, dzP);
    else
        head_backward_kernel<32, 1><<<dim3((K + 63) / 64, N, parts), 64, (size_t)B * 32 * 4, s>>>(
            B, K, C, st->A[L - 1], X, h->ld, m.w_off[L - 1], st->dzL, G, st->dwp, dzP);
    DBW_LAUNCHED();
    // backward through the tensor-core layers
    for (int l = L - 2; l >= 0; --l) {
        const int in = m.dims[l], out = m.dims[l + 1];
        TcArgs w{};
        w.M = out; w.N = in; w.K = B; w.epi = EPI_DW;
        w.outf = G + m.w_off[l]; w.outf_z = h->ld; w.outf_pitch = in;
        w.status = h->d_status;
        if ((rc = run_tc(h, st->dwA[l], st->dwB[l], w, N, s, true, true))) return rc;
        if (l >= 1) {
            TcArgs a{};
            a.M = B; a.N = in; a.K = out; a.epi = EPI_DA;
            a.out = st->dZ[l]; a.out_z = (long long)B * in; a.out_pitch = in;
            a.mask = st->A[l]; a.mask_z = (long long)B * in; a.mask_pitch = in;
            a.status = h->d_status;
            if ((rc = run_tc(h, st->daA[l], st->daB[l], a, N, s, false, true))) return rc;
        }
    }
    // the reductions over the batch that only the mix needs: bias gradients, last layer's dW and db, losses
    TailArgs t{};
    t.n_bias = L - 1;
    int next = 0;
    for (int l = 0; l <= L - 2; ++l) {
        t.first[l] = next;
        t.out_dim[l] = m.dims[l + 1];
        t.dz[l] = st->dZ[l + 1];
        t.b_off[l] = m.b_off[l];
        next += (m.dims[l + 1] + 127) / 128;
    }
    t.first[L - 1] = next;
    next += (std::max(C * K, C) + 255) / 256;
    t.first[L] = next;
    t.B = B; t.K = K; t.C = C; t.parts = parts; t.workers = N;
    t.dwp = st->dwp; t.dzL = st->dzL; t.loss_s = st->loss_s; t.loss = loss;
    t.G = G; t.ld = h->ld; t.w_off_last = m.w_off[L - 1]; t.b_off_last = m.b_off[L - 1];
    grad_tail_kernel<<<dim3(next + 1, N), 256, 0, s>>>(t);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
