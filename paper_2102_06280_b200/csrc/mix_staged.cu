// Mix kernel for many workers and many terms per output: one persistent CTA per
// SM, warp-specialised, with the NEXT column panel prefetched into tensor memory.
//
// With N of the order of 1000 a 32-column panel of all rows (N x 128 B) plus the neighbour lists
// fill shared memory, so there is no room for a second panel buffer, and with about 30 terms per
// output the gather out of shared memory takes longer than the HBM stream.  To overlap the two,
// eight producer warps stream the next panel of X and G from HBM (128-bit loads, x - lr*g formed
// in registers) and park it in the SM's tensor memory with tcgen05.st, while twenty-four consumer
// warps gather the current panel out of shared memory (the gather waits on shared-memory round
// trips, so it wants every warp the SM can hold).  When both are done the producers move the parked
// panel from tensor memory into shared memory (tcgen05.ld + 128-bit shared stores) and the roles
// repeat.  The neighbour lists (16-bit entries built once per launch from the mixing plan: a bare row
// index with uniform weights, a 10-bit index and a 6-bit weight code with the Metropolis weights) stay
// in shared memory for the whole launch.  HBM traffic is the algorithmic 12 bytes per element; a panel
// is fully staged before any of it is written and panels are disjoint, so X' may overwrite X.
#include "common.cuh"

namespace dbw {

namespace {

constexpr int kProdWarps = 8, kConsWarps = 24;
constexpr int kThreads = (kProdWarps + kConsWarps) * 32;  // 1024
constexpr int kTmemCols = 256;                            // 128 lanes x 256 columns x 4 B = one 1024 x 32 panel
constexpr int kMaxN = 1024;
constexpr int kZeroCode = 63;  // weight code of list padding (weighted lists): weight 0

// 1 / (1 + m) for the weight codes m = 0 .. 62 of the weighted lists (Assumption 1: the weight worker i puts on a kept
// neighbour j is 1 / (1 + max(p_i, p_j))), the same fp32 quotient the mixing plan holds; code 63 is weight 0.
__constant__ float c_weight[64] = {
    1.0f / 1,  1.0f / 2,  1.0f / 3,  1.0f / 4,  1.0f / 5,  1.0f / 6,  1.0f / 7,  1.0f / 8,  1.0f / 9,  1.0f / 10, 1.0f / 11,
    1.0f / 12, 1.0f / 13, 1.0f / 14, 1.0f / 15, 1.0f / 16, 1.0f / 17, 1.0f / 18, 1.0f / 19, 1.0f / 20, 1.0f / 21, 1.0f / 22,
    1.0f / 23, 1.0f / 24, 1.0f / 25, 1.0f / 26, 1.0f / 27, 1.0f / 28, 1.0f / 29, 1.0f / 30, 1.0f / 31, 1.0f / 32, 1.0f / 33,
    1.0f / 34, 1.0f / 35, 1.0f / 36, 1.0f / 37, 1.0f / 38, 1.0f / 39, 1.0f / 40, 1.0f / 41, 1.0f / 42, 1.0f / 43, 1.0f / 44,
    1.0f / 45, 1.0f / 46, 1.0f / 47, 1.0f / 48, 1.0f / 49, 1.0f / 50, 1.0f / 51, 1.0f / 52, 1.0f / 53, 1.0f / 54, 1.0f / 55,
    1.0f / 56, 1.0f / 57, 1.0f / 58, 1.0f / 59, 1.0f / 60, 1.0f / 61, 1.0f / 62, 1.0f / 63, 0.0f};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float4 (&v)[4]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "f"(v[0].x), "f"(v[0].y), "f"(v[0].z), "f"(v[0].w), "f"(v[1].x), "f"(v[1].y), "f"(v[1].z), "f"(v[1].w),
        "f"(v[2].x), "f"(v[2].y), "f"(v[2].z), "f"(v[2].w), "f"(v[3].x), "f"(v[3].y), "f"(v[3].z), "f"(v[3].w)
        : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float4 (&v)[4]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[0].z), "=f"(v[0].w), "=f"(v[1].x), "=f"(v[1].y), "=f"(v[1].z), "=f"(v[1].w),
          "=f"(v[2].x), "=f"(v[2].y), "=f"(v[2].z), "=f"(v[2].w), "=f"(v[3].x), "=f"(v[3].y), "=f"(v[3].z), "=f"(v[3].w)
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void add4(float4& a, const float4 v) {
    a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
}
__device__ __forceinline__ void fma4(float4& a, const float w, const float4 v) {
    a.x = fmaf(w, v.x, a.x); a.y = fmaf(w, v.y, a.y); a.z = fmaf(w, v.z, a.z); a.w = fmaf(w, v.w, a.w);
}

struct StagedArgs {
    int N, n_panels, mix_then_correct, plan_row;  // plan_row: 16-bit entries per neighbour-list row (multiple of 8)
    long long ld;
    const float* X;
    const float* G;
    float lr;
    const float* lr_pw;
    float* Xout;
    uint16_t* shadow;
    MixPlan plan;
};

// Shared memory: panel float4 [N + 1][8] (row N is all zero: the target of list padding), then the
// neighbour lists uint16 [N][plan_row + 8] (the 16-byte skew keeps four consecutive rows in distinct
// banks), then the per-row scale float [N], then the list lengths in blocks of 8, uint8 [N].
// WEIGHTED = false: uniform weights, a list entry is a bare 16-bit row index and the sum is scaled once per row.
// WEIGHTED = true: a list entry is a 10-bit row index and a 6-bit weight code; padding is (own row, weight 0).
template <bool WEIGHTED>
__global__ void __launch_bounds__(kThreads, 1) mix_staged_kernel(StagedArgs a) {
    extern __shared__ float4 smem4[];
    float4* panel = smem4;
    const int N = a.N;
    const int prow = a.plan_row + 8;  // uint16 per list row
    uint16_t* lists = reinterpret_cast<uint16_t*>(panel + (size_t)(N + 1) * 8);
    float* scale = reinterpret_cast<float*>(lists + (size_t)N * prow);
    uint8_t* nblk = reinterpret_cast<uint8_t*>(scale + N);
    float* wtab = reinterpret_cast<float*>(nblk + (N + 15) / 16 * 16);  // copy of c_weight (weighted lists)
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // neighbour lists, scales and the zero row: once per launch
    for (int e = tid; e < N * (prow / 8); e += kThreads) {
        const int i = e / (prow / 8), k0 = (e % (prow / 8)) * 8;
        const int cnt = a.plan.cnt[i];
        uint32_t w[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int k = k0 + 2 * h;
            auto entry = [&](int kk) -> uint32_t {
                if (!WEIGHTED) return kk < cnt ? (uint32_t)checked(a.plan.idx[(size_t)i * a.plan.stride + kk], N, a.plan.status) : (uint32_t)N;
                if (kk >= cnt) return (uint32_t)i | ((uint32_t)kZeroCode << 10);
                // the plan's weight is 1 / (1 + m): recover m (exact for m <= 62) and keep it as the code
                const int m = __float2int_rn(1.0f / a.plan.w[(size_t)i * a.plan.stride + kk]) - 1;
                return (uint32_t)checked(a.plan.idx[(size_t)i * a.plan.stride + kk], N, a.plan.status) | ((uint32_t)min(max(m, 0), kZeroCode - 1) << 10);
            };
            w[h] = entry(k) | (entry(k + 1) << 16);
        }
        *reinterpret_cast<uint4*>(lists + (size_t)i * prow + k0) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    for (int i = tid; i < N; i += kThreads) {
        scale[i] = a.plan.w_self[i];
        nblk[i] = (uint8_t)((a.plan.cnt[i] + 7) / 8);
    }
    if (WEIGHTED && tid < 64) wtab[tid] = c_weight[tid];
    if (tid < 8) panel[(size_t)N * 8 + tid] = make_float4(0.f, 0.f, 0.f, 0.f);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;

    const int n_its = (N + 31) / 32;  // a producer warp stages 4 rows per iteration, the eight warps 32
    const bool producer = warp < kProdWarps;
    // producer coordinates: row (within an iteration) and 16-byte slot of the 128-byte row segment
    const int p_row = warp * 4 + (lane >> 3), slot = lane & 7;
    const uint32_t p_taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    // consumer coordinates: 64 groups of 8 lanes, each group owns rows grp, grp + 64, ...
    const int grp = (warp - kProdWarps) * 4 + (lane >> 3);

    auto stage = [&](int pn) {  // HBM -> registers -> tensor memory
        const long long c = (long long)pn * 32 + 4 * slot;
        const bool c_ok = c < a.ld;
        for (int bt = 0; bt < n_its; bt += 4) {
            float4 x[4], g[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int r = (bt + u) * 32 + p_row;
                const bool ok = c_ok && r < N;
                x[u] = ok ? ldg4(a.X + (size_t)r * a.ld + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (a.G && !a.mix_then_correct) {  // G == nullptr: consensus-only round, G = 0
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int r = (bt + u) * 32 + p_row;
                    const bool ok = c_ok && r < N;
                    g[u] = ok ? ldg4(a.G + (size_t)r * a.ld + c) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int r = (bt + u) * 32 + p_row;
                    const float nlr = -((a.lr_pw && r < N) ? a.lr_pw[r] : a.lr);
                    x[u].x = fmaf(nlr, g[u].x, x[u].x);
                    x[u].y = fmaf(nlr, g[u].y, x[u].y);
                    x[u].z = fmaf(nlr, g[u].z, x[u].z);
                    x[u].w = fmaf(nlr, g[u].w, x[u].w);
                }
            }
            tmem_st16(p_taddr + (uint32_t)(4 * bt), x);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    };
    auto unpark = [&]() {  // tensor memory -> shared-memory panel
        for (int bt = 0; bt < n_its; bt += 4) {
            float4 x[4];
            tmem_ld16(p_taddr + (uint32_t)(4 * bt), x);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int r = (bt + u) * 32 + p_row;
                if (r < N) panel[(size_t)r * 8 + slot] = x[u];
            }
        }
    };
    auto gather = [&](int pn) {  // every output row of the panel out of shared memory
        const long long c = (long long)pn * 32 + 4 * slot;
        // Flattened loop over (row, list block) with the NEXT block's indices (of this row, or of the
        // group's next row together with that row's own segment) fetched before the current block's
        // eight rows are gathered, so that no shared-memory round trip sits between two gathers.
        int i = grp;
        if (i >= N) return;
        const uint4* lp = reinterpret_cast<const uint4*>(lists + (size_t)i * prow);
        int nb = max((int)nblk[i], 1), kb = 0;  // a row without kept neighbours gathers one all-padding block
        uint4 u = lp[0];
        auto first = [&](int row) {  // uniform: the own row, scaled with the sum at the end; weighted: own weight x own row
            float4 v = panel[(size_t)row * 8 + slot];
            if (WEIGHTED) {
                const float ws = scale[row];
                v.x *= ws; v.y *= ws; v.z *= ws; v.w *= ws;
            }
            return v;
        };
        float4 acc = first(i);
        while (true) {
            const bool last = kb + 1 >= nb;
            const int i2 = i + kConsWarps * 4;
            const bool more = !last || i2 < N;
            const uint4* lp2 = last ? reinterpret_cast<const uint4*>(lists + (size_t)i2 * prow) : lp;
            uint4 un = u;
            float4 acc2 = acc;
            if (more) un = lp2[last ? 0 : kb + 1];
            if (last && i2 < N) acc2 = first(i2);
            constexpr uint32_t kIdx = WEIGHTED ? 0x3ffu : 0xffffu;
            const float4 v0 = panel[(size_t)(u.x & kIdx) * 8 + slot], v1 = panel[(size_t)((u.x >> 16) & kIdx) * 8 + slot];
            const float4 v2 = panel[(size_t)(u.y & kIdx) * 8 + slot], v3 = panel[(size_t)((u.y >> 16) & kIdx) * 8 + slot];
            const float4 v4 = panel[(size_t)(u.z & kIdx) * 8 + slot], v5 = panel[(size_t)((u.z >> 16) & kIdx) * 8 + slot];
            const float4 v6 = panel[(size_t)(u.w & kIdx) * 8 + slot], v7 = panel[(size_t)((u.w >> 16) & kIdx) * 8 + slot];
            if (!WEIGHTED) {
                add4(acc, v0); add4(acc, v1); add4(acc, v2); add4(acc, v3);
                add4(acc, v4); add4(acc, v5); add4(acc, v6); add4(acc, v7);
            } else {  // weights out of a 64-entry table in shared memory (one wavefront for the warp's four codes), list order
                fma4(acc, wtab[(u.x >> 10) & 63u], v0); fma4(acc, wtab[u.x >> 26], v1);
                fma4(acc, wtab[(u.y >> 10) & 63u], v2); fma4(acc, wtab[u.y >> 26], v3);
                fma4(acc, wtab[(u.z >> 10) & 63u], v4); fma4(acc, wtab[u.z >> 26], v5);
                fma4(acc, wtab[(u.w >> 10) & 63u], v6); fma4(acc, wtab[u.w >> 26], v7);
            }
            u = un;
            if (!last) {
                ++kb;
                continue;
            }
            if (!WEIGHTED) {
                const float w = scale[i];
                acc.x *= w; acc.y *= w; acc.z *= w; acc.w *= w;
            }
            if (c < a.ld) {
                if (a.G && a.mix_then_correct) {
                    const float4 gi = ldg4(a.G + (size_t)i * a.ld + c);
                    const float nlr = -(a.lr_pw ? a.lr_pw[i] : a.lr);
                    acc.x = fmaf(nlr, gi.x, acc.x); acc.y = fmaf(nlr, gi.y, acc.y);
                    acc.z = fmaf(nlr, gi.z, acc.z); acc.w = fmaf(nlr, gi.w, acc.w);
                }
                *reinterpret_cast<float4*>(a.Xout + (size_t)i * a.ld + c) = acc;
                if (a.shadow) *reinterpret_cast<uint2*>(a.shadow + (size_t)i * a.ld + c) = pack_bf16x4_rn(acc.x, acc.y, acc.z, acc.w);
            }
            if (i2 >= N) break;
            i = i2;
            lp = lp2;
            nb = max((int)nblk[i], 1);
            kb = 0;
            acc = acc2;
        }
    };

    int pn = blockIdx.x;
    if (pn < a.n_panels) {
        if (producer) {
            stage(pn);
            unpark();
        }
        __syncthreads();
        while (true) {
            const int next = pn + gridDim.x;
            const bool more = next < a.n_panels;
            if (producer) {
                if (more) stage(next);
            } else {
                gather(pn);
            }
            __syncthreads();  // panel pn consumed, panel `next` parked
            if (!more) break;
            if (producer) unpark();
            __syncthreads();  // panel `next` in shared memory
            pn = next;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

size_t staged_smem(const dbw_handle* h, int plan_row) {
    const size_t N = (size_t)h->N;
    return (N + 1) * 128 + N * (size_t)(plan_row + 8) * 2 + N * 4 + ((N + 15) / 16) * 16 + 256;
}

}  // namespace

// Usable when every worker's panel row fits the tensor-memory staging area and the shared memory holds
// panel and lists; with uniform weights a list entry is a bare 16-bit index (one scale per row), with
// the Metropolis weights it carries a 6-bit weight code next to a 10-bit index (degrees up to 62).
bool mix_staged_usable(const dbw_handle* h) {
    if (h->N > kMaxN || h->N < 64) return false;
    if (!(h->flags & DBW_WEIGHT_UNIFORM) && h->maxdeg > kZeroCode - 1) return false;
    const int plan_row = (h->maxdeg + 7) / 8 * 8;
    if (plan_row > 248) return false;
    return staged_smem(h, plan_row) + 256 <= (size_t)h->smem_optin;
}

int launch_mix_staged(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
                      uint16_t* shadow, cudaStream_t s) {
    StagedArgs a{};
    a.N = h->N;
    a.ld = h->ld;
    a.n_panels = (int)((h->ld + 31) / 32);
    a.mix_then_correct = (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0;
    a.plan_row = (h->maxdeg + 7) / 8 * 8;
    a.X = X; a.G = G; a.lr = lr; a.lr_pw = lr_pw; a.Xout = X_out; a.shadow = shadow; a.plan = h->plan;
    const size_t smem = staged_smem(h, a.plan_row);
    static PerDeviceOnce once;
    const int rc = once.run(h->device, [h]() -> int {
        DBW_CUDA(cudaFuncSetAttribute(mix_staged_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 256));
        DBW_CUDA(cudaFuncSetAttribute(mix_staged_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 256));
        return DBW_OK;
    });
    if (rc) return rc;
    const int grid = a.n_panels < h->sm_count ? a.n_panels : h->sm_count;
    if (h->flags & DBW_WEIGHT_UNIFORM)
        mix_staged_kernel<false><<<grid, kThreads, smem, s>>>(a);
    else
        mix_staged_kernel<true><<<grid, kThreads, smem, s>>>(a);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
