// Mix kernel on the tensor cores, for uniform weights (opt-in: dbw_set_mix_panel(h, 2)).
//
// With uniform weights (Eq. 5 with P_ij = 1/(1+p_i) on the kept set) a mixed row is
//   x'_i = s_i * sum_j S_ij x~_j,   S_ij = 1 if j = i or j is a kept neighbour of i, else 0,
// i.e. X' = diag(s) (S X~) with a 0/1 selection matrix S.  When a worker keeps about 30 neighbours
// out of 1000, gathering 30 operands per output out of shared memory is bound by the shared-memory
// data pipe; the dense product S X~ on the tensor cores needs no per-operand delivery to the CUDA
// cores at all, but 97 % of its multiplications are by zero.  Measured on the 1024-worker workload it
// runs at 1.2 PFLOP/s of dense BF16 work, close to what the power limit lets a dense GEMM reach, and
// that is not faster than the gather kernel: it stays an option, not the default.
//
// fp32 accuracy on BF16 tensor cores: every x~ = x - lr*g (fp32) is split exactly into three BF16
// pieces hi + mid + lo (8 significand bits each, 24 together); S is exact in BF16; the products are
// exact and the accumulation is the tensor core's fp32.  The three pieces are three MMAs into the
// same accumulator.  (A non-finite x~ makes NaN pieces, and 0 x NaN = NaN reaches every row of that
// column, not only the rows that keep the worker.)
//
// Work split: a pair of CTAs (one cluster, tcgen05 cta_group::2, MMA shape 256 x 256 x 16) owns a
// work item = (panel of 256 columns, group of 512 output workers).  The accumulators of the item fill
// tensor memory (each CTA: 2 row tiles x 256 columns; CTA r of the pair holds rows 256 t + 128 r ..
// + 127 of tile t), so X~ is streamed through shared memory once per item, 64 input workers at a time.
// With more than 512 workers the row groups of a panel go to neighbouring pairs, which run side by
// side, so the second reader of the panel's X and G finds them in L2; then X' must not alias X.
//   warp 0      TMA: S tiles (128 rows x 64 inputs, K-major, 128-byte swizzle) out of L2, 3-stage ring;
//               L2 prefetch of the X and G boxes a few chunks ahead
//   warp 1      MMA issue (leader CTA) + tensor-memory allocation (both CTAs)
//   warps 2-5   epilogue: tcgen05.ld, row scale, 128-byte-swizzled 32 x 32 blocks in shared memory,
//               TMA stores
//   warps 6-21  producers: x and g (each CTA its own 128 columns: 512-byte row segments), x~ and its
//               three pieces, stored as MN-major 128-byte-swizzled BF16 tiles, 4-stage ring of 32 inputs
// HBM traffic is the algorithmic 12 bytes per element; S (2 MB) is re-read from L2 for every item.
// Every mbarrier wait is bounded; the first wait that runs out sets DBW_STATUS_WAIT_TIMEOUT and the abort
// word of both CTAs, after which every role stops issuing work and reaches the end, where tensor memory
// is released.
#include <new>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace dbw {

namespace {

constexpr int kPanel = 256;  // columns per CTA pair (the N of one MMA)
constexpr int kHalf = 128;   // columns staged by one CTA
constexpr int kKC = 64;      // input workers per K chunk
constexpr int kKB = 32;      // input workers per stage of the piece ring (half a K chunk)
constexpr int kAStages = 3, kBStages = 4;
constexpr int kTiles = 2;                        // row tiles of 256 output workers (128 per CTA) per work item
constexpr int kRowsPerItem = 256 * kTiles;       // 512 output workers
constexpr int kTileBytes = 128 * kKC * 2;        // 16 KiB: 128 rows of S x 64 inputs
constexpr int kAStageBytes = kTiles * kTileBytes;
constexpr int kPieceBytes = kKB * kHalf * 2;     // 8 KiB: 32 inputs x 128 columns of one piece (two 64-column chunks of 4 KiB)
constexpr int kBStageBytes = 3 * kPieceBytes;
constexpr int kProdWarps = 16, kEpiWarps = 4;
constexpr int kThreads = (2 + kEpiWarps + kProdWarps) * 32;  // 704
constexpr int kStagingBytes = kEpiWarps * 2 * 4096;          // per epilogue warp two 32 x 32 fp32 blocks
constexpr int kMaxN = 1024;
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kAStages * kAStageBytes + (size_t)kBStages * kBStageBytes +
                              (size_t)kStagingBytes + 256 /*barriers*/;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr int kPrefetchAhead = 4;  // K chunks of X and G requested into L2 ahead of the producers
// kind::f16: D = f32, A = B = bf16, A K-major, B MN-major, N = 256, M = 256 (two CTAs)
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kPanel >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

using namespace ptx;

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Every wait is bounded and shares the CTA's abort word (set by the first wait that runs out, in both
// CTAs of the pair): after one expired wait all roles of the pair drain at once.
// Waits that are not on the MMA thread's critical path poll with a pause in between: a tight poll
// loop floods the memory-instruction queue its scheduler shares with the warps that do the work.
struct WaitCtx {
    volatile uint32_t* abort;  // this CTA's abort word (shared memory)
    uint32_t peer_abort;       // shared::cluster address of the other CTA's abort word
    uint32_t* status;
};
__device__ __forceinline__ void raise_peer(const WaitCtx& w) {
    asm volatile("st.relaxed.cluster.shared::cluster.u32 [%0], %1;" ::"r"(w.peer_abort), "r"(1u) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
    if (mbar_wait_bounded<true>(bar, parity, kSpinLimit, 0, w.abort, w.status)) return true;
    raise_peer(w);
    return false;
}
__device__ __forceinline__ bool mbar_wait_paused(uint64_t* bar, uint32_t parity, const WaitCtx& w, unsigned pause_ns) {
    if (mbar_wait_bounded<true>(bar, parity, kSpinLimit / 4, pause_ns, w.abort, w.status)) return true;
    raise_peer(w);
    return false;
}
// One lane polls for the whole warp; the result is warp-uniform.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, const WaitCtx& w, unsigned pause_ns) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait_paused(bar, parity, w, pause_ns);
    return __all_sync(0xffffffffu, ok);
}
// 2-D tiled TMA load into this CTA's shared memory; the bytes are counted on the barrier at
// `bar_cluster_addr`, which may belong to the other CTA of the pair (no multicast).
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
        : "memory");
}
// asks for one box of a tensor to be brought into L2 (no shared memory, no completion to wait for)
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int c0, int c1) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(c0), "r"(c1) : "memory");
}
// arrives on the barrier at this shared-memory offset in BOTH CTAs once all MMAs issued so far are complete
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
        : "memory");
}
// MN-major piece tiles of this file: chunks of 64 columns x kKB K rows
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t smem_addr) { return mnmajor_sw128_desc(smem_addr, kKB * 128); }

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16_lo_as_float(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi_as_float(uint32_t packed) { return __uint_as_float(packed & 0xffff0000u); }

struct TcMixArgs {
    int N, n_halves, n_kc, n_panels, mix_then_correct, stagger_clocks;
    long long ld;
    const float* X;
    const float* G;
    float lr;
    const float* lr_pw;
    float* Xout;
    uint16_t* shadow;
    const float* scale;  // per-row weight 1/(1+p_i)
    uint32_t* status;
};

struct Barriers {
    uint64_t a_full[kAStages], a_empty[kAStages];
    uint64_t b_full[kBStages], b_empty[kBStages];
    uint64_t acc_full[kTiles], acc_empty[kTiles];
    uint64_t drain;  // shutdown after an expired wait: completion of the MMAs issued so far
    uint32_t tmem_slot;
    uint32_t abort;  // set (in both CTAs) by the first wait that runs out
};

// A work item is (panel of 256 columns, group of 512 output workers).  With more than 512 workers
// the row groups of one panel go to neighbouring CTA pairs, which run side by side, so that the
// second reader of the panel's X and G finds them in L2.
__global__ void __launch_bounds__(kThreads, 1)
mix_tc_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmX,
              const __grid_constant__ CUtensorMap tmG, TcMixArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ringA = smem;
    uint8_t* ringB = ringA + kAStages * kAStageBytes;
    uint8_t* staging = ringB + kBStages * kBStageBytes;
    Barriers* bars = reinterpret_cast<Barriers*>(staging + kStagingBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();  // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int groups = n_pairs / a.n_halves;             // pairs working on different panels at a time
    const int group = pair / a.n_halves, half = pair % a.n_halves;
    const int my_items = (group < groups && a.n_panels > group) ? (a.n_panels - group + groups - 1) / groups : 0;
    const int row_base = half * kRowsPerItem;            // first output worker of this pair's row group
    const int n_tiles = min(kTiles, (a.N - row_base + 255) / 256);

    if (tid == 0) {
        bars->abort = 0u;
        mbar_init(&bars->drain, 1);
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(&bars->a_full[s], 1);   // the leader's expect_tx arrival; TMA bytes of both CTAs
            mbar_init(&bars->a_empty[s], 1);  // one commit
        }
        for (int s = 0; s < kBStages; ++s) {
            mbar_init(&bars->b_full[s], kProdWarps);  // one arrival per warp of the producer group (eight warps) of both CTAs
            mbar_init(&bars->b_empty[s], 1);
        }
        for (int t = 0; t < kTiles; ++t) {
            mbar_init(&bars->acc_full[t], 1);
            mbar_init(&bars->acc_empty[t], 2 * kEpiWarps);  // one arrival per epilogue warp of both CTAs
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // both CTAs: all 512 columns of each CTA's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx wc{&bars->abort, map_to_cta(smem_u32(&bars->abort), rank ^ 1u), a.status};

    // All pairs would otherwise reach their epilogues at the same moment and the whole GPU would store
    // in bursts: start the groups of pairs spread over about one work item's time.
    if (a.stagger_clocks > 0) {
        const long long t0 = clock64(), delay = (long long)(group & 7) * a.stagger_clocks;
        while (clock64() - t0 < delay) __nanosleep(256);
    }

    if (warp == 0) {
        // ---------------- S tiles by TMA; X and G boxes prefetched into L2 a few chunks ahead ----------------
        if (lane == 0) {
            const int total = my_items * a.n_kc;
            auto prefetch = [&](int ch) {  // this CTA's 64 workers x 128 columns of chunk ch
                if (ch >= total) return;
                const int w = ch / a.n_kc, kc = ch % a.n_kc;
                const long long col = (long long)(group + w * groups) * kPanel + (long long)rank * kHalf;
                if (col >= a.ld) return;
                tma_prefetch_2d(&tmX, (int)col, kc * kKC);
                if (a.G && !a.mix_then_correct) tma_prefetch_2d(&tmG, (int)col, kc * kKC);
            };
            for (int ch = 0; ch < kPrefetchAhead; ++ch) prefetch(ch);
            int it = 0;
            bool live = true;
            for (int w = 0; w < my_items && live; ++w)
                for (int kc = 0; kc < a.n_kc; ++kc, ++it) {
                    prefetch(it + kPrefetchAhead);
                    const int s = it % kAStages;
                    if (it >= kAStages && !mbar_wait_paused(&bars->a_empty[s], ((it / kAStages) - 1) & 1, wc, 64)) {
                        live = false;  // a wait ran out somewhere in the pair: issue nothing more
                        break;
                    }
                    if (rank == 0) mbar_expect_tx(&bars->a_full[s], (uint32_t)(2 * n_tiles * kTileBytes));
                    const uint32_t full_addr = map_to_cta(smem_u32(&bars->a_full[s]), 0);
                    for (int t = 0; t < n_tiles; ++t)
                        tma_load_2d_pair(ringA + s * kAStageBytes + t * kTileBytes, &tmS, kc * kKC, row_base + t * 256 + (int)rank * 128,
                                         full_addr);
                }
            // The copies of both CTAs are counted on the leader's barriers: the leader sees the last ones land
            // before the pair meets at the final cluster barrier, so neither CTA leaves with a copy in flight.
            if (rank == 0)
                for (int j = it > kAStages ? it - kAStages : 0; j < it; ++j) mbar_wait_quiet<true>(&bars->a_full[j % kAStages], (j / kAStages) & 1, 1u << 20);
        }
    } else if (warp == 1) {
        // ---------------- MMA issue (leader CTA only) ----------------
        if (rank == 0 && lane == 0) {
            int it = 0;
            bool live = true;
            for (int w = 0; w < my_items && live; ++w)
                for (int kc = 0; kc < a.n_kc && live; ++kc, ++it) {
                    const int sa = it % kAStages;
                    if (!mbar_wait(&bars->a_full[sa], (it / kAStages) & 1, wc)) {
                        live = false;
                        break;
                    }
                    const uint32_t baseA = smem_u32(ringA + sa * kAStageBytes);
#pragma unroll
                    for (int hb = 0; hb < kKC / kKB; ++hb) {  // the two halves of the K chunk: one piece-ring stage each
                        const int ib = it * (kKC / kKB) + hb, sb = ib % kBStages;
                        if (!mbar_wait(&bars->b_full[sb], (ib / kBStages) & 1, wc)) {
                            live = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t baseB = smem_u32(ringB + sb * kBStageBytes);
                        for (int t = 0; t < n_tiles; ++t) {
                            if (kc == 0 && hb == 0 && w > 0) {  // the epilogues of both CTAs have drained this tile's accumulator
                                if (!mbar_wait(&bars->acc_empty[t], (w - 1) & 1, wc)) {
                                    live = false;
                                    break;
                                }
                                tc_fence_after();
                            }
                            const uint64_t da = kmajor_sw128_desc(baseA + t * kTileBytes) + (uint64_t)(hb * (kKB / 16) * 2);
#pragma unroll
                            for (int pc = 0; pc < 3; ++pc) {
                                const uint64_t db = mnmajor_desc(baseB + pc * kPieceBytes);
#pragma unroll
                                for (int k = 0; k < kKB / 16; ++k)  // 16 inputs further: 32 bytes (K-major), 16 rows of 128 bytes (MN-major)
                                    tc_mma_pair(tmem_base + (uint32_t)(t * kPanel), da + (uint64_t)(k * 2), db + (uint64_t)(k * 128),
                                                (kc > 0 || hb > 0 || pc > 0 || k > 0) ? 1u : 0u);
                            }
                            if (kc == a.n_kc - 1 && hb == kKC / kKB - 1) tc_commit_pair(&bars->acc_full[t]);
                        }
                        if (!live) break;
                        tc_commit_pair(&bars->b_empty[sb]);
                    }
                    if (live) tc_commit_pair(&bars->a_empty[sa]);
                }
            if (bars->abort) {  // shutdown after an expired wait: the MMAs issued so far are complete before tensor memory is freed
                tc_commit_pair(&bars->drain);
                mbar_wait_quiet<true>(&bars->drain, 0, 1u << 20);
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ---------------- epilogue: this warp owns accumulator lanes 32 q .. 32 q + 31 ----------------
        // Per 32-column block: tcgen05.ld (lane = row), row scale, into a 128-byte-swizzled 32 x 32
        // block in shared memory, written to X' by one TMA store (rows past N and columns past ld are
        // clipped by the tensor map).  With the Eq. 3 order or a BF16 shadow the block is read back
        // row-contiguous and stored with plain 128-bit stores instead.
        const int q = warp & 3;
        uint8_t* stg = staging + (warp - 2) * 8192;
        const bool plain = a.mix_then_correct || a.shadow;
        float sc[kTiles];
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
            const int r = row_base + t * 256 + (int)rank * 128 + q * 32 + lane;
            sc[t] = (t < n_tiles && r < a.N) ? a.scale[r] : 0.f;
        }
        int blk = 0;
        for (int w = 0; w < my_items; ++w) {
            const long long col0 = (long long)(group + w * groups) * kPanel;
#pragma unroll
            for (int t = 0; t < kTiles; ++t) {
                if (t >= n_tiles) break;
                if (!mbar_wait_warp(&bars->acc_full[t], w & 1, wc, 256)) break;
                tc_fence_after();
                const int row0 = row_base + t * 256 + (int)rank * 128 + q * 32;
                for (int c = 0; c < kPanel / 32; ++c, ++blk) {
                    uint8_t* buf = stg + (blk & 1) * 4096;
                    // the TMA store that last read this buffer (two blocks ago) has finished reading it
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                    uint32_t r[32];
                    tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(t * kPanel + c * 32), r);
#pragma unroll
                    for (int j = 0; j < 8; ++j)  // 16-byte chunk j of row `lane` sits at chunk j ^ (lane mod 8)
                        *reinterpret_cast<float4*>(buf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                            make_float4(sc[t] * __uint_as_float(r[4 * j]), sc[t] * __uint_as_float(r[4 * j + 1]),
                                        sc[t] * __uint_as_float(r[4 * j + 2]), sc[t] * __uint_as_float(r[4 * j + 3]));
                    const long long colb = col0 + c * 32;
                    if (!plain) {
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) {
                            if (row0 < a.N && colb < a.ld)
                                asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                             ::"l"(&tmOut), "r"((int)colb), "r"(row0), "r"(smem_u32(buf)) : "memory");
                            // one group per block, empty or not: "at most one group pending" above then always means
                            // that the store which last read THIS buffer, two blocks ago, is done with it
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    } else {
                        __syncwarp();
                        const int f4 = lane & 7;
                        const long long col = colb + 4 * f4;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = 4 * i + (lane >> 3);
                            const int gi = row0 + rr;
                            float4 v = *reinterpret_cast<const float4*>(buf + rr * 128 + ((f4 ^ (rr & 7)) << 4));
                            if (gi < a.N && col < a.ld) {
                                if (a.mix_then_correct && a.G) {
                                    const float4 g = __ldg(reinterpret_cast<const float4*>(a.G + (size_t)gi * a.ld + col));
                                    const float nlr = -(a.lr_pw ? a.lr_pw[gi] : a.lr);
                                    v.x = fmaf(nlr, g.x, v.x); v.y = fmaf(nlr, g.y, v.y);
                                    v.z = fmaf(nlr, g.z, v.z); v.w = fmaf(nlr, g.w, v.w);
                                }
                                *reinterpret_cast<float4*>(a.Xout + (size_t)gi * a.ld + col) = v;
                                if (a.shadow) *reinterpret_cast<uint2*>(a.shadow + (size_t)gi * a.ld + col) = pack_bf16x4_rn(v.x, v.y, v.z, v.w);
                            }
                        }
                        __syncwarp();
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[t]), 0));
            }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // all of this warp's stores are complete
    } else {
        // ---------------- producers: x~ pieces of this CTA's 128 columns ----------------
        // Two groups of eight warps take alternate half chunks (32 input workers x 128 columns = one stage
        // of the piece ring), so that one group's loads are in flight while the other converts, and with
        // four stages each group may run a stage ahead of the MMA.  A warp owns four rows of the half
        // chunk.  Every load instruction of a warp reads one whole 512-byte row segment (lane l: columns
        // 4l .. 4l+3) and every store instruction writes one row of a piece (8 bytes per lane; no shuffles:
        // anything that goes through the shared-memory pipe competes with the MMA's operand reads).  All
        // loads of a half chunk are issued before the first conversion, and the proxy fence that publishes
        // the stage to the MMA comes when none of the thread's loads is in flight any more.
        const int pw = warp - 2 - kEpiWarps;
        const int grp = pw >> 3, gw = pw & 7;   // half-chunk parity this warp works on, warp within the group
        const int total = my_items * a.n_kc * (kKC / kKB);  // half chunks
        const int j0 = (gw >> 2) * 8 + (gw & 3);  // rows j0, j0 + 4, j0 + 16, j0 + 20 of the half chunk
        const int c16 = lane >> 1;  // a lane's four columns are one half (8 bytes) of a 16-byte chunk
        for (int hc = grp; hc < total; hc += 2) {
            const int ch = hc / (kKC / kKB), w = ch / a.n_kc, kc = ch % a.n_kc;
            const int row_lo = kc * kKC + (hc % (kKC / kKB)) * kKB;
            const long long col = (long long)(group + w * groups) * kPanel + (long long)rank * kHalf + 4 * lane;
            float4 x[4], g[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int row = row_lo + j0 + 4 * (q & 1) + 16 * (q >> 1);
                const bool ok = row < a.N && col < a.ld;
                x[q] = ok ? __ldg(reinterpret_cast<const float4*>(a.X + (size_t)row * a.ld + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
                g[q] = (ok && a.G && !a.mix_then_correct) ? __ldg(reinterpret_cast<const float4*>(a.G + (size_t)row * a.ld + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const int sb = hc % kBStages;
            if (hc >= kBStages && !mbar_wait_warp(&bars->b_empty[sb], ((hc / kBStages) - 1) & 1, wc, 64)) break;
            uint8_t* stage = ringB + sb * kBStageBytes;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = j0 + 4 * (q & 1) + 16 * (q >> 1);
                const int row = row_lo + r;
                const float nlr = -((a.lr_pw && row < a.N) ? a.lr_pw[row] : a.lr);
                const float v[4] = {fmaf(nlr, g[q].x, x[q].x), fmaf(nlr, g[q].y, x[q].y), fmaf(nlr, g[q].z, x[q].z), fmaf(nlr, g[q].w, x[q].w)};
                uint32_t pc[3][2];  // [piece][packed pair]
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p0 = v[2 * e], p1 = v[2 * e + 1];
                    const uint32_t hi = pack_bf16x2_rn(p0, p1);
                    const float r0 = p0 - bf16_lo_as_float(hi), r1 = p1 - bf16_hi_as_float(hi);
                    const uint32_t mid = pack_bf16x2_rn(r0, r1);
                    const float s0 = r0 - bf16_lo_as_float(mid), s1 = r1 - bf16_hi_as_float(mid);
                    pc[0][e] = hi;
                    pc[1][e] = mid;
                    pc[2][e] = pack_bf16x2_rn(s0, s1);
                }
                // 64-column chunk, then the 128-byte swizzle: 16-byte chunk index XOR (row mod 8) inside each 8-row, 1024-byte group
                const uint32_t off = (uint32_t)((c16 >> 3) * (kKB * 128) + (r >> 3) * 1024 + (r & 7) * 128 + (((c16 & 7) ^ (r & 7)) << 4) + (lane & 1) * 8);
#pragma unroll
                for (int p = 0; p < 3; ++p) *reinterpret_cast<uint2*>(stage + p * kPieceBytes + off) = make_uint2(pc[p][0], pc[p][1]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> visible to the MMA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->b_full[sb]), 0));
        }
    }
    // both CTAs are done with each other's shared and tensor memory before either leaves
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

// S as BF16 [rows_pad][k_pad]: row i has ones at i and at its kept neighbours.
__global__ void __launch_bounds__(128)
build_selection_kernel(int N, int k_pad, MixPlan plan, uint16_t* S) {
    const int i = blockIdx.x;
    uint4* row = reinterpret_cast<uint4*>(S + (size_t)i * k_pad);
    for (int e = threadIdx.x; e < k_pad / 8; e += blockDim.x) row[e] = make_uint4(0u, 0u, 0u, 0u);
    if (i >= N) return;
    __syncthreads();
    const int cnt = plan.cnt[i];
    for (int k = threadIdx.x; k < cnt; k += blockDim.x) S[(size_t)i * k_pad + checked(plan.idx[(size_t)i * plan.stride + k], N, plan.status)] = 0x3F80u;
    if (threadIdx.x == 0) S[(size_t)i * k_pad + i] = 0x3F80u;
}

// launch configuration of `ctas` CTAs in clusters of two
void pair_launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int ctas, cudaStream_t s) {
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(ctas);
    cfg->blockDim = dim3(kThreads);
    cfg->dynamicSmemBytes = kSmemBytes;
    cfg->stream = s;
    attr->id = cudaLaunchAttributeClusterDimension;
    attr->val.clusterDim.x = 2;
    attr->val.clusterDim.y = 1;
    attr->val.clusterDim.z = 1;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
}

}  // namespace

struct TcMixState {
    uint16_t* S = nullptr;  // [rows_pad][k_pad] BF16
    int rows_pad = 0, k_pad = 0, n_pairs = 0;
    CUtensorMap map;        // S, box 64 inputs x 128 rows
    CUtensorMap out_map;    // X' as last launched: box 32 columns x 32 rows
    CUtensorMap x_map, g_map;  // X and G as last launched: box 128 columns x 64 rows (L2 prefetch)
    const float* out_ptr = nullptr;
    const float* x_ptr = nullptr;
    const float* g_ptr = nullptr;
};

void mix_tc_free(dbw_handle* h) {
    if (!h->mix_tc) return;
    if (h->mix_tc->S) cudaFree(h->mix_tc->S);
    delete h->mix_tc;
    h->mix_tc = nullptr;
}

// Uniform weights (S is 0/1 and the weight a per-row scale), all output rows of two row groups fit
// the tensor memory of neighbouring CTA pairs, and enough rows that the dense product beats the gather.
bool mix_tc_usable(const dbw_handle* h) {
    if (!(h->flags & DBW_WEIGHT_UNIFORM)) return false;
    if (h->N > kMaxN || h->N < 256) return false;
    return kSmemBytes <= (size_t)h->smem_optin;
}

// With more than one row group per panel another CTA pair still reads the panel's old rows while
// this one stores its new ones: X' must then be a different buffer.
bool mix_tc_in_place_ok(const dbw_handle* h) { return h->N <= kRowsPerItem; }

static int mix_tc_prepare(dbw_handle* h) {
    if (h->mix_tc) return DBW_OK;
    TcMixState* st = new (std::nothrow) TcMixState();
    if (!st) return DBW_ERR_CUDA;
    h->mix_tc = st;
    st->rows_pad = (h->N + 255) / 256 * 256;
    st->k_pad = (h->N + kKC - 1) / kKC * kKC;
    DBW_CUDA(cudaMalloc(reinterpret_cast<void**>(&st->S), (size_t)st->rows_pad * st->k_pad * 2));
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return DBW_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)st->k_pad, (cuuint64_t)st->rows_pad};
    cuuint64_t strides[1] = {(cuuint64_t)st->k_pad * 2};
    cuuint32_t box[2] = {(cuuint32_t)kKC, 128};
    cuuint32_t estr[2] = {1, 1};
    if (fn(&st->map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, st->S, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DBW_ERR_CUDA;
    DBW_CUDA(cudaFuncSetAttribute(mix_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    // how many CTA pairs can be resident at once (the two CTAs of a cluster share one group of SMs)
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    pair_launch_config(&cfg, &attr, 2 * h->sm_count, nullptr);
    int clusters = 0;
    DBW_CUDA(cudaOccupancyMaxActiveClusters(&clusters, mix_tc_kernel, &cfg));
    if (clusters < 1) return DBW_ERR_BAD_SHAPE;
    st->n_pairs = clusters;
    return DBW_OK;
}

int launch_mix_tc(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out, uint16_t* shadow,
                  cudaStream_t s) {
    int rc = mix_tc_prepare(h);
    if (rc != DBW_OK) return rc;
    TcMixState* st = h->mix_tc;
    // tensor maps of X' (the epilogue's stores) and of X and G (L2 prefetch), [N][ld] fp32; rebuilt when a pointer changes
    auto encode = [&](CUtensorMap* map, const float* base, cuuint32_t box_cols, cuuint32_t box_rows, CUtensorMapSwizzle sw) {
        EncodeTiledFn fn = encode_tiled_fn();
        cuuint64_t dims[2] = {(cuuint64_t)h->ld, (cuuint64_t)h->N};
        cuuint64_t strides[1] = {(cuuint64_t)h->ld * 4};
        cuuint32_t box[2] = {box_cols, box_rows};
        cuuint32_t estr[2] = {1, 1};
        return fn && fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        sw, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    if (st->out_ptr != X_out) {
        if (!encode(&st->out_map, X_out, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return DBW_ERR_CUDA;
        st->out_ptr = X_out;
    }
    if (st->x_ptr != X) {
        if (!encode(&st->x_map, X, kHalf, kKC, CU_TENSOR_MAP_SWIZZLE_NONE)) return DBW_ERR_CUDA;
        st->x_ptr = X;
    }
    if (G && st->g_ptr != G) {  // G == nullptr (consensus only): the kernel never touches the map
        if (!encode(&st->g_map, G, kHalf, kKC, CU_TENSOR_MAP_SWIZZLE_NONE)) return DBW_ERR_CUDA;
        st->g_ptr = G;
    }
    build_selection_kernel<<<st->rows_pad, 128, 0, s>>>(h->N, st->k_pad, h->plan, st->S);
    DBW_LAUNCHED();
    TcMixArgs a{};
    a.N = h->N;
    a.n_halves = (st->rows_pad + kRowsPerItem - 1) / kRowsPerItem;
    a.n_kc = st->k_pad / kKC;
    a.n_panels = (int)((h->ld + kPanel - 1) / kPanel);
    a.mix_then_correct = (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0;
    a.ld = h->ld;
    a.X = X; a.G = G; a.lr = lr; a.lr_pw = lr_pw; a.Xout = X_out; a.shadow = shadow;
    a.scale = h->plan.w_self;
    // an eighth of a work item's time (about 100 clocks per MMA, 24 MMAs per K chunk) between groups of pairs
    a.stagger_clocks = a.n_panels * a.n_halves > st->n_pairs ? a.n_kc * 24 * 100 / 8 : 0;
    a.status = h->d_status;
    if (st->n_pairs < a.n_halves) return DBW_ERR_BAD_SHAPE;
    int pairs = a.n_panels * a.n_halves < st->n_pairs ? a.n_panels * a.n_halves : st->n_pairs;
    pairs -= pairs % a.n_halves;  // whole groups of neighbouring pairs
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    pair_launch_config(&cfg, &attr, 2 * pairs, s);
    DBW_CUDA(cudaLaunchKernelEx(&cfg, mix_tc_kernel, st->map, st->out_map, st->x_map, st->g_map, a));
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
