// Mix kernel on the tensor cores with 2:4 structured sparsity, for uniform weights.
//
// With uniform weights (Eq. 5 with P_ij = 1/(1+p_i) on the kept set) a mixed row is
//   x'_i = s_i * sum_j S_ij x~_j,   S_ij = 1 if j = i or j is a kept neighbour of i, else 0,
// i.e. X' = diag(s) (S X~) with a 0/1 selection matrix S whose row i is supported on {i} and N_i.  The
// gather kernels deliver every one of the ~30 operands of an output through the shared-memory data
// pipe, which bounds them; the dense product on the tensor cores (mix_tc.cu) multiplies 97 % zeros and
// is bound by the dense BF16 rate.  Here the zeros pay half: the workers are given an order (fixed per
// graph, found on the host at the first launch) in which no row of S has more than two of its possible
// non-zeros in any aligned group of four consecutive workers, so S is a 2:4 structured-sparse operand
// whatever the kept masks are: tcgen05.mma.sp reads S compressed to half its width plus two index bits
// per kept value, and runs the same product at twice the dense rate.
//
// fp32 accuracy: every x~ = x - lr*g (fp32) is split exactly into three BF16 pieces hi + mid + lo (8
// significand bits each, 24 together); S is exact in BF16; products are exact, accumulation is the tensor
// core's fp32.  The three pieces are three MMAs into the same accumulator.  (A non-finite x~ makes NaN
// pieces, and 0 x NaN = NaN reaches every row of that column.)
//
// Work split: a pair of CTAs (one cluster, cta_group::2, MMA shape 256 x 224 x 32) owns a work item =
// (panel of 224 columns, group of 512 output workers).  Each CTA's tensor memory holds the accumulators
// of two row tiles (2 x 224 columns; CTA r of the pair holds rows 256 t + 128 r .. + 127 of tile t) and,
// in its last 64 columns, the sparsity metadata of its 256 rows for all inputs (written once per launch).
//   warp 0      TMA: compressed S tiles (128 rows x 128 inputs = 64 values, K-major, 128-byte swizzle) out
//               of L2, 2-stage ring
//   warp 1      MMA issue (leader CTA) + tensor-memory allocation (both CTAs)
//   warps 2-5   metadata into tensor memory (once), then the epilogue: tcgen05.ld, row scale,
//               128-byte-swizzled 32 x 32 blocks in shared memory, TMA stores
//   warps 6-21  producers: x and g rows in the 2:4 order (each CTA its own 112 columns), x~ and its three
//               pieces, stored as MN-major 128-byte-swizzled BF16 tiles, 4-stage ring of 32 inputs
// HBM traffic is the algorithmic 12 bytes per element; compressed S (1 MB) is re-read from L2 per item.
// Every mbarrier wait is bounded; the first wait that runs out sets DBW_STATUS_WAIT_TIMEOUT and the abort
// word of both CTAs, after which every role stops issuing work and reaches the end, where tensor memory
// is released.  No TMA load is multicast; every tensor map covers this GPU's memory only.
#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace dbw {

namespace {

constexpr int kPanel = 224;  // columns per CTA pair (the N of one MMA)
constexpr int kHalf = 112;   // columns staged by one CTA
constexpr int kHalfAlloc = 128;  // columns a piece tile has room for (two 64-column swizzle chunks)
constexpr int kKA = 128;     // input workers per stage of the S ring (64 compressed values per row)
constexpr int kKB = 32;      // input workers per stage of the piece ring = the K of one sparse MMA
constexpr int kAStages = 2, kBStages = 4;
constexpr int kTiles = 2;                        // row tiles of 256 output workers (128 per CTA) per work item
constexpr int kRowsPerItem = 256 * kTiles;       // 512 output workers
constexpr int kTileBytes = 128 * (kKA / 2) * 2;  // 16 KiB: 128 rows of S x 64 compressed values
constexpr int kAStageBytes = kTiles * kTileBytes;
constexpr int kPieceBytes = kKB * kHalfAlloc * 2;  // 8 KiB: 32 inputs x 128 columns of one piece (two chunks of 4 KiB)
constexpr int kBStageBytes = 3 * kPieceBytes;
constexpr int kProdWarps = 16, kEpiWarps = 4;
constexpr int kThreads = (2 + kEpiWarps + kProdWarps) * 32;  // 704
constexpr int kStagingBytes = kEpiWarps * 2 * 4096;          // per epilogue warp two 32 x 32 fp32 blocks
constexpr int kMaxN = 1024;                                  // metadata of all inputs: 32 columns per row tile
constexpr int kMetaCol = kTiles * kPanel;                    // first metadata column (448)
constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kAStages * kAStageBytes + (size_t)kBStages * kBStageBytes +
                              (size_t)kStagingBytes + 256 /*barriers*/;
constexpr uint32_t kSpinLimit = 1u << 24;
// kind::f16, sparse: D = f32, A = B = bf16, A K-major (compressed), B MN-major, N = 224, M = 256 (two CTAs)
constexpr uint32_t kIdesc = (1u << 2) | (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(kPanel >> 3) << 17) |
                            ((uint32_t)(256 >> 4) << 24);

using namespace ptx;

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
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
// Waits off the MMA thread's critical path poll with a pause in between (a tight poll loop floods the
// memory-instruction queue its scheduler shares with the warps that do the work).
__device__ __forceinline__ bool mbar_wait_paused(uint64_t* bar, uint32_t parity, const WaitCtx& w, unsigned pause_ns) {
    if (mbar_wait_bounded<true>(bar, parity, kSpinLimit / 4, pause_ns, w.abort, w.status)) return true;
    raise_peer(w);
    return false;
}
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
// Arrives on the barrier at this shared-memory offset in BOTH CTAs once all MMAs issued so far are complete
// (a barrier arrive sent to the two CTAs of the pair; no data moves).
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
// D (+)= A_sparse * B: A compressed 2:4 along K, its metadata in tensor memory at column `meta_col`
// (the instruction takes the even column and the low bit of the column as a selector).
__device__ __forceinline__ void tc_mma_sp_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t meta_taddr, uint32_t accumulate) {
    const uint32_t idesc = kIdesc | (meta_taddr & 1u);
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(meta_taddr & ~1u), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
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

struct SpMixArgs {
    int N, n_halves, n_ka, n_panels, mix_then_correct, stagger_clocks;
    long long ld;
    const float* X;
    const float* G;
    float lr;
    const float* lr_pw;
    float* Xout;
    uint16_t* shadow;
    const float* scale;       // per-row weight 1/(1+p_i)
    const int32_t* order;     // [k_pad] worker at input position k, -1 = empty position
    const uint16_t* meta16;   // [rows_pad][k_pad / 16] metadata of 16 input positions (4 groups of four) per entry
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

__global__ void __launch_bounds__(kThreads, 1)
mix_sp_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmOut, SpMixArgs a) {
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
    const int n_kb = a.n_ka * (kKA / kKB);               // piece stages (sparse MMA K steps) per item

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
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx wc{&bars->abort, map_to_cta(smem_u32(&bars->abort), rank ^ 1u), a.status};

    // Sparsity metadata of this CTA's rows, all inputs, once per launch.  For the MMA of K step s on row
    // tile t the tensor core reads column kMetaCol + 32 t + s: lane l holds, in its low half, the sixteen
    // index bits (four groups of four inputs, two 2-bit indices each) of row (l mod 8) + 16 (l / 16) for the
    // inputs 32 s + 16 ((l / 8) mod 2) .. + 15, and in its high half the same for the row eight further on.
    if (warp >= 2 && warp < 2 + kEpiWarps) {
        const int l = (warp & 3) * 32 + lane;
        const int k1 = (l >> 3) & 1;
        const int per_row = a.n_ka * (kKA / 16);  // 16-bit entries per row of meta16
        for (int t = 0; t < n_tiles; ++t) {
            const int row_lo = row_base + t * 256 + (int)rank * 128 + (l & 7) + 16 * (l >> 4);
            const uint16_t* m_lo = a.meta16 + (size_t)row_lo * per_row;
            const uint16_t* m_hi = a.meta16 + (size_t)(row_lo + 8) * per_row;
            uint32_t r[32];
#pragma unroll
            for (int s = 0; s < 32; ++s) {
                const int e = 2 * s + k1;
                r[s] = e < per_row ? ((uint32_t)m_lo[e] | ((uint32_t)m_hi[e] << 16)) : 0x44444444u;
            }
            tmem_st32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(kMetaCol + 32 * t), r);
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();

    // All pairs would otherwise reach their epilogues at the same moment and the whole GPU would store
    // in bursts: start the groups of pairs spread over about one work item's time.
    if (a.stagger_clocks > 0) {
        const long long t0 = clock64(), delay = (long long)(group & 7) * a.stagger_clocks;
        while (clock64() - t0 < delay) __nanosleep(256);
    }

    if (warp == 0) {
        // ---------------- compressed S tiles by TMA ----------------
        int it = 0;
        bool live = true;
        for (int w = 0; w < my_items && live; ++w)
            for (int ka = 0; ka < a.n_ka; ++ka, ++it) {
                const int s = it % kAStages;
                bool ok = true;
                if (lane == 0 && it >= kAStages) ok = mbar_wait_paused(&bars->a_empty[s], ((it / kAStages) - 1) & 1, wc, 64);
                if (!__all_sync(0xffffffffu, ok)) {
                    live = false;  // a wait ran out somewhere in the pair: issue nothing more
                    break;
                }
                if (lane == 0) {
                    if (rank == 0) mbar_expect_tx(&bars->a_full[s], (uint32_t)(2 * n_tiles * kTileBytes));
                    const uint32_t full_addr = map_to_cta(smem_u32(&bars->a_full[s]), 0);
                    for (int t = 0; t < n_tiles; ++t)
                        tma_load_2d_pair(ringA + s * kAStageBytes + t * kTileBytes, &tmS, ka * (kKA / 2), row_base + t * 256 + (int)rank * 128,
                                         full_addr);
                }
            }
        // The copies of both CTAs are counted on the leader's barriers: the leader sees the last ones land
        // before the pair meets at the final cluster barrier, so neither CTA leaves with a copy in flight.
        if (rank == 0 && lane == 0)
            for (int j = it > kAStages ? it - kAStages : 0; j < it; ++j) mbar_wait_quiet<true>(&bars->a_full[j % kAStages], (j / kAStages) & 1, 1u << 20);
    } else if (warp == 1) {
        // ---------------- MMA issue (leader CTA only) ----------------
        if (rank == 0 && lane == 0) {
            int it = 0;
            bool live = true;
            for (int w = 0; w < my_items && live; ++w)
                for (int ka = 0; ka < a.n_ka && live; ++ka, ++it) {
                    const int sa = it % kAStages;
                    if (!mbar_wait(&bars->a_full[sa], (it / kAStages) & 1, wc)) {
                        live = false;
                        break;
                    }
                    const uint32_t baseA = smem_u32(ringA + sa * kAStageBytes);
#pragma unroll
                    for (int hb = 0; hb < kKA / kKB; ++hb) {  // four K steps of 32 inputs: one piece-ring stage each
                        const int ib = it * (kKA / kKB) + hb, sb = ib % kBStages;
                        if (!mbar_wait(&bars->b_full[sb], (ib / kBStages) & 1, wc)) {
                            live = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t baseB = smem_u32(ringB + sb * kBStageBytes);
                        const int kstep = ka * (kKA / kKB) + hb;
                        for (int t = 0; t < n_tiles; ++t) {
                            if (kstep == 0 && w > 0) {  // the epilogues of both CTAs have drained this tile's accumulator
                                if (!mbar_wait(&bars->acc_empty[t], (w - 1) & 1, wc)) {
                                    live = false;
                                    break;
                                }
                                tc_fence_after();
                            }
                            // 32 inputs further along K: 16 compressed values = 32 bytes inside the swizzle atom
                            const uint64_t da = kmajor_sw128_desc(baseA + t * kTileBytes) + (uint64_t)(hb * 2);
                            const uint32_t meta = tmem_base + (uint32_t)(kMetaCol + 32 * t + kstep);
#pragma unroll
                            for (int pc = 0; pc < 3; ++pc)
                                tc_mma_sp_pair(tmem_base + (uint32_t)(t * kPanel), da, mnmajor_desc(baseB + pc * kPieceBytes), meta,
                                               (kstep > 0 || pc > 0) ? 1u : 0u);
                            if (kstep == n_kb - 1) tc_commit_pair(&bars->acc_full[t]);
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
        const bool plain = (a.mix_then_correct && a.G) || a.shadow;
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
        // ---------------- producers: x~ pieces of this CTA's 112 columns ----------------
        // Two groups of eight warps take alternate piece stages (32 inputs x 112 columns), so that one
        // group's loads are in flight while the other converts, and with four stages each group may run a
        // stage ahead of the MMA.  A warp owns four inputs of the stage; the worker at an input position
        // comes from the 2:4 order.  Every load instruction of a warp reads one 448-byte row segment (lanes
        // 0 .. 27: columns 4l .. 4l+3) and every store instruction writes one row of a piece (8 bytes per lane;
        // no shuffles: anything that goes through the shared-memory pipe competes with the MMA's operand
        // reads).  All loads of a stage are issued before the first conversion, and the proxy fence that
        // publishes the stage to the MMA comes when none of the thread's loads is in flight any more.
        const int pw = warp - 2 - kEpiWarps;
        const int grp = pw >> 3, gw = pw & 7;   // stage parity this warp works on, warp within the group
        const int total = my_items * n_kb;
        const int j0 = (gw >> 2) * 8 + (gw & 3);  // inputs j0, j0 + 4, j0 + 16, j0 + 20 of the stage
        const int c16 = lane >> 1;  // a lane's four columns are one half (8 bytes) of a 16-byte chunk
        const bool col_lane = lane < kHalf / 4;
        for (int hc = grp; hc < total; hc += 2) {
            const int w = hc / n_kb, kb = hc % n_kb;
            const long long col = (long long)(group + w * groups) * kPanel + (long long)rank * kHalf + 4 * lane;
            float4 x[4], g[4];
            int rows[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = j0 + 4 * (q & 1) + 16 * (q >> 1);
                rows[q] = __ldg(a.order + kb * kKB + r);
                if (rows[q] >= 0) rows[q] = checked(rows[q], a.N, a.status);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool ok = col_lane && rows[q] >= 0 && col < a.ld;
                x[q] = ok ? __ldg(reinterpret_cast<const float4*>(a.X + (size_t)rows[q] * a.ld + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
                g[q] = (ok && a.G && !a.mix_then_correct) ? __ldg(reinterpret_cast<const float4*>(a.G + (size_t)rows[q] * a.ld + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const int sb = hc % kBStages;
            if (hc >= kBStages && !mbar_wait_warp(&bars->b_empty[sb], ((hc / kBStages) - 1) & 1, wc, 64)) break;
            uint8_t* stage = ringB + sb * kBStageBytes;
            if (col_lane) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int r = j0 + 4 * (q & 1) + 16 * (q >> 1);
                    const float nlr = -((a.lr_pw && rows[q] >= 0) ? a.lr_pw[rows[q]] : a.lr);
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

// Compressed selection matrix and its metadata for one launch.  Row i of S is supported on the input
// positions pos[i] (self) and pos[j] of the kept neighbours j; the 2:4 order guarantees at most two of
// them in any aligned group of four positions.  Per group of four: the two kept values (BF16 1.0 or 0)
// in position order and the two 2-bit position indices idx0 < idx1 as one nibble idx0 | idx1 << 2.
// A thread handles 16 positions: eight values (16 bytes) and one 16-bit metadata entry.
__global__ void __launch_bounds__(64)
build_sparse_selection_kernel(int N, int k_pad, MixPlan plan, const int32_t* __restrict__ pos, uint16_t* __restrict__ Sc,
                              uint16_t* __restrict__ meta16, uint32_t* status) {
    __shared__ uint8_t mark[kMaxN];
    const int i = blockIdx.x;
    for (int k = threadIdx.x; k < k_pad; k += blockDim.x) mark[k] = 0;
    __syncthreads();
    if (i < N) {
        const int cnt = plan.cnt[i];
        for (int k = threadIdx.x; k < cnt; k += blockDim.x) mark[checked(pos[checked(plan.idx[(size_t)i * plan.stride + k], N, status)], k_pad, status)] = 1;
        if (threadIdx.x == 0) mark[checked(pos[i], k_pad, status)] = 1;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < k_pad / 16; e += blockDim.x) {
        uint32_t vals[4];
        uint32_t meta = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint8_t* m = mark + 16 * e + 4 * c;
            int i0 = -1, i1 = -1, n = 0;
#pragma unroll
            for (int p = 0; p < 4; ++p)
                if (m[p]) {
                    if (n == 0) i0 = p;
                    else if (n == 1) i1 = p;
                    ++n;
                }
            if (n > 2) atomicOr(status, DBW_STATUS_INTERNAL);  // the order does not fit this graph: cannot happen after the host check
            uint32_t v0 = 0, v1 = 0;
            if (n == 0) {
                i0 = 0; i1 = 1;
            } else if (n == 1) {  // one kept value and one explicit zero, indices ascending
                if (i0 < 3) { i1 = i0 + 1; v0 = 0x3F80u; }
                else { i1 = 3; i0 = 2; v1 = 0x3F80u; }
            } else {
                v0 = v1 = 0x3F80u;
            }
            vals[c] = v0 | (v1 << 16);
            meta |= (uint32_t)(i0 | (i1 << 2)) << (4 * c);
        }
        *reinterpret_cast<uint4*>(Sc + (size_t)i * (k_pad / 2) + 8 * e) = make_uint4(vals[0], vals[1], vals[2], vals[3]);
        meta16[(size_t)i * (k_pad / 16) + e] = (uint16_t)meta;
    }
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

// ---- the 2:4 order (host) -------------------------------------------------------------------------
// Workers are placed on k_pad input positions (-1 = empty) so that for every worker i no aligned group of
// four positions holds more than two members of {i} + N_i.  Local search from the identity placement:
// while some group is in conflict, move one of its conflicting members to a random other group (swap) if
// that does not raise the number of conflicts of the two groups.  Deterministic (fixed-seed generator).
struct OrderSearch {
    int N, k_pad;
    const int32_t* rowptr;
    const int32_t* col;
    std::vector<int32_t> order;  // [k_pad]
    std::vector<int> count;      // scratch [N], all zero between calls
    uint64_t rng = 0x9E3779B97F4A7C15ull;

    uint32_t next() {
        rng ^= rng << 13; rng ^= rng >> 7; rng ^= rng << 17;
        return (uint32_t)(rng >> 32);
    }
    // number of workers i with three or more members of {i} + N_i in group g; *culprit = a member that takes part
    int conflicts(int g, int* culprit) {
        int bad = 0;
        for (int s = 0; s < 4; ++s) {
            const int v = order[4 * g + s];
            if (v < 0) continue;
            auto bump = [&](int i) {
                if (++count[i] == 3) {
                    ++bad;
                    if (culprit) *culprit = v;
                }
            };
            bump(v);
            for (int e = rowptr[v]; e < rowptr[v + 1]; ++e) bump(col[e]);
        }
        for (int s = 0; s < 4; ++s) {
            const int v = order[4 * g + s];
            if (v < 0) continue;
            count[v] = 0;
            for (int e = rowptr[v]; e < rowptr[v + 1]; ++e) count[col[e]] = 0;
        }
        return bad;
    }
    bool run() {
        const int groups = k_pad / 4;
        order.assign(k_pad, -1);
        count.assign(N, 0);
        if (k_pad >= 2 * N) {  // two workers per group: nothing can conflict
            for (int v = 0; v < N; ++v) order[4 * (v / 2) + (v & 1)] = v;
            return true;
        }
        for (int v = 0; v < N; ++v) order[v] = v;
        std::vector<int> bad_groups;
        for (long long iter = 0; iter < 400ll * k_pad; ++iter) {
            if (bad_groups.empty()) {
                for (int g = 0; g < groups; ++g)
                    if (conflicts(g, nullptr)) bad_groups.push_back(g);
                if (bad_groups.empty()) return true;
            }
            const int g = bad_groups.back();
            int culprit = -1;
            const int before_g = conflicts(g, &culprit);
            if (!before_g) {
                bad_groups.pop_back();
                continue;
            }
            int slot = 4 * g;
            while (order[slot] != culprit) ++slot;
            const int g2 = (int)(next() % (uint32_t)groups);
            if (g2 == g) continue;
            const int slot2 = 4 * g2 + (int)(next() & 3u);
            const int before = before_g + conflicts(g2, nullptr);
            std::swap(order[slot], order[slot2]);
            const int after = conflicts(g, nullptr) + conflicts(g2, nullptr);
            if (after > before || (after == before && (next() & 3u))) std::swap(order[slot], order[slot2]);  // undo
            else if (conflicts(g2, nullptr)) bad_groups.insert(bad_groups.begin(), g2);
        }
        for (int g = 0; g < groups; ++g)
            if (conflicts(g, nullptr)) return false;
        return true;
    }
};

}  // namespace

struct SpMixState {
    bool feasible = false;
    int rows_pad = 0, k_pad = 0, n_pairs = 0;
    int32_t* d_order = nullptr;  // [k_pad]
    int32_t* d_pos = nullptr;    // [N]
    uint16_t* Sc = nullptr;      // [rows_pad][k_pad / 2] BF16, compressed S of the current launch
    uint16_t* meta16 = nullptr;  // [rows_pad][k_pad / 16]
    CUtensorMap map;             // Sc, box 64 values x 128 rows
    CUtensorMap out_map;         // X' as last launched: box 32 columns x 32 rows
    const float* out_ptr = nullptr;
};

void mix_sp_free(dbw_handle* h) {
    if (!h->mix_sp) return;
    void* ptrs[] = {h->mix_sp->d_order, h->mix_sp->d_pos, h->mix_sp->Sc, h->mix_sp->meta16};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    delete h->mix_sp;
    h->mix_sp = nullptr;
}

// Host part of the set-up, done at dbw_init for graphs the kernel could serve: the 2:4 order.
static bool mix_sp_search(dbw_handle* h, std::vector<int32_t>* order, int* k_pad) {
    for (int attempt = 0; attempt < 2; ++attempt) {
        OrderSearch s;
        s.N = h->N;
        s.k_pad = attempt == 0 ? (h->N + kKA - 1) / kKA * kKA : (2 * h->N + kKA - 1) / kKA * kKA;
        if (s.k_pad > kMaxN) return false;
        s.rowptr = h->h_rowptr.data();
        s.col = h->h_col.data();
        if (s.run()) {
            *order = s.order;
            *k_pad = s.k_pad;
            return true;
        }
    }
    return false;
}

// Uniform weights (S is 0/1 and the weight a per-row scale), the metadata of all inputs fits the 64 spare
// columns of tensor memory, enough rows that the product beats the gather, and a 2:4 order exists.
static bool mix_sp_eligible(const dbw_handle* h) {
    if (!(h->flags & DBW_WEIGHT_UNIFORM)) return false;
    if (h->N > kMaxN || h->N < 256) return false;
    return kSmemBytes <= (size_t)h->smem_optin;
}

bool mix_sp_usable(const dbw_handle* h) { return h->mix_sp && h->mix_sp->feasible; }

// Set-up at dbw_init (the handle's device is current): the 2:4 order on the host, then the device copies,
// the buffers of the compressed matrix and the kernel's attributes.  A graph without such an order, or a
// failed allocation, leaves the kernel unusable (the other mix kernels serve); never an error.
void mix_sp_prepare(dbw_handle* h) {
    if (!mix_sp_eligible(h) || h->mix_sp) return;
    SpMixState* st = new (std::nothrow) SpMixState();
    if (!st) return;
    h->mix_sp = st;
    std::vector<int32_t> order;
    if (!mix_sp_search(h, &order, &st->k_pad)) return;
    st->rows_pad = (h->N + 255) / 256 * 256;
    std::vector<int32_t> pos(h->N, 0);
    for (int k = 0; k < st->k_pad; ++k)
        if (order[k] >= 0) pos[order[k]] = k;
    bool ok = cuda_ok(cudaMalloc(reinterpret_cast<void**>(&st->d_order), (size_t)st->k_pad * 4)) &&
              cuda_ok(cudaMalloc(reinterpret_cast<void**>(&st->d_pos), (size_t)h->N * 4)) &&
              cuda_ok(cudaMalloc(reinterpret_cast<void**>(&st->Sc), (size_t)st->rows_pad * (st->k_pad / 2) * 2)) &&
              cuda_ok(cudaMalloc(reinterpret_cast<void**>(&st->meta16), (size_t)st->rows_pad * (st->k_pad / 16) * 2)) &&
              cuda_ok(cudaMemcpy(st->d_order, order.data(), (size_t)st->k_pad * 4, cudaMemcpyHostToDevice)) &&
              cuda_ok(cudaMemcpy(st->d_pos, pos.data(), (size_t)h->N * 4, cudaMemcpyHostToDevice));
    EncodeTiledFn fn = encode_tiled_fn();
    if (ok && fn) {
        cuuint64_t dims[2] = {(cuuint64_t)(st->k_pad / 2), (cuuint64_t)st->rows_pad};
        cuuint64_t strides[1] = {(cuuint64_t)(st->k_pad / 2) * 2};
        cuuint32_t box[2] = {(cuuint32_t)(kKA / 2), 128};
        cuuint32_t estr[2] = {1, 1};
        ok = fn(&st->map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, st->Sc, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    } else {
        ok = false;
    }
    if (ok) ok = cuda_ok(cudaFuncSetAttribute(mix_sp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
    if (ok) {  // how many CTA pairs can be resident at once (the two CTAs of a cluster share one group of SMs)
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr;
        pair_launch_config(&cfg, &attr, 2 * h->sm_count, nullptr);
        int clusters = 0;
        ok = cuda_ok(cudaOccupancyMaxActiveClusters(&clusters, mix_sp_kernel, &cfg)) && clusters >= (h->N + kRowsPerItem - 1) / kRowsPerItem;
        st->n_pairs = clusters;
    }
    st->feasible = ok;
}

// With more than one row group per panel another CTA pair still reads the panel's old rows while
// this one stores its new ones: X' must then be a different buffer.
bool mix_sp_in_place_ok(const dbw_handle* h) { return h->N <= kRowsPerItem; }

int launch_mix_sp(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out, uint16_t* shadow,
                  cudaStream_t s) {
    if (!mix_sp_usable(h)) return DBW_ERR_BAD_SHAPE;
    SpMixState* st = h->mix_sp;
    if (st->out_ptr != X_out) {  // tensor map of X' (the epilogue's stores), [N][ld] fp32; rebuilt when the pointer changes
        EncodeTiledFn fn = encode_tiled_fn();
        cuuint64_t dims[2] = {(cuuint64_t)h->ld, (cuuint64_t)h->N};
        cuuint64_t strides[1] = {(cuuint64_t)h->ld * 4};
        cuuint32_t box[2] = {32, 32};
        cuuint32_t estr[2] = {1, 1};
        if (!fn || fn(&st->out_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, X_out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DBW_ERR_CUDA;
        st->out_ptr = X_out;
    }
    build_sparse_selection_kernel<<<st->rows_pad, 64, 0, s>>>(h->N, st->k_pad, h->plan, st->d_pos, st->Sc, st->meta16, h->d_status);
    DBW_LAUNCHED();
    SpMixArgs a{};
    a.N = h->N;
    a.n_halves = (st->rows_pad + kRowsPerItem - 1) / kRowsPerItem;
    a.n_ka = st->k_pad / kKA;
    a.n_panels = (int)((h->ld + kPanel - 1) / kPanel);
    a.mix_then_correct = (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0;
    a.ld = h->ld;
    a.X = X; a.G = G; a.lr = lr; a.lr_pw = lr_pw; a.Xout = X_out; a.shadow = shadow;
    a.scale = h->plan.w_self;
    a.order = st->d_order;
    a.meta16 = st->meta16;
    // an eighth of a work item's time (about 120 clocks per MMA, 6 MMAs per K step) between groups of pairs
    a.stagger_clocks = a.n_panels * a.n_halves > st->n_pairs ? a.n_ka * (kKA / kKB) * 6 * 120 / 8 : 0;
    a.status = h->d_status;
    int pairs = a.n_panels * a.n_halves < st->n_pairs ? a.n_panels * a.n_halves : st->n_pairs;
    pairs -= pairs % a.n_halves;  // whole groups of neighbouring pairs
    if (pairs < a.n_halves) return DBW_ERR_BAD_SHAPE;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    pair_launch_config(&cfg, &attr, 2 * pairs, s);
    DBW_CUDA(cudaLaunchKernelEx(&cfg, mix_sp_kernel, st->map, st->out_map, a));
    DBW_LAUNCHED();
    return DBW_OK;
}

// The 2:4 order of a graph on the host (no GPU needed): order[k_pad] receives the worker at each input
// position (-1 = empty); returns k_pad, or 0 when no order with k_pad <= 1024 was found.
int mix_sp_order_host(int N, const int32_t* rowptr, const int32_t* col, int32_t* order, int capacity) {
    for (int attempt = 0; attempt < 2; ++attempt) {
        OrderSearch s;
        s.N = N;
        s.k_pad = attempt == 0 ? (N + kKA - 1) / kKA * kKA : (2 * N + kKA - 1) / kKA * kKA;
        if (s.k_pad > kMaxN || s.k_pad > capacity) return 0;
        s.rowptr = rowptr;
        s.col = col;
        if (s.run()) {
            std::copy(s.order.begin(), s.order.end(), order);
            return s.k_pad;
        }
    }
    return 0;
}

}  // namespace dbw
