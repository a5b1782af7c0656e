// Masked consensus mix fused with the SGD step (Eqs. 4-5, or Eq. 3 over the kept set).
//
// Panel kernel: a CTA owns a panel of `4*GS` consecutive columns of ALL N rows.  It streams the
// panel of X and G from HBM once (128-bit loads), forms the locally updated rows x - lr*g on
// the fly and parks them in shared memory; then every output row of the panel is a weighted sum
// of shared-memory rows, written once with 128-bit stores.  Each element of X and G is read from
// HBM once and each element of X' is written once (12 bytes per parameter element).  A panel is
// fully staged before any of it is written and panels are disjoint, so X' may overwrite X.
// G == nullptr in any of the kernels means G = 0 (a consensus-only round): nothing of G is read, 8 bytes
// per element.
#include "common.cuh"
#include "round_dev.cuh"

namespace dbw {

namespace {

constexpr int kMixThreads = 512;

using namespace dev;

template <int GS>
__global__ void __launch_bounds__(kMixThreads, 3)
mix_panel_kernel(int N, long long ld, const float* X, const float* __restrict__ G, float lr,
                 const float* __restrict__ lr_pw, float* Xout, uint16_t* __restrict__ shadow, MixPlan plan,
                 int mix_then_correct, int n_panels) {
    extern __shared__ float4 sm[];  // [N][GS]
    for (int panel = blockIdx.x; panel < n_panels; panel += gridDim.x) {
        mix_panel_body<GS, kMixThreads>(panel, sm, N, ld, X, G, lr, lr_pw, Xout, shadow, plan, mix_then_correct);
        __syncthreads();
    }
}

// Fallback for graphs too large for a shared-memory panel: neighbour rows are re-read through L2.
// A work item is one output row of one column panel; a block computes it with consecutive lanes on
// consecutive columns (every neighbour read of a warp is one contiguous 512-byte segment).  Items are
// numbered row-fastest inside a panel and handed out in order, so the blocks that run at the same
// time work on the same column panel, whose X and G segments (N x panel_cols x 8 bytes, sized to a
// small share of L2) are fetched from HBM once and re-read out of L2 by the rows that keep them.  Out of place only.
__global__ void __launch_bounds__(256)
mix_direct_kernel(int N, long long ld, const float* __restrict__ X, const float* __restrict__ G, float lr,
                  const float* __restrict__ lr_pw, float* __restrict__ Xout, uint16_t* __restrict__ shadow,
                  MixPlan plan, int mix_then_correct, int panel_cols, long long n_items) {
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int i = (int)(item % N);
        const long long c = (item / N) * panel_cols + 4 * (long long)threadIdx.x;
        if (c >= ld) continue;
        auto stepped = [&](int r) {
            float4 v = ldg4(X + (size_t)r * ld + c);
            if (G && !mix_then_correct) v = fma4(-(lr_pw ? lr_pw[r] : lr), ldg4(G + (size_t)r * ld + c), v);
            return v;
        };
        const float ws = plan.w_self[i];
        const float4 self = stepped(i);
        float4 acc = make_float4(ws * self.x, ws * self.y, ws * self.z, ws * self.w);
        const int cnt = plan.cnt[i];
        const int* pi = plan.idx + (size_t)i * plan.stride;
        const float* pw = plan.w + (size_t)i * plan.stride;
        int k = 0;
        for (; k + 4 <= cnt; k += 4) {  // four neighbour rows in flight, added in list order
            const float4 v0 = stepped(checked(pi[k], N, plan.status)), v1 = stepped(checked(pi[k + 1], N, plan.status)),
                         v2 = stepped(checked(pi[k + 2], N, plan.status)), v3 = stepped(checked(pi[k + 3], N, plan.status));
            acc = fma4(pw[k], v0, acc);
            acc = fma4(pw[k + 1], v1, acc);
            acc = fma4(pw[k + 2], v2, acc);
            acc = fma4(pw[k + 3], v3, acc);
        }
        for (; k < cnt; ++k) acc = fma4(pw[k], stepped(checked(pi[k], N, plan.status)), acc);
        if (G && mix_then_correct) acc = fma4(-(lr_pw ? lr_pw[i] : lr), ldg4(G + (size_t)i * ld + c), acc);
        *reinterpret_cast<float4*>(Xout + (size_t)i * ld + c) = acc;
        if (shadow) *reinterpret_cast<uint2*>(shadow + (size_t)i * ld + c) = pack_bf16x4_rn(acc.x, acc.y, acc.z, acc.w);
    }
}

int auto_group_size(const dbw_handle* h) {
    if (h->mix_panel_cols < 0) return 0;  // direct kernel forced
    if (h->mix_panel_cols >= 1 && h->mix_panel_cols <= 3) return 0;  // staged / tensor-core kernels forced (handled by the caller)
    if (h->mix_panel_cols) return ((size_t)h->N * h->mix_panel_cols * 4 <= (size_t)h->smem_optin) ? h->mix_panel_cols / 4 : 0;
    // few workers and a matrix that streams from HBM (well beyond L2): 256-column panels (1 KB row segments) while
    // three CTAs still share an SM
    if ((size_t)h->N * 64 * 16 <= (size_t)(h->smem_optin) / 3 - 1024 && (size_t)h->N * h->ld * 4 > ((size_t)256 << 20)) return 64;
    // widest panel whose staging buffer still lets two CTAs share an SM
    const size_t budget = (size_t)(h->smem_optin) / 2 - 1024;
    for (int gs = 32; gs >= 4; gs >>= 1)
        if ((size_t)h->N * gs * 16 <= budget) return gs;
    return ((size_t)h->N * 4 * 16 <= (size_t)h->smem_optin) ? 4 : 0;
}

template <int GS>
int launch_panel(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
                 uint16_t* shadow, cudaStream_t s) {
    const size_t smem = (size_t)h->N * GS * 16;
    static PerDeviceOnce once;
    const int rc = once.run(h->device, [h]() -> int {
        DBW_CUDA(cudaFuncSetAttribute(mix_panel_kernel<GS>, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin));
        return DBW_OK;
    });
    if (rc) return rc;
    int per_sm = 0;
    DBW_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mix_panel_kernel<GS>, kMixThreads, smem));
    if (per_sm < 1) return DBW_ERR_BAD_SHAPE;
    const int n_panels = (int)((h->ld + 4 * GS - 1) / (4 * GS));
    const int grid = n_panels < per_sm * h->sm_count ? n_panels : per_sm * h->sm_count;
    mix_panel_kernel<GS><<<grid, kMixThreads, smem, s>>>(h->N, h->ld, X, G, lr, lr_pw, X_out, shadow, h->plan,
                                                        (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0,
                                                        n_panels);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace

constexpr bool kSparseByDefault = false;

// The tensor-memory staged kernel takes over when it applies and the plain panel kernel could not
// keep a 32-column (128-byte segment) panel with two CTAs per SM.
static bool use_staged(const dbw_handle* h) {
    if (!mix_staged_usable(h)) return false;
    if (h->mix_panel_cols == 1) return true;
    return h->mix_panel_cols == 0 && auto_group_size(h) < 8;
}

// The tensor-core kernel (dense 0/1 selection product) when asked for and applicable.
static bool use_tc(const dbw_handle* h) { return h->mix_panel_cols == 2 && mix_tc_usable(h); }

// The 2:4 structured-sparse tensor-core kernel: when asked for, or automatically where the staged kernel
// would otherwise run with uniform weights (many workers, many kept neighbours) and a 2:4 order exists.
static bool use_sp(const dbw_handle* h) {
    if (!mix_sp_usable(h)) return false;
    if (h->mix_panel_cols == 3) return true;
    return h->mix_panel_cols == 0 && kSparseByDefault && h->N >= 512 && use_staged(h);
}

bool mix_panel_fits(const dbw_handle* h) {
    if (use_sp(h)) return mix_sp_in_place_ok(h);
    return use_tc(h) ? mix_tc_in_place_ok(h) : (use_staged(h) || auto_group_size(h) != 0);
}
int mix_kernel_kind(const dbw_handle* h) { return use_sp(h) ? 4 : use_tc(h) ? 3 : use_staged(h) ? 2 : (auto_group_size(h) != 0 ? 1 : 0); }

int launch_mix(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
               cudaStream_t s) {
    // With parameter tracking the bf16 shadow of X' is written alongside; any other mix call leaves
    // the shadow stale for the buffer it describes.
    uint16_t* shadow = (h->track_params && h->d_shadow) ? h->d_shadow : nullptr;
    h->shadow_valid = shadow != nullptr;
    h->shadow_of = X_out;
    if (use_sp(h)) return launch_mix_sp(h, X, G, lr, lr_pw, X_out, shadow, s);
    if (use_tc(h)) return launch_mix_tc(h, X, G, lr, lr_pw, X_out, shadow, s);
    if (use_staged(h)) return launch_mix_staged(h, X, G, lr, lr_pw, X_out, shadow, s);
    switch (auto_group_size(h)) {
        case 64: return launch_panel<64>(h, X, G, lr, lr_pw, X_out, shadow, s);
        case 32: return launch_panel<32>(h, X, G, lr, lr_pw, X_out, shadow, s);
        case 16: return launch_panel<16>(h, X, G, lr, lr_pw, X_out, shadow, s);
        case 8: return launch_panel<8>(h, X, G, lr, lr_pw, X_out, shadow, s);
        case 4: return launch_panel<4>(h, X, G, lr, lr_pw, X_out, shadow, s);
        default: break;
    }
    if (X_out == X) return DBW_ERR_BAD_SHAPE;
    // panel width: the widest of 1024 / 512 / 256 columns whose X and G segments of all rows stay within
    // 12 MB (measured: a small share of L2 keeps the re-reads hitting while the rest of the grid streams
    // through; 128-column panels leave too few threads per block), and no wider than the matrix needs
    int panel_cols = 1024;
    while (panel_cols > 128 && ((panel_cols > 256 && (long long)h->N * panel_cols * 8 > (12ll << 20)) || panel_cols / 2 >= h->ld)) panel_cols >>= 1;
    const long long n_items = ((h->ld + panel_cols - 1) / panel_cols) * h->N;
    long long blocks = (long long)h->sm_count * (2048 / (panel_cols / 4) > 16 ? 16 : 2048 / (panel_cols / 4));
    if (blocks > n_items) blocks = n_items;
    mix_direct_kernel<<<(int)blocks, panel_cols / 4, 0, s>>>(h->N, h->ld, X, G, lr, lr_pw, X_out, shadow, h->plan,
                                                           (h->flags & DBW_ORDER_MIX_THEN_CORRECT) ? 1 : 0, panel_cols, n_items);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
