// Fastest-neighbour selection (Section 2.2), iteration times (Section 3.2.2) and the per-round
// mixing plan with the weights of Assumption 1.  One warp per worker.
#include "common.cuh"
#include "round_dev.cuh"

namespace dbw {

namespace {

constexpr int kWarpsPerBlock = 4;

using namespace dev;

// Selection: one warp per worker (dev::select_worker); the last block to finish computes the per-worker and
// per-round times, which need to know who is waited for by whom.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
select_kernel(int N, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
              const double* __restrict__ t, const double* __restrict__ t_edge, const int32_t* __restrict__ b,
              uint8_t* __restrict__ kept,
              double* __restrict__ T_nbr_ws, double* T_nbr_out, double* T_worker, double* T_round,
              uint32_t* waited, uint32_t* ticket, uint32_t* status, MixPlan plan, int build_plan,
              int uniform) {
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (i < N) select_worker(i, lane, rowptr, col, t, t_edge, b, kept, T_nbr_ws, waited, status, plan, build_plan, uniform);

    // ---- last block: T_worker, T_round ----
    __shared__ bool is_last;
    __shared__ double red[kWarpsPerBlock];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double tr = round_times_part(N, rowptr, t, b, T_nbr_ws, T_nbr_out, T_worker, waited, status);
    tr = warp_max(tr);
    if (lane == 0) red[threadIdx.x >> 5] = tr;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 1; k < kWarpsPerBlock; ++k) tr = fmax(tr, red[k]);
        if (T_round) *T_round = tr;
        *ticket = 0u;
    }
}

// Plan from a caller-supplied kept mask (dbw_mix on its own).  With uniform weights the weight is
// 1 / (1 + number of kept entries in the mask), so a row's weights sum to one whatever the mask holds;
// a mask whose count differs from deg_i - b_i is reported (DBW_STATUS_BAD_B).  The weights of Assumption 1
// use the nominal counts p = deg - b of both ends and keep the rows stochastic through w_ii = 1 - sum.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
plan_kernel(int N, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
            const uint8_t* __restrict__ kept, const int32_t* __restrict__ b, uint32_t* status, MixPlan plan,
            int uniform) {
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (i >= N) return;
    const int lo = rowptr[i], hi = rowptr[i + 1], deg = hi - lo;
    int p = deg - clamped_b(b, i, deg, status);
    int n_kept = 0;
    for (int base = 0; base < deg; base += 32) {
        const int e = lo + base + lane;
        n_kept += __popc(__ballot_sync(0xffffffffu, e < hi && kept[e] != 0));
    }
    if (n_kept != p && lane == 0) atomicOr(status, DBW_STATUS_BAD_B);
    if (uniform) p = n_kept;
    float wsum = 0.f;
    int running = 0;
    for (int base = 0; base < deg; base += 32) {
        const int e = lo + base + lane;
        const bool keep = e < hi && kept[e] != 0;
        const int j = e < hi ? checked(col[e], N, status) : 0;
        float w = 0.f;
        if (keep) {
            const int dj = rowptr[j + 1] - rowptr[j];
            w = edge_weight(uniform, p, dj - clamped_b(b, j, dj, status));
            wsum += w;
        }
        plan_append(plan, i, lane, keep, j, w, running);
    }
    wsum = warp_sum(wsum);
    plan_finish(plan, i, lane, running, uniform ? 1.0f / (1.0f + (float)p) : 1.0f - wsum);
}

}  // namespace

int launch_select(dbw_handle* h, const double* t, const int32_t* b, uint8_t* kept, double* T_worker,
                  double* T_nbr, double* T_round, bool build_plan, cudaStream_t s) {
    const int blocks = (h->N + kWarpsPerBlock - 1) / kWarpsPerBlock;
    select_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(
        h->N, h->d_rowptr, h->d_col, t, h->t_edge, b, kept, h->d_Tnbr_ws, T_nbr, T_worker, T_round, h->d_waited,
        h->d_ticket, h->d_status, h->plan, build_plan ? 1 : 0, (h->flags & DBW_WEIGHT_UNIFORM) ? 1 : 0);
    DBW_LAUNCHED();
    return DBW_OK;
}

int launch_plan_from_kept(dbw_handle* h, const uint8_t* kept, const int32_t* b, cudaStream_t s) {
    const int blocks = (h->N + kWarpsPerBlock - 1) / kWarpsPerBlock;
    plan_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(h->N, h->d_rowptr, h->d_col, kept, b, h->d_status,
                                                       h->plan, (h->flags & DBW_WEIGHT_UNIFORM) ? 1 : 0);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw

// ---------------------------------------------------------------------------------------------
// Selection without a handle and without any allocation (dbw_select_static).
// ---------------------------------------------------------------------------------------------
namespace dbw {
namespace {

// Scratch of the allocation-free entry point, resident on every GPU that loads the library:
// [0,256) ticket and status words, then the "waited for" flags of N workers, then their T_nbr.
constexpr size_t kStaticFlagsOff = 256;
constexpr size_t kStaticTnbrOff = kStaticFlagsOff + sizeof(uint32_t) * DBW_SELECT_STATIC_MAX_N;
constexpr size_t kStaticBytes = kStaticTnbrOff + sizeof(double) * DBW_SELECT_STATIC_MAX_N;
static __device__ __align__(256) unsigned char g_select_scratch[kStaticBytes];

// Device address of the scratch on the current device (the symbol's name is only a host-side
// stand-in); looked up once per device, under a lock, so host threads may race for the first call.
int static_scratch(unsigned char** out) {
    static PerDeviceOnce once;
    static unsigned char* cache[64] = {};
    int dev = 0;
    DBW_CUDA(cudaGetDevice(&dev));
    const int rc = once.run(dev, [dev]() -> int {
        void* p = nullptr;
        DBW_CUDA(cudaGetSymbolAddress(&p, g_select_scratch));
        cache[dev] = static_cast<unsigned char*>(p);
        return DBW_OK;
    });
    if (rc) return rc;
    *out = cache[dev];
    return DBW_OK;
}

}  // namespace
}  // namespace dbw

extern "C" int dbw_select_static(int32_t N, const int32_t* rowptr, const int32_t* col, const double* t,
                                 const int32_t* b, uint8_t* kept, double* T_worker, double* T_nbr,
                                 double* T_round, uint32_t* status_out, void* stream) {
    if (!rowptr || !col || !t || !b || !kept) return DBW_ERR_NULL;
    if (N < 1) return DBW_ERR_BAD_SHAPE;
    if (N > DBW_SELECT_STATIC_MAX_N) return DBW_ERR_TOO_LARGE;
    unsigned char* base = nullptr;
    int rc = dbw::static_scratch(&base);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t* ticket = reinterpret_cast<uint32_t*>(base);
    uint32_t* status = ticket + 1;
    uint32_t* waited = reinterpret_cast<uint32_t*>(base + dbw::kStaticFlagsOff);
    double* tnbr = reinterpret_cast<double*>(base + dbw::kStaticTnbrOff);
    // the array keeps whatever the previous call left: ticket, status and flags must start at zero
    DBW_CUDA(cudaMemsetAsync(base, 0, dbw::kStaticFlagsOff + sizeof(uint32_t) * (size_t)N, s));
    const int blocks = (N + dbw::kWarpsPerBlock - 1) / dbw::kWarpsPerBlock;
    dbw::MixPlan no_plan{};
    no_plan.n = N;  // only the bounds-checked build looks at it: this entry point's CSR is not validated on the host
    dbw::select_kernel<<<blocks, dbw::kWarpsPerBlock * 32, 0, s>>>(N, rowptr, col, t, nullptr, b, kept, tnbr, T_nbr, T_worker,
                                                                   T_round, waited, ticket, status, no_plan, 0, 0);
    DBW_LAUNCHED();
    if (status_out) DBW_CUDA(cudaMemcpyAsync(status_out, status, sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    return DBW_OK;
}
