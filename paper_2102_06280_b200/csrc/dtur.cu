// Distributed threshold-based update rule (Section 4.1) and one iteration of Algorithm 2.
// One CTA: the state is N-1 flags and two counters, the work is O(N + nnz).
#include "common.cuh"

namespace dbw {

namespace {

constexpr int kThreads = 1024;

__device__ __forceinline__ double time_or_inf(double t, uint32_t* status) {
    if (t != t) {
        atomicOr(status, DBW_STATUS_NAN_TIME);
        return __longlong_as_double(0x7ff0000000000000LL);
    }
    return t;
}

__global__ void __launch_bounds__(kThreads)
update_backups_kernel(int N, const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                      const int32_t* __restrict__ links, int32_t* covered, int32_t* epoch,
                      const double* __restrict__ t, int32_t* __restrict__ b_out, double* theta_out,
                      uint32_t* status) {
    const int D = N - 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    // theta: earliest establishment time max(t_u, t_v) among the uncovered links, first on ties
    double best = inf;
    int best_pos = 0x7fffffff;
    for (int pos = tid; pos < D; pos += kThreads) {
        if (covered[pos]) continue;
        const double est = fmax(time_or_inf(t[checked(links[2 * pos], N, status)], status), time_or_inf(t[checked(links[2 * pos + 1], N, status)], status));
        if (est < best || (est == best && pos < best_pos)) {
            best = est;
            best_pos = pos;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int op = __shfl_xor_sync(0xffffffffu, best_pos, o);
        if (ob < best || (ob == best && op < best_pos)) {
            best = ob;
            best_pos = op;
        }
    }
    __shared__ double s_best[32];
    __shared__ int s_pos[32];
    __shared__ double s_theta;
    __shared__ int s_clear;
    if (lane == 0) {
        s_best[warp] = best;
        s_pos[warp] = best_pos;
    }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < kThreads / 32; ++w)
            if (s_best[w] < best || (s_best[w] == best && s_pos[w] < best_pos)) {
                best = s_best[w];
                best_pos = s_pos[w];
            }
        int clear = 0;
        if (best_pos != 0x7fffffff) {
            covered[best_pos] = 1;
            const int step = epoch[0] + 1;
            epoch[1] = best_pos;
            clear = step == D;
            epoch[0] = clear ? 0 : step;
        }
        s_theta = best;
        s_clear = clear;
        if (theta_out) *theta_out = best;
    }
    __syncthreads();
    const double theta = s_theta;
    if (s_clear)
        for (int pos = tid; pos < D; pos += kThreads) covered[pos] = 0;
    // threshold rule: on-time workers wait for their on-time neighbours, late workers for nobody
    for (int j = tid; j < N; j += kThreads) {
        const int lo = rowptr[j], hi = rowptr[j + 1];
        int p = 0;
        if (time_or_inf(t[j], status) <= theta)
            for (int e = lo; e < hi; ++e) p += time_or_inf(t[checked(col[e], N, status)], status) <= theta;
        b_out[j] = (hi - lo) - p;
    }
}

}  // namespace

int launch_update_backups(dbw_handle* h, const double* t, int32_t* b_out, double* theta_out, cudaStream_t s) {
    update_backups_kernel<<<1, kThreads, 0, s>>>(h->N, h->d_rowptr, h->d_col, h->d_links, h->d_covered,
                                                 h->d_epoch, t, b_out, theta_out, h->d_status);
    DBW_LAUNCHED();
    return DBW_OK;
}

}  // namespace dbw
