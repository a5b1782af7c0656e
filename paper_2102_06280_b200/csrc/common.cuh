// Shared declarations of the cb-DyBW round library: the handle and the host-side launchers
// each translation unit provides.  No device code crosses translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "dbw.h"

namespace dbw {

extern std::atomic<long long> g_launches;
extern std::atomic<int> g_last_cuda_error;

inline bool cuda_ok(cudaError_t e) {
    if (e != cudaSuccess) {
        g_last_cuda_error.store((int)e);
        return false;
    }
    return true;
}

#define DBW_CUDA(call)                                  \
    do {                                                \
        if (!::dbw::cuda_ok((call))) return DBW_ERR_CUDA; \
    } while (0)

// Counts a kernel launch and reports a launch-configuration failure.
#define DBW_LAUNCHED()                                         \
    do {                                                       \
        ::dbw::g_launches.fetch_add(1);                        \
        if (!::dbw::cuda_ok(cudaGetLastError())) return DBW_ERR_CUDA; \
    } while (0)

// One-time set-up per device (kernel attributes, symbol addresses), safe when several host threads
// make the first call at once: `f` runs under the lock until it has succeeded once on that device.
struct PerDeviceOnce {
    std::mutex mu;
    bool done[64] = {};
    template <class F>
    int run(int dev, F&& f) {
        if (dev < 0 || dev >= 64) return DBW_ERR_BAD_SHAPE;
        std::lock_guard<std::mutex> lock(mu);
        if (done[dev]) return DBW_OK;
        const int rc = f();
        if (rc == DBW_OK) done[dev] = true;
        return rc;
    }
};

// Per-round mixing plan (built on the device from kept and b): for each worker the compacted
// list of kept neighbours with their weights, padded to `stride` entries with (self, 0).
struct MixPlan {
    int* idx = nullptr;      // [N][stride]
    float* w = nullptr;      // [N][stride]
    float* w_self = nullptr; // [N]
    int* cnt = nullptr;      // [N]
    int stride = 0;
    int n = 0;                   // N (0 in a default-constructed plan: nothing to check against)
    uint32_t* status = nullptr;  // the handle's status word, for the index checks of the bounds-checked build
};

// Index check of the bounds-checked build (-DDBW_BOUNDS, libdbw_dbg.so): an index outside [0, limit) that a
// kernel read from its own data sets DBW_STATUS_BOUNDS and is replaced by 0, so that the access which follows
// stays inside its array (nothing traps).  The regular build compiles the check away.
__device__ __forceinline__ int checked(int idx, int limit, uint32_t* status) {
#ifdef DBW_BOUNDS
    if (limit > 0 && (idx < 0 || idx >= limit)) {
        if (status) atomicOr(status, DBW_STATUS_BOUNDS);
        return 0;
    }
#endif
    return idx;
}

struct BF16State;  // tensor-core gradient path (grad_bf16.cu)
struct TcMixState;  // tensor-core mix (mix_tc.cu)
struct SpMixState;  // tensor-core mix with 2:4 structured sparsity (mix_sp.cu)
struct FusedState;  // single-launch round for small networks (round_fused.cu)

}  // namespace dbw

struct dbw_handle {
    int N = 0;
    int64_t d = 0, ld = 0;
    int nnz = 0;
    int maxdeg = 0;
    uint32_t flags = 0;
    int device = 0;
    int sm_count = 0;
    int smem_optin = 0;  // max dynamic shared memory per block

    std::vector<int32_t> h_rowptr, h_col, h_links;  // host copies; links = (u,v) pairs of P
    int32_t* d_rowptr = nullptr;
    int32_t* d_col = nullptr;
    int32_t* d_links = nullptr;  // [2*(N-1)]

    // Algorithm 2 state, device resident: covered[N-1] flags then step counter
    int32_t* d_covered = nullptr;  // [N-1]
    int32_t* d_epoch = nullptr;    // [2]: links covered in this epoch, position of last credited link

    uint32_t* d_status = nullptr;    // [1]
    uint32_t* d_waited = nullptr;    // [N] scratch flags of the selection kernel (kept zero between calls)
    uint32_t* d_ticket = nullptr;    // [1] block ticket of the selection kernel (kept zero between calls)
    double* d_Tnbr_ws = nullptr;     // [N]

    const double* t_edge = nullptr;  // optional per-link arrival times (caller-owned, DEVICE, aligned with col)

    dbw::MixPlan plan;
    int mix_panel_cols = 0;  // 0 = automatic
    dbw::TcMixState* mix_tc = nullptr;  // selection matrix and tensor map of the tensor-core mix (lazy)
    dbw::SpMixState* mix_sp = nullptr;  // 2:4 order, compressed selection matrix and tensor maps of the sparse tensor-core mix (dbw_init)

    dbw::FusedState* fused = nullptr;   // single-launch round (dbw_init)
    int fused_mode = -1;                // -1 = where it is the faster path, 0 = never, 1 = wherever it applies

    // model / gradient path
    bool has_model = false;
    dbw_model_desc model{};
    const float* feat = nullptr;
    const int32_t* labels = nullptr;
    int32_t S = 0;
    float* d_act[DBW_MAX_LAYERS + 1] = {};  // fp32 path: A_0 (gathered batch) .. A_L (logits), [N][B][dims[l]]
    float* d_dz[DBW_MAX_LAYERS + 1] = {};   // fp32 path: dZ_l for l = 1..L, [N][B][dims[l]]
    int32_t* d_ylab = nullptr;              // [N][B] gathered labels
    float* d_G = nullptr;                   // [N][ld] gradient workspace of dbw_round (lazy)
    dbw::BF16State* bf16 = nullptr;
    // bf16 shadow of the parameter matrix, [N][ld], same layout as X (tensor-core path only).  The
    // mix writes it next to X' when parameter tracking is on; the next gradient call then skips the
    // weight cast if it is handed that very X'.
    uint16_t* d_shadow = nullptr;
    bool track_params = false;
    bool shadow_valid = false;
    const float* shadow_of = nullptr;

    // selection of dbw_round runs beside the gradient kernels on this stream (forked from and joined back
    // into the caller's stream by the two events)
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;

    // stage timing (dbw_profile): events[round][0..5] = start / end of the gradient, selection and mix stages
    bool profiling = false;
    std::vector<cudaEvent_t> prof_events;
    std::vector<cudaEvent_t> prof_gemm_events;  // pairs around every tensor-core GEMM launch while profiling
    int prof_gemm_used = 0;
    std::vector<char> prof_single;  // per recorded round: 1 = single-launch round (events 0 and 1 only)
    int prof_rounds = 0;

    // device staging of dbw_round_host
    double* s_t = nullptr;
    int32_t* s_b = nullptr;
    int32_t* s_bidx = nullptr;
    uint8_t* s_kept = nullptr;
    double* s_Tw = nullptr;
    double* s_Tr = nullptr;
    float* s_loss = nullptr;
};

namespace dbw {

// select.cu
int launch_select(dbw_handle* h, const double* t, const int32_t* b, uint8_t* kept, double* T_worker,
                  double* T_nbr, double* T_round, bool build_plan, cudaStream_t s);
int launch_plan_from_kept(dbw_handle* h, const uint8_t* kept, const int32_t* b, cudaStream_t s);

// mix.cu
int launch_mix(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
               cudaStream_t s);
// device helper shared by the mix kernels: four floats -> four bf16 (round to nearest even)
__device__ __forceinline__ uint2 pack_bf16x4_rn(float a, float b, float c, float d) {
    uint32_t lo, hi;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(b), "f"(a));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(d), "f"(c));
    return make_uint2(lo, hi);
}
bool mix_panel_fits(const dbw_handle* h);
int mix_kernel_kind(const dbw_handle* h);

// mix_staged.cu
bool mix_staged_usable(const dbw_handle* h);
int launch_mix_staged(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
                      uint16_t* shadow, cudaStream_t s);

// mix_tc.cu
bool mix_tc_usable(const dbw_handle* h);
bool mix_tc_in_place_ok(const dbw_handle* h);
void mix_tc_free(dbw_handle* h);
int launch_mix_tc(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
                  uint16_t* shadow, cudaStream_t s);

// mix_sp.cu
void mix_sp_prepare(dbw_handle* h);
bool mix_sp_usable(const dbw_handle* h);
bool mix_sp_in_place_ok(const dbw_handle* h);
void mix_sp_free(dbw_handle* h);
int launch_mix_sp(dbw_handle* h, const float* X, const float* G, float lr, const float* lr_pw, float* X_out,
                  uint16_t* shadow, cudaStream_t s);
int mix_sp_order_host(int N, const int32_t* rowptr, const int32_t* col, int32_t* order, int capacity);

// round_fused.cu
void round_fused_prepare(dbw_handle* h);
bool round_fused_usable(const dbw_handle* h);
void round_fused_free(dbw_handle* h);
int launch_round_fused(dbw_handle* h, const float* X, const double* t, const int32_t* b, const int32_t* batch_idx, float lr,
                       const float* lr_pw, float* X_out, uint8_t* kept, double* T_worker, double* T_nbr, double* T_round,
                       float* loss, cudaStream_t s);

// dtur.cu
int launch_update_backups(dbw_handle* h, const double* t, int32_t* b_out, double* theta_out, cudaStream_t s);

// grad_fp32.cu
// fp32 gradient path: shared memory of the last layer's backward step (the worker's dZ and its row offsets),
// and whether the last layer can take the small-output path (at most 32 classes, 16-byte rows).
inline size_t fp32_head_smem_bytes(int B, int C) { return (size_t)((B * C + 1) & ~1) * 4 + (size_t)B * 8; }
inline bool fp32_head_usable(const dbw_handle* h) {
    const dbw_model_desc& m = h->model;
    const int L = m.n_layers;
    if (L < 1) return false;
    return m.dims[L] <= 32 && (m.dims[L - 1] & 3) == 0 && (m.w_off[L - 1] & 3) == 0 && (h->ld & 3) == 0 &&
           ((uintptr_t)h->feat & 15) == 0 && fp32_head_smem_bytes(m.batch, m.dims[L]) <= 32768;
}
int grad_fp32_alloc(dbw_handle* h);
void grad_fp32_free(dbw_handle* h);
int launch_grad_fp32(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss,
                     cudaStream_t s);

// grad_bf16.cu
int grad_bf16_alloc(dbw_handle* h);
void grad_bf16_free(dbw_handle* h);
int launch_grad_bf16(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss,
                     cudaStream_t s);

}  // namespace dbw
