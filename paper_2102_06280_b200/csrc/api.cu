// C ABI entry points: argument checks on the host, workspace ownership, and the composition of
// one round (Algorithm 1) out of the stage launchers.
#include <algorithm>
#include <cstring>
#include <new>
#include <queue>

#include "common.cuh"

namespace dbw {
std::atomic<long long> g_launches{0};
std::atomic<int> g_last_cuda_error{0};
}  // namespace dbw

using namespace dbw;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        ok = cuda_ok(cudaGetDevice(&prev));
        if (ok && prev != dev) ok = cuda_ok(cudaSetDevice(dev));
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// Sorted, in range, no self loops, no duplicates, symmetric, connected.
bool valid_graph(int N, const int32_t* rowptr, const int32_t* col) {
    if (rowptr[0] != 0) return false;
    for (int i = 0; i < N; ++i) {
        if (rowptr[i + 1] < rowptr[i]) return false;
        for (int e = rowptr[i]; e < rowptr[i + 1]; ++e) {
            const int j = col[e];
            if (j < 0 || j >= N || j == i) return false;
            if (e > rowptr[i] && col[e - 1] >= j) return false;
        }
    }
    for (int i = 0; i < N; ++i)
        for (int e = rowptr[i]; e < rowptr[i + 1]; ++e) {
            const int j = col[e];
            int lo = rowptr[j], hi = rowptr[j + 1] - 1;
            bool found = false;
            while (lo <= hi) {
                const int mid = (lo + hi) / 2;
                if (col[mid] == i) { found = true; break; }
                if (col[mid] < i) lo = mid + 1; else hi = mid - 1;
            }
            if (!found) return false;
        }
    return true;
}

// Breadth-first spanning tree from worker 0, neighbours in ascending index, links in discovery
// order.  Returns false when the graph is not connected.
bool spanning_links(int N, const int32_t* rowptr, const int32_t* col, std::vector<int32_t>& links) {
    std::vector<char> seen(N, 0);
    std::queue<int> q;
    seen[0] = 1;
    q.push(0);
    links.clear();
    while (!q.empty()) {
        const int u = q.front();
        q.pop();
        for (int e = rowptr[u]; e < rowptr[u + 1]; ++e) {
            const int v = col[e];
            if (!seen[v]) {
                seen[v] = 1;
                links.push_back(u);
                links.push_back(v);
                q.push(v);
            }
        }
    }
    return (int)links.size() == 2 * (N - 1);
}

bool valid_model(const dbw_model_desc* m, int64_t d, int64_t ld) {
    if (m->n_layers < 1 || m->n_layers > DBW_MAX_LAYERS || m->batch < 1) return false;
    int64_t logical = 0;
    for (int l = 0; l <= m->n_layers; ++l)
        if (m->dims[l] < 1) return false;
    // every block inside the row, 32-float aligned, pairwise disjoint (checked in offset order)
    std::vector<std::pair<int64_t, int64_t>> blocks;
    for (int l = 0; l < m->n_layers; ++l) {
        const int64_t wsz = (int64_t)m->dims[l] * m->dims[l + 1];
        if (m->w_off[l] < 0 || m->b_off[l] < 0 || (m->w_off[l] & 31) || (m->b_off[l] & 31)) return false;
        blocks.push_back({m->w_off[l], wsz});
        blocks.push_back({m->b_off[l], m->dims[l + 1]});
        logical += wsz + m->dims[l + 1];
    }
    std::sort(blocks.begin(), blocks.end());
    int64_t end = 0;
    for (auto& b : blocks) {
        if (b.first < end) return false;
        end = b.first + b.second;
    }
    return end <= ld && logical == d;
}

template <typename T>
int dev_alloc(T** p, size_t n) {
    DBW_CUDA(cudaMalloc(reinterpret_cast<void**>(p), (n ? n : 1) * sizeof(T)));
    return DBW_OK;
}

void free_all(dbw_handle* h) {
    for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
    for (cudaEvent_t e : h->prof_gemm_events) cudaEventDestroy(e);
    h->prof_events.clear();
    h->prof_gemm_events.clear();
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->side) cudaStreamDestroy(h->side);
    h->ev_fork = h->ev_join = nullptr;
    h->side = nullptr;
    grad_fp32_free(h);
    grad_bf16_free(h);
    mix_tc_free(h);
    mix_sp_free(h);
    round_fused_free(h);
    void* ptrs[] = {h->d_rowptr, h->d_col, h->d_links, h->d_covered, h->d_epoch, h->d_status, h->d_waited,
                    h->d_ticket, h->d_Tnbr_ws, h->plan.idx, h->plan.w, h->plan.w_self, h->plan.cnt, h->d_G,
                    h->s_t, h->s_b, h->s_bidx, h->s_kept, h->s_Tw, h->s_Tr, h->s_loss};
    for (void* p : ptrs)
        if (p) cudaFree(p);
}

int ensure_G(dbw_handle* h) {
    if (h->d_G) return DBW_OK;
    int rc = dev_alloc(&h->d_G, (size_t)h->N * h->ld);
    if (rc != DBW_OK) return rc;
    DBW_CUDA(cudaMemset(h->d_G, 0, (size_t)h->N * h->ld * sizeof(float)));
    return DBW_OK;
}

int ensure_staging(dbw_handle* h) {
    if (h->s_t) return DBW_OK;
    int rc;
    if ((rc = dev_alloc(&h->s_t, h->N)) || (rc = dev_alloc(&h->s_b, h->N)) ||
        (rc = dev_alloc(&h->s_bidx, (size_t)h->N * (h->has_model ? h->model.batch : 1))) ||
        (rc = dev_alloc(&h->s_kept, h->nnz)) || (rc = dev_alloc(&h->s_Tw, h->N)) ||
        (rc = dev_alloc(&h->s_Tr, 1)) || (rc = dev_alloc(&h->s_loss, h->N)))
        return rc;
    return DBW_OK;
}

struct StateBlob {
    uint32_t magic;
    int32_t n_links;
    int32_t epoch[2];
    // followed by n_links int32 covered flags
};
constexpr uint32_t kStateMagic = 0x44425731u;  // "DBW1"
constexpr int kProfMaxRounds = 4096;

}  // namespace

extern "C" {

int dbw_model_layout(const int32_t* dims, int32_t n_layers, int32_t batch, dbw_model_desc* desc, int64_t* d,
                     int64_t* ld) {
    if (!dims || !desc || !d || !ld) return DBW_ERR_NULL;
    if (n_layers < 1 || n_layers > DBW_MAX_LAYERS || batch < 1) return DBW_ERR_BAD_MODEL;
    std::memset(desc, 0, sizeof(*desc));
    desc->n_layers = n_layers;
    desc->batch = batch;
    int64_t off = 0, logical = 0;
    for (int l = 0; l <= n_layers; ++l) {
        if (dims[l] < 1) return DBW_ERR_BAD_MODEL;
        desc->dims[l] = dims[l];
    }
    auto round32 = [](int64_t v) { return (v + 31) / 32 * 32; };
    for (int l = 0; l < n_layers; ++l) {
        const int64_t wsz = (int64_t)dims[l] * dims[l + 1];
        desc->w_off[l] = off;
        off = round32(off + wsz);
        desc->b_off[l] = off;
        off = round32(off + dims[l + 1]);
        logical += wsz + dims[l + 1];
    }
    *d = logical;
    *ld = off;
    return DBW_OK;
}

int dbw_init(dbw_handle** out, int32_t N, int64_t d, int64_t ld, const int32_t* h_rowptr, const int32_t* h_col,
             const dbw_model_desc* model, uint32_t flags, int device) {
    if (!out || !h_rowptr || !h_col) return DBW_ERR_NULL;
    *out = nullptr;
    if (N < 1 || d < 1 || ld < d || (ld & 3)) return DBW_ERR_BAD_SHAPE;
    if (!valid_graph(N, h_rowptr, h_col)) return DBW_ERR_BAD_GRAPH;
    if (model && !valid_model(model, d, ld)) return DBW_ERR_BAD_MODEL;
    dbw_handle* h = new (std::nothrow) dbw_handle();
    if (!h) return DBW_ERR_CUDA;
    h->N = N; h->d = d; h->ld = ld; h->flags = flags; h->device = device;
    h->nnz = h_rowptr[N];
    h->h_rowptr.assign(h_rowptr, h_rowptr + N + 1);
    h->h_col.assign(h_col, h_col + h->nnz);
    if (!spanning_links(N, h_rowptr, h_col, h->h_links)) {
        delete h;
        return DBW_ERR_BAD_GRAPH;
    }
    for (int i = 0; i < N; ++i) h->maxdeg = std::max(h->maxdeg, h_rowptr[i + 1] - h_rowptr[i]);

    DeviceGuard guard(device);
    int rc = guard.ok ? DBW_OK : DBW_ERR_CUDA;
    auto fail = [&](int code) {
        free_all(h);
        delete h;
        return code;
    };
    if (rc) return fail(rc);
    cudaDeviceProp prop;
    if (!cuda_ok(cudaGetDeviceProperties(&prop, device))) return fail(DBW_ERR_CUDA);
    h->sm_count = prop.multiProcessorCount;
    h->smem_optin = (int)prop.sharedMemPerBlockOptin;

    h->plan.stride = std::max(4, (h->maxdeg + 3) / 4 * 4);
    h->plan.n = N;
    const int D = N - 1;
    if ((rc = dev_alloc(&h->d_rowptr, N + 1)) || (rc = dev_alloc(&h->d_col, h->nnz)) ||
        (rc = dev_alloc(&h->d_links, 2 * D)) || (rc = dev_alloc(&h->d_covered, D)) ||
        (rc = dev_alloc(&h->d_epoch, 2)) || (rc = dev_alloc(&h->d_status, 1)) ||
        (rc = dev_alloc(&h->d_waited, N)) || (rc = dev_alloc(&h->d_ticket, 1)) ||
        (rc = dev_alloc(&h->d_Tnbr_ws, N)) || (rc = dev_alloc(&h->plan.idx, (size_t)N * h->plan.stride)) ||
        (rc = dev_alloc(&h->plan.w, (size_t)N * h->plan.stride)) || (rc = dev_alloc(&h->plan.w_self, N)) ||
        (rc = dev_alloc(&h->plan.cnt, N)))
        return fail(rc);
    bool ok = cuda_ok(cudaMemcpy(h->d_rowptr, h_rowptr, (N + 1) * sizeof(int32_t), cudaMemcpyHostToDevice)) &&
              cuda_ok(cudaMemcpy(h->d_col, h_col, (size_t)h->nnz * sizeof(int32_t), cudaMemcpyHostToDevice)) &&
              cuda_ok(cudaMemcpy(h->d_links, h->h_links.data(), (size_t)2 * D * sizeof(int32_t), cudaMemcpyHostToDevice)) &&
              cuda_ok(cudaMemset(h->d_covered, 0, (size_t)(D ? D : 1) * sizeof(int32_t))) &&
              cuda_ok(cudaMemset(h->d_epoch, 0, 2 * sizeof(int32_t))) &&
              cuda_ok(cudaMemset(h->d_status, 0, sizeof(uint32_t))) &&
              cuda_ok(cudaMemset(h->d_waited, 0, (size_t)N * sizeof(uint32_t))) &&
              cuda_ok(cudaMemset(h->d_ticket, 0, sizeof(uint32_t)));
    if (!ok) return fail(DBW_ERR_CUDA);
    h->plan.status = h->d_status;
    if (!cuda_ok(cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking)) ||
        !cuda_ok(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming)) ||
        !cuda_ok(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming)))
        return fail(DBW_ERR_CUDA);
    mix_sp_prepare(h);  // the 2:4 worker order of the sparse tensor-core mix, where that kernel can apply
    if (model) {
        h->has_model = true;
        h->model = *model;
        rc = (flags & DBW_GEMM_BF16) ? grad_bf16_alloc(h) : grad_fp32_alloc(h);
        if (rc) return fail(rc);
        round_fused_prepare(h);  // the single-launch round, for the networks it serves
    }
    *out = h;
    return DBW_OK;
}

int dbw_destroy(dbw_handle* h) {
    if (!h) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    cudaDeviceSynchronize();
    free_all(h);
    delete h;
    return DBW_OK;
}

int dbw_set_dataset(dbw_handle* h, const float* feat, const int32_t* labels, int32_t S) {
    if (!h || !feat || !labels) return DBW_ERR_NULL;
    if (!h->has_model) return DBW_ERR_BAD_MODEL;
    if (S < 1 || !aligned16(feat)) return DBW_ERR_BAD_SHAPE;
    h->feat = feat; h->labels = labels; h->S = S;
    return DBW_OK;
}

int dbw_set_edge_times(dbw_handle* h, const double* t_edge) {
    if (!h) return DBW_ERR_NULL;
    h->t_edge = t_edge;
    return DBW_OK;
}

int dbw_select(dbw_handle* h, const double* t, const int32_t* b, uint8_t* kept, double* T_worker, double* T_nbr,
               double* T_round, void* stream) {
    if (!h || !t || !b || !kept) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    return launch_select(h, t, b, kept, T_worker, T_nbr, T_round, false, (cudaStream_t)stream);
}

int dbw_grad(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss, void* stream) {
    if (!h || !X || !batch_idx || !G) return DBW_ERR_NULL;
    if (!h->has_model || !h->feat) return DBW_ERR_BAD_MODEL;
    if (!aligned16(X) || !aligned16(G)) return DBW_ERR_BAD_SHAPE;
    DeviceGuard guard(h->device);
    return (h->flags & DBW_GEMM_BF16) ? launch_grad_bf16(h, X, batch_idx, G, loss, (cudaStream_t)stream)
                                      : launch_grad_fp32(h, X, batch_idx, G, loss, (cudaStream_t)stream);
}

static int check_mix_args(dbw_handle* h, const float* X, const float* G, float* X_out) {
    if (!aligned16(X) || (G && !aligned16(G)) || !aligned16(X_out)) return DBW_ERR_BAD_SHAPE;
    const size_t bytes = (size_t)h->N * h->ld * sizeof(float);
    const char* a = reinterpret_cast<const char*>(X);
    const char* o = reinterpret_cast<const char*>(X_out);
    if (o != a && o < a + bytes && a < o + bytes) return DBW_ERR_BAD_SHAPE;  // partial overlap
    if (o == a && !mix_panel_fits(h)) return DBW_ERR_BAD_SHAPE;
    const char* g = reinterpret_cast<const char*>(G);
    if (g && o < g + bytes && g < o + bytes) return DBW_ERR_BAD_SHAPE;  // G is read only
    return DBW_OK;
}

int dbw_mix(dbw_handle* h, const float* X, const float* G, const uint8_t* kept, const int32_t* b, float lr,
            const float* lr_per_worker, float* X_out, void* stream) {
    if (!h || !X || !kept || !b || !X_out) return DBW_ERR_NULL;  // G == NULL: consensus only, G = 0
    int rc = check_mix_args(h, X, G, X_out);
    if (rc) return rc;
    DeviceGuard guard(h->device);
    if ((rc = launch_plan_from_kept(h, kept, b, (cudaStream_t)stream))) return rc;
    return launch_mix(h, X, G, lr, lr_per_worker, X_out, (cudaStream_t)stream);
}

int dbw_set_param_tracking(dbw_handle* h, int enable) {
    if (!h) return DBW_ERR_NULL;
    h->track_params = enable != 0;
    h->shadow_valid = false;
    h->shadow_of = nullptr;
    return DBW_OK;
}

int dbw_set_fused_round(dbw_handle* h, int enable) {
    if (!h) return DBW_ERR_NULL;
    h->fused_mode = enable < 0 ? -1 : (enable ? 1 : 0);
    return DBW_OK;
}

int dbw_round_is_fused(const dbw_handle* h) { return h ? (round_fused_usable(h) ? 1 : 0) : DBW_ERR_NULL; }

int dbw_mix_in_place_ok(const dbw_handle* h) { return h && mix_panel_fits(h) ? 1 : 0; }

int dbw_mix_kernel(const dbw_handle* h) { return h ? mix_kernel_kind(h) : DBW_ERR_NULL; }

int dbw_set_mix_panel(dbw_handle* h, int32_t cols) {
    if (!h) return DBW_ERR_NULL;
    if (!(cols == 0 || cols == -1 || cols == 1 || cols == 2 || cols == 3 || cols == 16 || cols == 32 || cols == 64 || cols == 128 || cols == 256)) return DBW_ERR_BAD_SHAPE;
    h->mix_panel_cols = cols;
    return DBW_OK;
}

int dbw_round(dbw_handle* h, const float* X, const double* t, const int32_t* b, const int32_t* batch_idx,
              const float* G_ext, float lr, const float* lr_per_worker, float* X_out, uint8_t* kept,
              double* T_worker, double* T_nbr, double* T_round, float* loss, void* stream) {
    if (!h || !X || !t || !b || !X_out || !kept) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    cudaStream_t s = (cudaStream_t)stream;
    int rc;
    const float* G = G_ext;  // NULL together with batch_idx == NULL: a consensus-only round, G = 0
    if (batch_idx) {
        if (!h->has_model || !h->feat) return DBW_ERR_BAD_MODEL;
        if ((rc = ensure_G(h))) return rc;
        G = h->d_G;
    }
    if ((rc = check_mix_args(h, X, G, X_out))) return rc;
    cudaEvent_t* ev = nullptr;
    if (h->profiling && h->prof_rounds < kProfMaxRounds) {
        while ((int)h->prof_events.size() < 6 * (h->prof_rounds + 1)) {
            cudaEvent_t e;
            DBW_CUDA(cudaEventCreate(&e));
            h->prof_events.push_back(e);
        }
        ev = &h->prof_events[6 * h->prof_rounds++];
        if ((int)h->prof_single.size() < h->prof_rounds) h->prof_single.resize(h->prof_rounds);
        h->prof_single[h->prof_rounds - 1] = 0;
    }
    if (batch_idx && round_fused_usable(h)) {
        // small fp32 network: the whole iteration in one cooperative launch (same bits as the launches below)
        if (ev) DBW_CUDA(cudaEventRecord(ev[0], s));
        rc = launch_round_fused(h, X, t, b, batch_idx, lr, lr_per_worker, X_out, kept, T_worker, T_nbr, T_round, loss, s);
        if (ev) {  // the stages are not separable: one pair of events, reported under "gradients"
            DBW_CUDA(cudaEventRecord(ev[1], s));
            h->prof_single[h->prof_rounds - 1] = 1;
        }
        h->shadow_valid = false;
        return rc;
    }
    // first error of the calls below; later calls still run so that a forked side stream is always joined
    int first = DBW_OK;
    auto note = [&](int code) {
        if (first == DBW_OK && code != DBW_OK) first = code;
    };
    auto cuda = [&](cudaError_t e) { note(cuda_ok(e) ? DBW_OK : DBW_ERR_CUDA); };
    // The selection needs only t and b, so with gradients to compute it runs beside them on the handle's
    // side stream: fork after everything the caller queued, join before the mix.
    cudaStream_t sel = s;
    bool forked = false;
    if (batch_idx) {
        cuda(cudaEventRecord(h->ev_fork, s));
        if (first == DBW_OK) cuda(cudaStreamWaitEvent(h->side, h->ev_fork, 0));
        if (first != DBW_OK) return first;  // nothing forked yet
        sel = h->side;
        forked = true;
    }
    if (ev) cuda(cudaEventRecord(ev[2], sel));
    note(launch_select(h, t, b, kept, T_worker, T_nbr, T_round, true, sel));
    if (ev) cuda(cudaEventRecord(ev[3], sel));
    if (ev) cuda(cudaEventRecord(ev[0], s));
    if (batch_idx && first == DBW_OK)
        note((h->flags & DBW_GEMM_BF16) ? launch_grad_bf16(h, X, batch_idx, h->d_G, loss, s)
                                        : launch_grad_fp32(h, X, batch_idx, h->d_G, loss, s));
    if (ev) cuda(cudaEventRecord(ev[1], s));
    if (forked) {  // whatever failed above, the side stream is joined back: it never dangles, a capture stays valid
        cuda(cudaEventRecord(h->ev_join, sel));
        cuda(cudaStreamWaitEvent(s, h->ev_join, 0));
    }
    if (first != DBW_OK) return first;
    if (ev) cuda(cudaEventRecord(ev[4], s));
    note(launch_mix(h, X, G, lr, lr_per_worker, X_out, s));
    if (ev) cuda(cudaEventRecord(ev[5], s));
    return first;
}

int dbw_profile(dbw_handle* h, int enable) {
    if (!h) return DBW_ERR_NULL;
    h->profiling = enable != 0;
    if (!h->profiling) h->prof_gemm_used = 0;
    return DBW_OK;
}

int dbw_profile_read(dbw_handle* h, double* ms, int32_t* rounds) {
    if (!h || !ms || !rounds) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    for (int r = 0; r < h->prof_rounds; ++r) {
        cudaEvent_t* ev = &h->prof_events[6 * r];
        if (h->prof_single[r]) {  // a single-launch round: one pair of events
            float v = 0.f;
            DBW_CUDA(cudaEventSynchronize(ev[1]));
            DBW_CUDA(cudaEventElapsedTime(&v, ev[0], ev[1]));
            ms[0] += v;
            continue;
        }
        DBW_CUDA(cudaEventSynchronize(ev[5]));
        for (int st = 0; st < 3; ++st) {  // gradients, selection (beside the gradients when there are any), mix
            float v = 0.f;
            DBW_CUDA(cudaEventElapsedTime(&v, ev[2 * st], ev[2 * st + 1]));
            ms[st] += v;
        }
    }
    for (int e = 0; e + 1 < h->prof_gemm_used; e += 2) {  // the tensor-core GEMM launches of those rounds
        float v = 0.f;
        DBW_CUDA(cudaEventSynchronize(h->prof_gemm_events[e + 1]));
        DBW_CUDA(cudaEventElapsedTime(&v, h->prof_gemm_events[e], h->prof_gemm_events[e + 1]));
        ms[3] += v;
    }
    h->prof_gemm_used = 0;
    *rounds = h->prof_rounds;
    h->prof_rounds = 0;
    return DBW_OK;
}

int dbw_round_host(dbw_handle* h, const float* X, const double* h_t, const int32_t* h_b,
                   const int32_t* h_batch_idx, const float* G_ext, float lr, float* X_out, uint8_t* h_kept,
                   double* h_T_worker, double* h_T_round, float* h_loss, int32_t* h_b_out, void* stream) {
    if (!h || !X || !h_t || !X_out) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    cudaStream_t s = (cudaStream_t)stream;
    int rc;
    if ((rc = ensure_staging(h))) return rc;
    DBW_CUDA(cudaMemcpyAsync(h->s_t, h_t, (size_t)h->N * sizeof(double), cudaMemcpyHostToDevice, s));
    if (h_b) {
        DBW_CUDA(cudaMemcpyAsync(h->s_b, h_b, (size_t)h->N * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    } else if ((rc = launch_update_backups(h, h->s_t, h->s_b, nullptr, s))) {
        return rc;
    }
    if (h_batch_idx) {
        if (!h->has_model) return DBW_ERR_BAD_MODEL;
        DBW_CUDA(cudaMemcpyAsync(h->s_bidx, h_batch_idx, (size_t)h->N * h->model.batch * sizeof(int32_t),
                                 cudaMemcpyHostToDevice, s));
    }
    rc = dbw_round(h, X, h->s_t, h->s_b, h_batch_idx ? h->s_bidx : nullptr, G_ext, lr, nullptr, X_out, h->s_kept,
                   h->s_Tw, nullptr, h->s_Tr, h->s_loss, stream);
    if (rc) return rc;
    if (h_kept) DBW_CUDA(cudaMemcpyAsync(h_kept, h->s_kept, (size_t)h->nnz, cudaMemcpyDeviceToHost, s));
    if (h_T_worker) DBW_CUDA(cudaMemcpyAsync(h_T_worker, h->s_Tw, (size_t)h->N * sizeof(double), cudaMemcpyDeviceToHost, s));
    if (h_T_round) DBW_CUDA(cudaMemcpyAsync(h_T_round, h->s_Tr, sizeof(double), cudaMemcpyDeviceToHost, s));
    if (h_b_out) DBW_CUDA(cudaMemcpyAsync(h_b_out, h->s_b, (size_t)h->N * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    if (h_loss && h_batch_idx) DBW_CUDA(cudaMemcpyAsync(h_loss, h->s_loss, (size_t)h->N * sizeof(float), cudaMemcpyDeviceToHost, s));
    return DBW_OK;
}

int dbw_update_backups(dbw_handle* h, const double* t_next, int32_t* b_out, double* theta_out, void* stream) {
    if (!h || !t_next || !b_out) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    return launch_update_backups(h, t_next, b_out, theta_out, (cudaStream_t)stream);
}

int dbw_reset_backups(dbw_handle* h, void* stream) {
    if (!h) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    const int D = h->N - 1;
    DBW_CUDA(cudaMemsetAsync(h->d_covered, 0, (size_t)(D ? D : 1) * sizeof(int32_t), (cudaStream_t)stream));
    DBW_CUDA(cudaMemsetAsync(h->d_epoch, 0, 2 * sizeof(int32_t), (cudaStream_t)stream));
    return DBW_OK;
}

int dbw_state_export(dbw_handle* h, void* buf, size_t* size, void* stream) {
    if (!h || !size) return DBW_ERR_NULL;
    const int D = h->N - 1;
    const size_t need = sizeof(StateBlob) + (size_t)D * sizeof(int32_t);
    if (!buf || *size < need) {
        *size = need;
        return buf ? DBW_ERR_STATE : DBW_OK;
    }
    DeviceGuard guard(h->device);
    StateBlob* blob = static_cast<StateBlob*>(buf);
    blob->magic = kStateMagic;
    blob->n_links = D;
    DBW_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    DBW_CUDA(cudaMemcpy(blob->epoch, h->d_epoch, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (D) DBW_CUDA(cudaMemcpy(blob + 1, h->d_covered, (size_t)D * sizeof(int32_t), cudaMemcpyDeviceToHost));
    *size = need;
    return DBW_OK;
}

int dbw_state_import(dbw_handle* h, const void* buf, size_t size, void* stream) {
    if (!h || !buf) return DBW_ERR_NULL;
    const int D = h->N - 1;
    const StateBlob* blob = static_cast<const StateBlob*>(buf);
    if (size != sizeof(StateBlob) + (size_t)D * sizeof(int32_t) || blob->magic != kStateMagic || blob->n_links != D)
        return DBW_ERR_STATE;
    DeviceGuard guard(h->device);
    DBW_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    DBW_CUDA(cudaMemcpy(h->d_epoch, blob->epoch, 2 * sizeof(int32_t), cudaMemcpyHostToDevice));
    if (D) DBW_CUDA(cudaMemcpy(h->d_covered, blob + 1, (size_t)D * sizeof(int32_t), cudaMemcpyHostToDevice));
    return DBW_OK;
}

int dbw_status(dbw_handle* h) {
    if (!h) return DBW_ERR_NULL;
    DeviceGuard guard(h->device);
    uint32_t v = 0;
    DBW_CUDA(cudaDeviceSynchronize());
    DBW_CUDA(cudaMemcpy(&v, h->d_status, sizeof(v), cudaMemcpyDeviceToHost));
    DBW_CUDA(cudaMemset(h->d_status, 0, sizeof(v)));
    return (int)v;
}

int dbw_get_links(const dbw_handle* h, int32_t* links) {
    if (!h || !links) return DBW_ERR_NULL;
    std::memcpy(links, h->h_links.data(), h->h_links.size() * sizeof(int32_t));
    return h->N - 1;
}

int dbw_graph_order_2of4(int32_t N, const int32_t* h_rowptr, const int32_t* h_col, int32_t* order, int32_t capacity) {
    if (!h_rowptr || !h_col || !order) return DBW_ERR_NULL;
    if (N < 1 || capacity < 1) return DBW_ERR_BAD_SHAPE;
    if (!valid_graph(N, h_rowptr, h_col)) return DBW_ERR_BAD_GRAPH;
    return mix_sp_order_host(N, h_rowptr, h_col, order, capacity);
}

int64_t dbw_launch_count(void) { return g_launches.load(); }
int dbw_last_cuda_error(void) { return g_last_cuda_error.load(); }

}  // extern "C"
