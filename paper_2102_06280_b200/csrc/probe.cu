// Self-test of the bounded pipeline wait: a wait that nothing will ever complete must give up after its
// poll limit, report it, and make every later wait of the CTA return at once.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace dbw {
namespace {

// out[0] = 1 if the first wait returned "not completed", out[1] = 1 if the second wait (after the
// abort word was set) returned "not completed", out[2] = clock ticks the second wait took.
__global__ void wait_probe_kernel(uint32_t polls, uint32_t* status, uint32_t* out) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0u;
        ptx::mbar_init(&bar, 1);  // one arrival expected; nobody arrives
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 32) {  // a second warp, as a pipeline role would be
        const bool first = ptx::mbar_wait_bounded<false>(&bar, 0, polls, 32, &abort_word, status);
        const long long t0 = clock64();
        const bool second = ptx::mbar_wait_bounded<false>(&bar, 0, 1u << 24, 0, &abort_word, status);
        const long long t1 = clock64();
        out[0] = first ? 0u : 1u;
        out[1] = second ? 0u : 1u;
        out[2] = (uint32_t)(t1 - t0);
    }
}

}  // namespace
}  // namespace dbw

extern "C" int dbw_debug_wait_probe(dbw_handle* h, uint32_t polls, uint32_t* out, void* stream) {
    if (!h || !out) return DBW_ERR_NULL;
    if (polls < 1 || polls > (1u << 20)) return DBW_ERR_BAD_SHAPE;
    int prev = -1;
    DBW_CUDA(cudaGetDevice(&prev));
    if (prev != h->device) DBW_CUDA(cudaSetDevice(h->device));
    dbw::wait_probe_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(polls, h->d_status, out);
    ::dbw::g_launches.fetch_add(1);
    const bool ok = ::dbw::cuda_ok(cudaGetLastError());
    if (prev != h->device) cudaSetDevice(prev);
    return ok ? DBW_OK : DBW_ERR_CUDA;
}
