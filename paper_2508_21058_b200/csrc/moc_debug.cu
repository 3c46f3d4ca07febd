// Test hooks that need a kernel of their own.
//
// moc_debug_wait_probe: the kernels of this library bound every wait on an mbarrier; when one runs out
// the block records MOC_ERR_TIMEOUT and a code in the workspace's status area and returns normally.
// Nothing in a healthy run makes a wait run out, so this probe does it on purpose in the one way that is
// harmless: a block waits on a barrier that no thread, copy or tensor-core operation will ever arrive
// on, through the same bounded wait as every other kernel, with the limit the workspace states.  It
// touches no other memory, holds no tensor memory and has no copy in flight, so giving up is all it does.
#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

__global__ void __launch_bounds__(32) wait_probe_kernel(int *status, int code, unsigned wait_us) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        status[ST_WAIT_US] = (int)wait_us;      // what routing with this plan would have stated
        __threadfence();
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        volatile int *abort_flag = &s_abort;
        // phase 0 of a freshly initialised barrier completes only after one arrival: none comes
        (void)tc::mbar_wait(tc::smem_u32(&bar), 0, abort_flag, status, code);
    }
    __syncwarp();
}

}  // namespace moc

extern "C" int moc_debug_wait_probe(const moc_plan *p, void *ws, int code, void *stream) {
    using namespace moc;
    if (!p) return MOC_ERR_NULL;
    if (!ws) return MOC_ERR_WORKSPACE;
    if (p->wait_us == 0 || p->wait_us > 100000u) return MOC_ERR_SHAPE;   // a probe never waits longer than 0.1 s
    wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ws_ptr<int>(ws, p->ws.status), code, p->wait_us);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}
