// Test support, not part of the public header: runs the bounded wait of the tensor-core kernels to its limit.
//
// Every wait of those kernels on an mbarrier gives up after a time limit, records TWN_ERR_TIMEOUT in the
// caller's status word, raises the block's abort flag so that the other roles leave their loops, and the
// kernel returns normally.  In a correct run no wait ever expires, so that path never executes; this entry
// point executes it on purpose, with a short limit, on a barrier that nothing ever arrives on.  Nothing here
// faults or waits without bound.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

__global__ void __launch_bounds__(96)
wait_timeout_kernel(int32_t *status, unsigned long long limit_ns, int *order)
{
    __shared__ unsigned long long bar;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);          // one arrival expected; none is ever made
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (warp == 0) {
        // a single-thread role (producer, MMA issuer): its wait runs out and raises the flag
        if (lane == 0) ok = mbar_wait(&bar, 0, &abort_flag, status, 64, limit_ns);
    } else if (warp == 1) {
        // a warp-wide role (decode, epilogue) with the full limit: it must leave because of the flag
        ok = mbar_wait_warp(&bar, 0, &abort_flag, status, 32);
    } else {
        // a warp-wide role with the short limit of its own
        ok = mbar_wait_warp(&bar, 0, &abort_flag, status, 32, limit_ns);
    }
    if (lane == 0) order[warp] = ok ? 1 : 0;
    __syncthreads();                 // the teardown barrier every role reaches
    if (threadIdx.x == 0) order[3] = abort_flag;
}

}  // namespace

// dev_status: device int32, zero before the call; receives TWN_ERR_TIMEOUT.  dev_out: device int[4]: whether
// each of the three waits reported success (all 0) and the block's abort flag (1).
extern "C" int twn_selftest_wait_timeout(int32_t *dev_status, int *dev_out, unsigned long long limit_ns, twn_stream_t stream)
{
    TWN_REQUIRE(dev_status && dev_out && limit_ns > 0 && limit_ns <= 100000000ull, TWN_ERR_INVALID_ARG);
    twn_device_info dev;
    const int rc = twn_current_device(&dev);
    if (rc != TWN_OK) return rc;
    wait_timeout_kernel<<<1, 96, 0, twn_cu(stream)>>>(dev_status, limit_ns, dev_out);
    TWN_CUDA_OK(cudaGetLastError());
    return TWN_OK;
}
