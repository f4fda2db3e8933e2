// Self-test of the bounded-wait machinery every tensor-core kernel of this library relies on.
//
// The pipelines hand tiles from role to role through mbarriers; every such wait has a time
// limit, and when one expires the waiting role records an error word, raises a CTA-wide abort
// flag that all other roles' waits poll, the producer waits (again bounded) for the copies it
// still has in flight, and the kernel returns normally.  In a healthy run none of this ever
// executes.  ta_selftest_wait_timeout runs exactly that sequence in a one-CTA kernel, on purpose
// and harmlessly: a barrier that nobody ever arrives at, waited on with a short limit given by
// the caller.  Nothing faults, nothing spins without limit, the context stays usable.
#include "ta_internal.h"
#include "ta_ptx.cuh"

namespace ta {
namespace {

__device__ __align__(128) unsigned char g_selftest_src[256];   // source of the copy in flight
__device__ unsigned int g_selftest_report[4];

// report[0]: 1 if the producer's wait on the orphan barrier returned false (expired)
// report[1]: 1 if the consumer's wait ended because it saw the abort flag (not its own limit)
// report[2]: 1 if the producer then saw its copy in flight complete (drain path)
// report[3]: nanoseconds the producer spent in the expired wait (saturated to 32 bits)
__global__ void __launch_bounds__(64, 1) wait_timeout_kernel(unsigned long long limit_ns) {
    __shared__ __align__(128) unsigned char tile[256];
    __shared__ __align__(8) unsigned long long bars[3];
    __shared__ unsigned int abort_word;
    const uint32_t full = smem_u32(&bars[0]), orphan_a = smem_u32(&bars[1]), orphan_b = smem_u32(&bars[2]);
    volatile uint32_t *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(full, 1);
        mbar_init(orphan_a, 1);
        mbar_init(orphan_b, 1);
        abort_word = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async_smem();
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0 && lane == 0) {
        // producer: one bulk copy in flight, then a wait for a slot nobody will ever hand back
        mbar_expect_tx(full, 256u);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_u32(tile)),
                     "l"(g_selftest_src), "r"(256u), "r"(full)
                     : "memory");
        const unsigned long long t0 = globaltimer_ns();
        const bool ok = mbar_wait_abortable(orphan_a, 0, 0xF0, abort_flag, limit_ns);
        const unsigned long long dt = globaltimer_ns() - t0;
        g_selftest_report[0] = ok ? 0u : 1u;
        g_selftest_report[3] = dt > 0xFFFFFFFFull ? 0xFFFFFFFFu : (unsigned int)dt;
        // leaving early: let the copy already issued land (bounded) before shared memory is released
        bool landed = false;
        const unsigned long long t1 = globaltimer_ns();
        while (!(landed = mbar_try_wait(full, 0)) && globaltimer_ns() - t1 < 10000000ull) {
        }
        g_selftest_report[2] = landed ? 1u : 0u;
    } else if (warp == 1 && lane == 0) {
        // another role, waiting (with the ordinary long limit) on something that will not come
        // either: it must leave as soon as the producer raises the flag
        const unsigned long long t0 = globaltimer_ns();
        const bool ok = mbar_wait_abortable(orphan_b, 0, 0xF1, abort_flag);
        const unsigned long long dt = globaltimer_ns() - t0;
        g_selftest_report[1] = (!ok && dt < kWaitLimitNs) ? 1u : 0u;
    }
    __syncthreads();
}

}  // namespace

int read_status_selftest(unsigned int *word) {
    if (cudaMemcpyFromSymbol(word, g_status_word, sizeof(*word)) != cudaSuccess) return TA_ERR_CUDA;
    if (*word != 0) {
        unsigned int z = 0;
        cudaMemcpyToSymbol(g_status_word, &z, sizeof(z));
    }
    return TA_OK;
}

}  // namespace ta

using namespace ta;

extern "C" int ta_selftest_wait_timeout(unsigned limit_us, unsigned *report, ta_stream_t stream) {
    if (limit_us == 0 || limit_us > 1000000u) return TA_ERR_INVALID_ARG;   // at most one second
    tl_last_cuda_error = 0;
    const cudaStream_t s = (cudaStream_t)stream;
    const unsigned int zero[4] = {0, 0, 0, 0};
    if (cudaMemcpyToSymbolAsync(g_selftest_report, zero, sizeof(zero), 0, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return cuda_fail(cudaGetLastError());
    const int rc = launch_kernel(wait_timeout_kernel, 1, 64, 0, s, false, (unsigned long long)limit_us * 1000ull);
    if (rc != TA_OK) return rc;
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    if (report) {
        e = cudaMemcpyFromSymbol(report, g_selftest_report, sizeof(zero));
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return TA_OK;
}
