// based_selftest_bounded_wait: exercises the failure path of the device-side waits without
// faulting or hanging the GPU.  A one-CTA kernel waits on an mbarrier that nothing ever arrives
// on, with a short limit; the wait gives up, the kernel records it in the sticky status word
// and exits normally, and based_poll_error then reports BASED_ERR_DEVICE_TIMEOUT.
#include "common.cuh"
#include "sm100.cuh"

namespace based {

__global__ void bounded_wait_probe_kernel(unsigned int* err, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        abort_flag = 0;
        sm100::fence_mbar_init();
    }
    __syncthreads();
    const bool ok = sm100::mbar_wait(&bar, 0, &abort_flag, limit_ns);   // phase 0 never completes
    if (!ok && threadIdx.x == 0) atomicOr(err, 1u);
}

}  // namespace based

extern "C" based_status based_selftest_bounded_wait(unsigned int limit_ms, void* cuda_stream) {
    if (limit_ms == 0 || limit_ms > 2000) return BASED_ERR_INVALID_ARG;
    unsigned int* err = nullptr;
    if (based::error_word_ptr(&err) != BASED_OK) return BASED_ERR_CUDA;
    based::bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        err, static_cast<unsigned long long>(limit_ms) * 1000000ull);
    based::note_launch();
    return based::check_launch("bounded_wait_probe_kernel");
}
