// Exercises the give-up path of the library's bounded waits without touching the attention kernels: a
// tiny kernel sets up an mbarrier on which nothing ever arrives and waits on it with mbar_wait, the same
// routine every wait of the tcgen05 kernels goes through, with a short limit.  The wait must run out,
// raise TTS_ERR_DEVICE_TIMEOUT in the status word and return; the kernel then ends normally, so the
// context stays usable.
#include "tts_internal.cuh"
#include "umma_ptx.cuh"

namespace tts {

namespace {

__global__ void __launch_bounds__(32) wait_probe_kernel(int32_t* status, long long limit_ns, int* gave_up) {
    __shared__ __align__(8) unsigned long long barrier_word;
    __shared__ int abort_flag;
    using namespace ptx;
    const uint32_t bar = smem_u32(&barrier_word);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const Abort ab{&abort_flag, status};
    bool done = true;
    if (threadIdx.x == 0) done = mbar_wait(bar, 0, ab, limit_ns);     // phase 0 never completes
    __syncwarp();
    // the other lanes see the abort flag exactly as the other roles of an attention kernel would
    if (threadIdx.x == 1 && gave_up) *gave_up = abort_flag;
    (void)done;
}

}  // namespace

cudaError_t launch_wait_probe(int32_t* status, long long limit_ns, int* gave_up, cudaStream_t st) {
    wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_ns, gave_up);
    return cudaGetLastError();
}

}  // namespace tts
