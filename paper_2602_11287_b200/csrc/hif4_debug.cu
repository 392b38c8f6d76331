// Test hook for the bounded-wait machinery of the tensor-core kernels: a one-block kernel that waits, with the
// library's own mbar_wait, on an mbarrier that nothing ever arrives on.  No copy and no MMA is in flight, so
// when the (short, caller-given) budget runs out the kernel only raises the library's device error word and
// returns; hif4_last_device_status then reports HIF4_ERR_DEVICE_TIMEOUT once and clears it.  This is the same
// give-up path that every TMA / MMA / epilogue role of the GEMM kernels takes after its 2 s budget.
#include "hif4_common.cuh"
#include "hif4_tc_common.cuh"

namespace hif4 {
namespace {

__global__ void __launch_bounds__(64)
debug_wait_timeout_kernel(uint64_t budget_ns, unsigned int* error_word) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_word;
  const uint32_t bar_addr = smem_u32(&bar);
  volatile uint32_t* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(bar_addr, 1);            // one arrival expected; nobody arrives
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // warp 0 waits on the barrier; warp 1 waits too and leaves as soon as warp 0 has given up (the abort word),
  // as the other roles of a GEMM CTA do
  const bool ok = mbar_wait(bar_addr, 0u, abort_flag, 32, budget_ns);
  __syncthreads();
  if (!ok && threadIdx.x == 0 && *abort_flag) atomicExch(error_word, 1u);
}

}  // namespace
}  // namespace hif4

extern "C" hif4_status hif4_debug_wait_timeout(uint64_t budget_ns, void* stream) {
  using namespace hif4;
  if (budget_ns == 0 || budget_ns > 100000000ull) return HIF4_ERR_SHAPE;     // at most 0.1 s: this is a test hook
  unsigned int* word = device_error_word();
  if (!word) return HIF4_ERR_CUDA;
  debug_wait_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(budget_ns, word);
  note_launch();
  return launch_status();
}
