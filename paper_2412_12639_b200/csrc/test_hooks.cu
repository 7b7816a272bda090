// falcon_test_poison: a test hook.  Every SM's shared memory and tensor memory are filled with a
// bit pattern, so that a kernel launched afterwards which reads on-chip memory it has not written
// itself (a tile row that was never loaded, an accumulator column that was never started) computes
// with that pattern instead of with whatever an earlier launch happened to leave: all ones are a
// NaN as bf16 and as fp32.  Nothing here can fault or wait: plain stores, one TMEM allocation that
// is given back before the kernel ends.
#include "tc_util.cuh"

namespace falcon {
namespace {
using namespace tc;

constexpr uint32_t kPoisonSmem = 227u * 1024u - 1024u;

__global__ void __launch_bounds__(128, 1) poison_kernel(uint32_t pattern) {
  extern __shared__ uint4 poison_smem[];
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  const uint4 v = make_uint4(pattern, pattern, pattern, pattern);
  for (uint32_t i = tid; i < kPoisonSmem / 16; i += 128) poison_smem[i] = v;
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t base = tmem_base_s + (static_cast<uint32_t>(warp * 32) << 16);  // this warp's lane quadrant
  uint32_t r[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = pattern;
  for (uint32_t c = 0; c < 512; c += 32) FALCON_TMEM_ST32(base + c, r);
  tmem_wait_st();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"(512u) : "memory");
  }
}

}  // namespace

int launch_test_poison(falcon_ctx* ctx, uint32_t pattern, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(poison_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kPoisonSmem));
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(poison_kernel)");
  // one CTA fills an SM (it takes all of its shared memory); several rounds so that every SM gets one
  poison_kernel<<<4 * ctx->sm_count, 128, kPoisonSmem, s>>>(pattern);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "poison_kernel launch");
  return FALCON_OK;
}

}  // namespace falcon
