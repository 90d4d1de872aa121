// Measurement aid: the ceiling of the contraction of Eq. 3 on this GPU.  One CTA per SM issues tcgen05.mma kind::i8
// (s8 x u8 -> s32, 128 x 256 x 32 per instruction) back to back from operands that stay in shared memory: no loads,
// no epilogue.  What it reaches is the number the fused convolution's tensor throughput is divided by, next to the
// nominal figure.  The operands are pseudo-random bytes (an integer hash): data-dependent power, hence clocks, are
// those of a real layer.  Every wait is bounded and reports through the handle's status word.
#include "hq_internal.cuh"

namespace {

constexpr int kRowsA = 128, kRowsB = 256, kRowBytes = 128;      // K-major tiles with 128-byte rows (one swizzle span)
constexpr unsigned long long kPeakWaitBudgetNs = 2000000000ull;

__device__ __forceinline__ uint32_t pk_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long pk_ns() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ bool pk_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t pk_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(((kRowBytes * 8) >> 4) & 0x3FFF) << 32;     // 8-row groups are 1024 bytes apart
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;                                     // 128-byte swizzle
  return d;
}

// `rounds` times: `blocks_per_round` K blocks of 128 bytes (4 instructions each) into two alternating accumulators,
// then one commit and a bounded wait for it (the queue of issued instructions stays finite).
__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int rounds, int blocks_per_round, uint32_t seed, uint32_t* status) {
  extern __shared__ uint8_t pk_raw[];
  __shared__ unsigned long long bar;
  __shared__ uint32_t tmem_base_s;
  const uint32_t base = (pk_smem(pk_raw) + 1023u) & ~1023u;
  uint8_t* tiles = pk_raw + (base - pk_smem(pk_raw));
  // operands: bytes of an integer hash of their address (any byte pattern is a valid s8 / u8 operand)
  uint32_t* words = (uint32_t*)tiles;
  for (int i = threadIdx.x; i < (kRowsA + kRowsB) * kRowBytes / 4; i += blockDim.x) {
    uint32_t x = (uint32_t)i * 2654435761u + seed + blockIdx.x * 40503u;
    x ^= x >> 15; x *= 2246822519u; x ^= x >> 13; x *= 3266489917u; x ^= x >> 16;
    words[i] = x;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(pk_smem(&bar)), "r"(1));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pk_smem(&tmem_base_s)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_base_s;
  if (threadIdx.x == 0) {
    // D = S32, A = s8, B = u8, both K-major, N = 256, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | ((uint32_t)(kRowsB >> 3) << 17) | ((uint32_t)(kRowsA >> 4) << 24);
    const uint64_t adesc0 = pk_desc(base), bdesc0 = pk_desc(base + kRowsA * kRowBytes);
    bool ok = true;
    for (int r = 0; r < rounds && ok; ++r) {
      for (int b = 0; b < blocks_per_round; ++b) {
        const uint32_t d = tmem + (uint32_t)(b & 1) * kRowsB;
        uint64_t adesc = adesc0, bdesc = bdesc0;
#pragma unroll
        for (int k = 0; k < 4; ++k, adesc += 2, bdesc += 2) {
          const uint32_t acc = (r | b | k) ? 1u : 0u;
          asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                       ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
        }
      }
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(pk_smem(&bar)) : "memory");
      const unsigned long long t0 = pk_ns();
      while (!pk_try_wait(pk_smem(&bar), (uint32_t)(r & 1))) {
        if (pk_ns() - t0 > kPeakWaitBudgetNs) { atomicCAS(status, 0u, (uint32_t)HQ_DEV_TIMEOUT_MMA); ok = false; break; }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

}  // namespace

extern "C" hq_status hq_mma_peak_launch(hq_handle* h, int32_t rounds, int32_t blocks_per_round, int64_t* ops, void* stream) {
  if (!h || rounds < 1 || blocks_per_round < 1 || rounds > (1 << 20) || blocks_per_round > (1 << 16)) return HQ_ERR_INVALID_ARG;
  // 120 KiB although 49 KiB are used: one CTA per SM, so that no second CTA waits for tensor-memory columns
  const size_t smem = 120 * 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(mma_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return HQ_ERR_CUDA;
    attr_set = true;
  }
  mma_peak_kernel<<<h->sm_count, 128, smem, (cudaStream_t)stream>>>(rounds, blocks_per_round, 12345u, h->dev_status);
  if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  if (ops) *ops = (int64_t)2 * kRowsA * kRowsB * kRowBytes * (int64_t)blocks_per_round * rounds * h->sm_count;
  return HQ_OK;
}
