// Measurement kernel: the rate at which one SM's tensor cores retire tcgen05.mma kind::i8 when nothing else
// is in the way -- operands resident in shared memory (no loads in the loop), two TMEM accumulators, one
// elected thread issuing back to back.  It is the ceiling the integer GEMM of the layer is measured against
// (the paper has no counterpart: it is a property of the machine, taken on the machine that runs the benchmark).
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace stamp {

constexpr int PEAK_THREADS = 64;
constexpr int PEAK_SMEM = (128 + 256) * 128 + 1024;   // a 128 x 128 and a 256 x 128 int8 tile, 1024-byte aligned
constexpr int PEAK_BATCH = 64;                         // MMAs between two commits

// Every CTA issues `nbatch` batches of PEAK_BATCH instructions of shape M128 x N256 x K32 (int8 x int8 -> int32)
// on tiles of zeros and waits (bounded) for each batch's commit before it issues the batch after the next, so at
// most two batches are queued.  Work per CTA: nbatch * PEAK_BATCH * 2 * 128 * 256 * 32 integer operations.
__global__ void __launch_bounds__(PEAK_THREADS, 1) k_peak_mma_i8(int nbatch) {
  extern __shared__ uint8_t peak_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(peak_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ uint32_t abort_word;
  for (int i = threadIdx.x; i < (128 + 256) * 128 / 16; i += blockDim.x) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar[0], 1);
    ptx::mbar_init(&bar[1], 1);
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  ptx::fence_proxy_async_smem();   // the zeros were written by ordinary stores; the MMA reads through the async proxy
  if (threadIdx.x < 32) {
    ptx::tmem_alloc(&tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  if (threadIdx.x < 32 && ptx::elect_one()) {
    constexpr uint32_t idesc = ptx::make_i8_idesc(128, 256);
    const uint32_t wa = ptx::smem_u32(smem);
    const uint32_t xa = wa + 128 * 128;
    bool ok = true;
    for (int b = 0; b < nbatch && ok; ++b) {
      const int s = b & 1;
      if (b >= 2 && !ptx::mbar_wait_bounded(&bar[s], static_cast<uint32_t>(((b >> 1) - 1) & 1), &abort_word, 2000000000LL)) {
        ok = false;
        break;
      }
#pragma unroll 4
      for (int i = 0; i < PEAK_BATCH; ++i) {
        const int k = i & 3;
        const uint64_t adesc = ptx::make_kmajor_sw128_desc(wa + k * 32);
        const uint64_t bdesc = ptx::make_kmajor_sw128_desc(xa + k * 32);
        ptx::mma_i8_ss(tmem_base + static_cast<uint32_t>(((i >> 2) & 1) * 256), adesc, bdesc, idesc, 1u);
      }
      ptx::tc_commit(&bar[s]);
    }
    // drain: the last (up to) two batches
    for (int b = max(nbatch - 2, 0); b < nbatch && ok; ++b)
      if (!ptx::mbar_wait_bounded(&bar[b & 1], static_cast<uint32_t>((b >> 1) & 1), &abort_word, 2000000000LL)) ok = false;
    if (!ok) raise_device_status(STAMP_ERR_TIMEOUT);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Test kernel for the failure path every kernel of the library shares: one thread waits, with the bounded wait
// the product kernels use, on an mbarrier that nobody will ever complete.  After `limit_cycles` SM clocks the
// wait gives up, the thread records STAMP_ERR_TIMEOUT in the device status word and the kernel returns normally:
// nothing faults, traps or hangs, and the context stays usable.
__global__ void __launch_bounds__(32, 1) k_expire_wait(long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0 && !ptx::mbar_wait_bounded(&bar, 0u, &abort_word, limit_cycles)) {
    abort_word = 1;
    raise_device_status(STAMP_ERR_TIMEOUT);
  }
}

}  // namespace stamp
