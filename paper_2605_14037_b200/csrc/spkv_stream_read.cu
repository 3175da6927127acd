// Measurement aid (no counterpart in the paper): how fast can this GPU READ from HBM with the
// copy mechanism the decode kernel uses?  The decode path only reads its K/V pages, while the
// usual bandwidth figure is a copy (half reads, half writes); this kernel streams a buffer
// through shared memory in 32 KB bulk copies, five in flight per block, one block per SM, and does
// nothing else with it (one word per page goes into a checksum so that the copies are not dead).
#include "spkv_internal.cuh"
#include "spkv_mma.cuh"

namespace spkv {

namespace {
constexpr int kReadStages = 5;
constexpr int kReadSmem = kReadStages * kPageBytes + 64;
}  // namespace

// grid = SMs, 32 threads.  Pages are handed out one at a time by an atomic counter (sink[1]) rather
// than split evenly: SMs do not draw from HBM at the same rate -- under full load, with the same
// bytes in flight, the fastest takes about a fifth more pages than the mean and the slowest a
// fifth less, the same SMs in every run -- and an even split ends when the slowest SM does
// (measured on one B200: 7.30 TB/s with an even split, 7.54 TB/s with the counter).  Every block
// claims until the counter has run past n_pages, i.e. fails exactly once; the claim that brings
// it to n_pages + gridDim.x is the launch's last and its owner leaves the counter at zero.
// status[0] != 0 on a timed-out wait.
__global__ void __launch_bounds__(32) stream_read_kernel(const unsigned char *buf, long long n_pages,
                                                         unsigned long long *sink, int *status) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kReadStages * kPageBytes);
  if (threadIdx.x == 0) {
    for (int i = 0; i < kReadStages; ++i) mbar_init(&full[i], 1);
    mbar_fence_init();
  }
  __syncwarp();
  if (threadIdx.x != 0) return;
  unsigned long long sum = 0;
  long long k = 0;
  bool failed = false;
  for (;; ++k) {
    const long long p = (long long)atomicAdd(&sink[1], 1ULL);
    if (p >= n_pages) {
      if (p == n_pages + (long long)gridDim.x - 1) sink[1] = 0;
      break;
    }
    const int s = (int)(k % kReadStages);
    if (k >= kReadStages) {  // the copy that used this stage before has landed
      if (!mbar_wait_bounded(&full[s], (uint32_t)((k / kReadStages) - 1) & 1)) { failed = true; break; }
      sum += *reinterpret_cast<const unsigned int *>(smem + s * kPageBytes);
      // the generic-proxy read above is ordered before the next bulk copy into the stage
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    mbar_arrive_expect_tx(&full[s], kPageBytes);
    bulk_load(smem + s * kPageBytes, buf + p * (long long)kPageBytes, kPageBytes, &full[s]);
  }
  // do not leave while copies may still be landing
  for (long long j = k > kReadStages ? k - kReadStages : 0; j < k; ++j) {
    const int s = (int)(j % kReadStages);
    if (!mbar_wait_bounded(&full[s], (uint32_t)(j / kReadStages) & 1)) failed = true;
    else sum += *reinterpret_cast<const unsigned int *>(smem + s * kPageBytes);
  }
  if (failed) atomicExch(status, SPKV_E_TIMEOUT);
  atomicAdd(sink, sum);
}

// Self-test of the bounded waits, the error path every copy pipeline of the library shares: one
// thread arms an mbarrier for 64 bytes more than the one 32 KB bulk copy it issues will ever
// deliver, so the wait must run out after `limit` clocks.  It then records SPKV_E_TIMEOUT,
// closes the phase by counting the missing bytes in itself and waits (bounded again, default
// limit) for the copy that IS in flight, so that nothing lands in shared memory after the block
// has gone -- what the real kernels do before they leave.  status: [0] SPKV_E_TIMEOUT if the first
// wait ran out, 0 if it did not; [1] 1 if the copy was then seen complete; [2] clocks the first
// wait lasted; [3] 1 if the first word in shared memory equals the first word of the buffer.
__global__ void __launch_bounds__(32) wait_selftest_kernel(const unsigned char *buf, long long limit, int *status) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t *bar = reinterpret_cast<uint64_t *>(smem + kPageBytes);
  if (threadIdx.x != 0) return;
  mbar_init(bar, 1);
  mbar_fence_init();
  mbar_arrive_expect_tx(bar, kPageBytes + 64);
  bulk_load(smem, buf, kPageBytes, bar);
  const long long t0 = clock64();
  const bool arrived = mbar_wait_bounded(bar, 0, limit);
  status[2] = (int)min(clock64() - t0, (long long)0x7fffffff);
  status[0] = arrived ? 0 : SPKV_E_TIMEOUT;
  if (!arrived) mbar_complete_tx(bar, 64);
  const bool drained = mbar_wait_bounded(bar, 0);
  status[1] = drained ? 1 : 0;
  status[3] = drained && *reinterpret_cast<const unsigned int *>(smem) == *reinterpret_cast<const unsigned int *>(buf);
}

}  // namespace spkv

using namespace spkv;

extern "C" int spkv_wait_selftest(const void *d_buf, long long limit_clocks, int32_t *d_status, spkv_stream_t stream) {
  if (!d_buf || !d_status || ((uintptr_t)d_buf & 15) || limit_clocks < 1) return SPKV_E_INVALID;
  if (cudaFuncSetAttribute(wait_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPageBytes + 64) !=
      cudaSuccess)
    return SPKV_E_CUDA;
  wait_selftest_kernel<<<1, 32, kPageBytes + 64, as_stream(stream)>>>(static_cast<const unsigned char *>(d_buf),
                                                                     limit_clocks, d_status);
  return check_stream_error(cudaGetLastError());
}

extern "C" int spkv_stream_read(const void *d_buf, size_t bytes, unsigned long long *d_sink, int32_t *d_status,
                                spkv_stream_t stream) {
  if (!d_buf || !d_sink || !d_status || ((uintptr_t)d_buf & 15)) return SPKV_E_INVALID;
  const long long n_pages = (long long)(bytes / kPageBytes);
  if (n_pages == 0) return SPKV_OK;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SPKV_E_CUDA;
  if (cudaFuncSetAttribute(stream_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kReadSmem) != cudaSuccess)
    return SPKV_E_CUDA;
  stream_read_kernel<<<sms, 32, kReadSmem, as_stream(stream)>>>(static_cast<const unsigned char *>(d_buf), n_pages,
                                                               d_sink, d_status);
  return check_stream_error(cudaGetLastError());
}
