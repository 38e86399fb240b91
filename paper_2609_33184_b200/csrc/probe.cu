// Read-bandwidth probe: the practical ceiling for a kernel that streams device memory once.
//
// A measurement aid, not a step of the method: bench.py runs it over the same history buffers
// as the verification round, in the same process and clock state, so that the round's KV GB/s
// can be read against what a plain streaming read reaches on this GPU right now.
#include "ss_internal.h"
#include "tc_ptx.cuh"

namespace {

constexpr int kThreads = 512;
constexpr int kUnroll = 8;               // independent 16-byte loads in flight per thread
constexpr int kSlabVec = kThreads * 16;  // 16-byte vectors per CTA: a contiguous 128 KiB slab
constexpr int kMaxSegments = 64;

struct Segments {
  const uint4* ptr[kMaxSegments];
  unsigned long long n_vec[kMaxSegments];
  unsigned int first_slab[kMaxSegments + 1];  // running count of 128 KiB slabs
  int n;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Four CTAs per SM walk the slabs of all segments round-robin; one atomic per CTA at the end.
__global__ void __launch_bounds__(kThreads) probe_read_kernel(const Segments seg,
                                                              unsigned long long* sink) {
  __shared__ uint32_t warp_acc[kThreads / 32];
  const unsigned total = seg.first_slab[seg.n];
  uint32_t acc = 0;
  int y = 0;
  for (unsigned slab = blockIdx.x; slab < total; slab += gridDim.x) {
    while (slab >= seg.first_slab[y + 1]) ++y;
    const uint4* src = seg.ptr[y];
    const size_t n_vec = seg.n_vec[y];
    const size_t lo = (size_t)(slab - seg.first_slab[y]) * kSlabVec;
    const size_t hi = lo + kSlabVec < n_vec ? lo + kSlabVec : n_vec;
    size_t i = lo + threadIdx.x;
    for (; i + (kUnroll - 1) * kThreads < hi; i += kUnroll * kThreads) {
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream(src + i + u * kThreads);
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < hi; i += kThreads) {
      const uint4 v = ld_stream(src + i);
      acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) warp_acc[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t a = 0;
    for (int w = 0; w < kThreads / 32; ++w) a ^= warp_acc[w];
    if (a) atomicXor(sink, (unsigned long long)a);
  }
}

}  // namespace

extern "C" ss_status ss_probe_read(const void* const* srcs, const size_t* bytes, int32_t n,
                                   uint64_t* sink, void* stream) {
  if (!srcs || !bytes || !sink || n < 0) return SS_ERR_ARG;
  if (n > kMaxSegments) return SS_ERR_CAPACITY;
  if ((uintptr_t)sink & 7) return SS_ERR_ALIGN;
  Segments seg;
  seg.n = n;
  seg.first_slab[0] = 0;
  for (int i = 0; i < n; ++i) {
    if (!srcs[i]) return SS_ERR_ARG;
    if (((uintptr_t)srcs[i] & 15) || (bytes[i] & 15)) return SS_ERR_ALIGN;
    seg.ptr[i] = static_cast<const uint4*>(srcs[i]);
    seg.n_vec[i] = bytes[i] / 16;
    const size_t slabs = (bytes[i] / 16 + kSlabVec - 1) / kSlabVec;
    if (slabs + seg.first_slab[i] > 0x7fffffffu) return SS_ERR_CAPACITY;
    seg.first_slab[i + 1] = seg.first_slab[i] + (unsigned)slabs;
  }
  const unsigned total = seg.first_slab[n];
  if (total == 0) return SS_OK;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SS_ERR_CUDA;
  const unsigned full = (unsigned)sms * 4;  // four CTAs of 512 threads per SM: every warp slot taken
  probe_read_kernel<<<total < full ? total : full, kThreads, 0, (cudaStream_t)stream>>>(
      seg, reinterpret_cast<unsigned long long*>(sink));
  return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}

namespace ss {
uint32_t* ctx_status_word(ss_ctx* c);  // api.cu
}
namespace {
// A wait nothing will ever satisfy: every thread waits on an mbarrier whose phase never
// completes, with the kernels' own bounded wait and a short limit.
__global__ void __launch_bounds__(64) wait_expiry_kernel(uint32_t* status, unsigned long long limit_ns,
                                                         uint32_t* gave_up) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t abort_word;
  if (threadIdx.x == 0) {
    ss::tc::mbar_init(&bar, 1);
    abort_word = 0;
    ss::tc::fence_barrier_init();
  }
  __syncthreads();
  const bool ok = ss::tc::mbar_wait_abortable(&bar, 0, &abort_word, status, limit_ns);
  if (!ok) atomicAdd(gave_up, 1u);
}
}  // namespace

extern "C" ss_status ss_selftest_wait_expiry(ss_ctx* ctx, int32_t limit_ms, uint32_t* gave_up, void* stream) {
  if (!ctx || !gave_up || limit_ms <= 0 || limit_ms > 1000) return SS_ERR_ARG;
  wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(ss::ctx_status_word(ctx),
                                                         (unsigned long long)limit_ms * 1000000ull, gave_up);
  return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
