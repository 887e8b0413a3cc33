// Stand-alone eviction kernel: one CTA per (sample, kv-head) cache.  Used after a prefill block
// (candidates = cached pairs + the block's pairs) and by bm_evict (candidates = cached pairs).
#include "evict.cuh"

namespace bm {
namespace {

constexpr int kEvictThreads = 512;

template <typename T, int D, bool FILL>
__global__ void __launch_bounds__(kEvictThreads) evict_kernel(CacheView c, EvictArgs e) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int unit = blockIdx.x;
  evict_body_impl<T, D, kEvictThreads, FILL>(c, unit, unit / c.Hkv, unit % c.Hkv, e, smem_raw);
}

template <typename T, int D, bool FILL>
cudaError_t launch_f(const CacheView& c, const EvictArgs& e, cudaStream_t st) {
  const size_t smem = evict_smem_bytes(c.n_old + e.I, e.target);
  static SmemConfigured configured;
  if (cudaError_t err = configured.ensure(evict_kernel<T, D, FILL>, smem); err != cudaSuccess) return err;
  ProfileScope prof(kEvict, st);
  evict_kernel<T, D, FILL><<<c.nsamples * c.Hkv, kEvictThreads, smem, st>>>(c, e);
  count_launch();
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_t(const CacheView& c, const EvictArgs& e, cudaStream_t st) {
  return c.fill ? launch_f<T, D, true>(c, e, st) : launch_f<T, D, false>(c, e, st);
}

}  // namespace

// Self-test of the checked build's row test: asks it about the first row index past the cache (nothing is accessed).
__global__ void row_check_selftest(CacheView c) { (void)row_ok(c, c.cap); }

cudaError_t launch_row_check_selftest(const CacheView& c, cudaStream_t st) {
  row_check_selftest<<<1, 1, 0, st>>>(c);
  count_launch();
  return cudaGetLastError();
}

size_t evict_smem_bytes(int n_cand, int target) { return evict_smem_layout(nullptr, n_cand, target, nullptr); }

cudaError_t launch_evict(int dtype, int d, const CacheView& c, const EvictArgs& e, cudaStream_t st) {
  if (dtype == 0 && d == 64) return launch_t<float, 64>(c, e, st);
  if (dtype == 0 && d == 128) return launch_t<float, 128>(c, e, st);
  if (dtype == 1 && d == 64) return launch_t<__nv_bfloat16, 64>(c, e, st);
  if (dtype == 1 && d == 128) return launch_t<__nv_bfloat16, 128>(c, e, st);
  return cudaErrorInvalidValue;
}

}  // namespace bm
