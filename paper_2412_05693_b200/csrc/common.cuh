// Shared declarations of the CUDA path: cache view, launcher prototypes, small device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bm {

// Device-side view of one layer's slabs for a contiguous range of samples (Sec. 3: one cache per
// attention head and sample).  Unit u = local_sample * Hkv + kv_head; its rows start at u * cap.
struct CacheView {
  void* k_slab;        // [units][cap][d] elements of the cache dtype
  void* v_slab;        // [units][cap][d]
  float* sum_weights;  // [units][cap]
  int32_t* kv_ids;     // [units][cap]
  int32_t cap;
  int32_t n_old;       // pairs cached before this call (equal for every unit of the range)
  int32_t Hq, Hkv, g;
  int32_t nsamples;
  int32_t* status;     // device status word
  const int32_t* left_pad;  // [nsamples] padding positions at the start of each sample of the range, or null
  unsigned long long* moved;  // [16] counters of rows moved by compactions (unit & 15), or null when not counting
  int32_t rule;             // 0 average attention (Sec. 3.2); Sec. 2: 1 sum + window of recent pairs, 2 current query,
                            // 3 last-window sums, pooled, recent window kept, 4 average + standard deviation
  int32_t fill;             // 1: unordered cache -- pairs that stay never move, new pairs fill the freed rows
  float* sum_sq;            // [units][cap] sums of squared attention weights (rule 4), else null
  int32_t window, pool;     // rule 3: queries observed / recent pairs kept; width of the max-pooling (odd)
  int32_t std_permille;     // rule 4: share of the kept pairs chosen by standard deviation, in 1/1000
};

// Rules that rank by recent queries only (Sec. 2): sum_weights is overwritten by every pass, and only the rows of the
// pass's last inputs count -- its last input (rule 2) or its last min(window, I) inputs (rule 3).
__host__ __device__ inline bool rule_overwrites(int rule) { return rule == 2 || rule == 3; }
__host__ __device__ inline int rule_first_counted_row(int rule, int window, int I, int g) {
  const int inputs = rule == 2 ? 1 : (rule == 3 ? (window < I ? window : I) : I);
  return (I - inputs) * g;
}

// Left padding (Sec. 3): positions below the sample's count are padding.  A padding pair is masked for every
// real query; a padding query produces a zero output row and no attention weights.
__device__ inline int sample_left_pad(const CacheView& c, int smp) {
  return c.left_pad != nullptr ? c.left_pad[smp] : 0;
}

// Checked build (-DBM_DEBUG, libbatchmax_debug.so): every cache row index a kernel is about to write with plain
// stores is tested against the cache's capacity first; a bad index records BM_ERR_BOUNDS in the status word and the
// access is skipped (nothing traps).  In the ordinary build the test is the constant `true`.
constexpr int kErrBounds = 7;   // BM_ERR_BOUNDS
#ifdef BM_DEBUG
__device__ inline bool row_ok(const CacheView& c, long long r) {
  if (r >= 0 && r < c.cap) return true;
  atomicExch(c.status, kErrBounds);
  return false;
}
#else
__device__ __forceinline__ constexpr bool row_ok(const CacheView&, long long) { return true; }
#endif

// One forward pass over a block (I inputs) for the range.
struct BlockArgs {
  const void* q;    // [nsamples][I][Hq][d]
  const void* k;    // [nsamples][I][Hkv][d]
  const void* v;    // [nsamples][I][Hkv][d]
  void* out;        // [nsamples][I][Hq][d]
  float* lse;       // workspace: [units][I*g]  natural-log-sum-exp of every query row
  float* new_sum;   // workspace: [units][I]    column sums of the block's own pairs
  float* new_sq;    // workspace: [units][I]    column sums of squares of the block's own pairs (rule 4), else null
  int32_t I;
  int32_t pos0;
  float scale;
};

struct EvictArgs {
  const void* blk_k;     // block K/V when the new pairs still live in the caller's buffers, else null
  const void* blk_v;
  const float* new_sum;  // [units][I] when I > 0
  const float* new_sq = nullptr;  // [units][I] when I > 0 under rule 4
  int32_t I;             // candidates = n_old + I
  int32_t pos0;
  int32_t curr_id;       // last processed position
  int32_t target;        // pairs to keep (<= n_old + I)
  int32_t recent = 0;    // 1: keep the `target` most recent candidates instead of ranking by ave_weights
};

// Launchers (host).  All enqueue on `st` and return the CUDA error of the launch.
cudaError_t launch_attn_simt(int dtype, int d, const CacheView& c, const BlockArgs& a, cudaStream_t st);
cudaError_t launch_score_simt(int dtype, int d, const CacheView& c, const BlockArgs& a, cudaStream_t st);
cudaError_t launch_evict(int dtype, int d, const CacheView& c, const EvictArgs& e, cudaStream_t st);
cudaError_t launch_decode(int dtype, int d, const CacheView& c, const void* q, const void* k, const void* v,
                          void* out, int32_t pos, float scale, int32_t target /* <0: none */, cudaStream_t st);
cudaError_t launch_decode_mma(int d, const CacheView& c, const void* q, const void* k, const void* v, void* out,
                              int32_t pos, float scale, int32_t target /* <0: none */, cudaStream_t st);
size_t decode_mma_smem_bytes(int d, int g, int n_rows, int target);
size_t evict_smem_bytes(int n_cand, int target);
size_t decode_smem_bytes(int d, int g, int n_rows, int target);
bool tc_path_available();
cudaError_t launch_wait_timeout_selftest(int* status, cudaStream_t st);
cudaError_t launch_row_check_selftest(const CacheView& c, cudaStream_t st);
cudaError_t launch_attn_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used);
cudaError_t launch_score_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used);

// cudaFuncSetAttribute applies to the current device only, so the largest dynamic shared-memory size a kernel has
// been configured for is remembered per device (a process may hold handles on several GPUs).
struct SmemConfigured {
  size_t bytes[64] = {};
  template <typename Kernel>
  cudaError_t ensure(Kernel kernel, size_t smem) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (smem > bytes[dev]) {
      e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      bytes[dev] = smem;
    }
    return cudaSuccess;
  }
};

// Launch as a programmatic dependent of the stream's previous kernel: the grid may be started while that kernel is
// still running; the kernel itself must execute pdl_wait() before it touches anything the predecessor may have
// written, and pdl_release() lets its own successor start.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

extern unsigned long long g_launch_count;
inline void count_launch(int n = 1) { g_launch_count += (unsigned long long)n; }

// Optional per-launch timing: when enabled, a ProfileScope brackets a launch with two CUDA events.
enum KernelClass { kAttnFwd = 0, kScore = 1, kEvict = 2, kDecode = 3, kNumKernelClasses = 4 };
void profile_begin(int cls, cudaStream_t st);
void profile_end(int cls, cudaStream_t st);
struct ProfileScope {
  int cls; cudaStream_t st;
  ProfileScope(int c, cudaStream_t s) : cls(c), st(s) { profile_begin(cls, st); }
  ~ProfileScope() { profile_end(cls, st); }
};

// ---- element helpers -------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kVec = 4;  // elements per 16-byte load
  __device__ static inline void unpack(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
    f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
  }
  __device__ static inline float to_out(float x) { return x; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static inline void unpack(const uint4& r, float* f) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // bf16 -> fp32 is a 16-bit shift
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static inline __nv_bfloat16 to_out(float x) { return __float2bfloat16_rn(x); }
};

__device__ inline uint4 ld_global_16(const void* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ inline void st_global_16(void* p, const uint4& v) { *reinterpret_cast<uint4*>(p) = v; }

}  // namespace bm
