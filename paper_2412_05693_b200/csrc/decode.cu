// One decoding step (Algorithm 1 "generate token", Sec. 3.2 with I = 1) for every (sample, kv-head)
// cache of a range, in one bandwidth-bound pass: append the step's pair, g one-query attentions over
// the n+1 cached rows (K and V streamed once per group with 128-bit loads), sum_weights update, and an
// optional eviction back to `target` rows.  One CTA per cache.
#include "evict.cuh"

namespace bm {
namespace {

constexpr int kDecThreads = 512;
constexpr int kDecWarps = kDecThreads / 32;

struct DecodeArgs {
  const void* q;  // [nsamples][Hq][d]
  const void* k;  // [nsamples][Hkv][d]
  const void* v;
  void* out;      // [nsamples][Hq][d]
  int32_t pos;
  float scale;
  int32_t target;  // < 0: no eviction
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecThreads) decode_kernel(CacheView c, DecodeArgs a) {
  constexpr int V = Elem<T>::kVec;
  constexpr int LPR = D / V;                 // lanes that share one row (one 16-byte piece each)
  constexpr int SLOTS = kDecThreads / LPR;   // rows in flight per pass over the CTA
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n1 = c.n_old + 1;
  const int n1p = (n1 + 3) & ~3;
  float* sQ = reinterpret_cast<float*>(smem_raw);     // [G][D]
  float* sP = sQ + G * D;                             // [G][n1p]
  float* sRed = sP + G * n1p;                         // [warps][G][D]

  const int unit = blockIdx.x, smp = unit / c.Hkv, kh = unit % c.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t base = (size_t)unit * c.cap;
  T* kslab = reinterpret_cast<T*>(c.k_slab) + base * D;
  T* vslab = reinterpret_cast<T*>(c.v_slab) + base * D;

  // queries of the group -> smem (fp32); the step's pair -> row n_old of the cache
  for (int t = tid; t < G * D; t += kDecThreads) {
    const T* qp = reinterpret_cast<const T*>(a.q) + ((size_t)smp * c.Hq + kh * G) * D;
    sQ[t] = (float)qp[t];
  }
  if (tid < 2 * LPR) {
    const int pc = tid % LPR;
    const T* src = reinterpret_cast<const T*>(tid < LPR ? a.k : a.v) + ((size_t)smp * c.Hkv + kh) * D + pc * V;
    T* dst = (tid < LPR ? kslab : vslab) + (size_t)c.n_old * D + pc * V;
    st_global_16(dst, ld_global_16(src));
  }
  if (tid == 0) c.kv_ids[base + c.n_old] = a.pos;
  __syncthreads();

  const int slot = tid / LPR, lr = tid % LPR;
  float qr[G][V];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int e = 0; e < V; ++e) qr[h][e] = sQ[h * D + lr * V + e];

  // ---- logits: scale * <q_h, k_j>
  constexpr int UNR = 4;
  const int n_iter = (n1 + SLOTS * UNR - 1) / (SLOTS * UNR);  // same trip count for every thread
  for (int it = 0; it < n_iter; ++it) {
    const int j0 = it * SLOTS * UNR + slot;
    uint4 raw[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int j = j0 + u * SLOTS;
      if (j < n1) raw[u] = ld_global_16(kslab + (size_t)j * D + lr * V);
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int j = j0 + u * SLOTS;
      float kf[V];
      if (j < n1) Elem<T>::unpack(raw[u], kf);
      else {
#pragma unroll
        for (int e = 0; e < V; ++e) kf[e] = 0.f;
      }
      float dot[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < V; ++e) s = fmaf(qr[h][e], kf[e], s);
        dot[h] = s;
      }
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1)
#pragma unroll
        for (int h = 0; h < G; ++h) dot[h] += __shfl_xor_sync(0xffffffffu, dot[h], off);
      if (lr == 0 && j < n1) {
#pragma unroll
        for (int h = 0; h < G; ++h) sP[h * n1p + j] = dot[h] * a.scale;
      }
    }
  }
  __syncthreads();

  // ---- softmax per head: warp h normalises head h
  if (warp < G) {
    float* p = sP + warp * n1p;
    float m = -INFINITY;
    for (int j = lane; j < n1; j += 32) m = fmaxf(m, p[j]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float sum = 0.f;
    for (int j = lane; j < n1; j += 32) { const float e = expf(p[j] - m); p[j] = e; sum += e; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const float inv = 1.f / sum;
    for (int j = lane; j < n1; j += 32) p[j] *= inv;
  }
  __syncthreads();

  // ---- sum_weights += attn_weights (added over the group's heads in a fixed order)
  for (int j = tid; j < n1; j += kDecThreads) {
    float add = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h) add += sP[h * n1p + j];
    const float old = (j < c.n_old) ? c.sum_weights[base + j] : 0.f;
    c.sum_weights[base + j] = old + add;
  }

  // ---- out_h = sum_j p_h[j] v_j
  float acc[G][V];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int e = 0; e < V; ++e) acc[h][e] = 0.f;
  for (int it = 0; it < n_iter; ++it) {
    const int j0 = it * SLOTS * UNR + slot;
    uint4 raw[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int j = j0 + u * SLOTS;
      if (j < n1) raw[u] = ld_global_16(vslab + (size_t)j * D + lr * V);
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int j = j0 + u * SLOTS;
      if (j < n1) {
        float vf[V];
        Elem<T>::unpack(raw[u], vf);
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float p = sP[h * n1p + j];
#pragma unroll
          for (int e = 0; e < V; ++e) acc[h][e] = fmaf(p, vf[e], acc[h][e]);
        }
      }
    }
  }
  // rows of one warp first (lanes lr, lr+LPR, ...), then across warps through smem, fixed order
#pragma unroll
  for (int off = 16; off >= LPR; off >>= 1)
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int e = 0; e < V; ++e) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], off);
  if (lane < LPR) {
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int e = 0; e < V; ++e) sRed[(warp * G + h) * D + lr * V + e] = acc[h][e];
  }
  __syncthreads();
  for (int t = tid; t < G * D; t += kDecThreads) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) tot += sRed[w * G * D + t];
    T* op = reinterpret_cast<T*>(a.out) + ((size_t)smp * c.Hq + kh * G) * D;
    op[t] = Elem<T>::to_out(tot);
  }

  // ---- optional eviction back to `target` rows (all candidates live in the cache now)
  if (a.target >= 0 && n1 > a.target) {
    __syncthreads();  // sum_weights / appended row visible to the whole CTA; smem reusable
    CacheView cv = c;
    cv.n_old = n1;
    EvictArgs e;
    e.blk_k = nullptr; e.blk_v = nullptr; e.new_sum = nullptr;
    e.I = 0; e.pos0 = 0; e.curr_id = a.pos; e.target = a.target;
    evict_body<T, D, kDecThreads>(cv, unit, smp, kh, e, smem_raw);
  }
}

template <typename T, int D, int G>
cudaError_t launch_t(const CacheView& c, const DecodeArgs& a, cudaStream_t st) {
  const size_t smem = decode_smem_bytes(D, G, c.n_old + 1, a.target);
  static size_t configured = 0;
  if (smem > configured) {
    cudaError_t err = cudaFuncSetAttribute(decode_kernel<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    configured = smem;
  }
  ProfileScope prof(kDecode, st);
  decode_kernel<T, D, G><<<c.nsamples * c.Hkv, kDecThreads, smem, st>>>(c, a);
  count_launch();
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_g(const CacheView& c, const DecodeArgs& a, cudaStream_t st) {
  switch (c.g) {
    case 1: return launch_t<T, D, 1>(c, a, st);
    case 2: return launch_t<T, D, 2>(c, a, st);
    case 4: return launch_t<T, D, 4>(c, a, st);
    case 8: return launch_t<T, D, 8>(c, a, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

size_t decode_smem_bytes(int d, int g, int n_rows, int target) {
  const size_t n1p = (size_t)((n_rows + 3) & ~3);
  const size_t attn = sizeof(float) * ((size_t)g * d + (size_t)g * n1p + (size_t)kDecWarps * g * d);
  const size_t ev = (target >= 0 && n_rows > target) ? evict_smem_bytes(n_rows, target) : 0;
  return attn > ev ? attn : ev;
}

cudaError_t launch_decode(int dtype, int d, const CacheView& c, const void* q, const void* k, const void* v,
                          void* out, int32_t pos, float scale, int32_t target, cudaStream_t st) {
  DecodeArgs a{q, k, v, out, pos, scale, target};
  if (dtype == 0 && d == 64) return launch_g<float, 64>(c, a, st);
  if (dtype == 0 && d == 128) return launch_g<float, 128>(c, a, st);
  if (dtype == 1 && d == 64) return launch_g<__nv_bfloat16, 64>(c, a, st);
  if (dtype == 1 && d == 128) return launch_g<__nv_bfloat16, 128>(c, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace bm
