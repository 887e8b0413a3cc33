// One decoding step (the token-generation step of Algorithm 1; Sec. 3.2 with I = 1) for every (sample, kv-head)
// cache of a range, in one bandwidth-bound pass per cache (one CTA):
//   append the step's pair -> logits (K streamed once for the g heads, 128-bit loads) -> softmax ->
//   sum_weights update -> choice of the pair to evict -> P.V (V streamed once) with the one-row
//   compaction of V fused into the same pass -> one-row compaction of K.
// With growth 1 (evict after every step) exactly one pair leaves, so the top-k select is an arg-min over
// ave_weights (ties: the higher position leaves) and the stable compaction is a one-row shift of the rows
// behind the hole.  Any other target falls back to the general select + compaction of evict_body.
#include "evict.cuh"

namespace bm {
namespace {

constexpr int kDecThreads = 512;
constexpr int kDecWarps = kDecThreads / 32;
constexpr int kUnroll = 4;   // rows in flight per thread and pass
constexpr float kLog2e = 1.4426950408889634f;

struct DecodeArgs {
  const void* q;  // [nsamples][Hq][d]
  const void* k;  // [nsamples][Hkv][d]
  const void* v;
  void* out;      // [nsamples][Hq][d]
  int32_t pos;
  float scale;
  int32_t target;  // < 0: no eviction
};

struct DecSmem {
  float* q;       // [G][D]
  float* p;       // [G][n1p]   logits, then probabilities
  float* score;   // [n1p]      updated sum_weights
  int32_t* id;    // [n1p]
  float* wred;    // [2][G][warps]
  float* best;    // [warps] + int [warps]
  float* ored;    // [warps][G][D]
};

__host__ __device__ inline size_t dec_smem_layout(unsigned char* base, int d, int g, int n1, DecSmem* s) {
  const size_t n1p = (size_t)((n1 + 3) & ~3);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) & ~size_t(15); return o; };
  const size_t oq = take(4 * (size_t)g * d), op = take(4 * (size_t)g * n1p), os = take(4 * n1p), oi = take(4 * n1p);
  const size_t ow = take(4 * 2 * (size_t)g * kDecWarps), ob = take(4 * 2 * kDecWarps);
  const size_t oo = take(4 * (size_t)kDecWarps * g * d);
  if (s != nullptr) {
    s->q = reinterpret_cast<float*>(base + oq);
    s->p = reinterpret_cast<float*>(base + op);
    s->score = reinterpret_cast<float*>(base + os);
    s->id = reinterpret_cast<int32_t*>(base + oi);
    s->wred = reinterpret_cast<float*>(base + ow);
    s->best = reinterpret_cast<float*>(base + ob);
    s->ored = reinterpret_cast<float*>(base + oo);
  }
  return off;
}

__device__ inline float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecThreads) decode_kernel(CacheView c, DecodeArgs a) {
  constexpr int V = Elem<T>::kVec;
  constexpr int LPR = D / V;                 // lanes that share one row (one 16-byte piece each)
  constexpr int SLOTS = kDecThreads / LPR;   // rows covered by one load per thread
  constexpr int RPI = SLOTS * kUnroll;       // rows per iteration of the CTA
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n1 = c.n_old + 1;
  const int n1p = (n1 + 3) & ~3;
  DecSmem s;
  dec_smem_layout(smem_raw, D, G, n1, &s);

  const int unit = blockIdx.x, smp = unit / c.Hkv, kh = unit % c.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t base = (size_t)unit * c.cap;
  T* kslab = reinterpret_cast<T*>(c.k_slab) + base * D;
  T* vslab = reinterpret_cast<T*>(c.v_slab) + base * D;
  // (an unordered cache takes the general path for every cut: there the new pair fills the freed row)
  const bool evict_one = (a.target == n1 - 1) && !c.fill && c.rule < 3;   // rules 3, 4 rank by more than one value per pair
  const bool evict_general = (a.target >= 0 && a.target < n1 && !evict_one);
  // left-padded sample: padding pairs are masked and leave first; a query at a padding position (not a real
  // decode step) gets a zero output and no weights
  const int pad = sample_left_pad(c, smp);
  const bool q_real = a.pos >= pad;

  // queries of the group -> smem (fp32); the step's pair -> row n_old of the cache
  for (int t = tid; t < G * D; t += kDecThreads) {
    const T* qp = reinterpret_cast<const T*>(a.q) + ((size_t)smp * c.Hq + kh * G) * D;
    s.q[t] = (float)qp[t];
  }
  if (tid < 2 * LPR) {
    const int pc = tid % LPR;
    const T* src = reinterpret_cast<const T*>(tid < LPR ? a.k : a.v) + ((size_t)smp * c.Hkv + kh) * D + pc * V;
    T* dst = (tid < LPR ? kslab : vslab) + (size_t)c.n_old * D + pc * V;
    if (row_ok(c, c.n_old)) st_global_16(dst, ld_global_16(src));
  }
  for (int j = tid; j < n1; j += kDecThreads) s.id[j] = (j < c.n_old) ? c.kv_ids[base + j] : a.pos;
  __syncthreads();

  const int slot = tid / LPR, lr = tid % LPR;
  const float sc2 = a.scale * kLog2e;
  const int n_iter = (n1 + RPI - 1) / RPI;  // same trip count for every thread
  {
    float qr[G][V];
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int e = 0; e < V; ++e) qr[h][e] = s.q[h * D + lr * V + e];
    // ---- logits (log2 domain): scale * log2(e) * <q_h, k_j>
    for (int it = 0; it < n_iter; ++it) {
      const int j0 = it * RPI + slot;
      uint4 raw[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int j = j0 + u * SLOTS;
        if (j < n1) raw[u] = ld_global_16(kslab + (size_t)j * D + lr * V);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
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
          float acc = 0.f;
#pragma unroll
          for (int e = 0; e < V; ++e) acc = fmaf(qr[h][e], kf[e], acc);
          dot[h] = acc;
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1)
#pragma unroll
          for (int h = 0; h < G; ++h) dot[h] += __shfl_xor_sync(0xffffffffu, dot[h], off);
        if (lr == 0 && j < n1) {
          const bool masked = q_real && s.id[j] < pad;
#pragma unroll
          for (int h = 0; h < G; ++h) s.p[h * n1p + j] = masked ? -INFINITY : dot[h] * sc2;
        }
      }
    }
  }
  __syncthreads();

  // ---- softmax over the n1 rows, all threads: row max, then exp2 and row sum, per head
  float mx[G], sm[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float m = -INFINITY;
    for (int j = tid; j < n1; j += kDecThreads) m = fmaxf(m, s.p[h * n1p + j]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (lane == 0) s.wred[h * kDecWarps + warp] = m;
  }
  __syncthreads();
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) m = fmaxf(m, s.wred[h * kDecWarps + w]);
    mx[h] = m;
    float t = 0.f;
    for (int j = tid; j < n1; j += kDecThreads) {
      const float e = ex2f(s.p[h * n1p + j] - m);
      s.p[h * n1p + j] = e;
      t += e;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    if (lane == 0) s.wred[(G + h) * kDecWarps + warp] = t;
  }
  __syncthreads();
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) t += s.wred[(G + h) * kDecWarps + w];  // fixed order
    sm[h] = q_real ? 1.f / t : 0.f;
  }
  (void)mx;

  // ---- normalise, sum_weights += attn_weights (group's heads added in a fixed order), eviction candidate
  float best_ave = INFINITY;
  int best_j = -1;
  for (int j = tid; j < n1; j += kDecThreads) {
    float add = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float p = s.p[h * n1p + j] * sm[h];
      s.p[h * n1p + j] = p;
      add += p;
    }
    // rules 2 and 3 (recent queries only) keep this step's weights only
    const float sw = ((j < c.n_old && !rule_overwrites(c.rule)) ? c.sum_weights[base + j] : 0.f) + add;
    if (c.sum_sq != nullptr) {                                       // rule 4: sum of squared weights as well
      float add_sq = 0.f;
#pragma unroll
      for (int h = 0; h < G; ++h) add_sq = fmaf(s.p[h * n1p + j], s.p[h * n1p + j], add_sq);
      c.sum_sq[base + j] = (j < c.n_old ? c.sum_sq[base + j] : 0.f) + add_sq;
    }
    s.score[j] = sw;
    if (evict_one) {
      float ave;   // ranking value: average attention (Sec. 3.2), or the raw weights with / without a recent window
      if (s.id[j] < pad) ave = -1.f;
      else if (c.rule == 0) ave = sw / ((float)G * (float)(a.pos + 1 - s.id[j]));
      else ave = (c.rule == 1 && j >= n1 - a.target / 2) ? INFINITY : sw;
      if (ave <= best_ave) { best_ave = ave; best_j = j; }   // j ascends: ties move to the higher position
    } else if (row_ok(c, j)) {
      c.sum_weights[base + j] = sw;
    }
  }
  int hole = n1;  // no row leaves
  if (evict_one) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float oa = __shfl_xor_sync(0xffffffffu, best_ave, off);
      const int oj = __shfl_xor_sync(0xffffffffu, best_j, off);
      if (oa < best_ave || (oa == best_ave && oj > best_j)) { best_ave = oa; best_j = oj; }
    }
    if (lane == 0) { s.best[warp] = best_ave; reinterpret_cast<int*>(s.best)[kDecWarps + warp] = best_j; }
    __syncthreads();
    best_ave = s.best[0];
    best_j = reinterpret_cast<int*>(s.best)[kDecWarps];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) {
      const float oa = s.best[w];
      const int oj = reinterpret_cast<int*>(s.best)[kDecWarps + w];
      if (oa < best_ave || (oa == best_ave && oj > best_j)) { best_ave = oa; best_j = oj; }
    }
    hole = best_j;
    if (c.moved != nullptr && tid == 0) atomicAdd(&c.moved[unit & 15], (unsigned long long)(n1 - 1 - hole));
    // sum_weights / kv_ids in their final places: rows behind the hole move up by one
    for (int j = tid; j < n1; j += kDecThreads) {
      if (j < hole) { if (j >= 0) c.sum_weights[base + j] = s.score[j]; }
      else if (j > hole) { c.sum_weights[base + j - 1] = s.score[j]; c.kv_ids[base + j - 1] = s.id[j]; }
    }
    if (hole >= c.n_old && tid == 0) { /* the new pair itself leaves: nothing to record */ }
  } else {
    if (tid == 0) c.kv_ids[base + c.n_old] = a.pos;
    __syncthreads();
  }

  // ---- out_h = sum_j p_h[j] v_j ; rows behind the hole are written back one row up while they are in registers
  float acc[G][V];
#pragma unroll
  for (int h = 0; h < G; ++h)
#pragma unroll
    for (int e = 0; e < V; ++e) acc[h][e] = 0.f;
  for (int it = 0; it < n_iter; ++it) {
    const int j0 = it * RPI + slot;
    uint4 raw[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = j0 + u * SLOTS;
      if (j < n1) raw[u] = ld_global_16(vslab + (size_t)j * D + lr * V);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = j0 + u * SLOTS;
      if (j < n1) {
        float vf[V];
        Elem<T>::unpack(raw[u], vf);
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float p = s.p[h * n1p + j];
#pragma unroll
          for (int e = 0; e < V; ++e) acc[h][e] = fmaf(p, vf[e], acc[h][e]);
        }
      }
    }
    if (evict_one && (it + 1) * RPI > hole) {   // uniform over the CTA
      __syncthreads();                          // every load of rows < (it+1)*RPI has completed
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int j = j0 + u * SLOTS;
        if (j < n1 && j > hole && row_ok(c, j - 1)) st_global_16(vslab + (size_t)(j - 1) * D + lr * V, raw[u]);
      }
    }
  }
  // K rows behind the hole: same one-row shift (re-read, mostly from L2: the logits pass just streamed them)
  if (evict_one) {
    for (int it = hole / RPI; it < n_iter; ++it) {
      const int j0 = it * RPI + slot;
      uint4 raw[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int j = j0 + u * SLOTS;
        if (j < n1 && j > hole) raw[u] = ld_global_16(kslab + (size_t)j * D + lr * V);
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int j = j0 + u * SLOTS;
        if (j < n1 && j > hole && row_ok(c, j - 1)) st_global_16(kslab + (size_t)(j - 1) * D + lr * V, raw[u]);
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
      for (int e = 0; e < V; ++e) s.ored[(warp * G + h) * D + lr * V + e] = acc[h][e];
  }
  __syncthreads();
  for (int t = tid; t < G * D; t += kDecThreads) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) tot += s.ored[w * G * D + t];
    T* op = reinterpret_cast<T*>(a.out) + ((size_t)smp * c.Hq + kh * G) * D;
    op[t] = Elem<T>::to_out(tot);
  }

  // ---- any other target: general select + compaction over the cache (all candidates live in it now)
  if (evict_general) {
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
  static SmemConfigured configured;
  if (cudaError_t err = configured.ensure(decode_kernel<T, D, G>, smem); err != cudaSuccess) return err;
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
  const size_t attn = dec_smem_layout(nullptr, d, g, n_rows, nullptr);
  const size_t ev = (target >= 0 && target < n_rows) ? evict_smem_bytes(n_rows, target) : 0;
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
