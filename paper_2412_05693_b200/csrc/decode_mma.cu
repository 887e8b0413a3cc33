// bf16 decoding step (the token-generation step of Algorithm 1; Sec. 3.2 with I = 1), one CTA per (sample, kv-head) cache.
// Same steps as the fp32 kernel in decode.cu, but the two contractions run on warp-level tensor-core MMAs
// (m16n8k16, bf16 in, fp32 accumulate) fed straight from 128-bit global loads, so that the kernel issues few
// enough instructions to be limited by HBM bandwidth:
//   logits^T [16 keys x heads] = K-tile [16 keys x d] . q^T          (heads padded to 8 columns)
//   out^T    [16 d    x heads] = V-tile^T [16 d x 16 keys] . p^T
// Both contractions are invariant under a permutation of the contracted index, and the output index of the
// second one can be un-permuted when it is written, so every thread loads whole 16-byte pieces of cache
// rows (coalesced) and the MMA fragment slots are assigned to whatever elements those loads delivered.
// The instance for grids of at most one cache per SM (KD > 1 below) differs in how rows travel: K is loaded once and
// kept in registers, V is staged in shared memory by TMA while the softmax phases run and read back with
// transposing ldmatrix (standard fragment layout), and the rows behind the pair that leaves are written from there.
#include "evict.cuh"
#include "tc_common.cuh"

namespace bm {
namespace {

// CTA size NT (template parameter): 256 threads, two CTAs per SM, when the grid is at most about two CTAs per SM --
// a step's time is then one CTA's latency, and eight warps finish a cache sooner; 128 threads, four CTAs per SM,
// for larger grids -- four independent caches per SM keep the memory pipe busy while others sit in their
// softmax / arg-min / reduction phases (0.85 against 0.71 of the HBM copy peak at 16384 caches of 512 pairs) -- as
// long as four of them fit into shared memory, which grows with the cache length; beyond that the larger CTA is
// faster again (0.84 against 0.65 at 2048 caches of 2048 pairs).  One CTA of 512 threads per SM measured worst at
// every size.
constexpr int kMaxWarps = 8;
constexpr float kLog2e = 1.4426950408889634f;

struct DecodeArgs {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int32_t pos;
  float scale;
  int32_t target;
};

struct Smem {
  float* p;       // [G][n1t]  logits, then probabilities (zero beyond n1)
  float* score;   // [n1t]
  int32_t* id;    // [n1t]
  float* wred;    // [2][G][warps]
  float* best;    // [3][warps]
  float* ored;    // [warps][G][D]
};

__host__ __device__ inline size_t smem_layout(unsigned char* base, int d, int g, int n1, int kWarps, Smem* s) {
  const size_t n1t = (size_t)((n1 + 15) & ~15);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) & ~size_t(15); return o; };
  const size_t op = take(4 * (size_t)g * n1t), os = take(4 * n1t), oi = take(4 * n1t);
  const size_t ow = take(4 * 2 * (size_t)g * kWarps), ob = take(4 * 3 * kWarps), oo = take(4 * (size_t)kWarps * g * d);
  if (s != nullptr) {
    s->p = reinterpret_cast<float*>(base + op);
    s->score = reinterpret_cast<float*>(base + os);
    s->id = reinterpret_cast<int32_t*>(base + oi);
    s->wred = reinterpret_cast<float*>(base + ow);
    s->best = reinterpret_cast<float*>(base + ob);
    s->ored = reinterpret_cast<float*>(base + oo);
  }
  return off;
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg16_or_zero(const __nv_bfloat16* p, bool ok) {
  return ok ? ld_global_16(p) : make_uint4(0u, 0u, 0u, 0u);
}
// 32 bytes (16 elements) with one 256-bit load: the four lanes that share a key row then cover a whole 128-byte
// line per request instead of half of one
__device__ __forceinline__ void ldg32_or_zero(const __nv_bfloat16* p, bool ok, uint4& lo, uint4& hi) {
  lo = make_uint4(0u, 0u, 0u, 0u);
  hi = lo;
  if (ok)
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
                 : "l"(p) : "memory");
}

__device__ __forceinline__ void stg32(__nv_bfloat16* p, const uint4& lo, const uint4& hi) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
}

// PLAIN: no left padding and the paper's own eviction rule -- the instance the common case runs, free of those
// branches.
// KD: 1 = every warp keeps one tile of rows in flight beyond the one it multiplies (fits the register budget of two
// or four CTAs per SM).  KD > 1 = one CTA per SM with the whole register file, for caches of at most KD tiles per
// warp in grids of at most one CTA per SM: all of K is loaded at once and stays in registers until the pair that
// leaves is known, so that the rows behind it are written one row up straight from registers.  Such a grid's step
// lasts as long as its slowest CTA, which is the one that has to move most of its cache; re-reading K for the move
// (as the KD = 1 instances do) made that CTA 4.7 us slower than the fastest one at 128 caches of 512 pairs.
template <int D, int G, int NT, bool PLAIN, int KD>
__global__ void __launch_bounds__(NT, KD > 1 ? 1 : 512 / NT) decode_mma_kernel(CacheView c, DecodeArgs a, const __grid_constant__ CUtensorMap vmap) {
  using T = __nv_bfloat16;
  constexpr int kThreads = NT, kWarps = NT / 32;
  constexpr int kRowsPerIter = kWarps * 16;   // one 16-key tile per warp and iteration
  constexpr int QR = D / 32;   // 32-element rounds of the logits contraction
  constexpr int VR = D / 64;   // 64-element rounds of the output contraction
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n1 = c.n_old + 1;
  const int n1t = (n1 + 15) & ~15;
  Smem s;
  smem_layout(smem_raw, D, G, n1, kWarps, &s);

  const int unit = blockIdx.x, smp = unit / c.Hkv, kh = unit % c.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, tq = lane & 3;   // MMA fragment coordinates: group id, thread in group
  const size_t base = (size_t)unit * c.cap;
  T* kslab = reinterpret_cast<T*>(c.k_slab) + base * D;
  T* vslab = reinterpret_cast<T*>(c.v_slab) + base * D;
  // (an unordered cache under the rule with a window of recent pairs takes the general path for every cut: the
  // window is a select on kv_ids there)
  // (so do the rules whose ranking is more than one value per pair: pooled window sums, deviation-protected averages)
  const bool evict_one = (a.target == n1 - 1) && (PLAIN || !((c.fill && c.rule == 1) || c.rule >= 3));
  const bool evict_general = (a.target >= 0 && a.target < n1 && !evict_one);

  // Programmatic dependent launch: this grid may have been started while its predecessor in the stream was still
  // running (so that the launch latency of back-to-back decode steps is hidden); nothing that the predecessor may
  // have written -- the cache, and the inputs too -- is touched before this point.  The grid that follows may be
  // started right away: it waits at the same point for this one to complete.
  pdl_wait();
  pdl_release();
  if constexpr (KD > 1) {   // barriers of the V tiles (initialised by the thread that issues the copies)
    if (tid == 0) {
      const uint32_t st0 = (tc::smem_u32(smem_raw) + (uint32_t)smem_layout(nullptr, D, G, n1, kWarps, nullptr) + 1023u) & ~1023u;
      unsigned char* st = smem_raw + (st0 - tc::smem_u32(smem_raw));
      for (int u = 0; u < KD; ++u) tc::mbar_init(reinterpret_cast<uint64_t*>(st) + u, 1);
      *reinterpret_cast<volatile int*>(st + 64) = 0;
      tc::mbar_fence_init();
    }
  }

  // the step's pair -> row n_old of the cache; ids -> smem
  if (tid < 2 * (D / 8)) {
    const int pc = tid % (D / 8);
    const T* src = reinterpret_cast<const T*>(tid < D / 8 ? a.k : a.v) + ((size_t)smp * c.Hkv + kh) * D + pc * 8;
    T* dst = (tid < D / 8 ? kslab : vslab) + (size_t)c.n_old * D + pc * 8;
    if (row_ok(c, c.n_old)) st_global_16(dst, ld_global_16(src));
  }
  for (int j = tid; j < n1t; j += kThreads) s.id[j] = (j < c.n_old) ? c.kv_ids[base + j] : a.pos;
  // q fragments: thread (gid, tq) holds, for every pair of rounds (2R, 2R+1), the 16 elements [64R + 16tq, +16) of
  // head gid -- the k-slots of an MMA may stand for any elements as long as both operands agree
  uint32_t qf[QR][4];
  {
    const T* qp = reinterpret_cast<const T*>(a.q) + ((size_t)smp * c.Hq + kh * G + gid) * D;
#pragma unroll
    for (int r = 0; r < QR; ++r) {
      const uint4 w = ldg16_or_zero(qp + 64 * (r >> 1) + 16 * tq + 8 * (r & 1), gid < G);
      qf[r][0] = w.x; qf[r][1] = w.y; qf[r][2] = w.z; qf[r][3] = w.w;
    }
  }
  const float sc2 = a.scale * kLog2e;
  const int n_iter = (n1 + kRowsPerIter - 1) / kRowsPerIter;   // same trip count for every thread

  // ---- logits (log2 domain).  Tile rows gid and gid+8; the k-slots of thread tq are its own 8 elements.
  // The loads of iteration it+1 are issued before the MMAs of iteration it (one round trip in flight).
  // (batched mode reads the step's own pair from the caller's buffers, so that no load waits for the barrier that
  // publishes the appended row)
  const T* k_new = reinterpret_cast<const T*>(a.k) + ((size_t)smp * c.Hkv + kh) * D;
  const T* v_new = reinterpret_cast<const T*>(a.v) + ((size_t)smp * c.Hkv + kh) * D;
  auto k_row = [&](int j) { return (KD > 1 && j == c.n_old) ? k_new : kslab + (size_t)j * D; };
  auto v_row = [&](int j) { return (KD > 1 && j == c.n_old) ? v_new : vslab + (size_t)j * D; };
  auto load_k = [&](int it, uint4 (&xx)[QR], uint4 (&yy)[QR]) {
    const int j0 = it * kRowsPerIter + warp * 16 + gid, j1 = j0 + 8;
#pragma unroll
    for (int R = 0; R < QR / 2; ++R) {   // elements [64R + 16tq, +16) of both rows, 32 bytes per load
      ldg32_or_zero(k_row(j0) + 64 * R + 16 * tq, j0 < n1, xx[2 * R], xx[2 * R + 1]);
      ldg32_or_zero(k_row(j1) + 64 * R + 16 * tq, j1 < n1, yy[2 * R], yy[2 * R + 1]);
    }
  };
  auto store_logits = [&](int it, const float (&cacc)[4]) {
    // cacc[0], cacc[1]: key j0, heads 2tq, 2tq+1 ; cacc[2], cacc[3]: key j1
    const int j0 = it * kRowsPerIter + warp * 16 + gid, j1 = j0 + 8;
    if (2 * tq < G) {
      if (j0 < n1) s.p[(2 * tq) * n1t + j0] = cacc[0] * sc2;
      if (j1 < n1) s.p[(2 * tq) * n1t + j1] = cacc[2] * sc2;
    }
    if (2 * tq + 1 < G) {
      if (j0 < n1) s.p[(2 * tq + 1) * n1t + j0] = cacc[1] * sc2;
      if (j1 < n1) s.p[(2 * tq + 1) * n1t + j1] = cacc[3] * sc2;
    }
  };
  // rows of V for iteration `it`: thread (gid, tq) loads, from the 4 rows tb + 4tq + {0..3}, elements [64r + 8gid, +8)
  auto load_v = [&](int it, uint4 (&zz)[VR][4]) {
    const int jr = it * kRowsPerIter + warp * 16 + 4 * tq;
#pragma unroll
    for (int r = 0; r < VR; ++r)
#pragma unroll
      for (int sx = 0; sx < 4; ++sx)
        zz[r][sx] = ldg16_or_zero(v_row(jr + sx) + 64 * r + 8 * gid, jr + sx < n1);
  };
  uint4 xk[KD > 1 ? KD : 1][QR], yk[KD > 1 ? KD : 1][QR];   // KD > 1: the whole cache's K rows (n_iter <= KD)
  if constexpr (KD > 1) {
#pragma unroll
    for (int u = 0; u < KD; ++u) load_k(u, xk[u], yk[u]);   // tiles beyond the last hold no row: no load issued
#pragma unroll
    for (int u = 0; u < KD; ++u) {
      if (u < n_iter) {
        float cacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int r = 0; r < QR; ++r) {
          mma16816(cacc, xk[u][r].x, yk[u][r].x, xk[u][r].y, yk[u][r].y, qf[r][0], qf[r][1]);
          mma16816(cacc, xk[u][r].z, yk[u][r].z, xk[u][r].w, yk[u][r].w, qf[r][2], qf[r][3]);
        }
        store_logits(u, cacc);
      }
    }
  } else {
    uint4 x[QR], y[QR];
    // the first tile of K does not contain the row appended above unless the cache is still tiny, so its loads
    // are issued before the barrier that publishes that row
    const bool early = c.n_old >= kRowsPerIter;
    if (early) load_k(0, x, y);
    __syncthreads();
    if (!early) load_k(0, x, y);
    for (int it = 0; it < n_iter; ++it) {
      uint4 xn[QR], yn[QR];
      if (it + 1 < n_iter) load_k(it + 1, xn, yn);
      float cacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int r = 0; r < QR; ++r) {
        mma16816(cacc, x[r].x, y[r].x, x[r].y, y[r].y, qf[r][0], qf[r][1]);
        mma16816(cacc, x[r].z, y[r].z, x[r].w, y[r].w, qf[r][2], qf[r][3]);
      }
      store_logits(it, cacc);
      if (it + 1 < n_iter) {
#pragma unroll
        for (int r = 0; r < QR; ++r) { x[r] = xn[r]; y[r] = yn[r]; }
      }
    }
  }
  // first V tile and the old sum_weights start loading now; they are needed only after the softmax
  uint4 z[VR][4];
  // KD > 1: all of V starts on its way into shared memory now, as TMA tiles of 128 rows x 64 elements (128-byte
  // swizzle; rows past n_old arrive as zeros), one mbarrier per 128 rows; the tiles of each half of the row lie
  // one behind the other, so that each half is one array of 128-byte rows.  The copies stream while the softmax
  // phases run and pass by the register file, whose write-back path those phases need (the same rows prefetched
  // into registers made the phases longer by the time the loads took; per-thread cp.async stalled at issue).
  const uint32_t stage0 = (tc::smem_u32(smem_raw) + (uint32_t)smem_layout(nullptr, D, G, n1, kWarps, nullptr) + 1023u) & ~1023u;
  unsigned char* stage = smem_raw + (stage0 - tc::smem_u32(smem_raw));   // [0, 1024): barriers; then the tiles
  uint64_t* vbar = reinterpret_cast<uint64_t*>(stage);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(stage + 64);
  constexpr int kBoxBytes = 128 * 128;   // 128 rows x 64 bf16
  if constexpr (KD > 1) {
    if (tid == 0) {
#pragma unroll
      for (int u = 0; u < KD; ++u)
        if (u < n_iter) {
          tc::mbar_expect_tx(&vbar[u], 2 * kBoxBytes);
          tc::tma_load_3d(stage + 1024 + u * kBoxBytes, &vmap, 0, u * 128, unit, &vbar[u]);
          tc::tma_load_3d(stage + 1024 + (KD + u) * kBoxBytes, &vmap, 64, u * 128, unit, &vbar[u]);
        }
    }
  } else {
    load_v(0, z);
  }
  constexpr int kSwPrefetch = 4;
  float sw_old[kSwPrefetch];
#pragma unroll
  for (int u = 0; u < kSwPrefetch; ++u) {
    const int j = tid + u * kThreads;
    sw_old[u] = (j < c.n_old) ? c.sum_weights[base + j] : 0.f;
  }
  __syncthreads();

  // ---- softmax statistics over the n1 rows with one barrier: every thread folds its own logits into a
  // (maximum, sum of exp2 relative to that maximum) pair per head, pairs are merged across the warp by shuffles
  // and across warps through shared memory in a fixed order.
  // left-padded sample: padding pairs are masked and leave first (each thread masks the rows whose ids it
  // loaded itself); a query at a padding position, which no real decode step is, gets zero output and no weights
  const int pad = PLAIN ? 0 : sample_left_pad(c, smp);
  const int rule = PLAIN ? 0 : c.rule;
  const bool q_real = PLAIN || a.pos >= pad;
  if (!PLAIN && pad > 0 && q_real) {
    for (int j = tid; j < n1; j += kThreads)
      if (s.id[j] < pad) {
#pragma unroll
        for (int h = 0; h < G; ++h) s.p[h * n1t + j] = -INFINITY;
      }
  }
  float inv[G], mfin[G];
  {
    float m[G], t[G];
#pragma unroll
    for (int h = 0; h < G; ++h) m[h] = -INFINITY;
    for (int j = tid; j < n1; j += kThreads)
#pragma unroll
      for (int h = 0; h < G; ++h) m[h] = fmaxf(m[h], s.p[h * n1t + j]);
    // the warp's maximum first (plain max shuffles), then every lane sums relative to it: no exponentials inside
    // the shuffle chain
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
#pragma unroll
      for (int h = 0; h < G; ++h) m[h] = fmaxf(m[h], __shfl_xor_sync(0xffffffffu, m[h], off));
#pragma unroll
    for (int h = 0; h < G; ++h) t[h] = 0.f;
    for (int j = tid; j < n1; j += kThreads)
#pragma unroll
      for (int h = 0; h < G; ++h)   // a warp whose rows are all masked carries (-inf, 0): no inf - inf
        t[h] += ex2f(s.p[h * n1t + j] - (m[h] == -INFINITY ? 0.f : m[h]));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
#pragma unroll
      for (int h = 0; h < G; ++h) t[h] += __shfl_xor_sync(0xffffffffu, t[h], off);   // a + b == b + a: lanes agree
    if (lane == 0)
#pragma unroll
      for (int h = 0; h < G; ++h) { s.wred[h * kWarps + warp] = m[h]; s.wred[(G + h) * kWarps + warp] = t[h]; }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float mm = -INFINITY;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, s.wred[h * kWarps + w]);
      float tt = 0.f;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {   // fixed order
        const float mw = s.wred[h * kWarps + w];
        tt += (mw == -INFINITY) ? 0.f : s.wred[(G + h) * kWarps + w] * ex2f(mw - mm);
      }
      mfin[h] = mm;
      inv[h] = q_real ? 1.f / tt : 0.f;
    }
  }

  // ---- normalise, sum_weights += attn_weights (heads added in a fixed order), candidate for eviction
  float best_ave = INFINITY;
  int best_j = -1, best_id = -1;
  for (int j = tid, u = 0; j < n1t; j += kThreads, ++u) {
    if (j >= n1) {
#pragma unroll
      for (int h = 0; h < G; ++h) s.p[h * n1t + j] = 0.f;   // padding keys carry no weight
      continue;
    }
    float add = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float p = ex2f(s.p[h * n1t + j] - mfin[h]) * inv[h];
      s.p[h * n1t + j] = p;
      add += p;
    }
    float old_sw = 0.f;
    if (u < kSwPrefetch) {
#pragma unroll
      for (int uu = 0; uu < kSwPrefetch; ++uu) old_sw = (uu == u) ? sw_old[uu] : old_sw;
    } else if (j < c.n_old) {
      old_sw = c.sum_weights[base + j];
    }
    const float sw = (rule_overwrites(rule) ? 0.f : old_sw) + add;   // rules 2, 3 keep this step's weights only
    if (!PLAIN && c.sum_sq != nullptr) {                             // rule 4: sum of squared weights as well
      float add_sq = 0.f;
#pragma unroll
      for (int h = 0; h < G; ++h) add_sq = fmaf(s.p[h * n1t + j], s.p[h * n1t + j], add_sq);
      c.sum_sq[base + j] = (j < c.n_old ? c.sum_sq[base + j] : 0.f) + add_sq;
    }
    s.score[j] = sw;
    if (evict_one) {
      float ave;   // ranking value: average attention (Sec. 3.2), or the raw weights with / without a recent window
      if (!PLAIN && s.id[j] < pad) ave = -1.f;
      // fast division: the IEEE routine takes a slow path for the tiny sums of long-evicted histories (4 % of the step)
      else if (rule == 0) ave = __fdividef(sw, (float)G * (float)(a.pos + 1 - s.id[j]));
      else ave = (rule == 1 && j >= n1 - a.target / 2) ? INFINITY : sw;
      // ties: the higher position leaves (kv_ids, not rows: the rows of an unordered cache are in no order)
      if (ave < best_ave || (ave == best_ave && s.id[j] > best_id)) { best_ave = ave; best_j = j; best_id = s.id[j]; }
    } else if (row_ok(c, j)) {
      c.sum_weights[base + j] = sw;
    }
  }
  int hole = n1;  // no row leaves
  if (evict_one) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float oa = __shfl_xor_sync(0xffffffffu, best_ave, off);
      const int oj = __shfl_xor_sync(0xffffffffu, best_j, off), oi = __shfl_xor_sync(0xffffffffu, best_id, off);
      if (oa < best_ave || (oa == best_ave && oi > best_id)) { best_ave = oa; best_j = oj; best_id = oi; }
    }
    if (lane == 0) {
      s.best[warp] = best_ave;
      reinterpret_cast<int*>(s.best)[kWarps + warp] = best_j;
      reinterpret_cast<int*>(s.best)[2 * kWarps + warp] = best_id;
    }
    __syncthreads();
    best_ave = s.best[0];
    best_j = reinterpret_cast<int*>(s.best)[kWarps];
    best_id = reinterpret_cast<int*>(s.best)[2 * kWarps];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) {
      const float oa = s.best[w];
      const int oj = reinterpret_cast<int*>(s.best)[kWarps + w], oi = reinterpret_cast<int*>(s.best)[2 * kWarps + w];
      if (oa < best_ave || (oa == best_ave && oi > best_id)) { best_ave = oa; best_j = oj; best_id = oi; }
    }
    hole = best_j;
    if (c.fill) {
      // unordered cache: every pair stays where it is and the step's own pair takes the row of the pair that leaves
      if (c.moved != nullptr && tid == 0 && hole < c.n_old) atomicAdd(&c.moved[unit & 15], 1ull);
      for (int j = tid; j < c.n_old; j += kThreads) {
        if (j != hole) c.sum_weights[base + j] = s.score[j];
        else { c.sum_weights[base + j] = s.score[c.n_old]; c.kv_ids[base + j] = a.pos; }
      }
    } else {
      if (c.moved != nullptr && tid == 0) atomicAdd(&c.moved[unit & 15], (unsigned long long)(n1 - 1 - hole));
      // sum_weights / kv_ids in their final places: rows behind the hole move up by one
      for (int j = tid; j < n1; j += kThreads) {
        if (!row_ok(c, j)) continue;
        if (j < hole) c.sum_weights[base + j] = s.score[j];
        else if (j > hole) { c.sum_weights[base + j - 1] = s.score[j]; c.kv_ids[base + j - 1] = s.id[j]; }
      }
    }
  } else {
    if (tid == 0) c.kv_ids[base + c.n_old] = a.pos;
    __syncthreads();
  }

  // ---- out^T = V^T p^T.  Thread (gid, tq) loads, from the 4 rows tb + 4tq + {0..3}, the 8 elements
  // [64r + 8gid, +8); MMA m uses element m as fragment row gid and element m+4 as row gid+8.
  float oacc[VR][4][4];
#pragma unroll
  for (int r = 0; r < VR; ++r)
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
      for (int e = 0; e < 4; ++e) oacc[r][m][e] = 0.f;
  // one tile of 16 rows per warp: its MMAs, then -- once the hole lies in or before the tile -- its rows' move up
  auto pv_tile = [&](int it, const uint4 (&zt)[VR][4]) {
    const int tb = it * kRowsPerIter + warp * 16;
    const int jr = tb + 4 * tq;   // first of this thread's 4 rows
    // p^T fragment: (head gid; keys jr, jr+1) and (head gid; keys jr+2, jr+3)
    uint32_t pb0 = 0u, pb1 = 0u;
    if (gid < G && jr < n1t) {
      const float4 pv = *reinterpret_cast<const float4*>(&s.p[gid * n1t + jr]);
      pb0 = pack2(pv.x, pv.y);
      pb1 = pack2(pv.z, pv.w);
    }
#pragma unroll
    for (int r = 0; r < VR; ++r) {
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        // element m of the 8 loaded: 32-bit word m/2, half m%2 ; element m+4: word 2 + m/2, same half
        const uint32_t sel = (m & 1) ? 0x7632u : 0x5410u;
        const uint32_t w0 = (m < 2) ? zt[r][0].x : zt[r][0].y, w1 = (m < 2) ? zt[r][1].x : zt[r][1].y;
        const uint32_t w2 = (m < 2) ? zt[r][2].x : zt[r][2].y, w3 = (m < 2) ? zt[r][3].x : zt[r][3].y;
        const uint32_t u0 = (m < 2) ? zt[r][0].z : zt[r][0].w, u1 = (m < 2) ? zt[r][1].z : zt[r][1].w;
        const uint32_t u2 = (m < 2) ? zt[r][2].z : zt[r][2].w, u3 = (m < 2) ? zt[r][3].z : zt[r][3].w;
        mma16816(oacc[r][m], prmt(w0, w1, sel), prmt(u0, u1, sel), prmt(w2, w3, sel), prmt(u2, u3, sel), pb0, pb1);
      }
    }
    if (evict_one && !c.fill && (it + 1) * kRowsPerIter > hole) {   // uniform over the CTA
      __syncthreads();                                   // every load of rows < (it+1)*kRowsPerIter has completed
#pragma unroll
      for (int r = 0; r < VR; ++r)
#pragma unroll
        for (int sx = 0; sx < 4; ++sx) {
          const int j = jr + sx;
          if (j < n1 && j > hole && row_ok(c, j - 1)) st_global_16(vslab + (size_t)(j - 1) * D + 64 * r + 8 * gid, zt[r][sx]);
        }
    }
  };
  if constexpr (KD > 1) {
    if (evict_one && !c.fill) {   // K rows behind the hole, one row up, from the registers that fed the logits
#pragma unroll
      for (int u = 0; u < KD; ++u) {
        const int j0 = u * kRowsPerIter + warp * 16 + gid, j1 = j0 + 8;
#pragma unroll
        for (int R = 0; R < QR / 2; ++R) {
          if (j0 < n1 && j0 > hole && row_ok(c, j0 - 1)) stg32(kslab + (size_t)(j0 - 1) * D + 64 * R + 16 * tq, xk[u][2 * R], xk[u][2 * R + 1]);
          if (j1 < n1 && j1 > hole && row_ok(c, j1 - 1)) stg32(kslab + (size_t)(j1 - 1) * D + 64 * R + 16 * tq, yk[u][2 * R], yk[u][2 * R + 1]);
        }
      }
    }
    // V has arrived (every thread observes every tile's barrier itself: what it reads below, and what it overwrites
    // in global memory, has been read by the copies)
#pragma unroll
    for (int u = 0; u < KD; ++u)
      if (u < n_iter) tc::mbar_wait(&vbar[u], 0, abort_flag, c.status);
    auto v_piece = [&](int j, int piece) -> uint4* {   // 16 bytes [8 piece, +8) of row j in the swizzled tiles
      return reinterpret_cast<uint4*>(stage + 1024 + (piece >> 3) * (KD * kBoxBytes) + j * 128 + (((piece & 7) ^ (j & 7)) << 4));
    };
    if (tid < D / 8) {   // the step's own row
      *v_piece(c.n_old, tid) = ld_global_16(v_new + tid * 8);
      tc::fence_async_smem();   // the TMA stores below read it
    }
    __syncthreads();
    if (evict_one && !c.fill) {
      // V rows behind the hole, one row up, from shared memory: up to the next multiple of 8 rows (the swizzle's
      // period) by plain stores, the rest as TMA tiles of 128 rows written one row higher than they were read
      // (rows past n_old - 1 are clipped by the map); they drain under the MMAs below.  A tile that would read past
      // the staged rows is not stored: the rows from r_tail on (fewer than 128) leave by plain stores as well.
      const int r8 = (hole + 8) & ~7;
      const int r_tail = r8 > (KD - 1) * 128 ? r8 : r8 + 128 * (((KD - 1) * 128 - r8) / 128 + 1);
      const int pieces = (min(r8, n1) - 1 - hole) * (D / 8);
      if (tid < pieces) {
        const int j = hole + 1 + tid / (D / 8), pc = tid % (D / 8);
        if (row_ok(c, j - 1)) st_global_16(vslab + (size_t)(j - 1) * D + pc * 8, *v_piece(j, pc));
      }
      for (int x = tid; x < (n1 - r_tail) * (D / 8); x += kThreads) {
        const int j = r_tail + x / (D / 8), pc = x % (D / 8);
        if (row_ok(c, j - 1)) st_global_16(vslab + (size_t)(j - 1) * D + pc * 8, *v_piece(j, pc));
      }
      if (tid == 0) {
        for (int r0 = r8; r0 < min(n1, r_tail); r0 += 128) {
          tc::tma_store_3d(&vmap, stage + 1024 + r0 * 128, 0, r0 - 1, unit);
          tc::tma_store_3d(&vmap, stage + 1024 + KD * kBoxBytes + r0 * 128, 64, r0 - 1, unit);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
    // out^T tiles of 16 elements x heads: A = V^T (transposing ldmatrix), B = p^T of keys tb + {2tq, 2tq+1, 2tq+8, 2tq+9}
#pragma unroll
    for (int u = 0; u < KD; ++u) {
      const int tb = u * kRowsPerIter + warp * 16;
      if (u < n_iter && tb < n1t) {   // warp-uniform
        uint32_t pb0 = 0u, pb1 = 0u;
        if (gid < G) {
          const float2 p0 = *reinterpret_cast<const float2*>(&s.p[gid * n1t + tb + 2 * tq]);
          const float2 p1 = *reinterpret_cast<const float2*>(&s.p[gid * n1t + tb + 2 * tq + 8]);
          pb0 = pack2(p0.x, p0.y);
          pb1 = pack2(p1.x, p1.y);
        }
        // lane l addresses row l%8 of matrix l/8: keys tb + 8(l/16) + l%8, elements 16 dt + 8((l/8)%2) + [0, 8)
        const int krow = tb + ((lane >> 4) << 3) + (lane & 7);
#pragma unroll
        for (int dt = 0; dt < D / 16; ++dt) {
          uint32_t a0, a1, a2, a3;
          const uint32_t addr = tc::smem_u32(v_piece(krow, 2 * dt + ((lane >> 3) & 1)));
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                       : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr) : "memory");
          mma16816(oacc[dt / 4][dt % 4], a0, a1, a2, a3, pb0, pb1);
        }
      }
    }
  } else {
    for (int it = 0; it < n_iter; ++it) {
      uint4 zn[VR][4];
      if (it + 1 < n_iter) load_v(it + 1, zn);   // next iteration's rows load while this one is multiplied
      pv_tile(it, z);
      if (it + 1 < n_iter) {
#pragma unroll
        for (int r = 0; r < VR; ++r)
#pragma unroll
          for (int sx = 0; sx < 4; ++sx) z[r][sx] = zn[r][sx];
      }
    }
  }
  // K rows behind the hole: one-row shift (re-read, mostly from L2: the logits pass just streamed them)
  if (evict_one && c.fill) {
    // unordered cache: the step's own pair takes the row of the pair that leaves (every read of that row is over)
    __syncthreads();
    if (hole < c.n_old && tid < 2 * (D / 8)) {
      const int pc = tid % (D / 8);
      T* dst = (tid < D / 8 ? kslab : vslab) + (size_t)hole * D + pc * 8;
      if (row_ok(c, hole)) st_global_16(dst, ld_global_16((tid < D / 8 ? k_new : v_new) + pc * 8));
    }
  } else if (KD == 1 && evict_one) {
    constexpr int PR = D / 8;                 // 16-byte pieces per row
    constexpr int RPI = kThreads / PR * 8;    // rows per iteration, 8 pieces per thread
    const int slot = tid / PR, pc = tid % PR;
    for (int r0 = (hole / RPI) * RPI; r0 < n1; r0 += RPI) {
      uint4 raw[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = r0 + slot + u * (kThreads / PR);
        if (j < n1 && j > hole) raw[u] = ld_global_16(kslab + (size_t)j * D + pc * 8);
      }
      __syncthreads();
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = r0 + slot + u * (kThreads / PR);
        if (j < n1 && j > hole && row_ok(c, j - 1)) st_global_16(kslab + (size_t)(j - 1) * D + pc * 8, raw[u]);
      }
    }
  }

  // ---- combine the warps' partial outputs in a fixed order.  oacc[r][m][0..1]: element 64r + 8gid + m of heads
  // 2tq, 2tq+1; oacc[r][m][2..3]: element 64r + 8gid + m + 4.
#pragma unroll
  for (int r = 0; r < VR; ++r)
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int h = 2 * tq + (e & 1);
        // KD > 1: tile dt = 4r + m holds elements 16 dt + gid (+ 8)
        const int dd = KD > 1 ? 16 * (4 * r + m) + gid + ((e & 2) ? 8 : 0) : 64 * r + 8 * gid + m + ((e & 2) ? 4 : 0);
        if (h < G) s.ored[(warp * G + h) * D + dd] = oacc[r][m][e];
      }
  __syncthreads();
  for (int t = tid; t < G * D; t += kThreads) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) tot += s.ored[w * G * D + t];
    T* op = reinterpret_cast<T*>(a.out) + ((size_t)smp * c.Hq + kh * G) * D;
    op[t] = __float2bfloat16_rn(tot);
  }

  if constexpr (KD > 1) {   // the TMA stores have read their rows out of shared memory
    if (tid == 0 && evict_one && !c.fill) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
  }
  if (evict_general) {
    __syncthreads();
    CacheView cv = c;
    cv.n_old = n1;
    EvictArgs e;
    e.blk_k = nullptr; e.blk_v = nullptr; e.new_sum = nullptr;
    e.I = 0; e.pos0 = 0; e.curr_id = a.pos; e.target = a.target;
    evict_body<T, D, kThreads>(cv, unit, smp, kh, e, smem_raw);
  }
}

constexpr size_t kMaxDynamicSmem = 227 * 1024;
// barriers + alignment slack + KD x 128 rows of V
constexpr size_t stage_bytes(int d, int nt, int kd) { return 2048 + (size_t)kd * (nt / 32) * 16 * d * 2; }
constexpr int kBatchTiles = 5;   // tiles per warp of the one-CTA-per-SM instance (160 registers of K rows): 640 pairs

template <int D, int G, int NT, bool PLAIN, int KD>
cudaError_t launch_nt_p(const CacheView& c, const DecodeArgs& a, cudaStream_t st, const CUtensorMap& vmap) {
  // sized for the larger CTA; the one-CTA-per-SM instance stages all of V behind it
  const size_t smem = decode_mma_smem_bytes(D, G, c.n_old + 1, a.target) + (KD > 1 ? stage_bytes(D, NT, KD) : 0);
  static SmemConfigured configured;
  if (cudaError_t err = configured.ensure(decode_mma_kernel<D, G, NT, PLAIN, KD>, smem); err != cudaSuccess) return err;
  ProfileScope prof(kDecode, st);
  const cudaError_t err =
      launch_dependent(decode_mma_kernel<D, G, NT, PLAIN, KD>, dim3(c.nsamples * c.Hkv), dim3(NT), smem, st, c, a, vmap);
  count_launch();
  return err != cudaSuccess ? err : cudaGetLastError();
}

template <int D, int G, int NT>
cudaError_t launch_nt(const CacheView& c, const DecodeArgs& a, cudaStream_t st, bool one_per_sm) {
  const bool plain = c.left_pad == nullptr && c.rule == 0;
  if constexpr (NT == 256 && D == 128) {
    if (one_per_sm && c.n_old + 1 <= kBatchTiles * (NT / 32) * 16 &&
        decode_mma_smem_bytes(D, G, c.n_old + 1, a.target) + stage_bytes(D, NT, kBatchTiles) <= kMaxDynamicSmem) {
      CUtensorMap vmap;
      if (encode_slab_rows_map(&vmap, c.v_slab, D, c.n_old, c.cap, c.nsamples * c.Hkv, 128))
        return plain ? launch_nt_p<D, G, NT, true, kBatchTiles>(c, a, st, vmap)
                     : launch_nt_p<D, G, NT, false, kBatchTiles>(c, a, st, vmap);
    }
  }
  static const CUtensorMap no_map = {};   // the other instances take no tensor map
  return plain ? launch_nt_p<D, G, NT, true, 1>(c, a, st, no_map) : launch_nt_p<D, G, NT, false, 1>(c, a, st, no_map);
}

int sm_count() {   // of the current device
  static int count[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (count[dev] == 0 && cudaDeviceGetAttribute(&count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    count[dev] = 148;
  return count[dev];
}

template <int D, int G>
cudaError_t launch_t(const CacheView& c, const DecodeArgs& a, cudaStream_t st) {
  // four small CTAs per SM only pay for short caches: all four must fit into shared memory (up to about 1500 pairs
  // at g = 4), and beyond that length the larger CTA measured faster at every group size (g = 1, 4096 pairs, 2000
  // caches: 0.96 against 0.69)
  const bool four_fit = c.n_old + 1 <= 1536 && smem_layout(nullptr, D, G, c.n_old + 1, 4, nullptr) <= 56 * 1024;
  const bool small_ctas = four_fit && c.nsamples * c.Hkv > 2 * sm_count();
  // a grid that leaves every CTA an SM of its own: the instance that keeps K in registers
  const bool one_per_sm = c.nsamples * c.Hkv <= sm_count();
  return small_ctas ? launch_nt<D, G, 128>(c, a, st, false) : launch_nt<D, G, 256>(c, a, st, one_per_sm);
}

template <int D>
cudaError_t launch_g(const CacheView& c, const DecodeArgs& a, cudaStream_t st) {
  switch (c.g) {
    case 1: return launch_t<D, 1>(c, a, st);
    case 2: return launch_t<D, 2>(c, a, st);
    case 4: return launch_t<D, 4>(c, a, st);
    case 8: return launch_t<D, 8>(c, a, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

size_t decode_mma_smem_bytes(int d, int g, int n_rows, int target) {
  const size_t attn = smem_layout(nullptr, d, g, n_rows, kMaxWarps, nullptr);
  const size_t ev = (target >= 0 && target < n_rows) ? evict_smem_bytes(n_rows, target) : 0;
  return attn > ev ? attn : ev;
}

cudaError_t launch_decode_mma(int d, const CacheView& c, const void* q, const void* k, const void* v, void* out,
                              int32_t pos, float scale, int32_t target, cudaStream_t st) {
  DecodeArgs a{q, k, v, out, pos, scale, target};
  if (d == 64) return launch_g<64>(c, a, st);
  if (d == 128) return launch_g<128>(c, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace bm
