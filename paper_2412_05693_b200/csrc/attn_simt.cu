// fp32 SIMT forward pass over a block of inputs (Sec. 3.2): tiled attention with an online softmax
// (outputs + log-sum-exp), and the transposed score pass that turns the normalised weights into the
// column sums  sum_weights += sum_i attn_weights[i].  This is the production path for fp32 caches
// (fp32 accuracy rules out the bf16 tensor-core kernels) and the fallback shape coverage for bf16.
#include "common.cuh"

namespace bm {
namespace {

constexpr int kTile = 64;     // query rows per CTA tile and keys per tile
constexpr int kThreads = 256;

// Loads 64 rows of D elements (fp32-widened) into smem with row stride D+1.  `row_ptr(r)` returns the
// global address of tile row r or nullptr for a row that does not exist (filled with zeros).
template <typename T, int D, typename F>
__device__ inline void load_tile(float* dst, int tid, F row_ptr) {
  constexpr int V = Elem<T>::kVec;
  constexpr int CH = D / V;  // 16-byte chunks per row
  for (int idx = tid; idx < kTile * CH; idx += kThreads) {
    const int r = idx / CH, cv = idx % CH;
    const T* p = row_ptr(r);
    float f[V];
    if (p != nullptr) {
      Elem<T>::unpack(ld_global_16(p + cv * V), f);
    } else {
#pragma unroll
      for (int e = 0; e < V; ++e) f[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < V; ++e) dst[r * (D + 1) + cv * V + e] = f[e];
  }
}

// 64x64 tile of dot products: thread (ty, tx) owns rows ty+16a, columns tx+16b.
template <int D>
__device__ inline void dot_tile(const float* sA, const float* sB, int ty, int tx, float (&acc)[4][4]) {
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 8
  for (int c = 0; c < D; ++c) {
    float av[4], bv[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) av[a] = sA[(ty + 16 * a) * (D + 1) + c];
#pragma unroll
    for (int b = 0; b < 4; ++b) bv[b] = sB[(tx + 16 * b) * (D + 1) + c];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
  }
}

template <typename T, int D>
__device__ inline const T* key_row_ptr(const CacheView& c, const void* slab, const void* blk, int unit,
                                       int smp, int kh, int I, int j) {
  if (j < c.n_old) return reinterpret_cast<const T*>(slab) + ((size_t)unit * c.cap + j) * D;
  const int jj = j - c.n_old;
  if (jj < I) return reinterpret_cast<const T*>(blk) + ((size_t)(smp * I + jj) * c.Hkv + kh) * D;
  return nullptr;
}

template <typename T, int D>
__device__ inline const T* query_row_ptr(const CacheView& c, const BlockArgs& a, int smp, int kh, int row) {
  if (row >= a.I * c.g) return nullptr;
  const int i = row / c.g, h = row % c.g;
  return reinterpret_cast<const T*>(a.q) + ((size_t)(smp * a.I + i) * c.Hq + kh * c.g + h) * D;
}

// ------------------------------------------------------------------------------------------------
// Forward: out = softmax(scale * q k^T) v over the n_old cached pairs and the block's causal pairs.
// Grid: (row tiles of the unit's I*g query rows, units).  Row r of a unit = (input r / g, head r % g).
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) attn_fwd_simt(CacheView c, BlockArgs a) {
  constexpr int LD = D + 1;
  extern __shared__ float sm[];
  float* sQ = sm;
  float* sKV = sQ + kTile * LD;
  float* sS = sKV + kTile * LD;        // [64][65]
  float* sM = sS + kTile * (kTile + 1);
  float* sL = sM + kTile;
  float* sAl = sL + kTile;
  int* sKp = reinterpret_cast<int*>(sAl + kTile);   // [64] 1 = the tile's key is a padding pair

  const int unit = blockIdx.y, smp = unit / c.Hkv, kh = unit % c.Hkv;
  const int pad = sample_left_pad(c, smp);
  const int R = a.I * c.g, row0 = blockIdx.x * kTile;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4, lane = tid & 31, warp = tid >> 5;

  load_tile<T, D>(sQ, tid, [&](int r) { return query_row_ptr<T, D>(c, a, smp, kh, row0 + r); });
  if (tid < kTile) { sM[tid] = -INFINITY; sL[tid] = 0.f; }

  float o[4][D / 16];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < D / 16; ++y) o[x][y] = 0.f;

  const int last_row = min(R - 1, row0 + kTile - 1);
  const int n_keys = c.n_old + last_row / c.g + 1;  // keys visible to the tile's last row
  for (int j0 = 0; j0 < n_keys; j0 += kTile) {
    __syncthreads();  // previous iteration finished with sKV / sS
    load_tile<T, D>(sKV, tid, [&](int r) { return key_row_ptr<T, D>(c, c.k_slab, a.k, unit, smp, kh, a.I, j0 + r); });
    if (tid < kTile) {
      const int j = j0 + tid;
      int is_pad = 0;
      if (pad > 0 && j < c.n_old + a.I)
        is_pad = (j < c.n_old ? c.kv_ids[(size_t)unit * c.cap + j] : a.pos0 + (j - c.n_old)) < pad;
      sKp[tid] = is_pad;
    }
    __syncthreads();
    float acc[4][4];
    dot_tile<D>(sQ, sKV, ty, tx, acc);
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) sS[(ty + 16 * x) * (kTile + 1) + tx + 16 * y] = acc[x][y] * a.scale;
    __syncthreads();
    load_tile<T, D>(sKV, tid, [&](int r) { return key_row_ptr<T, D>(c, c.v_slab, a.v, unit, smp, kh, a.I, j0 + r); });
    // online softmax: warp w owns rows 8w .. 8w+7, lane owns columns lane and lane+32
    for (int rr = 0; rr < 8; ++rr) {
      const int r = warp * 8 + rr, row = row0 + r;
      const int vis = (row < R) ? (c.n_old + row / c.g + 1) : 1;
      // a real query does not see padding pairs; a padding query's row is computed over everything and dropped
      const bool real = (row < R) && (a.pos0 + row / c.g >= pad);
      const bool ok0 = (j0 + lane) < vis && !(real && sKp[lane]);
      const bool ok1 = (j0 + lane + 32) < vis && !(real && sKp[lane + 32]);
      const float s0 = ok0 ? sS[r * (kTile + 1) + lane] : -INFINITY;
      const float s1 = ok1 ? sS[r * (kTile + 1) + lane + 32] : -INFINITY;
      float mt = fmaxf(s0, s1);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, off));
      const float m_old = sM[r];
      const float m_new = fmaxf(m_old, mt);
      const float p0 = ok0 ? expf(s0 - m_new) : 0.f;
      const float p1 = ok1 ? expf(s1 - m_new) : 0.f;
      float ps = p0 + p1;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      const float alpha = (m_new == -INFINITY) ? 1.f : expf(m_old - m_new);
      __syncwarp();
      sS[r * (kTile + 1) + lane] = p0;
      sS[r * (kTile + 1) + lane + 32] = p1;
      if (lane == 0) { sM[r] = m_new; sL[r] = sL[r] * alpha + ps; sAl[r] = alpha; }
    }
    __syncthreads();
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const float al = sAl[ty + 16 * x];
#pragma unroll
      for (int y = 0; y < D / 16; ++y) o[x][y] *= al;
    }
#pragma unroll 4
    for (int j = 0; j < kTile; ++j) {
      float pv[4], vv[D / 16];
#pragma unroll
      for (int x = 0; x < 4; ++x) pv[x] = sS[(ty + 16 * x) * (kTile + 1) + j];
#pragma unroll
      for (int y = 0; y < D / 16; ++y) vv[y] = sKV[j * LD + tx + 16 * y];
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < D / 16; ++y) o[x][y] = fmaf(pv[x], vv[y], o[x][y]);
    }
  }
  __syncthreads();
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int r = ty + 16 * x, row = row0 + r;
    if (row >= R) continue;
    const int i = row / c.g, h = row % c.g;
    const bool real = a.pos0 + i >= pad;          // a padding query: zero output, and +inf so that it has no weights
    const float inv = real ? 1.f / sL[r] : 0.f;
    T* op = reinterpret_cast<T*>(a.out) + ((size_t)(smp * a.I + i) * c.Hq + kh * c.g + h) * D;
#pragma unroll
    for (int y = 0; y < D / 16; ++y) op[tx + 16 * y] = Elem<T>::to_out(o[x][y] * inv);
    if (tx == 0) a.lse[(size_t)unit * R + row] = real ? sM[r] + logf(sL[r]) : INFINITY;
  }
}

// ------------------------------------------------------------------------------------------------
// Score pass: for every candidate pair j (cached or new) the column sum over all query rows of the
// block of exp(scale * q.k_j - lse_row), i.e. sum_i attn_weights[i][j] added over the group's heads.
// Grid: (key tiles, units).  Sums are formed in a fixed order (deterministic, no float atomics).
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) score_simt(CacheView c, BlockArgs a) {
  constexpr int LD = D + 1;
  extern __shared__ float sm[];
  float* sQ = sm;
  float* sK = sQ + kTile * LD;
  float* sRed = sK + kTile * LD;  // [16][64]
  float* sLse = sRed + 16 * kTile;

  const int unit = blockIdx.y, smp = unit / c.Hkv, kh = unit % c.Hkv;
  const int R = a.I * c.g, j0 = blockIdx.x * kTile, n_c = c.n_old + a.I;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  load_tile<T, D>(sK, tid, [&](int r) { return key_row_ptr<T, D>(c, c.k_slab, a.k, unit, smp, kh, a.I, j0 + r); });
  float col[4] = {0.f, 0.f, 0.f, 0.f}, col_sq[4] = {0.f, 0.f, 0.f, 0.f};
  const int counted_from = rule_first_counted_row(c.rule, c.window, a.I, c.g);   // rules that look at the last queries only
  const int first_row = (j0 > c.n_old) ? (j0 - c.n_old) * c.g : 0;  // earlier rows cannot see this tile
  for (int row0 = (first_row / kTile) * kTile; row0 < R; row0 += kTile) {
    __syncthreads();
    load_tile<T, D>(sQ, tid, [&](int r) { return query_row_ptr<T, D>(c, a, smp, kh, row0 + r); });
    if (tid < kTile)
      sLse[tid] = (row0 + tid < R && row0 + tid >= counted_from) ? a.lse[(size_t)unit * R + row0 + tid] : INFINITY;
    __syncthreads();
    float acc[4][4];
    dot_tile<D>(sQ, sK, ty, tx, acc);
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = j0 + tx + 16 * y;
      float part = 0.f, part_sq = 0.f;
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int r = ty + 16 * x, row = row0 + r;
        const bool vis = (row < R) && (j < c.n_old + row / c.g + 1);
        const float w = vis ? expf(acc[x][y] * a.scale - sLse[r]) : 0.f;
        part += w;
        part_sq = fmaf(w, w, part_sq);
      }
      col[y] += part;
      col_sq[y] += part_sq;
    }
  }
  __syncthreads();
#pragma unroll
  for (int y = 0; y < 4; ++y) sRed[ty * kTile + tx + 16 * y] = col[y];
  __syncthreads();
  if (tid < kTile) {
    const int j = j0 + tid;
    if (j < n_c) {
      float tot = 0.f;
#pragma unroll
      for (int t = 0; t < 16; ++t) tot += sRed[t * kTile + tid];
      const int pad = sample_left_pad(c, smp);
      if (pad > 0 && (j < c.n_old ? c.kv_ids[(size_t)unit * c.cap + j] : a.pos0 + (j - c.n_old)) < pad)
        tot = 0.f;                                  // a padding pair is masked for every query
      if (j < c.n_old) {
        if (rule_overwrites(c.rule)) c.sum_weights[(size_t)unit * c.cap + j] = tot;   // nothing is carried over
        else c.sum_weights[(size_t)unit * c.cap + j] += tot;
      }
      else a.new_sum[(size_t)unit * a.I + (j - c.n_old)] = tot;
    }
  }
  if (c.sum_sq != nullptr) {    // rule 4: the same reduction over the squares
    __syncthreads();
#pragma unroll
    for (int y = 0; y < 4; ++y) sRed[ty * kTile + tx + 16 * y] = col_sq[y];
    __syncthreads();
    if (tid < kTile && j0 + tid < n_c) {
      const int j = j0 + tid;
      float tot = 0.f;
#pragma unroll
      for (int t = 0; t < 16; ++t) tot += sRed[t * kTile + tid];
      if (j < c.n_old) c.sum_sq[(size_t)unit * c.cap + j] += tot;
      else a.new_sq[(size_t)unit * a.I + (j - c.n_old)] = tot;
    }
  }
}

template <typename T, int D>
cudaError_t launch_attn_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  const size_t smem = sizeof(float) * (2 * kTile * (D + 1) + kTile * (kTile + 1) + 4 * kTile);
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(attn_fwd_simt<T, D>, (size_t)(smem)); e != cudaSuccess) return e;
  const int R = a.I * c.g;
  dim3 grid((R + kTile - 1) / kTile, c.nsamples * c.Hkv);
  ProfileScope prof(kAttnFwd, st);
  attn_fwd_simt<T, D><<<grid, kThreads, smem, st>>>(c, a);
  count_launch();
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch_score_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  const size_t smem = sizeof(float) * (2 * kTile * (D + 1) + 16 * kTile + kTile);
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(score_simt<T, D>, (size_t)(smem)); e != cudaSuccess) return e;
  dim3 grid((c.n_old + a.I + kTile - 1) / kTile, c.nsamples * c.Hkv);
  ProfileScope prof(kScore, st);
  score_simt<T, D><<<grid, kThreads, smem, st>>>(c, a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_simt(int dtype, int d, const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  if (dtype == 0 && d == 64) return launch_attn_t<float, 64>(c, a, st);
  if (dtype == 0 && d == 128) return launch_attn_t<float, 128>(c, a, st);
  if (dtype == 1 && d == 64) return launch_attn_t<__nv_bfloat16, 64>(c, a, st);
  if (dtype == 1 && d == 128) return launch_attn_t<__nv_bfloat16, 128>(c, a, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_score_simt(int dtype, int d, const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  if (dtype == 0 && d == 64) return launch_score_t<float, 64>(c, a, st);
  if (dtype == 0 && d == 128) return launch_score_t<float, 128>(c, a, st);
  if (dtype == 1 && d == 64) return launch_score_t<__nv_bfloat16, 64>(c, a, st);
  if (dtype == 1 && d == 128) return launch_score_t<__nv_bfloat16, 128>(c, a, st);
  return cudaErrorInvalidValue;
}

}  // namespace bm
