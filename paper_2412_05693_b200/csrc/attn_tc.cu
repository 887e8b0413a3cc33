// bf16 tensor-core path of the block forward pass (Sec. 3.2) for sm_100a:
//   attn_fwd_split (attn_fwd_split.cuh): out = softmax(scale q k^T) v over the cached pairs and the block's causal
//                 pairs, plus the log2-sum-exp of every query row.  QK^T and PV run on tcgen05 with TMA-staged
//                 tiles and TMEM accumulators; one CTA owns one tile of 128 query rows, two CTAs share an SM.
//   score_tc    : sum_weights += sum_i attn_weights[i].  Recomputes the transposed logits S^T = K Q^T so that
//                 a TMEM lane is a key; each thread then sums exp2(s - lse) over the queries of its own key
//                 in a fixed order (deterministic, no atomics).
// Query rows of a unit are ordered r = i * g + h (input i, head h of the group), so a tile of 128 rows shares
// its K/V tiles among the g heads of the group.
#include <type_traits>

#include "tc_common.cuh"
#include "common.cuh"

namespace bm {
namespace {

using namespace tc;

constexpr int kTileM = 128;      // query rows per tile
constexpr int kTileN = 128;      // keys per tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // stale row max is kept until the true max exceeds it by 2^8

struct TcMaps {
  CUtensorMap q;       // 5-d: (d, g, Hkv, I, nsamples)
  CUtensorMap o;       // same shape over the output
  CUtensorMap k_slab;  // 3-d: (d, n_old, units)
  CUtensorMap v_slab;
  CUtensorMap k_blk;   // 4-d: (d, Hkv, I, nsamples)
  CUtensorMap v_blk;
};

struct TcArgs {
  int n_old, I, g, Hq, Hkv;
  float scale_log2;  // softmax scale * log2(e)
  float* lse2;       // [units][I*g] log2-sum-exp (log2 domain, scaled logits)
  float* sum_weights;
  float* new_sum;
  int cap;
  int* status;
  // left-padded samples: padding counts of the range's samples (null: none), cached ids, the block's first position
  const int* left_pad;
  const int* kv_ids;
  int pos0;
  int rule;
  int first_row;     // query rows below it add nothing to the column sums (rules that look at the last queries only)
  int overwrite;     // 1: the column sums replace sum_weights instead of being added
  float* sum_sq;     // rule 4: sums of squared weights (cached pairs / the block's pairs), else null
  float* new_sq;
};

#include "attn_fwd_split.cuh"
#include "attn_onepass.cuh"

// ------------------------------------------------------------------------------------------------------
// Score pass.  CTA = (tile of 128 candidate keys, unit).  A = the key tile (loaded once), B = the unit's query
// tiles streamed through a ring; S^T lands in TMEM with lane = key, column = query row.  The pass is bound by
// one exponential per visible pair, so two reducer warpgroups (one TMEM buffer each, query tiles taken round
// robin) keep the special-function units busy; their partial sums are added in a fixed order.
constexpr int kScoreWG = 2;                              // reducer warpgroups == TMEM buffers of 128 columns
constexpr int kScoreThreads = 128 * kScoreWG + 64;       // + warp 4*WG: MMA + TMEM owner, warp 4*WG+1: TMA
constexpr int kQStages = 2;

template <int D>
struct ScoreSmem {
  static constexpr int kChunks = D / 64;
  static constexpr int kTileBytes = kChunks * 16384;
  static constexpr int kK = 0;
  static constexpr int kQ = kK + kTileBytes;
  static constexpr int kLse = kQ + kQStages * kTileBytes;      // [WG][128] floats
  static constexpr int kPart = kLse + kScoreWG * 128 * 4;      // [WG][128] floats: partial sums
  static constexpr int kBars = kPart + kScoreWG * 128 * 4;
  static constexpr int kTotal = kBars + 256 + 1024;
};
enum { C_KFULL = 0, C_QFULL = 1, C_QEMPTY = C_QFULL + kQStages, C_SFULL = C_QEMPTY + kQStages,
       C_SFREE = C_SFULL + kScoreWG, C_COUNT = C_SFREE + kScoreWG };

// SQ: the sums of squared weights are taken as well (rule 4; an instance of its own, so that the others carry none of it)
template <int D, bool SQ, int EMU>
__global__ void __launch_bounds__(kScoreThreads, 2)
score_tc(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = ScoreSmem<D>;
  constexpr int kMmaWarp = 4 * kScoreWG, kTmaWarp = 4 * kScoreWG + 1;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sLse = reinterpret_cast<float*>(sm + L::kLse);
  float* sPart = reinterpret_cast<float*>(sm + L::kPart);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.y, smp = unit / a.Hkv, kh = unit % a.Hkv;
  const int R = a.I * a.g;
  const int t_old = (a.n_old + kTileN - 1) / kTileN;
  const int kt = blockIdx.x;                       // key tile: old tiles first, then the block's own
  const bool is_old = kt < t_old;
  const int c0 = is_old ? 0 : (kt - t_old) * kTileN;  // first block position of a new-key tile
  const int qpt = kTileM / a.g;
  const int n_qt = (R + kTileM - 1) / kTileM;
  const int qt0 = is_old ? 0 : c0 / qpt;           // earlier query tiles cannot see these keys
  const int T = n_qt - qt0;

  auto load_k = [&]() {
    mbar_expect_tx(&bars[C_KFULL], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c) {
      if (is_old) tma_load_3d(sm + L::kK + c * 16384, &maps.k_slab, c * 64, kt * kTileN, unit, &bars[C_KFULL]);
      else tma_load_4d(sm + L::kK + c * 16384, &maps.k_blk, c * 64, kh, c0, smp, &bars[C_KFULL]);
    }
  };
  auto load_q = [&](int t) {
    const int s = t % kQStages;
    mbar_expect_tx(&bars[C_QFULL + s], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c)
      tma_load_5d(sm + L::kQ + s * L::kTileBytes + c * 16384, &maps.q, c * 64, 0, kh, (qt0 + t) * qpt, smp,
                  &bars[C_QFULL + s]);
  };
  if (warp == kTmaWarp && lane == 0) {   // barriers and the first loads before the CTA-wide barrier (overlaps TMEM allocation)
    *abort_flag = 0;
    mbar_init(&bars[C_KFULL], 1);
    for (int s = 0; s < kQStages; ++s) { mbar_init(&bars[C_QFULL + s], 1); mbar_init(&bars[C_QEMPTY + s], 1); }
    for (int b = 0; b < kScoreWG; ++b) { mbar_init(&bars[C_SFULL + b], 1); mbar_init(&bars[C_SFREE + b], 128); }
    mbar_fence_init();
    load_k();
    for (int t = 0; t < min(kQStages, T); ++t) load_q(t);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, 128 * kScoreWG);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == kTmaWarp) {
    if (lane == 0) {
      for (int t = kQStages; t < T; ++t) {
        mbar_wait(&bars[C_QEMPTY + t % kQStages], ((t / kQStages) - 1) & 1, abort_flag, a.status);
        load_q(t);
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kTileN, kTileM, 0, 0);
      const uint64_t d_hi = smem_desc(0, 16, 1024) & 0xffffffff00000000ull;
      const uint32_t d_lo = (uint32_t)(smem_desc(0, 16, 1024) & 0xffffffffull);
      const uint32_t k_lo = d_lo + (smem_u32(sm + L::kK) >> 4);
      mbar_wait(&bars[C_KFULL], 0, abort_flag, a.status);
      for (int t = 0; t < T; ++t) {
        const int s = t % kQStages, b = t % kScoreWG;
        mbar_wait(&bars[C_QFULL + s], (t / kQStages) & 1, abort_flag, a.status);
        if (t >= kScoreWG) mbar_wait(&bars[C_SFREE + b], ((t / kScoreWG) - 1) & 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t q_lo = d_lo + ((smem_u32(sm + L::kQ) >> 4) + s * (L::kTileBytes >> 4));
        const uint32_t ts = tmem + b * 128;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {   // only the start-address word of the descriptors changes
          const uint32_t off = (ks >> 2) * 1024 + (ks & 3) * 2;
          mma_ss(ts, d_hi | (k_lo + off), d_hi | (q_lo + off), idesc, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[C_SFULL + b]);
        mma_commit(&bars[C_QEMPTY + s]);
      }
    }
  } else {
    const int wg = warp >> 2;                      // reducer warpgroup: takes query tiles t = wg, wg + WG, ...
    const int quad = warp & 3;
    const int key = quad * 32 + lane;              // key inside the tile == TMEM lane
    const uint32_t ts = tmem + wg * 128 + ((uint32_t)(quad * 32) << 16);
    const float* lse_w = sLse + wg * 128;
    float acc = 0.f, acc_sq = 0.f;
    for (int t = wg; t < T; t += kScoreWG) {
      const int qrow0 = (qt0 + t) * kTileM;
      // this tile's log2-sum-exp values; +inf for rows past the block's end (weight 0)
      {
        const int rr = qrow0 + key;
        sLse[wg * 128 + key] = (rr < R && rr >= a.first_row) ? a.lse2[(size_t)unit * R + rr] : INFINITY;
      }
      named_bar_sync(1 + wg, 128);
      mbar_wait(&bars[C_SFULL + wg], (t / kScoreWG) & 1, abort_flag, a.status);
      tc_fence_after();
      // first query row of the tile that may see this key (causal mask inside the block)
      const int first_vis = is_old ? 0 : max(0, (c0 + key) * a.g - qrow0);
      const bool nomask = __all_sync(0xffffffffu, first_vis == 0);
      float p0 = 0.f, p1 = 0.f, q0 = 0.f, q1 = 0.f;
      // (the loop exists with and without the causal mask: as one loop with a test inside, the compiler evaluated
      // the mask of every tile, two more instructions per exponential)
      auto reduce_tile = [&](auto masked) {
        uint32_t cur[32], nxt[32];
        tmem_ld32(ts, cur);
        tmem_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          if (cc < 3) tmem_ld32(ts + (cc + 1) * 32, nxt);   // next chunk loads while this one is used
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const int col = cc * 32 + e;
            float x0, x1;
            fma2v(x0, x1, __uint_as_float(cur[e]), __uint_as_float(cur[e + 1]), a.scale_log2, -lse_w[col], -lse_w[col + 1]);
            float e0, e1;
            if (EMU > 0 && ((e >> 1) % EMU) == EMU - 1) ex2_poly2(x0, x1, e0, e1);   // a share of the pairs off the special-function unit
            else { e0 = ex2(x0); e1 = ex2(x1); }
            if (decltype(masked)::value) {
              e0 = col >= first_vis ? e0 : 0.f;
              e1 = col + 1 >= first_vis ? e1 : 0.f;
            }
            add2(p0, p1, e0, e1);
            if (SQ) { q0 = fmaf(e0, e0, q0); q1 = fmaf(e1, e1, q1); }
          }
          if (cc < 3) {
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) cur[e] = nxt[e];
          }
        }
      };
      if (nomask) reduce_tile(std::false_type{});
      else reduce_tile(std::true_type{});
      acc += p0 + p1;
      if (SQ) acc_sq += q0 + q1;
      tc_fence_before();
      mbar_arrive(&bars[C_SFREE + wg]);
      named_bar_sync(1 + wg, 128);                 // everyone is done with this tile's sLse before it is rewritten
    }
    sPart[wg * 128 + key] = acc;
    if (SQ) sLse[wg * 128 + key] = acc_sq;         // (the last tile's values are no longer needed: barrier above)
    named_bar_sync(1 + kScoreWG, 128 * kScoreWG);
    if (wg == 0) {
      float tot = 0.f, tot_sq = 0.f;
#pragma unroll
      for (int w = 0; w < kScoreWG; ++w) tot += sPart[w * 128 + key];   // fixed order
      if (SQ) {
#pragma unroll
        for (int w = 0; w < kScoreWG; ++w) tot_sq += sLse[w * 128 + key];
      }
      const int j = is_old ? kt * kTileN + key : c0 + key;
      if (a.left_pad != nullptr) {                  // a padding pair is masked for every query
        const int pad = a.left_pad[smp];
        const bool in_range = is_old ? j < a.n_old : j < a.I;
        if (pad > 0 && in_range && (is_old ? a.kv_ids[(size_t)unit * a.cap + j] : a.pos0 + j) < pad) tot = 0.f;
      }
      if (is_old) {
        if (j < a.n_old) {
          if (a.overwrite) a.sum_weights[(size_t)unit * a.cap + j] = tot;   // nothing is carried over
          else a.sum_weights[(size_t)unit * a.cap + j] += tot;
          if (SQ) a.sum_sq[(size_t)unit * a.cap + j] += tot_sq;
        }
      }
      else if (j < a.I) {
        a.new_sum[(size_t)unit * a.I + j] = tot;
        if (SQ) a.new_sq[(size_t)unit * a.I + j] = tot_sq;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem, 128 * kScoreWG);
}

// ------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool encode(CUtensorMap* m, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
            const cuuint32_t* box) {
  cuuint32_t es[5] = {1, 1, 1, 1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes,
                     box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps of one call.  Rows past n_old (slab) or past I (block, queries) read as zeros; output rows past I
// are clipped.
bool build_maps(int d, const CacheView& c, const BlockArgs& a, TcMaps* m) {
  const cuuint64_t D = (cuuint64_t)d, e = 2;
  const cuuint64_t units = (cuuint64_t)c.nsamples * c.Hkv;
  {
    cuuint64_t dims[5] = {D, (cuuint64_t)c.g, (cuuint64_t)c.Hkv, (cuuint64_t)a.I, (cuuint64_t)c.nsamples};
    cuuint64_t str[4] = {D * e, (cuuint64_t)c.g * D * e, (cuuint64_t)c.Hq * D * e, (cuuint64_t)a.I * c.Hq * D * e};
    cuuint32_t box[5] = {64, (cuuint32_t)c.g, 1, (cuuint32_t)(kTileM / c.g), 1};
    if (!encode(&m->q, a.q, 5, dims, str, box)) return false;
    if (!encode(&m->o, a.out, 5, dims, str, box)) return false;
  }
  {
    cuuint64_t dims[3] = {D, (cuuint64_t)(c.n_old > 0 ? c.n_old : 1), units};
    cuuint64_t str[2] = {D * e, (cuuint64_t)c.cap * D * e};
    cuuint32_t box[3] = {64, kTileN, 1};
    if (!encode(&m->k_slab, c.k_slab, 3, dims, str, box)) return false;
    if (!encode(&m->v_slab, c.v_slab, 3, dims, str, box)) return false;
  }
  {
    cuuint64_t dims[4] = {D, (cuuint64_t)c.Hkv, (cuuint64_t)a.I, (cuuint64_t)c.nsamples};
    cuuint64_t str[3] = {D * e, (cuuint64_t)c.Hkv * D * e, (cuuint64_t)a.I * c.Hkv * D * e};
    cuuint32_t box[4] = {64, 1, kTileN, 1};
    if (!encode(&m->k_blk, a.k, 4, dims, str, box)) return false;
    if (!encode(&m->v_blk, a.v, 4, dims, str, box)) return false;
  }
  return true;
}

TcArgs make_args(const CacheView& c, const BlockArgs& a) {
  TcArgs t;
  t.n_old = c.n_old; t.I = a.I; t.g = c.g; t.Hq = c.Hq; t.Hkv = c.Hkv;
  t.scale_log2 = a.scale * kLog2e;
  t.lse2 = a.lse; t.sum_weights = c.sum_weights; t.new_sum = a.new_sum;
  t.cap = c.cap; t.status = c.status;
  t.left_pad = c.left_pad; t.kv_ids = c.kv_ids; t.pos0 = a.pos0; t.rule = c.rule;
  t.first_row = rule_first_counted_row(c.rule, c.window, a.I, c.g);
  t.overwrite = rule_overwrites(c.rule) ? 1 : 0;
  t.sum_sq = c.sum_sq; t.new_sq = a.new_sq;
  return t;
}

// maps of the call in flight: built by the forward launcher, reused by the score launcher
thread_local TcMaps g_maps;            // per thread: handles used from different threads do not share them
thread_local const void* g_maps_q = nullptr;

template <int D, bool PAD>
cudaError_t launch_fwd_split(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  using L = SplitSmem<D>;
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(attn_fwd_split<D, PAD>, (size_t)(L::kTotal)); e != cudaSuccess) return e;
  const int R = a.I * c.g;
  dim3 grid((R + kTileM - 1) / kTileM, c.nsamples * c.Hkv);
  ProfileScope prof(kAttnFwd, st);
  attn_fwd_split<D, PAD><<<grid, L::kThreads, L::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
}

// the forward launch of the call in flight has taken the column sums as well: no score pass follows
thread_local bool g_scores_done = false;

// A block of at most one tile of query rows against at most four tiles of keys (cached + new), without padding and
// under a rule that accumulates every row's weights: forward pass and column sums in one kernel (attn_onepass.cuh).
bool onepass_applies(const CacheView& c, const BlockArgs& a) {
  const int t_old = (c.n_old + kTileN - 1) / kTileN, t_new = (a.I + kTileN - 1) / kTileN;
  return c.left_pad == nullptr && c.rule <= 1 && a.I * c.g <= kTileM && t_old + t_new <= 4;
}

template <int D>
cudaError_t launch_onepass(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  using L = OnePassSmem<D>;
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(attn_block_onepass<D>, (size_t)(L::kTotal)); e != cudaSuccess) return e;
  ProfileScope prof(kAttnFwd, st);
  attn_block_onepass<D><<<dim3(c.nsamples * c.Hkv), L::kThreads, L::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  g_scores_done = true;
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_fwd_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  if (onepass_applies(c, a)) return launch_onepass<D>(c, a, st);
  return c.left_pad != nullptr ? launch_fwd_split<D, true>(c, a, st) : launch_fwd_split<D, false>(c, a, st);
}

template <int D, bool SQ, int EMU>
cudaError_t launch_score_emu(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(score_tc<D, SQ, EMU>, (size_t)(ScoreSmem<D>::kTotal)); e != cudaSuccess) return e;
  const int t_old = (c.n_old + kTileN - 1) / kTileN, t_new = (a.I + kTileN - 1) / kTileN;
  dim3 grid(t_old + t_new, c.nsamples * c.Hkv);
  ProfileScope prof(kScore, st);
  score_tc<D, SQ, EMU><<<grid, kScoreThreads, ScoreSmem<D>::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
}
// Every fourth pair of exponentials of the score pass runs as a polynomial on the FMA and integer pipes
// (ex2_poly2): the pass is bound by the special-function unit, and a quarter is where the instruction issue the
// polynomial costs stops paying (measured at the cfg3 shape: -3.6 % at an eighth, -5.9 % at a quarter, -4.7 % at a
// third, -0.6 % at a half).
constexpr int kScoreEmu = 4;
template <int D, bool SQ>
cudaError_t launch_score_sq(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  return launch_score_emu<D, SQ, kScoreEmu>(c, a, st);
}
template <int D>
cudaError_t launch_score_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  return c.sum_sq != nullptr ? launch_score_sq<D, true>(c, a, st) : launch_score_sq<D, false>(c, a, st);
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever arrives on.  The wait gives up
// after its poll limit, records BM_ERR_TIMEOUT in the status word and the kernel ends normally.
__global__ void wait_timeout_selftest(int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { abort_flag = 0; mbar_init(&bar, 1); mbar_fence_init(); }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, &abort_flag, status, 1 << 16);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(int* status, cudaStream_t st) {
  wait_timeout_selftest<<<1, 32, 0, st>>>(status);
  count_launch();
  return cudaGetLastError();
}

bool tc_path_available() { return encode_fn() != nullptr; }

// Map over the first `rows` rows of every cache of a slab, as tiles of `box_rows` rows x 64 elements (128-byte
// swizzle); rows past `rows` read as zeros.  False when the driver's encoder is unavailable or refuses.
bool encode_slab_rows_map(CUtensorMap* m, const void* slab, int d, int rows, int cap, int units, int box_rows) {
  if (encode_fn() == nullptr) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)(rows > 0 ? rows : 1), (cuuint64_t)units};
  const cuuint64_t str[2] = {(cuuint64_t)d * 2, (cuuint64_t)cap * d * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  return encode(m, slab, 3, dims, str, box);
}

cudaError_t launch_attn_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used) {
  *used = 0;
  g_maps_q = nullptr;
  g_scores_done = false;
  if (!(d == 64 || d == 128) || c.g > 8 || (kTileM % c.g) != 0) return cudaSuccess;
  if (!build_maps(d, c, a, &g_maps)) return cudaSuccess;  // fall back to the SIMT kernels
  g_maps_q = a.q;
  *used = onepass_applies(c, a) ? 2 : 1;
  return d == 64 ? launch_fwd_t<64>(c, a, st) : launch_fwd_t<128>(c, a, st);
}

cudaError_t launch_score_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used) {
  *used = 0;
  if (g_maps_q != a.q) return cudaSuccess;  // the forward pass of this call did not take the tensor-core path
  *used = 1;
  if (g_scores_done) return cudaSuccess;    // ... or it has taken the column sums itself
  return d == 64 ? launch_score_t<64>(c, a, st) : launch_score_t<128>(c, a, st);
}

}  // namespace bm
