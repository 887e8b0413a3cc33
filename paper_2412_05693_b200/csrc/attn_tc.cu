// bf16 tensor-core path of the block forward pass (Sec. 3.2) for sm_100a:
//   attn_fwd_tc : out = softmax(scale q k^T) v over the cached pairs and the block's causal pairs, plus the
//                 log2-sum-exp of every query row.  QK^T and PV run on tcgen05 with TMA-staged tiles and
//                 TMEM accumulators; a warp-specialised CTA (TMA producer / MMA issuer / 4 softmax warps)
//                 handles one tile of 128 query rows.
//   score_tc    : sum_weights += sum_i attn_weights[i].  Recomputes the transposed logits S^T = K Q^T so that
//                 a TMEM lane is a key; each thread then sums exp2(s - lse) over the queries of its own key
//                 in a fixed order (deterministic, no atomics).
// Query rows of a (sample, kv-head) unit are ordered r = i * g + h (input i, head h of the group), so one
// tile of 128 rows shares every K/V tile it loads among the g heads of the group.
#include "tc_common.cuh"
#include "common.cuh"

namespace bm {
namespace {

using namespace tc;

constexpr int kTileM = 128;      // query rows per CTA tile
constexpr int kTileN = 128;      // keys per tile
constexpr int kFwdThreads = 192; // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: softmax / epilogue
constexpr int kStages = 2;       // K/V ring depth
constexpr int kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;  // stale row max is kept until the true max exceeds it by 2^8

struct TcMaps {
  CUtensorMap q;       // 5-d: (d, g, Hkv, I, nsamples)
  CUtensorMap k_slab;  // 3-d: (d, n_old, units)
  CUtensorMap v_slab;
  CUtensorMap k_blk;   // 4-d: (d, Hkv, I, nsamples)
  CUtensorMap v_blk;
};

struct TcArgs {
  int n_old, I, g, Hq, Hkv;
  float scale_log2;  // softmax scale * log2(e)
  void* out;
  float* lse2;       // [units][I*g] log2-sum-exp (log2 domain, scaled logits)
  float* sum_weights;
  float* new_sum;
  int cap;
  int* status;
};

template <int D>
struct FwdSmem {
  static constexpr int kChunks = D / 64;                 // 64-element (128-byte) column chunks per row
  static constexpr int kTileBytes = kChunks * 16384;     // 128 rows x D bf16
  static constexpr int kQ = 0;
  static constexpr int kK = kQ + kTileBytes;
  static constexpr int kV = kK + kStages * kTileBytes;
  static constexpr int kP = kV + kStages * kTileBytes;   // 128 x 128 bf16 probabilities
  static constexpr int kBars = kP + 2 * 16384;
  static constexpr int kTotal = kBars + 256 + 1024;      // + barriers + alignment slack
};

// barrier indices
enum { B_QFULL = 0, B_KFULL = 1, B_VFULL = B_KFULL + kStages, B_KVEMPTY = B_VFULL + kStages,
       B_SFULL = B_KVEMPTY + kStages, B_SFREE = B_SFULL + 2, B_PFULL = B_SFREE + 2, B_PVDONE = B_PFULL + 1,
       B_COUNT = B_PVDONE + 1 };

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_tc(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = FwdSmem<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.y, smp = unit / a.Hkv, kh = unit % a.Hkv;
  const int R = a.I * a.g;
  const int row0 = blockIdx.x * kTileM;
  const int qpt = kTileM / a.g;                  // inputs (positions) covered by one row tile
  const int i0 = blockIdx.x * qpt;
  const int i_last = min(a.I - 1, i0 + qpt - 1);
  const int t_old = (a.n_old + kTileN - 1) / kTileN;
  const int t_new = i_last / kTileN + 1;
  const int T = t_old + t_new;

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(&bars[B_QFULL], 1);
    for (int s = 0; s < kStages; ++s) { mbar_init(&bars[B_KFULL + s], 1); mbar_init(&bars[B_VFULL + s], 1); mbar_init(&bars[B_KVEMPTY + s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars[B_SFULL + b], 1); mbar_init(&bars[B_SFREE + b], 128); }
    mbar_init(&bars[B_PFULL], 128);
    mbar_init(&bars[B_PVDONE], 1);
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s[2] = {tmem, tmem + 128};
  const uint32_t tm_o = tmem + 256;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(&bars[B_QFULL], L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c)
        tma_load_5d(sm + L::kQ + c * 16384, &maps.q, c * 64, 0, kh, i0, smp, &bars[B_QFULL]);
      for (int j = 0; j < T; ++j) {
        const int s = j % kStages;
        if (j >= kStages) mbar_wait(&bars[B_KVEMPTY + s], ((j / kStages) - 1) & 1, abort_flag, a.status);
        unsigned char* kd = sm + L::kK + s * L::kTileBytes;
        unsigned char* vd = sm + L::kV + s * L::kTileBytes;
        mbar_expect_tx(&bars[B_KFULL + s], L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          if (j < t_old) tma_load_3d(kd + c * 16384, &maps.k_slab, c * 64, j * kTileN, unit, &bars[B_KFULL + s]);
          else tma_load_4d(kd + c * 16384, &maps.k_blk, c * 64, kh, (j - t_old) * kTileN, smp, &bars[B_KFULL + s]);
        }
        mbar_expect_tx(&bars[B_VFULL + s], L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          if (j < t_old) tma_load_3d(vd + c * 16384, &maps.v_slab, c * 64, j * kTileN, unit, &bars[B_VFULL + s]);
          else tma_load_4d(vd + c * 16384, &maps.v_blk, c * 64, kh, (j - t_old) * kTileN, smp, &bars[B_VFULL + s]);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one thread)
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(kTileM, kTileN, 0, 0);
      const uint32_t idesc_pv = instr_desc(kTileM, D, 0, 1);  // V is MN-major: d contiguous, keys along K
      const uint32_t q_addr = smem_u32(sm + L::kQ), p_addr = smem_u32(sm + L::kP);
      auto issue_pv = [&](int i) {
        const int s = i % kStages;
        mbar_wait(&bars[B_VFULL + s], (i / kStages) & 1, abort_flag, a.status);
        mbar_wait(&bars[B_PFULL], i & 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t v_addr = smem_u32(sm + L::kV + s * L::kTileBytes);
#pragma unroll
        for (int ks = 0; ks < kTileN / 16; ++ks) {
          const uint64_t da = smem_desc(p_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(v_addr + ks * 2048, 16384, 1024);
          mma_ss(tm_o, da, db, idesc_pv, (i > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(&bars[B_PVDONE]);
        mma_commit(&bars[B_KVEMPTY + s]);
      };
      mbar_wait(&bars[B_QFULL], 0, abort_flag, a.status);
      for (int j = 0; j < T; ++j) {
        const int s = j % kStages, b = j & 1;
        mbar_wait(&bars[B_KFULL + s], (j / kStages) & 1, abort_flag, a.status);
        if (j >= 2) mbar_wait(&bars[B_SFREE + b], ((j >> 1) - 1) & 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t k_addr = smem_u32(sm + L::kK + s * L::kTileBytes);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t da = smem_desc(q_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(k_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
          mma_ss(tm_s[b], da, db, idesc_qk, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[B_SFULL + b]);
        if (j >= 1) issue_pv(j - 1);
      }
      issue_pv(T - 1);
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue: thread = query row
    const int quad = warp & 3;
    const int r = quad * 32 + lane;               // row inside the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int row = row0 + r;
    const int i_row = min(a.I - 1, i0 + r / a.g);  // rows past the block's end behave like its last input
    float m_used = -INFINITY, l = 0.f;
    unsigned char* sP = sm + L::kP;
    for (int j = 0; j < T; ++j) {
      const int b = j & 1;
      mbar_wait(&bars[B_SFULL + b], (j >> 1) & 1, abort_flag, a.status);
      tc_fence_after();
      float sv[kTileN];
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t raw[32];
        tmem_ld32(tm_s[b] + lane_addr + cc * 32, raw);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) sv[cc * 32 + e] = __uint_as_float(raw[e]);
      }
      tc_fence_before();
      mbar_arrive(&bars[B_SFREE + b]);
      // number of visible columns of this tile for this row
      const int nvis = (j < t_old) ? min(kTileN, a.n_old - j * kTileN)
                                   : max(0, min(kTileN, i_row - (j - t_old) * kTileN + 1));
      float mx = -INFINITY;
#pragma unroll
      for (int e = 0; e < kTileN; ++e) mx = fmaxf(mx, e < nvis ? sv[e] : -INFINITY);
      const float mx2 = mx * a.scale_log2;
      float alpha = 1.f;
      bool rescale = false;
      if (j == 0) m_used = mx2;
      else if (mx2 > m_used + kRescaleThreshold) { alpha = ex2(m_used - mx2); m_used = mx2; rescale = true; }
      if (j > 0) {
        if (__any_sync(0xffffffffu, rescale)) {
          // O is only safe to touch once the previous P V product has completed
          mbar_wait(&bars[B_PVDONE], (j - 1) & 1, abort_flag, a.status);
          tc_fence_after();
#pragma unroll
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t raw[32];
            tmem_ld32(tm_o + lane_addr + cc * 32, raw);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) raw[e] = __float_as_uint(__uint_as_float(raw[e]) * alpha);
            tmem_st32(tm_o + lane_addr + cc * 32, raw);
          }
          tmem_wait_st();
          l *= alpha;
        }
      }
      float psum = 0.f;
#pragma unroll
      for (int e = 0; e < kTileN; ++e) {
        const float p = e < nvis ? ex2(fmaf(sv[e], a.scale_log2, -m_used)) : 0.f;
        sv[e] = p;
        psum += p;
      }
      l += psum;
      if (j > 0) mbar_wait(&bars[B_PVDONE], (j - 1) & 1, abort_flag, a.status);  // previous product done with sP
#pragma unroll
      for (int pc = 0; pc < kTileN / 8; ++pc) {
        uint4 w;
        w.x = pack_bf16(sv[pc * 8 + 0], sv[pc * 8 + 1]);
        w.y = pack_bf16(sv[pc * 8 + 2], sv[pc * 8 + 3]);
        w.z = pack_bf16(sv[pc * 8 + 4], sv[pc * 8 + 5]);
        w.w = pack_bf16(sv[pc * 8 + 6], sv[pc * 8 + 7]);
        *reinterpret_cast<uint4*>(sP + (pc >> 3) * 16384 + sw128_offset(r, pc & 7)) = w;
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(&bars[B_PFULL]);
    }
    // epilogue: O / l -> bf16, log2-sum-exp
    mbar_wait(&bars[B_PVDONE], (T - 1) & 1, abort_flag, a.status);
    tc_fence_after();
    const float inv = 1.f / l;
    const bool live = row < R;
    const int ii = row / a.g, hh = row % a.g;
    __nv_bfloat16* op = reinterpret_cast<__nv_bfloat16*>(a.out) + ((size_t)(smp * a.I + ii) * a.Hq + kh * a.g + hh) * D;
#pragma unroll
    for (int cc = 0; cc < D / 32; ++cc) {
      uint32_t raw[32];
      tmem_ld32(tm_o + lane_addr + cc * 32, raw);
      tmem_wait_ld();
      if (live) {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint4 w;
          w.x = pack_bf16(__uint_as_float(raw[q4 * 8 + 0]) * inv, __uint_as_float(raw[q4 * 8 + 1]) * inv);
          w.y = pack_bf16(__uint_as_float(raw[q4 * 8 + 2]) * inv, __uint_as_float(raw[q4 * 8 + 3]) * inv);
          w.z = pack_bf16(__uint_as_float(raw[q4 * 8 + 4]) * inv, __uint_as_float(raw[q4 * 8 + 5]) * inv);
          w.w = pack_bf16(__uint_as_float(raw[q4 * 8 + 6]) * inv, __uint_as_float(raw[q4 * 8 + 7]) * inv);
          *reinterpret_cast<uint4*>(op + cc * 32 + q4 * 8) = w;
        }
      }
    }
    if (live) a.lse2[(size_t)unit * R + row] = m_used + log2f(l);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------------
// Score pass.  CTA = (tile of 128 candidate keys, unit).  A = the key tile (loaded once), B = the unit's query
// tiles streamed through a ring; S^T lands in TMEM with lane = key, column = query row.
constexpr int kScoreThreads = 192;
constexpr int kQStages = 3;

template <int D>
struct ScoreSmem {
  static constexpr int kChunks = D / 64;
  static constexpr int kTileBytes = kChunks * 16384;
  static constexpr int kK = 0;
  static constexpr int kQ = kK + kTileBytes;
  static constexpr int kLse = kQ + kQStages * kTileBytes;      // 2 x 128 floats
  static constexpr int kBars = kLse + 2 * 128 * 4;
  static constexpr int kTotal = kBars + 256 + 1024;
};
enum { C_KFULL = 0, C_QFULL = 1, C_QEMPTY = C_QFULL + kQStages, C_SFULL = C_QEMPTY + kQStages, C_SFREE = C_SFULL + 2,
       C_COUNT = C_SFREE + 2 };

template <int D>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_tc(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = ScoreSmem<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sLse = reinterpret_cast<float*>(sm + L::kLse);

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

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(&bars[C_KFULL], 1);
    for (int s = 0; s < kQStages; ++s) { mbar_init(&bars[C_QFULL + s], 1); mbar_init(&bars[C_QEMPTY + s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars[C_SFULL + b], 1); mbar_init(&bars[C_SFREE + b], 128); }
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(tmem_slot, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s[2] = {tmem, tmem + 128};

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(&bars[C_KFULL], L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c) {
        if (is_old) tma_load_3d(sm + L::kK + c * 16384, &maps.k_slab, c * 64, kt * kTileN, unit, &bars[C_KFULL]);
        else tma_load_4d(sm + L::kK + c * 16384, &maps.k_blk, c * 64, kh, c0, smp, &bars[C_KFULL]);
      }
      for (int t = 0; t < T; ++t) {
        const int s = t % kQStages;
        if (t >= kQStages) mbar_wait(&bars[C_QEMPTY + s], ((t / kQStages) - 1) & 1, abort_flag, a.status);
        mbar_expect_tx(&bars[C_QFULL + s], L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c)
          tma_load_5d(sm + L::kQ + s * L::kTileBytes + c * 16384, &maps.q, c * 64, 0, kh, (qt0 + t) * qpt, smp,
                      &bars[C_QFULL + s]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kTileN, kTileM, 0, 0);
      const uint32_t k_addr = smem_u32(sm + L::kK);
      mbar_wait(&bars[C_KFULL], 0, abort_flag, a.status);
      for (int t = 0; t < T; ++t) {
        const int s = t % kQStages, b = t & 1;
        mbar_wait(&bars[C_QFULL + s], (t / kQStages) & 1, abort_flag, a.status);
        if (t >= 2) mbar_wait(&bars[C_SFREE + b], ((t >> 1) - 1) & 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t q_addr = smem_u32(sm + L::kQ + s * L::kTileBytes);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t da = smem_desc(k_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc(q_addr + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
          mma_ss(tm_s[b], da, db, idesc, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[C_SFULL + b]);
        mma_commit(&bars[C_QEMPTY + s]);
      }
    }
  } else {
    const int quad = warp & 3;
    const int key = quad * 32 + lane;              // key inside the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int t128 = tid - 64;                     // 0..127 among the reducer threads
    float acc = 0.f;
    for (int t = 0; t < T; ++t) {
      const int b = t & 1;
      const int qrow0 = (qt0 + t) * kTileM;
      // this tile's log2-sum-exp values; +inf for rows past the block's end (weight 0)
      {
        const int rr = qrow0 + t128;
        sLse[b * 128 + t128] = rr < R ? a.lse2[(size_t)unit * R + rr] : INFINITY;
      }
      named_bar_sync(1, 128);
      mbar_wait(&bars[C_SFULL + b], (t >> 1) & 1, abort_flag, a.status);
      tc_fence_after();
      // first query row of the tile that may see this key (causal mask inside the block)
      const int first_vis = is_old ? 0 : max(0, (c0 + key) * a.g - qrow0);
      float part = 0.f;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t raw[32];
        tmem_ld32(tm_s[b] + lane_addr + cc * 32, raw);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int col = cc * 32 + e;
          const float p = ex2(fmaf(__uint_as_float(raw[e]), a.scale_log2, -sLse[b * 128 + col]));
          part += col >= first_vis ? p : 0.f;
        }
      }
      acc += part;
      tc_fence_before();
      mbar_arrive(&bars[C_SFREE + b]);
    }
    const int j = is_old ? kt * kTileN + key : c0 + key;
    if (is_old) { if (j < a.n_old) a.sum_weights[(size_t)unit * a.cap + j] += acc; }
    else if (j < a.I) a.new_sum[(size_t)unit * a.I + j] = acc;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256);
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

// Tensor maps of one call.  Rows past n_old (slab) or past I (block, queries) read as zeros.
bool build_maps(int d, const CacheView& c, const BlockArgs& a, TcMaps* m) {
  const cuuint64_t D = (cuuint64_t)d, e = 2;
  const cuuint64_t units = (cuuint64_t)c.nsamples * c.Hkv;
  {
    cuuint64_t dims[5] = {D, (cuuint64_t)c.g, (cuuint64_t)c.Hkv, (cuuint64_t)a.I, (cuuint64_t)c.nsamples};
    cuuint64_t str[4] = {D * e, (cuuint64_t)c.g * D * e, (cuuint64_t)c.Hq * D * e, (cuuint64_t)a.I * c.Hq * D * e};
    cuuint32_t box[5] = {64, (cuuint32_t)c.g, 1, (cuuint32_t)(kTileM / c.g), 1};
    if (!encode(&m->q, a.q, 5, dims, str, box)) return false;
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
  t.out = a.out; t.lse2 = a.lse; t.sum_weights = c.sum_weights; t.new_sum = a.new_sum;
  t.cap = c.cap; t.status = c.status;
  return t;
}

// maps of the call in flight: built by the forward launcher, reused by the score launcher
TcMaps g_maps;
const void* g_maps_q = nullptr;

template <int D>
cudaError_t launch_fwd_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int R = a.I * c.g;
  dim3 grid((R + kTileM - 1) / kTileM, c.nsamples * c.Hkv);
  ProfileScope prof(kAttnFwd, st);
  attn_fwd_tc<D><<<grid, kFwdThreads, FwdSmem<D>::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_score_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(score_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScoreSmem<D>::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int t_old = (c.n_old + kTileN - 1) / kTileN, t_new = (a.I + kTileN - 1) / kTileN;
  dim3 grid(t_old + t_new, c.nsamples * c.Hkv);
  ProfileScope prof(kScore, st);
  score_tc<D><<<grid, kScoreThreads, ScoreSmem<D>::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
}

}  // namespace

bool tc_path_available() { return encode_fn() != nullptr; }

cudaError_t launch_attn_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used) {
  *used = 0;
  g_maps_q = nullptr;
  if (!(d == 64 || d == 128) || c.g > 8 || (kTileM % c.g) != 0) return cudaSuccess;
  if (!build_maps(d, c, a, &g_maps)) return cudaSuccess;  // fall back to the SIMT kernels
  g_maps_q = a.q;
  *used = 1;
  return d == 64 ? launch_fwd_t<64>(c, a, st) : launch_fwd_t<128>(c, a, st);
}

cudaError_t launch_score_tc(int d, const CacheView& c, const BlockArgs& a, cudaStream_t st, int* used) {
  *used = 0;
  if (g_maps_q != a.q) return cudaSuccess;  // the forward pass of this call did not take the tensor-core path
  *used = 1;
  return d == 64 ? launch_score_t<64>(c, a, st) : launch_score_t<128>(c, a, st);
}

}  // namespace bm
