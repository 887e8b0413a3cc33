// bf16 tensor-core path of the block forward pass (Sec. 3.2) for sm_100a:
//   attn_fwd_tc : out = softmax(scale q k^T) v over the cached pairs and the block's causal pairs, plus the
//                 log2-sum-exp of every query row.  QK^T and PV run on tcgen05 with TMA-staged tiles and TMEM
//                 accumulators.  One CTA owns two tiles of 128 query rows of the same (sample, kv-head) unit;
//                 two softmax warpgroups work on them alternately so that one tile's exponentials overlap the
//                 other tile's MMAs, and both tiles share every K/V tile that is loaded.
//   score_tc    : sum_weights += sum_i attn_weights[i].  Recomputes the transposed logits S^T = K Q^T so that
//                 a TMEM lane is a key; each thread then sums exp2(s - lse) over the queries of its own key
//                 in a fixed order (deterministic, no atomics).
// Query rows of a unit are ordered r = i * g + h (input i, head h of the group), so a tile of 128 rows shares
// its K/V tiles among the g heads of the group.
#include <cstdlib>

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
  int rule;          // 2: only the rows of the block's last input contribute to the column sums, which replace sum_weights
};

#include "attn_fwd_split.cuh"

// ------------------------------------------------------------------------------------------------------
// Forward, NT query tiles per CTA.  NT = 2 (large grids): warps 0-3 / 4-7 are the softmax warpgroups of tiles A / B,
// warp 8 issues the MMAs and owns the tensor memory, warp 9 is the TMA producer; one CTA per SM, both tiles share
// every K/V tile.  NT = 1 (small grids): four softmax warps + MMA warp + TMA warp, half the shared and tensor
// memory, two CTAs per SM, so that one CTA's prologue and epilogue overlap the other's main loop.
// TMEM: S tiles (fp32 logits, overwritten in place by the bf16 probabilities that feed P.V as the tensor-memory
// operand), then the O accumulators.
template <int D, int NT>
struct FwdSmem {
  static constexpr int kStages = NT == 2 ? 4 : 2;        // ring of K/V tiles: entry 2j = K_j, entry 2j+1 = V_j
  static constexpr int kChunks = D / 64;                 // 64-element (128-byte) column chunks per row
  static constexpr int kTileBytes = kChunks * 16384;     // 128 rows x D bf16
  static constexpr int kQ = 0;                           // query tiles (reused to stage the outputs)
  static constexpr int kKV = kQ + NT * kTileBytes;
  static constexpr int kBars = kKV + kStages * kTileBytes;
  static constexpr int kTotal = kBars + 256 + 1024;      // + barriers + alignment slack
  static constexpr int kThreads = 128 * NT + 64;
};

// PAD: the range has left-padded samples (a separate instance, so that the common case carries none of its masks).
template <int D, int NT, bool PAD>
__global__ void __launch_bounds__(128 * NT + 64, NT == 2 ? 1 : 2)
attn_fwd_tc(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = FwdSmem<D, NT>;
  constexpr int kKvStages = L::kStages;
  constexpr int kMmaWarp = 4 * NT, kTmaWarp = 4 * NT + 1;
  constexpr int kTmemCols = 256 * NT;
  constexpr int B_QFULL = 0, B_KVFULL = 2, B_KVEMPTY = B_KVFULL + kKvStages, B_SFULL = B_KVEMPTY + kKvStages,
                B_PFULL = B_SFULL + 2, B_ODONE = B_PFULL + 2, B_COUNT = B_ODONE + 2;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* np_slot = reinterpret_cast<int*>(tmem_slot + 2);   // [2] cached padding pairs, counted per query tile

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.y, smp = unit / a.Hkv, kh = unit % a.Hkv;
  const int R = a.I * a.g;
  const int qpt = kTileM / a.g;                  // inputs (positions) covered by one row tile
  const int t_old = (a.n_old + kTileN - 1) / kTileN;
  int row0[2], i0[2], T[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    row0[x] = (blockIdx.x * NT + x) * kTileM;
    i0[x] = (blockIdx.x * NT + x) * qpt;
    const int i_last = min(a.I - 1, i0[x] + qpt - 1);
    T[x] = t_old + i_last / kTileN + 1;          // cached-key tiles + block-key tiles up to the tile's last input
  }
  const bool active_b = NT == 2 && row0[1] < R;
  if (!active_b) T[1] = 0;
  const int t_max = active_b ? T[1] : T[0];      // tile B sees at least as many key tiles as tile A

  // The producer warp initialises the barriers and starts the first loads at once; tensor-memory allocation
  // and the CTA-wide barrier below overlap their latency.
  auto load_q = [&](int x) {
    mbar_expect_tx(&bars[B_QFULL + x], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c)
      tma_load_5d(sm + L::kQ + x * L::kTileBytes + c * 16384, &maps.q, c * 64, 0, kh, i0[x], smp, &bars[B_QFULL + x]);
  };
  auto load_kv = [&](int e) {   // ring entry e: K_j for even e, V_j for odd e, j = e / 2
    const int j = e >> 1, s = e % kKvStages;
    const bool is_v = e & 1;
    unsigned char* dst = sm + L::kKV + s * L::kTileBytes;
    mbar_expect_tx(&bars[B_KVFULL + s], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c) {
      if (j < t_old)
        tma_load_3d(dst + c * 16384, is_v ? &maps.v_slab : &maps.k_slab, c * 64, j * kTileN, unit, &bars[B_KVFULL + s]);
      else
        tma_load_4d(dst + c * 16384, is_v ? &maps.v_blk : &maps.k_blk, c * 64, kh, (j - t_old) * kTileN, smp,
                    &bars[B_KVFULL + s]);
    }
  };
  if (warp == kTmaWarp && lane == 0) {
    *abort_flag = 0;
    np_slot[0] = 0;
    np_slot[1] = 0;
    for (int x = 0; x < 2; ++x) {
      mbar_init(&bars[B_QFULL + x], 1);
      mbar_init(&bars[B_SFULL + x], 1);
      mbar_init(&bars[B_PFULL + x], 128);
      mbar_init(&bars[B_ODONE + x], 1);
    }
    for (int s = 0; s < kKvStages; ++s) { mbar_init(&bars[B_KVFULL + s], 1); mbar_init(&bars[B_KVEMPTY + s], 1); }
    mbar_fence_init();
    load_q(0);
    load_kv(0);
    if (active_b) load_q(1);
    for (int e = 1; e < min(kKvStages, 2 * t_max); ++e) load_kv(e);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s[2] = {tmem, tmem + 128};
  const uint32_t tm_o[2] = {tmem + 128 * NT, tmem + 128 * NT + 128};

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int e = kKvStages; e < 2 * t_max; ++e) {
        mbar_wait(&bars[B_KVEMPTY + e % kKvStages], ((e / kKvStages) - 1) & 1, abort_flag, a.status);
        load_kv(e);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer (one thread)
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(kTileM, kTileN, 0, 0);
      const uint32_t idesc_pv = instr_desc(kTileM, D, 0, 1);  // V is MN-major: d contiguous, keys along K
      auto wait_kv = [&](int e) { mbar_wait(&bars[B_KVFULL + e % kKvStages], (e / kKvStages) & 1, abort_flag, a.status); };
      // Descriptors differ between MMAs only in the start-address field (low word, 16-byte units), so the
      // issuing thread adds small constants to precomputed words instead of rebuilding 64-bit descriptors.
      const uint64_t dk_hi = smem_desc(0, 16, 1024) & 0xffffffff00000000ull;      // K-major operands (Q, K)
      const uint32_t dk_lo = (uint32_t)(smem_desc(0, 16, 1024) & 0xffffffffull);
      const uint64_t dv_hi = smem_desc(0, 16384, 1024) & 0xffffffff00000000ull;   // MN-major operand (V)
      const uint32_t dv_lo = (uint32_t)(smem_desc(0, 16384, 1024) & 0xffffffffull);
      const uint32_t q_lo[2] = {dk_lo + (smem_u32(sm + L::kQ) >> 4), dk_lo + (smem_u32(sm + L::kQ + L::kTileBytes) >> 4)};
      const uint32_t kv_lo0 = smem_u32(sm + L::kKV) >> 4;
      auto issue_qk = [&](int x, int j) {   // S_x = Q_x K_j^T
        const uint32_t k_lo = dk_lo + kv_lo0 + ((2 * j) % kKvStages) * (L::kTileBytes >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks >> 2) * 1024 + (ks & 3) * 2;   // (chunk * 16384 + kstep * 32) / 16
          mma_ss(tm_s[x], dk_hi | (q_lo[x] + off), dk_hi | (k_lo + off), idesc_qk, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[B_SFULL + x]);
      };
      auto issue_pv = [&](int x, int j) {   // O_x += P_x V_j, P_x read from tensor memory (over S_x)
        mbar_wait(&bars[B_PFULL + x], j & 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t v_lo = dv_lo + kv_lo0 + ((2 * j + 1) % kKvStages) * (L::kTileBytes >> 4);
        const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
        for (int ks = 0; ks < kTileN / 16; ++ks)   // 16 keys = 2 row groups of 1024 bytes per step
          mma_ts(tm_o[x], tm_s[x] + ks * 8, dv_hi | (v_lo + ks * 128), idesc_pv, ks > 0 ? 1u : acc0);
        mma_commit(&bars[B_ODONE + x]);
      };
      mbar_wait(&bars[B_QFULL + 0], 0, abort_flag, a.status);
      if (active_b) mbar_wait(&bars[B_QFULL + 1], 0, abort_flag, a.status);
      wait_kv(0);
      tc_fence_after();
      issue_qk(0, 0);
      if (active_b) issue_qk(1, 0);
      mma_commit(&bars[B_KVEMPTY + 0]);
      for (int j = 1; j <= t_max; ++j) {       // products of key tile j-1, logits of key tile j
        wait_kv(2 * j - 1);
        if (j < t_max) wait_kv(2 * j);
        tc_fence_after();
        if (j - 1 < T[0]) issue_pv(0, j - 1);
        if (j < T[0]) issue_qk(0, j);
        if (active_b) {
          issue_pv(1, j - 1);
          if (j < T[1]) issue_qk(1, j);
        }
        mma_commit(&bars[B_KVEMPTY + (2 * j - 1) % kKvStages]);
        if (j < t_max) mma_commit(&bars[B_KVEMPTY + (2 * j) % kKvStages]);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue: thread = query row
    const int x = warp >> 2;                      // tile A or B
    if (x == 0 || active_b) {
      const int quad = warp & 3;
      const int r = quad * 32 + lane;             // row inside the tile == TMEM lane
      const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
      const int row = row0[x] + r;
      const int i_row = min(a.I - 1, i0[x] + r / a.g);  // rows past the block's end behave like its last input
      // Left-padded sample: the cached padding pairs are the first n_pad rows (ids ascend), counted here by the
      // tile's 128 threads; a real query masks them and the block's padding positions, a padding query is
      // computed over everything and dropped in the epilogue.
      int pad = 0, n_pad = 0;
      if (PAD) {
        pad = a.left_pad[smp];
        const int* ids = a.kv_ids + (size_t)unit * a.cap;
        if (pad > 0 && a.n_old > 0 && ids[0] < pad) {          // uniform over the tile's threads
          int cnt = 0;
          for (int t = r; t < min(a.n_old, pad); t += 128) cnt += ids[t] < pad;
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
          if (lane == 0 && cnt > 0) atomicAdd(&np_slot[x], cnt);
          named_bar_sync(1 + x, 128);
          n_pad = np_slot[x];
        }
      }
      const bool real_row = !PAD || a.pos0 + i_row >= pad;
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < T[x]; ++j) {
        mbar_wait(&bars[B_SFULL + x], j & 1, abort_flag, a.status);
        tc_fence_after();
        // visible columns of this key tile for this row: [nlo, nvis)
        const int nvis = (j < t_old) ? min(kTileN, a.n_old - j * kTileN)
                                     : max(0, min(kTileN, i_row - (j - t_old) * kTileN + 1));
        const int nlo = (!PAD || !real_row) ? 0
                        : (j < t_old) ? max(0, min(kTileN, n_pad - j * kTileN))
                                      : max(0, min(kTileN, pad - a.pos0 - (j - t_old) * kTileN));
        const bool full = __all_sync(0xffffffffu, nvis >= kTileN && nlo == 0);   // warp-uniform: nothing to mask
        float mx = -INFINITY;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {                              // two TMEM loads in flight
          uint32_t ra[32], rb[32];
          tmem_ld32(tm_s[x] + lane_addr + hh * 64, ra);
          tmem_ld32(tm_s[x] + lane_addr + hh * 64 + 32, rb);
          tmem_wait_ld();
          if (full) {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              mx = max3(mx, __uint_as_float(ra[e]), __uint_as_float(ra[e + 1]));
              mx = max3(mx, __uint_as_float(rb[e]), __uint_as_float(rb[e + 1]));
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              mx = fmaxf(mx, (hh * 64 + e < nvis && hh * 64 + e >= nlo) ? __uint_as_float(ra[e]) : -INFINITY);
              mx = fmaxf(mx, (hh * 64 + 32 + e < nvis && hh * 64 + 32 + e >= nlo) ? __uint_as_float(rb[e]) : -INFINITY);
            }
          }
        }
        const float mx2 = mx * a.scale_log2;
        float alpha = 1.f;
        bool rescale = false;
        if (j == 0) m_used = mx2;
        else if (mx2 > m_used + kRescaleThreshold) { alpha = ex2(m_used - mx2); m_used = mx2; rescale = true; }
        // S_x(j) being complete implies the previous P.V into O_x has completed, so O_x may be touched here
        if (j > 0 && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t raw[32];
            tmem_ld32(tm_o[x] + lane_addr + cc * 32, raw);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) raw[e] = __float_as_uint(__uint_as_float(raw[e]) * alpha);
            tmem_st32(tm_o[x] + lane_addr + cc * 32, raw);
          }
          l *= alpha;
        }
        float ps0 = 0.f, ps1 = 0.f;
        const float neg_m = -m_used;
        uint32_t cur[32], nxt[32];
        tmem_ld32(tm_s[x] + lane_addr, cur);
        tmem_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          if (cc < 3) tmem_ld32(tm_s[x] + lane_addr + (cc + 1) * 32, nxt);   // next chunk loads while this one is used
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(cur[2 * e]), __uint_as_float(cur[2 * e + 1]), a.scale_log2, neg_m);
            float p0 = ex2(x0), p1 = ex2(x1);
            if (!full) {
              const int c0 = cc * 32 + 2 * e;
              p0 = (c0 < nvis && c0 >= nlo) ? p0 : 0.f;
              p1 = (c0 + 1 < nvis && c0 + 1 >= nlo) ? p1 : 0.f;
            }
            ps0 += p0;
            ps1 += p1;
            pk[e] = pack_bf16(p0, p1);
          }
          // bf16 pairs of columns [32cc, 32cc+32) land in columns [16cc, 16cc+16): logits already consumed
          tmem_st16(tm_s[x] + lane_addr + cc * 16, pk);
          if (cc < 3) {
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) cur[e] = nxt[e];
          }
        }
        l += ps0 + ps1;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars[B_PFULL + x]);
      }
      // epilogue: O / l -> bf16 -> swizzled tile in the (now idle) query buffer -> TMA store; log2-sum-exp
      mbar_wait(&bars[B_ODONE + x], (T[x] - 1) & 1, abort_flag, a.status);
      tc_fence_after();
      const float inv = real_row ? 1.f / l : 0.f;     // a padding query's output row is zero
      unsigned char* stage = sm + L::kQ + x * L::kTileBytes;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t raw[32];
        tmem_ld32(tm_o[x] + lane_addr + cc * 32, raw);
        tmem_wait_ld();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint4 w;
          w.x = pack_bf16(__uint_as_float(raw[q4 * 8 + 0]) * inv, __uint_as_float(raw[q4 * 8 + 1]) * inv);
          w.y = pack_bf16(__uint_as_float(raw[q4 * 8 + 2]) * inv, __uint_as_float(raw[q4 * 8 + 3]) * inv);
          w.z = pack_bf16(__uint_as_float(raw[q4 * 8 + 4]) * inv, __uint_as_float(raw[q4 * 8 + 5]) * inv);
          w.w = pack_bf16(__uint_as_float(raw[q4 * 8 + 6]) * inv, __uint_as_float(raw[q4 * 8 + 7]) * inv);
          const int piece = cc * 4 + q4;            // 16-byte piece of the row: chunk = piece / 8
          *reinterpret_cast<uint4*>(stage + (piece >> 3) * 16384 + sw128_offset(r, piece & 7)) = w;
        }
      }
      if (row < R) a.lse2[(size_t)unit * R + row] = real_row ? m_used + log2f(l) : INFINITY;  // +inf: no weights
      fence_async_smem();
      named_bar_sync(1 + x, 128);
      if (r == 0) {
        for (int c = 0; c < L::kChunks; ++c) tma_store_5d(&maps.o, stage + c * 16384, c * 64, 0, kh, i0[x], smp);
        tma_store_commit_and_wait();
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------------
// Score pass.  CTA = (tile of 128 candidate keys, unit).  A = the key tile (loaded once), B = the unit's query
// tiles streamed through a ring; S^T lands in TMEM with lane = key, column = query row.  The pass is bound by
// one exponential per visible pair, so four reducer warpgroups (one TMEM buffer each, query tiles taken round
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

template <int D>
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
    float acc = 0.f;
    for (int t = wg; t < T; t += kScoreWG) {
      const int qrow0 = (qt0 + t) * kTileM;
      // this tile's log2-sum-exp values; +inf for rows past the block's end (weight 0)
      {
        const int rr = qrow0 + key;
        sLse[wg * 128 + key] = (rr < R && (a.rule != 2 || rr >= R - a.g)) ? a.lse2[(size_t)unit * R + rr] : INFINITY;
      }
      named_bar_sync(1 + wg, 128);
      mbar_wait(&bars[C_SFULL + wg], (t / kScoreWG) & 1, abort_flag, a.status);
      tc_fence_after();
      // first query row of the tile that may see this key (causal mask inside the block)
      const int first_vis = is_old ? 0 : max(0, (c0 + key) * a.g - qrow0);
      const bool nomask = __all_sync(0xffffffffu, first_vis == 0);
      float p0 = 0.f, p1 = 0.f;
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
          float e0 = ex2(x0), e1 = ex2(x1);
          if (!nomask) {
            e0 = col >= first_vis ? e0 : 0.f;
            e1 = col + 1 >= first_vis ? e1 : 0.f;
          }
          add2(p0, p1, e0, e1);
        }
        if (cc < 3) {
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) cur[e] = nxt[e];
        }
      }
      acc += p0 + p1;
      tc_fence_before();
      mbar_arrive(&bars[C_SFREE + wg]);
      named_bar_sync(1 + wg, 128);                 // everyone is done with this tile's sLse before it is rewritten
    }
    sPart[wg * 128 + key] = acc;
    named_bar_sync(1 + kScoreWG, 128 * kScoreWG);
    if (wg == 0) {
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kScoreWG; ++w) tot += sPart[w * 128 + key];   // fixed order
      const int j = is_old ? kt * kTileN + key : c0 + key;
      if (a.left_pad != nullptr) {                  // a padding pair is masked for every query
        const int pad = a.left_pad[smp];
        const bool in_range = is_old ? j < a.n_old : j < a.I;
        if (pad > 0 && in_range && (is_old ? a.kv_ids[(size_t)unit * a.cap + j] : a.pos0 + j) < pad) tot = 0.f;
      }
      if (is_old) {
        if (j < a.n_old) {
          if (a.rule == 2) a.sum_weights[(size_t)unit * a.cap + j] = tot;   // nothing is carried over
          else a.sum_weights[(size_t)unit * a.cap + j] += tot;
        }
      }
      else if (j < a.I) a.new_sum[(size_t)unit * a.I + j] = tot;
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
  return t;
}

// maps of the call in flight: built by the forward launcher, reused by the score launcher
thread_local TcMaps g_maps;            // per thread: handles used from different threads do not share them
thread_local const void* g_maps_q = nullptr;

template <int D, int NT, bool PAD>
cudaError_t launch_fwd_nt(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  using L = FwdSmem<D, NT>;
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(attn_fwd_tc<D, NT, PAD>, (size_t)(L::kTotal)); e != cudaSuccess) return e;
  const int R = a.I * c.g;
  dim3 grid((R + NT * kTileM - 1) / (NT * kTileM), c.nsamples * c.Hkv);
  ProfileScope prof(kAttnFwd, st);
  attn_fwd_tc<D, NT, PAD><<<grid, L::kThreads, L::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
}

// One query tile per CTA with two CTAs per SM measured faster than two tiles per CTA on every shape tried
// (cfg2: 530 vs 507 TFLOP/s, cfg3 shape at b=256: 789 vs 776): overlapping one CTA's first loads and epilogue
// with the other's main loop is worth more than sharing K/V tiles.  BM_FWD_TILES=2 selects the other variant.
int g_fwd_tiles_override = 0;

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

int g_fwd_kernel = 0;   // 0: two threads per row; 1 / 2: one thread per row, one / two query tiles per CTA (BM_FWD_KERNEL)

template <int D>
cudaError_t launch_fwd_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  // (the one-thread-per-row kernels take cached padding to be a prefix of the rows: not so in an unordered cache)
  if (g_fwd_kernel == 0 || (c.fill && c.left_pad != nullptr))
    return c.left_pad != nullptr ? launch_fwd_split<D, true>(c, a, st) : launch_fwd_split<D, false>(c, a, st);
  if (c.left_pad != nullptr)
    return g_fwd_tiles_override == 2 ? launch_fwd_nt<D, 2, true>(c, a, st) : launch_fwd_nt<D, 1, true>(c, a, st);
  return g_fwd_tiles_override == 2 ? launch_fwd_nt<D, 2, false>(c, a, st) : launch_fwd_nt<D, 1, false>(c, a, st);
}

template <int D>
cudaError_t launch_score_t(const CacheView& c, const BlockArgs& a, cudaStream_t st) {
  static SmemConfigured configured;
  if (cudaError_t e = configured.ensure(score_tc<D>, (size_t)(ScoreSmem<D>::kTotal)); e != cudaSuccess) return e;
  const int t_old = (c.n_old + kTileN - 1) / kTileN, t_new = (a.I + kTileN - 1) / kTileN;
  dim3 grid(t_old + t_new, c.nsamples * c.Hkv);
  ProfileScope prof(kScore, st);
  score_tc<D><<<grid, kScoreThreads, ScoreSmem<D>::kTotal, st>>>(g_maps, make_args(c, a));
  count_launch();
  return cudaGetLastError();
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

bool tc_path_available() {
  static bool init = false;
  if (!init) {
    init = true;
    const char* e = std::getenv("BM_FWD_KERNEL");   // 0 (default) two threads per row; 1 / 2 one thread per row
    if (e != nullptr) { g_fwd_kernel = std::atoi(e); g_fwd_tiles_override = g_fwd_kernel; }
  }
  return encode_fn() != nullptr;
}

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
