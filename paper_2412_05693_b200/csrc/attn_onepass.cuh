// Forward pass AND column sums of a short block in one kernel, one exponential per visible pair (included by
// attn_tc.cu after TcMaps / TcArgs).
//
// The column sums of Sec. 3.2's update, sum_i attn_weights[i], need every row's final normaliser, which is why the
// general path recomputes the logits in a second kernel.  When the whole logit matrix of a cache fits tensor memory
// -- one tile of query rows (I * g <= 128) against at most four tiles of 128 keys (cached and new) -- nothing has to
// be recomputed: all logits are produced first and stay in tensor memory, a row's maximum and sum are exact before
// any probability is used, the un-normalised probabilities replace the logits in place (fp32), the column sums are
// taken from them (scaled by 1 / row sum) by a fixed-order butterfly across the rows of a warp and a fixed-order sum
// across the four warps, and only then are they rounded to bf16 for P.V.  This is the regime of Algorithm 1's own
// cadence (p inputs per pass, Sec. 3.1 / Sec. 4.1) on short caches.
//
// One CTA per cache, one CTA per SM (it owns all 512 tensor-memory columns): warps 0-7 hold the query rows, two
// threads per row (warps 0-3 key columns 0-63 of every tile, warps 4-7 columns 64-127; a warp may only touch the 32
// tensor-memory lanes of its quadrant), warp 8 issues the MMAs, warp 9 is the TMA producer.  Shared memory: Q | four tile slots (K_t, later V_t) |
// partial column sums.  Tensor memory: logits of key tile t in columns [128 t, +128); after the conversion the bf16
// probabilities of tile t sit in [128 t, +64) and the output accumulator takes freed columns: elements 0-63 of the
// head dimension in [64, 128), elements 64-127 in [192, 256).
#pragma once

template <int D>
struct OnePassSmem {
  static constexpr int kMaxKeyTiles = 4;
  static constexpr int kChunks = D / 64;
  static constexpr int kTileBytes = kChunks * 16384;     // 128 rows x D bf16
  static constexpr int kQ = 0;
  static constexpr int kKV = kTileBytes;                 // slot t: K_t, then V_t
  static constexpr int kPart = kKV + kMaxKeyTiles * kTileBytes;   // [4 row quadrants][512] floats
  static constexpr int kEx = kPart + 4 * 512 * 4;                 // [2][128] floats: the two threads of a row meet here
  static constexpr int kBars = kEx + 2 * 128 * 4;
  static constexpr int kTotal = kBars + 256 + 1024;
  static constexpr int kThreads = 320;
};

template <int D>
__global__ void __launch_bounds__(320, 1) attn_block_onepass(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = OnePassSmem<D>;
  constexpr int kMmaWarp = 8, kTmaWarp = 9;
  constexpr int kTmemCols = 512;
  constexpr int B_QFULL = 0, B_KVFULL = 1 /* 4 slots */, B_SFULL = 5 /* 4 tiles */, B_KDONE = 9, B_PFULL = 10, B_ODONE = 11,
                B_COUNT = 12;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* part = reinterpret_cast<float*>(sm + L::kPart);
  float* sEx = reinterpret_cast<float*>(sm + L::kEx);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, smp = unit / a.Hkv, kh = unit % a.Hkv;
  const int R = a.I * a.g;                                   // query rows of the block (<= 128)
  const int t_old = (a.n_old + kTileN - 1) / kTileN, t_new = (a.I + kTileN - 1) / kTileN;
  const int T = t_old + t_new;                               // <= 4 key tiles

  auto load_tile = [&](int t, bool is_v) {                   // key tile t into slot t
    unsigned char* dst = sm + L::kKV + t * L::kTileBytes;
    mbar_expect_tx(&bars[B_KVFULL + t], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c) {
      if (t < t_old)
        tma_load_3d(dst + c * 16384, is_v ? &maps.v_slab : &maps.k_slab, c * 64, t * kTileN, unit, &bars[B_KVFULL + t]);
      else
        tma_load_4d(dst + c * 16384, is_v ? &maps.v_blk : &maps.k_blk, c * 64, kh, (t - t_old) * kTileN, smp,
                    &bars[B_KVFULL + t]);
    }
  };
  if (warp == kTmaWarp && lane == 0) {
    *abort_flag = 0;
    mbar_init(&bars[B_QFULL], 1);
    for (int t = 0; t < 4; ++t) mbar_init(&bars[B_KVFULL + t], 1);
    for (int t = 0; t < 4; ++t) mbar_init(&bars[B_SFULL + t], 1);
    mbar_init(&bars[B_KDONE], 1);
    mbar_init(&bars[B_PFULL], 256);
    mbar_init(&bars[B_ODONE], 1);
    mbar_fence_init();
    mbar_expect_tx(&bars[B_QFULL], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c) tma_load_5d(sm + L::kQ + c * 16384, &maps.q, c * 64, 0, kh, 0, smp, &bars[B_QFULL]);
    for (int t = 0; t < T; ++t) load_tile(t, false);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == kTmaWarp) {
    // the value tiles follow into the same slots once every Q.K^T has read its key tile
    if (lane == 0) {
      mbar_wait(&bars[B_KDONE], 0, abort_flag, a.status);
      for (int t = 0; t < T; ++t) load_tile(t, true);
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(kTileM, kTileN, 0, 0);
      const uint32_t idesc_pv = instr_desc(kTileM, 64, 0, 1);   // V is MN-major; 64 elements of the head dimension per MMA
      const uint64_t dk_hi = smem_desc(0, 16, 1024) & 0xffffffff00000000ull;      // K-major operands (Q, K)
      const uint32_t dk_lo = (uint32_t)(smem_desc(0, 16, 1024) & 0xffffffffull);
      const uint64_t dv_hi = smem_desc(0, 16384, 1024) & 0xffffffff00000000ull;   // MN-major operand (V)
      const uint32_t dv_lo = (uint32_t)(smem_desc(0, 16384, 1024) & 0xffffffffull);
      const uint32_t q_lo = dk_lo + (smem_u32(sm + L::kQ) >> 4);
      mbar_wait(&bars[B_QFULL], 0, abort_flag, a.status);
      for (int t = 0; t < T; ++t) {                            // S_t = Q K_t^T, all tiles before any softmax
        mbar_wait(&bars[B_KVFULL + t], 0, abort_flag, a.status);
        tc_fence_after();
        const uint32_t k_lo = dk_lo + (smem_u32(sm + L::kKV + t * L::kTileBytes) >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks >> 2) * 1024 + (ks & 3) * 2;   // (chunk * 16384 + kstep * 32) / 16
          mma_ss(tmem + 128 * t, dk_hi | (q_lo + off), dk_hi | (k_lo + off), idesc_qk, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[B_SFULL + t]);                        // the row maxima are taken tile by tile as they land
      }
      mma_commit(&bars[B_KDONE]);
      mbar_wait(&bars[B_PFULL], 0, abort_flag, a.status);      // every probability is in place, columns are free
      tc_fence_after();
      for (int t = 0; t < T; ++t) {                            // O += P_t V_t
        mbar_wait(&bars[B_KVFULL + t], 1, abort_flag, a.status);
        tc_fence_after();
        const uint32_t v_lo = dv_lo + (smem_u32(sm + L::kKV + t * L::kTileBytes) >> 4);
#pragma unroll
        for (int ks = 0; ks < kTileN / 16; ++ks)
#pragma unroll
          for (int c = 0; c < L::kChunks; ++c)                 // elements [64 c, +64) -> accumulator columns 64 + 128 c
            mma_ts(tmem + 64 + 128 * c, tmem + 128 * t + ks * 8, dv_hi | (v_lo + c * 1024 + ks * 128), idesc_pv,
                   (t > 0 || ks > 0) ? 1u : 0u);
      }
      mma_commit(&bars[B_ODONE]);
    }
  } else {
    // ------------------------------------------------------------------ two threads per query row
    const int half = warp >> 2, quad = warp & 3;
    const int r = quad * 32 + lane;                            // row of the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int c_lo = 64 * half;                                // first key column of this thread in every tile
    const int i_row = min(a.I - 1, r / a.g);                   // rows past the block's end behave like its last input
    const bool live = r < R;                                   // ... but add nothing to the column sums
    auto n_visible = [&](int t) {                              // visible columns of key tile t for this row: [0, nvis)
      return t < t_old ? min(kTileN, a.n_old - t * kTileN) : max(0, min(kTileN, i_row - (t - t_old) * kTileN + 1));
    };
    // pass 1: the row's maximum over every visible logit (every lane takes part in every tensor-memory load)
    float mx = -INFINITY;
    for (int t = 0; t < T; ++t) {
      mbar_wait(&bars[B_SFULL + t], 0, abort_flag, a.status);
      tc_fence_after();
      const int nvis = n_visible(t);
      uint32_t s0[32], s1[32];
      tmem_ld32(tmem + lane_addr + 128 * t + c_lo, s0);
      tmem_ld32(tmem + lane_addr + 128 * t + c_lo + 32, s1);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        mx = fmaxf(mx, (c_lo + e < nvis) ? __uint_as_float(s0[e]) : -INFINITY);
        mx = fmaxf(mx, (c_lo + 32 + e < nvis) ? __uint_as_float(s1[e]) : -INFINITY);
      }
    }
    sEx[half * 128 + r] = mx;
    named_bar_sync(1, 256);
    mx = fmaxf(mx, sEx[(half ^ 1) * 128 + r]);
    const float neg_m = -mx * a.scale_log2;
    // pass 2: un-normalised probabilities replace the logits in place (fp32); exact row sum
    float l = 0.f;
    for (int t = 0; t < T; ++t) {
      const int nvis = n_visible(t);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t s[32];
        tmem_ld32(tmem + lane_addr + 128 * t + c_lo + 32 * ch, s);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const float p = (c_lo + 32 * ch + e < nvis) ? ex2(fmaf(__uint_as_float(s[e]), a.scale_log2, neg_m)) : 0.f;
          l += p;
          s[e] = __float_as_uint(p);
        }
        tmem_st32(tmem + lane_addr + 128 * t + c_lo + 32 * ch, s);
      }
    }
    named_bar_sync(1, 256);                                    // both threads of a row have read the other's maximum
    sEx[half * 128 + r] = l;
    named_bar_sync(1, 256);
    l = sEx[r] + sEx[128 + r];                                 // same order in both threads
    tmem_wait_st();
    const float inv = 1.f / l;                                 // l >= 1: every row sees at least its own key
    const float wgt = live ? inv : 0.f;
    // pass 3: column sums (fp32, normalised) and bf16 probabilities for P.V (un-normalised; O is divided at the end).
    // A chunk of 32 columns is reduced over the warp's 32 rows by a butterfly that halves the columns a lane still
    // carries at every step: after 5 steps lane c holds the sum of column c.
    for (int t = 0; t < T; ++t) {
      uint32_t sa[32], sb[32];
      tmem_ld32(tmem + lane_addr + 128 * t + c_lo, sa);
      tmem_ld32(tmem + lane_addr + 128 * t + c_lo + 32, sb);
      tmem_wait_ld();
      // The bf16 pairs of this thread's 64 keys go to columns [32 half, +32) of the tile, keys in order.  For half 1
      // that is where the row's other thread keeps logits, so both threads have loaded all of theirs first.
      named_bar_sync(2, 256);
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t pk[16];
        float v[32];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const uint32_t u0 = ch ? sb[2 * e] : sa[2 * e], u1 = ch ? sb[2 * e + 1] : sa[2 * e + 1];
          pk[e] = pack_bf16(__uint_as_float(u0), __uint_as_float(u1));
          v[2 * e] = __uint_as_float(u0) * wgt;
          v[2 * e + 1] = __uint_as_float(u1) * wgt;
        }
        tmem_st16(tmem + lane_addr + 128 * t + 32 * half + 16 * ch, pk);
#pragma unroll
        for (int w = 16; w >= 1; w >>= 1) {                    // lanes with bit w set keep the upper half of what is left
          const bool up = (lane & w) != 0;
#pragma unroll
          for (int e = 0; e < w; ++e) {
            const float mine = up ? v[e + w] : v[e], theirs = up ? v[e] : v[e + w];
            const float got = __shfl_xor_sync(0xffffffffu, theirs, w);
            v[e] = up ? got + mine : mine + got;               // lower lane's value first on both sides
          }
        }
        part[quad * 512 + 128 * t + c_lo + 32 * ch + lane] = v[0];
      }
    }
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(&bars[B_PFULL]);
    named_bar_sync(1, 256);
    // the four row quadrants' partial sums in a fixed order -> sum_weights (cached pairs) / new_sum (the block's pairs)
    for (int c = tid; c < 128 * T; c += 256) {
      const float tot = ((part[c] + part[512 + c]) + part[1024 + c]) + part[1536 + c];
      const int t = c >> 7, j = c & 127;
      if (t < t_old) {
        const int k = t * kTileN + j;
        if (k < a.n_old) a.sum_weights[(size_t)unit * a.cap + k] += tot;
      } else {
        const int k = (t - t_old) * kTileN + j;
        if (k < a.I) a.new_sum[(size_t)unit * a.I + k] = tot;
      }
    }
    // epilogue: O / l -> bf16 -> swizzled tile in the (idle) query buffer -> TMA store; each thread of a row
    // takes half of the row's output columns
    mbar_wait(&bars[B_ODONE], 0, abort_flag, a.status);
    tc_fence_after();
    unsigned char* stage = sm + L::kQ;
#pragma unroll
    for (int c2 = 0; c2 < D / 64; ++c2) {
      const int cc = half * (D / 64) + c2;                     // 32-column chunk of the output row
      uint32_t raw[32];
      tmem_ld32(tmem + lane_addr + 64 + 128 * (cc >> 1) + 32 * (cc & 1), raw);
      tmem_wait_ld();
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint4 w;
        w.x = pack_bf16(__uint_as_float(raw[q4 * 8 + 0]) * inv, __uint_as_float(raw[q4 * 8 + 1]) * inv);
        w.y = pack_bf16(__uint_as_float(raw[q4 * 8 + 2]) * inv, __uint_as_float(raw[q4 * 8 + 3]) * inv);
        w.z = pack_bf16(__uint_as_float(raw[q4 * 8 + 4]) * inv, __uint_as_float(raw[q4 * 8 + 5]) * inv);
        w.w = pack_bf16(__uint_as_float(raw[q4 * 8 + 6]) * inv, __uint_as_float(raw[q4 * 8 + 7]) * inv);
        const int piece = cc * 4 + q4;                         // 16-byte piece of the row: chunk = piece / 8
        *reinterpret_cast<uint4*>(stage + (piece >> 3) * 16384 + sw128_offset(r, piece & 7)) = w;
      }
    }
    fence_async_smem();
    named_bar_sync(1, 256);
    if (tid == 0) {
      for (int c = 0; c < L::kChunks; ++c) tma_store_5d(&maps.o, stage + c * 16384, c * 64, 0, kh, 0, smp);
      tma_store_commit_and_wait();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}
