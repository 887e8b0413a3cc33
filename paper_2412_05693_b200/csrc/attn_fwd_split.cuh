// Forward pass, one tile of 128 query rows per CTA with TWO threads per row (included by attn_tc.cu after
// TcMaps / TcArgs).  Warps 0-3 take key columns 0-63 of every 128-key tile, warps 4-7 columns 64-127 (a warp may
// only touch the 32 tensor-memory lanes of its quadrant, so the two warps of a row share lanes and split columns);
// warp 8 issues the MMAs and owns the tensor memory, warp 9 is the TMA producer.  The softmax of a tile is the
// serial link between its Q.K^T and its P.V, so halving its latency shortens the whole chain; the two threads of a
// row exchange their partial row maxima through shared memory (one named barrier per tile) and add their partial
// row sums in the epilogue.  A thread publishes its probabilities in two halves of 32 keys, so that the first half
// of P.V runs under the second half's exponentials.  Two CTAs per SM; tensor memory: S 128 columns (each thread's
// bf16 probabilities overwrite the first 32 of its own 64 logit columns) | O 128 columns.
#pragma once

template <int D>
struct SplitSmem {
  static constexpr int kChunks = D / 64;                 // 64-element (128-byte) column chunks per row
  static constexpr int kTileBytes = kChunks * 16384;     // 128 rows x D bf16
  static constexpr int kQ = 0;                           // query tile (reused to stage the output)
  static constexpr int kKV = kTileBytes;                 // ring of 2: entry 2j = K_j (slot 0), 2j+1 = V_j (slot 1)
  static constexpr int kEx = kKV + 2 * kTileBytes;       // [2][2][128] floats: row maxima (double-buffered), then row sums
  static constexpr int kBars = kEx + 2 * 2 * 128 * 4;
  static constexpr int kTotal = kBars + 256 + 1024;      // + barriers + alignment slack
  static constexpr int kThreads = 320;
};

template <int D, bool PAD>
__global__ void __launch_bounds__(320, 2) attn_fwd_split(const __grid_constant__ TcMaps maps, const TcArgs a) {
  using L = SplitSmem<D>;
  constexpr int kMmaWarp = 8, kTmaWarp = 9;
  constexpr int kTmemCols = 256;
  constexpr int B_QFULL = 0, B_KVFULL = 1, B_KVEMPTY = 3, B_SFULL = 5, B_PFULL = 6, B_ODONE = 7, B_PHALF = 8, B_COUNT = 9;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* sEx = reinterpret_cast<float*>(sm + L::kEx);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + L::kBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // [2][4] words: which keys of a cached tile are padding pairs (double-buffered over key tiles)
  uint32_t* pmask = reinterpret_cast<uint32_t*>(sm + L::kBars + 128);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.y, smp = unit / a.Hkv, kh = unit % a.Hkv;
  const int R = a.I * a.g;
  const int qpt = kTileM / a.g;                  // inputs (positions) covered by the row tile
  const int t_old = (a.n_old + kTileN - 1) / kTileN;
  // row tiles are handed out last first: a later tile sees more of the block's own keys, and the longest CTAs of a
  // cache should not be the ones that start last
  const int rt = gridDim.x - 1 - blockIdx.x;
  const int row0 = rt * kTileM, i0 = rt * qpt;
  const int T = t_old + min(a.I - 1, i0 + qpt - 1) / kTileN + 1;   // cached-key tiles + block-key tiles up to the last input

  auto load_kv = [&](int e) {   // ring entry e: K_j for even e, V_j for odd e, j = e / 2
    const int j = e >> 1, s = e & 1;
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
    mbar_init(&bars[B_QFULL], 1);
    mbar_init(&bars[B_SFULL], 1);
    mbar_init(&bars[B_PFULL], 256);
    mbar_init(&bars[B_PHALF], 256);   // the first half of every thread's probabilities is published on its own
    mbar_init(&bars[B_ODONE], 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&bars[B_KVFULL + s], 1); mbar_init(&bars[B_KVEMPTY + s], 1); }
    mbar_fence_init();
    mbar_expect_tx(&bars[B_QFULL], L::kTileBytes);
    for (int c = 0; c < L::kChunks; ++c)
      tma_load_5d(sm + L::kQ + c * 16384, &maps.q, c * 64, 0, kh, i0, smp, &bars[B_QFULL]);
    load_kv(0);
    load_kv(1);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s = tmem, tm_o = tmem + 128;

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int e = 2; e < 2 * T; ++e) {
        mbar_wait(&bars[B_KVEMPTY + (e & 1)], ((e >> 1) - 1) & 1, abort_flag, a.status);
        load_kv(e);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer (one thread)
    if (lane == 0) {
      const uint32_t idesc_qk = instr_desc(kTileM, kTileN, 0, 0);
      const uint32_t idesc_pv = instr_desc(kTileM, D, 0, 1);  // V is MN-major: d contiguous, keys along K
      const uint64_t dk_hi = smem_desc(0, 16, 1024) & 0xffffffff00000000ull;      // K-major operands (Q, K)
      const uint32_t dk_lo = (uint32_t)(smem_desc(0, 16, 1024) & 0xffffffffull);
      const uint64_t dv_hi = smem_desc(0, 16384, 1024) & 0xffffffff00000000ull;   // MN-major operand (V)
      const uint32_t dv_lo = (uint32_t)(smem_desc(0, 16384, 1024) & 0xffffffffull);
      const uint32_t q_lo = dk_lo + (smem_u32(sm + L::kQ) >> 4);
      const uint32_t k_lo = dk_lo + (smem_u32(sm + L::kKV) >> 4);
      const uint32_t v_lo = dv_lo + (smem_u32(sm + L::kKV + L::kTileBytes) >> 4);
      auto wait_kv = [&](int e) { mbar_wait(&bars[B_KVFULL + (e & 1)], (e >> 1) & 1, abort_flag, a.status); };
      auto issue_qk = [&]() {             // S = Q K_j^T
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks >> 2) * 1024 + (ks & 3) * 2;   // (chunk * 16384 + kstep * 32) / 16
          mma_ss(tm_s, dk_hi | (q_lo + off), dk_hi | (k_lo + off), idesc_qk, ks > 0 ? 1u : 0u);
        }
        mma_commit(&bars[B_KVEMPTY + 0]);
        mma_commit(&bars[B_SFULL]);
      };
      auto issue_pv = [&](int j) {        // O += P V_j, P read from tensor memory (over S)
        // The probabilities arrive in two halves: every thread's first 32 columns (keys 0-31 and 64-95: steps 0, 1,
        // 4, 5), then its last 32, each on a barrier of its own (one arrival per thread and key tile on either).  The
        // first half of P.V runs under the exponentials of the second.
#pragma unroll
        for (int ph = 0; ph < 2; ++ph) {
          mbar_wait(&bars[ph ? B_PFULL : B_PHALF], j & 1, abort_flag, a.status);
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int ks = (q >> 1) * 4 + ph * 2 + (q & 1);   // 16 keys per step; P of keys 64..127 sits at column 64
            mma_ts(tm_o, tm_s + (ks >> 2) * 64 + (ks & 3) * 8, dv_hi | (v_lo + ks * 128), idesc_pv,
                   (j > 0 || ph > 0 || q > 0) ? 1u : 0u);
          }
        }
        mma_commit(&bars[B_KVEMPTY + 1]);
      };
      mbar_wait(&bars[B_QFULL], 0, abort_flag, a.status);
      wait_kv(0);
      tc_fence_after();
      issue_qk();
      for (int j = 1; j <= T; ++j) {      // products of key tile j-1, logits of key tile j
        wait_kv(2 * j - 1);
        if (j < T) wait_kv(2 * j);
        tc_fence_after();
        issue_pv(j - 1);
        if (j < T) issue_qk();
      }
      mma_commit(&bars[B_ODONE]);
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue: two threads per row
    const int half = warp >> 2, quad = warp & 3;
    const int r = quad * 32 + lane;               // row inside the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int row = row0 + r;
    const int i_row = min(a.I - 1, i0 + r / a.g);  // rows past the block's end behave like its last input
    const int c_lo = 64 * half;                   // first key column of this thread
    // Left padding: a padding pair is masked for every real query.  Among the block's own keys padding is a prefix
    // of positions; among the cached pairs it is whatever kv_ids say (the rows of an unordered cache are in no
    // order), so warps 0-3 turn the kv_ids of each cached tile into a 128-bit mask one tile ahead.
    int pad = 0;
    const int* ids = a.kv_ids + (size_t)unit * a.cap;
    auto publish_pad_mask = [&](int jt) {   // tile jt < t_old, by the 128 threads of half 0
      if (half == 0) {
        const int k = jt * kTileN + r;
        const uint32_t w = __ballot_sync(0xffffffffu, k < a.n_old && ids[k] < pad);
        if (lane == 0) pmask[(jt & 1) * 4 + quad] = w;
      }
    };
    if (PAD) {
      pad = a.left_pad[smp];
      if (pad > 0 && t_old > 0) {
        publish_pad_mask(0);
        named_bar_sync(1, 256);
      }
    }
    const bool real_row = !PAD || a.pos0 + i_row >= pad;
    float m_used = -INFINITY, l = 0.f;
    for (int j = 0; j < T; ++j) {
      mbar_wait(&bars[B_SFULL], j & 1, abort_flag, a.status);
      tc_fence_after();
      // visible columns of this key tile for this row: [nlo, nvis)
      const int nvis = (j < t_old) ? min(kTileN, a.n_old - j * kTileN)
                                   : max(0, min(kTileN, i_row - (j - t_old) * kTileN + 1));
      // padding among this thread's 64 columns: a prefix [0, nlo) of a block tile, a bit mask of a cached tile
      const int nlo = (!PAD || !real_row || j < t_old) ? 0 : max(0, min(kTileN, pad - a.pos0 - (j - t_old) * kTileN));
      uint64_t pm = 0;
      if (PAD && pad > 0 && j < t_old) {
        if (real_row) pm = (uint64_t)pmask[(j & 1) * 4 + 2 * half] | ((uint64_t)pmask[(j & 1) * 4 + 2 * half + 1] << 32);
        if (j + 1 < t_old) publish_pad_mask(j + 1);   // read after this tile's exchange of maxima (a barrier)
      }
      const bool full = __all_sync(0xffffffffu, nvis >= kTileN && nlo == 0 && pm == 0);   // warp-uniform: nothing to mask
      uint32_t s0[32], s1[32];
      tmem_ld32(tm_s + lane_addr + c_lo, s0);
      tmem_ld32(tm_s + lane_addr + c_lo + 32, s1);
      tmem_wait_ld();
      float mx = -INFINITY;
      if (full) {
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          mx = max3(mx, __uint_as_float(s0[e]), __uint_as_float(s0[e + 1]));
          mx = max3(mx, __uint_as_float(s1[e]), __uint_as_float(s1[e + 1]));
        }
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          const int c0 = c_lo + e, c1 = c_lo + 32 + e;
          mx = fmaxf(mx, (c0 < nvis && c0 >= nlo && !((pm >> e) & 1)) ? __uint_as_float(s0[e]) : -INFINITY);
          mx = fmaxf(mx, (c1 < nvis && c1 >= nlo && !((pm >> (32 + e)) & 1)) ? __uint_as_float(s1[e]) : -INFINITY);
        }
      }
      // the row's other thread holds the maximum of the other 64 columns
      float* ex = sEx + (j & 1) * 256;
      ex[half * 128 + r] = mx;
      named_bar_sync(1, 256);
      mx = fmaxf(mx, ex[(half ^ 1) * 128 + r]);
      const float mx2 = mx * a.scale_log2;
      float alpha = 1.f;
      bool rescale = false;
      if (j == 0) m_used = mx2;
      else if (mx2 > m_used + kRescaleThreshold) { alpha = ex2(m_used - mx2); m_used = mx2; rescale = true; }
      // S(j) being complete implies the previous P.V into O has completed, so O may be touched here
      if (j > 0 && __any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int cc = 0; cc < D / 64; ++cc) {      // this thread's half of the row's output columns
          uint32_t raw[32];
          tmem_ld32(tm_o + lane_addr + half * (D / 2) + cc * 32, raw);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) raw[e] = __float_as_uint(__uint_as_float(raw[e]) * alpha);
          tmem_st32(tm_o + lane_addr + half * (D / 2) + cc * 32, raw);
        }
        l *= alpha;
      }
      float ps0 = 0.f, ps1 = 0.f;
      const float neg_m = -m_used;
      // second read of the logits, 32 columns at a time (keeps the register count inside two CTAs per SM); the
      // bf16 pairs of each chunk go over this thread's own logits: columns [64 half, 64 half + 32).  The loop exists
      // twice, with and without masks: as one loop with a test inside, the compiler evaluated the masks of every
      // tile (two more instructions per exponential on the fully visible tiles, which are most).
      auto exp_chunks = [&](auto masked) {
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t sv[32], pk[16];
          tmem_ld32(tm_s + lane_addr + c_lo + 32 * ch, sv);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(sv[2 * e]), __uint_as_float(sv[2 * e + 1]), a.scale_log2, neg_m);
            float p0 = ex2(x0), p1 = ex2(x1);
            if (decltype(masked)::value) {
              const int c0 = c_lo + 32 * ch + 2 * e;
              p0 = (c0 < nvis && c0 >= nlo && !((pm >> (32 * ch + 2 * e)) & 1)) ? p0 : 0.f;
              p1 = (c0 + 1 < nvis && c0 + 1 >= nlo && !((pm >> (32 * ch + 2 * e + 1)) & 1)) ? p1 : 0.f;
            }
            add2(ps0, ps1, p0, p1);
            pk[e] = pack_bf16(p0, p1);
          }
          tmem_st16(tm_s + lane_addr + c_lo + 16 * ch, pk);
          if (ch == 0) {                              // the first half may enter P.V now
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[B_PHALF]);
          }
        }
      };
      if (full) exp_chunks(std::false_type{});
      else exp_chunks(std::true_type{});
      l += ps0 + ps1;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars[B_PFULL]);
    }
    // epilogue: O / l -> bf16 -> swizzled tile in the (now idle) query buffer -> TMA store; log2-sum-exp
    float* exl = sEx;                               // row sums of the two threads of a row
    named_bar_sync(1, 256);                         // every read of the last tile's maxima is over
    exl[half * 128 + r] = l;
    named_bar_sync(1, 256);
    l = exl[r] + exl[128 + r];                      // same order in both threads
    mbar_wait(&bars[B_ODONE], 0, abort_flag, a.status);
    tc_fence_after();
    const float inv = real_row ? 1.f / l : 0.f;     // a padding query's output row is zero
    unsigned char* stage = sm + L::kQ;
#pragma unroll
    for (int c2 = 0; c2 < D / 64; ++c2) {
      const int cc = half * (D / 64) + c2;          // 32-column chunk of the output row
      uint32_t raw[32];
      tmem_ld32(tm_o + lane_addr + cc * 32, raw);
      tmem_wait_ld();
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint4 w;
        w.x = pack_bf16(__uint_as_float(raw[q4 * 8 + 0]) * inv, __uint_as_float(raw[q4 * 8 + 1]) * inv);
        w.y = pack_bf16(__uint_as_float(raw[q4 * 8 + 2]) * inv, __uint_as_float(raw[q4 * 8 + 3]) * inv);
        w.z = pack_bf16(__uint_as_float(raw[q4 * 8 + 4]) * inv, __uint_as_float(raw[q4 * 8 + 5]) * inv);
        w.w = pack_bf16(__uint_as_float(raw[q4 * 8 + 6]) * inv, __uint_as_float(raw[q4 * 8 + 7]) * inv);
        const int piece = cc * 4 + q4;              // 16-byte piece of the row: chunk = piece / 8
        *reinterpret_cast<uint4*>(stage + (piece >> 3) * 16384 + sw128_offset(r, piece & 7)) = w;
      }
    }
    if (half == 0 && row < R) a.lse2[(size_t)unit * R + row] = real_row ? m_used + log2f(l) : INFINITY;  // +inf: no weights
    fence_async_smem();
    named_bar_sync(1, 256);
    if (tid == 0) {
      for (int c = 0; c < L::kChunks; ++c) tma_store_5d(&maps.o, stage + c * 16384, c * 64, 0, kh, i0, smp);
      tma_store_commit_and_wait();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}
