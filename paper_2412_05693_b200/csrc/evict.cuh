// Average-attention eviction for one (sample, kv-head) cache, executed by one CTA (Sec. 3.2):
//   ave_weights = sum_weights / (g * (curr_id + 1 - kv_ids)),
// keep the `target` candidates ranking first under (ave_weights descending, kv_ids ascending),
// then compact rows, sum_weights and kv_ids to the front of the cache in ascending kv_ids order.
// (EvictArgs::recent selects the rule of the extreme decoding-only comparison instead, Algorithm 3:
// the `target` most recent candidates stay.)
// Candidates are the n_old cached pairs followed by I new pairs that still live in the caller's
// block buffers; both lists are ascending in kv_ids, so candidate index order is kv_ids order.
#pragma once
#include "common.cuh"

namespace bm {

struct EvictSmem {
  float* score;    // [n_cand]
  uint32_t* bits;  // [n_cand]   ranking value of every candidate as an ordered bit pattern (computed once)
  int32_t* id;     // [n_cand]
  int32_t* src;    // [target]   candidate index that lands in row r (fill mode: k-th candidate that has to move)
  int32_t* dst;    // [target]   fill mode: row the k-th moving candidate lands in
  uint32_t* hist;  // [256]
  int32_t* misc;   // [8]
  int32_t* wsum;   // [64]
};

__host__ __device__ inline size_t evict_smem_layout(unsigned char* base, int n_cand, int target, EvictSmem* s) {
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) & ~size_t(15); return o; };
  size_t o_score = take(sizeof(float) * n_cand), o_id = take(sizeof(int32_t) * n_cand);
  size_t o_bits = take(sizeof(uint32_t) * n_cand);
  size_t o_src = take(sizeof(int32_t) * (target > 0 ? target : 1)), o_dst = take(sizeof(int32_t) * (target > 0 ? target : 1));
  size_t o_hist = take(sizeof(uint32_t) * 256);
  size_t o_misc = take(sizeof(int32_t) * 8), o_wsum = take(sizeof(int32_t) * 64);
  if (s != nullptr) {
    s->score = reinterpret_cast<float*>(base + o_score);
    s->bits = reinterpret_cast<uint32_t*>(base + o_bits);
    s->id = reinterpret_cast<int32_t*>(base + o_id);
    s->src = reinterpret_cast<int32_t*>(base + o_src);
    s->dst = reinterpret_cast<int32_t*>(base + o_dst);
    s->hist = reinterpret_cast<uint32_t*>(base + o_hist);
    s->misc = reinterpret_cast<int32_t*>(base + o_misc);
    s->wsum = reinterpret_cast<int32_t*>(base + o_wsum);
  }
  return off;
}

// Exclusive block scan of two counters packed per thread; returns this thread's exclusive prefixes.
template <int NT>
__device__ inline void block_exclusive_scan2(int a, int b, int32_t* wsum /*[64]*/, int& ea, int& eb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int ta = __shfl_up_sync(0xffffffffu, ia, off), tb = __shfl_up_sync(0xffffffffu, ib, off);
    if (lane >= off) { ia += ta; ib += tb; }
  }
  if (lane == 31) { wsum[warp] = ia; wsum[32 + warp] = ib; }
  __syncthreads();
  int ba = 0, bb = 0;
  for (int w = 0; w < warp; ++w) { ba += wsum[w]; bb += wsum[32 + w]; }
  ea = ba + ia - a;
  eb = bb + ib - b;
  __syncthreads();
}

// FILL: the cache's rows are an unordered set (CacheView::fill); a template parameter, so that the instance for
// ordered rows carries none of that code (with both in one function the ordered instance ran 15 % slower).
template <typename T, int D, int NT, bool FILL>
__device__ inline void evict_body_impl(const CacheView& c, int unit, int smp, int kh, const EvictArgs& e,
                                  unsigned char* smem_raw) {
  const int tid = threadIdx.x;
  const int n_old = c.n_old, n_c = c.n_old + e.I, target = e.target;
  const size_t base = (size_t)unit * c.cap;
  EvictSmem s;
  evict_smem_layout(smem_raw, n_c, target, &s);

  for (int j = tid; j < n_c; j += NT) {
    if (j < n_old) { s.score[j] = c.sum_weights[base + j]; s.id[j] = c.kv_ids[base + j]; }
    else { s.score[j] = e.new_sum[(size_t)unit * e.I + (j - n_old)]; s.id[j] = e.pos0 + (j - n_old); }
  }
  __syncthreads();
  const float gf = (float)c.g;
  const int pad = sample_left_pad(c, smp);
  int id_win = 0x7fffffff;   // unordered cache, rule 1: pairs at positions >= id_win form the window of recent pairs
  // rule 3 (Sec. 2, SnapKV): the min(window, target) most recent candidates always stay; every other score is replaced
  // by the maximum over the `pool` neighbours centred on it, the window left out
  const int pool_body = n_c - min(c.window, target), pool_half = c.pool / 2;
  auto ave_bits = [&](int j) -> uint32_t {
    const float cnt = (float)(e.curr_id + 1 - s.id[j]);
    uint32_t b;   // ranking value >= 0: the bit pattern orders like the value
    if (c.rule == 0 || c.rule == 4) b = __float_as_uint(s.score[j] / (gf * cnt));   // average attention (Sec. 3.2)
    else if (c.rule == 1 && (FILL ? s.id[j] >= id_win : j >= n_c - target / 2)) b = 0x7f800000u;   // recent window: always kept
    else if (c.rule == 3) {
      if (j >= pool_body) b = 0x7f800000u;
      else {
        float m = s.score[j];
        for (int x = max(0, j - pool_half); x < min(pool_body, j + pool_half + 1); ++x) m = fmaxf(m, s.score[x]);
        b = __float_as_uint(m);
      }
    }
    else b = __float_as_uint(s.score[j]);                                // raw (sum of / current) weights
    if (pad == 0) return b;
    return s.id[j] < pad ? 0u : max(b, 1u);   // padding pairs rank below every real pair (left-padded samples)
  };

  // Radix select over the candidates `key_of` admits: the key of the need-th largest, and how many candidates equal
  // to that key belong to the `need` largest.  Four passes of 8 bits, histogram in shared memory.
  auto radix_kth_largest = [&](auto key_of, int need, uint32_t& out_key, int& out_need_eq) {
    uint32_t prefix = 0, mask = 0;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int t = tid; t < 256; t += NT) s.hist[t] = 0;
      __syncthreads();
      for (int j = tid; j < n_c; j += NT) {
        uint32_t b;
        if (key_of(j, b) && (b & mask) == prefix) atomicAdd(&s.hist[(b >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid < 32) {  // lane l owns digits 8l .. 8l+7; find the digit holding the need-th largest
        int loc = 0;
#pragma unroll
        for (int t = 0; t < 8; ++t) loc += (int)s.hist[tid * 8 + t];
        int incl = loc;  // suffix sums over lanes above
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, incl, off);
          if (tid + off < 32) incl += t;
        }
        const int above = incl - loc;
        if (above < need && need <= above + loc) {
          int cum = above, dg = 7;
          for (; dg >= 0; --dg) {
            const int h = (int)s.hist[tid * 8 + dg];
            if (cum + h >= need) break;
            cum += h;
          }
          s.misc[0] = tid * 8 + dg;
          s.misc[1] = need - cum;
        }
      }
      __syncthreads();
      prefix |= ((uint32_t)s.misc[0]) << shift;
      mask |= 255u << shift;
      need = s.misc[1];
      __syncthreads();
    }
    out_key = prefix;
    out_need_eq = need;
  };

  // Unordered cache: nothing that stays moves.  The candidates that stay but sit outside the first `target` rows
  // (new pairs, and cached pairs beyond row `target`) fill the rows that are freed or still empty, in ascending
  // order on both sides.
  auto fill_rows = [&](auto stays) {
    const int chunk = (n_c + NT - 1) / NT;
    const int jb = min(tid * chunk, n_c), je = min(jb + chunk, n_c);
    int nfree = 0, nsrc = 0;
    for (int j = jb; j < je; ++j) {
      const bool k = stays(j);
      nfree += (j < target && (j >= n_old || !k));
      nsrc += (k && (j >= target || j >= n_old));
    }
    int fb, sb;
    block_exclusive_scan2<NT>(nfree, nsrc, s.wsum, fb, sb);
    int nf = 0;
    for (int w = 0; w < NT / 32; ++w) nf += s.wsum[w];   // as many rows to fill as candidates to move
    for (int j = jb; j < je; ++j) {
      const bool k = stays(j);
      if (j < target && (j >= n_old || !k)) s.dst[fb++] = j;
      if (k && (j >= target || j >= n_old)) s.src[sb++] = j;
    }
    __syncthreads();
    if (c.moved != nullptr && tid == 0) atomicAdd(&c.moved[unit & 15], (unsigned long long)nf);
    for (int k = tid; k < nf; k += NT) {
      const int j = s.src[k], r = s.dst[k];
      if (!row_ok(c, r)) continue;
      c.sum_weights[base + r] = s.score[j];
      c.kv_ids[base + r] = s.id[j];
    }
    // sources lie outside the first `target` rows, destinations inside: no row is both read and written
    constexpr int PRF = D * (int)sizeof(T) / 16;
    T* kslab = reinterpret_cast<T*>(c.k_slab) + base * D;
    T* vslab = reinterpret_cast<T*>(c.v_slab) + base * D;
    for (int x0 = 0; x0 < nf * PRF; x0 += 4 * NT) {
      uint4 kb[4], vb[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int x = x0 + t * NT + tid;
        if (x < nf * PRF) {
          const int j = s.src[x / PRF], pc = x % PRF;
          if (j >= n_old) {
            const size_t off = ((size_t)(smp * e.I + (j - n_old)) * c.Hkv + kh) * D;
            kb[t] = ld_global_16(reinterpret_cast<const T*>(e.blk_k) + off + pc * (16 / sizeof(T)));
            vb[t] = ld_global_16(reinterpret_cast<const T*>(e.blk_v) + off + pc * (16 / sizeof(T)));
          } else {
            kb[t] = ld_global_16(kslab + (size_t)j * D + pc * (16 / sizeof(T)));
            vb[t] = ld_global_16(vslab + (size_t)j * D + pc * (16 / sizeof(T)));
          }
        }
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int x = x0 + t * NT + tid;
        if (x < nf * PRF) {
          const int r = s.dst[x / PRF], pc = x % PRF;
          if (!row_ok(c, r)) continue;
          st_global_16(kslab + (size_t)r * D + pc * (16 / sizeof(T)), kb[t]);
          st_global_16(vslab + (size_t)r * D + pc * (16 / sizeof(T)), vb[t]);
        }
      }
    }
  };

  if (target >= n_c) {
    for (int r = tid; r < n_c; r += NT) s.src[r] = r;
    __syncthreads();
  } else if (FILL && e.recent) {  // Algorithm 3's rule on an unordered cache: the `target` highest positions stay
    uint32_t key = 0;
    int unused;
    if (target > 0) radix_kth_largest([&](int j, uint32_t& k) { k = (uint32_t)s.id[j]; return true; }, target, key, unused);
    const int id_thr = target > 0 ? (int)key : 0x7fffffff;
    fill_rows([&](int j) { return s.id[j] >= id_thr; });
    return;
  } else if (e.recent) {  // Algorithm 3's rule: the most recent pairs stay, whatever their weights
    for (int r = tid; r < target; r += NT) s.src[r] = n_c - target + r;
    __syncthreads();
  } else {
    if (FILL && c.rule == 1 && target / 2 > 0) {   // the window's lowest position: the (target/2)-th highest
      uint32_t key;
      int unused;
      radix_kth_largest([&](int j, uint32_t& k) { k = (uint32_t)s.id[j]; return true; }, target / 2, key, unused);
      id_win = (int)key;
    }
    // ---- radix select: bit pattern `thr` of the target-th largest ave, and how many equal to it to keep
    uint32_t thr;
    int need_eq;
    const int n_std = c.rule == 4 ? (int)(((long long)target * c.std_permille) / 1000) : 0;
    if (n_std > 0) {
      // rule 4 (Sec. 2 / Sec. 3.2, RoCo): the n_std candidates whose weights have the largest standard deviation,
      // sqrt(E[w^2] - E[w]^2) over the g * (curr_id + 1 - kv_ids) weights received, stay whatever their average
      // (ties: lower position first); they enter the ranking below as +inf, the others with their average
      for (int j = tid; j < n_c; j += NT) {
        const float cnt = gf * (float)(e.curr_id + 1 - s.id[j]);
        const float sq = j < n_old ? c.sum_sq[base + j] : e.new_sq[(size_t)unit * e.I + (j - n_old)];
        const float mean = s.score[j] / cnt;
        s.bits[j] = __float_as_uint(sqrtf(fmaxf(sq / cnt - mean * mean, 0.f)));
      }
      __syncthreads();
      uint32_t thr_s;
      int need_s;
      radix_kth_largest([&](int j, uint32_t& key) { key = s.bits[j]; return true; }, n_std, thr_s, need_s);
      const int chunk = (n_c + NT - 1) / NT;
      const int jb = min(tid * chunk, n_c), je = min(jb + chunk, n_c);
      int eq = 0;
      for (int j = jb; j < je; ++j) eq += (s.bits[j] == thr_s);
      int unused, eq_before;
      block_exclusive_scan2<NT>(0, eq, s.wsum, unused, eq_before);
      for (int j = jb; j < je; ++j) {       // every thread rewrites its own chunk only
        const uint32_t b = s.bits[j];
        const bool prot = b > thr_s || (b == thr_s && eq_before < need_s);
        eq_before += (b == thr_s);
        s.bits[j] = prot ? 0x7f800000u : ave_bits(j);
      }
    } else {
      for (int j = tid; j < n_c; j += NT) s.bits[j] = ave_bits(j);   // one division per candidate, not one per pass
    }
    __syncthreads();
    radix_kth_largest([&](int j, uint32_t& key) { key = s.bits[j]; return true; }, target, thr, need_eq);
    if constexpr (FILL) {
      // ---- unordered cache: the rows of a cache are in no particular order, so (i) among the candidates equal to
      // the cut the need_eq lowest positions stay, found by a second select on kv_ids, and (ii) nothing that stays
      // moves: the candidates that stay but sit outside the first `target` rows (new pairs, and cached pairs beyond
      // row `target`) fill the rows that are freed or empty, in ascending order on both sides.
      const int eq_total = (int)s.hist[thr & 255u];   // the last pass counted the candidates equal to thr above the low digit
      int id_cut = 0x7fffffff;
      __syncthreads();   // the histogram is cleared by the next select
      if (need_eq < eq_total) {
        uint32_t key;
        int unused;
        radix_kth_largest([&](int j, uint32_t& k) { k = 0x7fffffffu - (uint32_t)s.id[j]; return s.bits[j] == thr; },
                          need_eq, key, unused);
        id_cut = (int)(0x7fffffffu - key);
      }
      fill_rows([&](int j) { const uint32_t b = s.bits[j]; return b > thr || (b == thr && s.id[j] <= id_cut); });
      return;
    }
    // ---- stable destinations: candidates above thr, plus the first need_eq equal to thr (lower id first)
    const int chunk = (n_c + NT - 1) / NT;
    const int jb = min(tid * chunk, n_c), je = min(jb + chunk, n_c);
    int gt = 0, eq = 0;
    for (int j = jb; j < je; ++j) {
      const uint32_t b = s.bits[j];
      gt += (b > thr);
      eq += (b == thr);
    }
    int gt_before, eq_before;
    block_exclusive_scan2<NT>(gt, eq, s.wsum, gt_before, eq_before);
    for (int j = jb; j < je; ++j) {
      const uint32_t b = s.bits[j];
      if (b > thr) { s.src[gt_before + min(eq_before, need_eq)] = j; ++gt_before; }
      else if (b == thr) {
        if (eq_before < need_eq) s.src[gt_before + eq_before] = j;
        ++eq_before;
      }
    }
    __syncthreads();
  }

  // ---- first row that changes (rows before it keep their place and their contents)
  if (tid == 0) s.misc[2] = target;
  __syncthreads();
  {
    int first = target;
    for (int r = tid; r < target; r += NT)
      if (s.src[r] != r || s.src[r] >= n_old) { first = r; break; }
    if (first < target) atomicMin(&s.misc[2], first);
  }
  __syncthreads();
  const int first_moved = s.misc[2];
  if (c.moved != nullptr && tid == 0 && first_moved < target)   // stable compaction: every row from there on moves
    atomicAdd(&c.moved[unit & 15], (unsigned long long)(target - first_moved));

  for (int r = first_moved + tid; r < target; r += NT) {
    const int j = s.src[r];
    if (!row_ok(c, r) || j < 0 || j >= n_c) continue;
    c.sum_weights[base + r] = s.score[j];
    c.kv_ids[base + r] = s.id[j];
  }
  if (c.sum_sq != nullptr) {
    // rule 4: the sums of squares take the same places; they pass through shared memory (the ranking values are no
    // longer needed), so that every load has completed before the first store
    for (int j = tid; j < n_c; j += NT)
      s.bits[j] = __float_as_uint(j < n_old ? c.sum_sq[base + j] : e.new_sq[(size_t)unit * e.I + (j - n_old)]);
    __syncthreads();
    for (int r = first_moved + tid; r < target; r += NT)
      if (row_ok(c, r)) c.sum_sq[base + r] = __uint_as_float(s.bits[s.src[r]]);
  }

  // ---- rows: ascending chunks, every source row index >= its destination, loads of a chunk complete
  // (barrier) before its stores; later chunks only read rows above everything written so far.
  constexpr int PR = D * (int)sizeof(T) / 16;  // 16-byte pieces per row
  constexpr int U = 4;                         // pieces per thread per tensor and chunk
  constexpr int RC = NT * U / PR;              // rows per chunk
  T* kslab = reinterpret_cast<T*>(c.k_slab) + base * D;
  T* vslab = reinterpret_cast<T*>(c.v_slab) + base * D;
  for (int r0 = first_moved; r0 < target; r0 += RC) {
    uint4 kb[U], vb[U];
    bool mv[U];
#pragma unroll
    for (int t = 0; t < U; ++t) {
      const int pidx = t * NT + tid, r = r0 + pidx / PR, pc = pidx % PR;
      mv[t] = false;
      if (r < target) {
        const int j = s.src[r];
        if (j >= n_old) {
          const size_t off = ((size_t)(smp * e.I + (j - n_old)) * c.Hkv + kh) * D;
          kb[t] = ld_global_16(reinterpret_cast<const T*>(e.blk_k) + off + pc * (16 / sizeof(T)));
          vb[t] = ld_global_16(reinterpret_cast<const T*>(e.blk_v) + off + pc * (16 / sizeof(T)));
          mv[t] = true;
        } else if (j != r) {
          kb[t] = ld_global_16(kslab + (size_t)j * D + pc * (16 / sizeof(T)));
          vb[t] = ld_global_16(vslab + (size_t)j * D + pc * (16 / sizeof(T)));
          mv[t] = true;
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < U; ++t) {
      if (mv[t]) {
        const int pidx = t * NT + tid, r = r0 + pidx / PR, pc = pidx % PR;
        if (!row_ok(c, r)) continue;
        st_global_16(kslab + (size_t)r * D + pc * (16 / sizeof(T)), kb[t]);
        st_global_16(vslab + (size_t)r * D + pc * (16 / sizeof(T)), vb[t]);
      }
    }
  }
}

template <typename T, int D, int NT>
__device__ inline void evict_body(const CacheView& c, int unit, int smp, int kh, const EvictArgs& e,
                                  unsigned char* smem_raw) {
  if (c.fill) evict_body_impl<T, D, NT, true>(c, unit, smp, kh, e, smem_raw);
  else evict_body_impl<T, D, NT, false>(c, unit, smp, kh, e, smem_raw);
}

}  // namespace bm
