// Host side of the C ABI: memory model and allocator (arena carving), argument validation, the host
// mirror of n / curr_id, and the stream-ordered launch sequence of every entry point.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <utility>
#include <algorithm>
#include <vector>

#include "../../include/batchmax.h"
#include "common.cuh"

namespace bm {
unsigned long long g_launch_count = 0;
int g_last_prefill_path = 0;

namespace {
bool g_profile_on = false;
std::vector<cudaEvent_t> g_event_pool;
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_pairs[kNumKernelClasses];
cudaEvent_t g_open_start = nullptr;
cudaEvent_t take_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
}  // namespace

void profile_begin(int, cudaStream_t st) {
  if (!g_profile_on) return;
  g_open_start = take_event();
  if (g_open_start) cudaEventRecord(g_open_start, st);
}
void profile_end(int cls, cudaStream_t st) {
  if (!g_profile_on || g_open_start == nullptr) return;
  cudaEvent_t stop = take_event();
  if (stop) cudaEventRecord(stop, st);
  g_pairs[cls].push_back({g_open_start, stop});
  g_open_start = nullptr;
}
}  // namespace bm

using namespace bm;

namespace {

// The CUDA error behind the most recent BM_ERR_CUDA of this thread (bm_last_cuda_error).
thread_local cudaError_t g_last_cuda_error = cudaSuccess;
bm_status_t cuda_fail(cudaError_t e) {
  g_last_cuda_error = e;
  return BM_ERR_CUDA;
}

#ifdef BM_DEBUG
// checked build: room for a 256-byte canary behind each of the (up to five) slabs as well
constexpr size_t kHeaderBytes = 4096;
constexpr size_t kCanaryBytes = 256;
#else
constexpr size_t kHeaderBytes = 1024;   // status word + room to align each of the four slabs to 256 B
constexpr size_t kCanaryBytes = 0;
#endif
constexpr int kCanaryByte = 0xA5;
constexpr int kMaxCandidates = 12288;   // candidates of one eviction must fit one CTA's shared memory
constexpr size_t kMaxSmem = 227 * 1024;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_size(int dtype) { return dtype == BM_BF16 ? 2 : 4; }

bool config_ok(const bm_config_t* c, bool need_batch) {
  if (c == nullptr) return false;
  if (need_batch && c->batch < 1) return false;
  if (c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads != 0) return false;
  const int g = c->n_q_heads / c->n_kv_heads;
  if (!(g == 1 || g == 2 || g == 4 || g == 8)) return false;
  if (!(c->head_dim == 64 || c->head_dim == 128)) return false;
  if (c->kv_max < 1 || c->block_max < 1 || c->growth < 1) return false;
  if (!(c->dtype == BM_F32 || c->dtype == BM_BF16)) return false;
  if (!(c->softmax_scale >= 0.f) || std::isinf(c->softmax_scale)) return false;
  if (c->device < 0 || c->max_call_samples < 0) return false;
  if (c->rule < 0 || c->rule > 4) return false;
  if (c->compaction < 0 || c->compaction > 1) return false;
  if (c->rule >= 3 && c->compaction != BM_COMPACT_STABLE) return false;   // both rank by the rows' position order
  if (c->rule == BM_RULE_WINDOW_POOLED && (c->window < 1 || c->pool < 1 || c->pool % 2 == 0 || c->pool > 255)) return false;
  if (c->rule == BM_RULE_AVERAGE_STD && (c->std_share_permille < 0 || c->std_share_permille > 1000)) return false;
  if ((long long)c->kv_max + c->growth > (1 << 24)) return false;
  return true;
}

size_t per_sample_bytes(const bm_config_t* c) {
  const size_t cap = (size_t)c->kv_max + c->growth;
  // key row, value row, sum_weights, kv_ids; under BM_RULE_AVERAGE_STD also the sum of squared weights
  const size_t per_row = 2 * (size_t)c->head_dim * elem_size(c->dtype) + 8 + (c->rule == BM_RULE_AVERAGE_STD ? 4 : 0);
  return (size_t)c->n_layers * c->n_kv_heads * cap * per_row;
}

int call_samples(const bm_config_t* c) { return c->max_call_samples > 0 ? c->max_call_samples : c->batch; }

size_t ws_lse_bytes(const bm_config_t* c) {
  return align_up(sizeof(float) * (size_t)call_samples(c) * c->n_q_heads * c->block_max, 256);
}
size_t ws_newsum_bytes(const bm_config_t* c) {
  return align_up(sizeof(float) * (size_t)call_samples(c) * c->n_kv_heads * c->block_max, 256);
}
size_t ws_pad_bytes(const bm_config_t* c) { return align_up(sizeof(int32_t) * (size_t)c->batch, 256); }
size_t ws_newsq_bytes(const bm_config_t* c) { return c->rule == BM_RULE_AVERAGE_STD ? ws_newsum_bytes(c) : 0; }

}  // namespace

struct bm_cache {
  bm_config_t cfg;
  int cap, g;
  size_t esz;
  float scale;
  char* k_slab;
  char* v_slab;
  float* sum_weights;
  float* sum_sq = nullptr;       // BM_RULE_AVERAGE_STD only
  int32_t* kv_ids;
  int32_t* status;
  float* ws_lse;
  float* ws_lse_own;             // the workspace's own (bm_prefill_block_static swaps ws_lse for the call)
  float* ws_new_sum;
  float* ws_new_sq = nullptr;    // BM_RULE_AVERAGE_STD only
  int32_t* left_pad = nullptr;   // [batch] device copy of the samples' padding counts (in the workspace)
  bool has_pad = false;          // some sample is left-padded
  // Padding leaves first at every eviction (under every rule), so how many padding pairs a sample's caches still
  // hold is a function of the calls made: the host tracks it and takes the kernels' padding-free instances again as
  // soon as a call's samples hold none and its block lies behind their padding.
  std::vector<int32_t> pad_host;  // [batch]
  std::vector<int32_t> npad;      // [L * b] padding pairs cached (kNpadUnknown after an import / set_len)
  bool count_moves = false;      // compactions add the rows they move to the counters in the status block
  std::vector<int32_t> n, curr_id;  // [L * b] host mirror
  std::vector<char*> canaries;      // checked build: the 256-byte guard behind each slab
  // host-fed calls run as a three-stage pipeline on streams owned by the handle -- input copies, the pass,
  // the output copy -- so that the three stages of consecutive calls overlap (PCIe is full duplex); the
  // caller's stream only waits for each call's output copy.  Up to four staging buffers can be in flight.
  cudaStream_t in_stream = nullptr, work_stream = nullptr, out_stream = nullptr;
  cudaEvent_t entry_ev = nullptr;
  struct Slot {
    void* staging = nullptr;
    cudaEvent_t in_done = nullptr, pass_done = nullptr, call_done = nullptr;
  };
  static constexpr int kSlots = 4;
  Slot slots[kSlots];
  int next_slot = 0;
  long dev_calls = 0, dev_calls_seen = -1;  // device-fed calls made / already ordered before the pipeline
};

namespace {

bm_status_t set_device(const bm_cache* c) {
  return cudaSetDevice(c->cfg.device) == cudaSuccess ? BM_OK : BM_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Range checks shared by the per-call entry points; returns the common n of the range in *n.
bm_status_t check_range(const bm_cache* c, int layer, int sample0, int nsamples, int* n, int* curr) {
  if (c == nullptr) return BM_ERR_INVALID;
  if (layer < 0 || layer >= c->cfg.n_layers) return BM_ERR_INVALID;
  if (sample0 < 0 || nsamples < 1 || (long long)sample0 + nsamples > c->cfg.batch) return BM_ERR_INVALID;
  if (nsamples > call_samples(&c->cfg)) return BM_ERR_INVALID;
  const size_t o = (size_t)layer * c->cfg.batch + sample0;
  for (int s = 1; s < nsamples; ++s)
    if (c->n[o + s] != c->n[o] || c->curr_id[o + s] != c->curr_id[o]) return BM_ERR_STATE;
  *n = c->n[o];
  *curr = c->curr_id[o];
  return BM_OK;
}

constexpr int32_t kNpadUnknown = 1 << 30;

// Does a call on this range, whose new pairs occupy positions [pos0, pos0 + I), meet any padding?
bool pad_active(const bm_cache* c, int layer, int sample0, int nsamples, int pos0, int I) {
  if (!c->has_pad) return false;
  const size_t o = (size_t)layer * c->cfg.batch + sample0;
  for (int s = 0; s < nsamples; ++s)
    if (c->npad[o + s] > 0 || (I > 0 && pos0 < c->pad_host[sample0 + s])) return true;
  return false;
}

// After a call that appended the positions [pos0, pos0 + I) and then removed `removed` pairs.
void pad_update(bm_cache* c, int layer, int sample0, int nsamples, int pos0, int I, int removed) {
  if (!c->has_pad) return;
  const size_t o = (size_t)layer * c->cfg.batch + sample0;
  for (int s = 0; s < nsamples; ++s) {
    int32_t& np = c->npad[o + s];
    if (np >= kNpadUnknown) continue;
    const int pad = c->pad_host[sample0 + s];
    const int added = I > 0 ? std::max(0, std::min(I, pad - pos0)) : 0;
    np = std::max(0, np + added - removed);
  }
}

CacheView make_view(const bm_cache* c, int layer, int sample0, int nsamples, int n_old, bool with_pad = true) {
  CacheView v;
  const size_t unit0 = ((size_t)layer * c->cfg.batch + sample0) * c->cfg.n_kv_heads;
  const size_t row0 = unit0 * c->cap;
  v.k_slab = c->k_slab + row0 * c->cfg.head_dim * c->esz;
  v.v_slab = c->v_slab + row0 * c->cfg.head_dim * c->esz;
  v.sum_weights = c->sum_weights + row0;
  v.kv_ids = c->kv_ids + row0;
  v.cap = c->cap;
  v.n_old = n_old;
  v.Hq = c->cfg.n_q_heads;
  v.Hkv = c->cfg.n_kv_heads;
  v.g = c->g;
  v.nsamples = nsamples;
  v.status = c->status;
  v.left_pad = (c->has_pad && with_pad) ? c->left_pad + sample0 : nullptr;
  v.rule = c->cfg.rule;
  v.fill = c->cfg.compaction == BM_COMPACT_FILL ? 1 : 0;
  v.sum_sq = c->sum_sq != nullptr ? c->sum_sq + row0 : nullptr;
  v.window = c->cfg.window; v.pool = c->cfg.pool; v.std_permille = c->cfg.std_share_permille;
  v.moved = c->count_moves ? reinterpret_cast<unsigned long long*>(c->status + 16) : nullptr;
  return v;
}

void set_mirror(bm_cache* c, int layer, int sample0, int nsamples, int n, int curr) {
  const size_t o = (size_t)layer * c->cfg.batch + sample0;
  for (int s = 0; s < nsamples; ++s) { c->n[o + s] = n; c->curr_id[o + s] = curr; }
}

}  // namespace

extern "C" {

bm_status_t bm_cache_bytes_per_sample(const bm_config_t* cfg, size_t* bytes) {
  if (!config_ok(cfg, false) || bytes == nullptr) return BM_ERR_INVALID;
  *bytes = per_sample_bytes(cfg);
  return BM_OK;
}

bm_status_t bm_arena_bytes(const bm_config_t* cfg, size_t* bytes) {
  if (!config_ok(cfg, true) || bytes == nullptr) return BM_ERR_INVALID;
  *bytes = kHeaderBytes + per_sample_bytes(cfg) * (size_t)cfg->batch;
  return BM_OK;
}

bm_status_t bm_max_batch(const bm_config_t* cfg, size_t hbm_budget_bytes, int32_t* b) {
  if (!config_ok(cfg, false) || b == nullptr) return BM_ERR_INVALID;
  if (hbm_budget_bytes <= kHeaderBytes) { *b = 0; return BM_OK; }
  const size_t q = (hbm_budget_bytes - kHeaderBytes) / per_sample_bytes(cfg);
  *b = (int32_t)(q > 0x7fffffff ? 0x7fffffff : q);
  return BM_OK;
}

bm_status_t bm_workspace_bytes(const bm_config_t* cfg, size_t* bytes) {
  if (!config_ok(cfg, true) || bytes == nullptr) return BM_ERR_INVALID;
  *bytes = ws_lse_bytes(cfg) + ws_newsum_bytes(cfg) + ws_pad_bytes(cfg) + ws_newsq_bytes(cfg);
  return BM_OK;
}

bm_status_t bm_cache_create(const bm_config_t* cfg, void* arena, size_t arena_bytes, void* workspace,
                            size_t workspace_bytes, void* cuda_stream, bm_cache_t** out) {
  if (!config_ok(cfg, true) || arena == nullptr || workspace == nullptr || out == nullptr) return BM_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return BM_ERR_INVALID;
  size_t need_arena = 0, need_ws = 0;
  bm_arena_bytes(cfg, &need_arena);
  bm_workspace_bytes(cfg, &need_ws);
  if (arena_bytes < need_arena || workspace_bytes < need_ws) return BM_ERR_OOM;
  if (cudaSetDevice(cfg->device) != cudaSuccess) return BM_ERR_CUDA;

  bm_cache* c = new (std::nothrow) bm_cache();
  if (c == nullptr) return BM_ERR_OOM;
  c->cfg = *cfg;
  c->cap = cfg->kv_max + cfg->growth;
  c->g = cfg->n_q_heads / cfg->n_kv_heads;
  c->esz = elem_size(cfg->dtype);
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  const size_t rows = (size_t)cfg->n_layers * cfg->batch * cfg->n_kv_heads * c->cap;
  const size_t slab = rows * cfg->head_dim * c->esz;  // multiple of 128 bytes
  char* p = static_cast<char*>(arena);
  c->status = reinterpret_cast<int32_t*>(p);
  // header = 256 B status block + up to 3 * 256 B of slab alignment padding
  size_t off = 256;
  auto guard = [&]() {   // checked build: a canary behind the slab that ends at `off`
    if (kCanaryBytes > 0) { c->canaries.push_back(p + off); off += kCanaryBytes; }
  };
  c->k_slab = p + off;                                   off = align_up(off + slab, 256);      guard();
  c->v_slab = p + off;                                   off = align_up(off + slab, 256);      guard();
  c->sum_weights = reinterpret_cast<float*>(p + off);    off = align_up(off + rows * 4, 256);  guard();
  c->kv_ids = reinterpret_cast<int32_t*>(p + off);       off = kCanaryBytes > 0 ? align_up(off + rows * 4, 256) : off + rows * 4;
  guard();
  if (cfg->rule == BM_RULE_AVERAGE_STD) {   // a fifth slab of 4-byte entries right behind the fourth
    c->sum_sq = reinterpret_cast<float*>(p + off);       off = kCanaryBytes > 0 ? align_up(off + rows * 4, 256) : off + rows * 4;
    guard();
  }
  if (off > need_arena) { delete c; return BM_ERR_OOM; }
  c->ws_lse = static_cast<float*>(workspace);
  c->ws_lse_own = c->ws_lse;
  c->ws_new_sum = reinterpret_cast<float*>(static_cast<char*>(workspace) + ws_lse_bytes(cfg));
  c->left_pad = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + ws_lse_bytes(cfg) + ws_newsum_bytes(cfg));
  if (cfg->rule == BM_RULE_AVERAGE_STD)
    c->ws_new_sq = reinterpret_cast<float*>(static_cast<char*>(workspace) + ws_lse_bytes(cfg) + ws_newsum_bytes(cfg) +
                                            ws_pad_bytes(cfg));
  c->n.assign((size_t)cfg->n_layers * cfg->batch, 0);
  c->curr_id.assign((size_t)cfg->n_layers * cfg->batch, -1);
  // Unwritten rows are read as zero-weight padding by the tiled kernels, so they must hold finite values.
  if (cudaMemsetAsync(arena, 0, need_arena, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    delete c;
    return BM_ERR_CUDA;
  }
  for (char* g : c->canaries)
    if (cudaMemsetAsync(g, kCanaryByte, kCanaryBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
      delete c;
      return BM_ERR_CUDA;
    }
  *out = c;
  return BM_OK;
}

bm_status_t bm_cache_destroy(bm_cache_t* cache) {
  if (cache == nullptr) return BM_ERR_INVALID;
  if (cache->in_stream != nullptr) {
    cudaSetDevice(cache->cfg.device);
    for (cudaStream_t st : {cache->in_stream, cache->work_stream, cache->out_stream})
      if (st != nullptr) { cudaStreamSynchronize(st); cudaStreamDestroy(st); }
    for (auto& sl : cache->slots)
      for (cudaEvent_t ev : {sl.in_done, sl.pass_done, sl.call_done})
        if (ev) cudaEventDestroy(ev);
    if (cache->entry_ev) cudaEventDestroy(cache->entry_ev);
  }
  delete cache;
  return BM_OK;
}

static bm_status_t run_evict(bm_cache* c, const CacheView& view, const EvictArgs& e, cudaStream_t st) {
  if (evict_smem_bytes(view.n_old + e.I, e.target) > kMaxSmem) return BM_ERR_CAPACITY;
  const cudaError_t err = launch_evict(c->cfg.dtype, c->cfg.head_dim, view, e, st);
  return err == cudaSuccess ? BM_OK : cuda_fail(err);
}

bm_status_t bm_prefill_block(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, const void* q,
                             const void* k, const void* v, int32_t I, int32_t pos0, void* out,
                             int32_t evict_to, void* cuda_stream) {
  int n_old = 0, curr = 0;
  bm_status_t s = check_range(c, layer, sample0, nsamples, &n_old, &curr);
  if (s != BM_OK) return s;
  ++c->dev_calls;  // a later host-fed call orders its pipeline after this one
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return BM_ERR_INVALID;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return BM_ERR_INVALID;
  if (I < 1 || I > c->cfg.block_max) return BM_ERR_INVALID;
  if ((long long)nsamples * c->cfg.n_kv_heads > 65535) return BM_ERR_CAPACITY;   // caches of a call index grid.y
  if (pos0 != curr + 1) return BM_ERR_STATE;
  const int n_c = n_old + I;
  const int target = (evict_to >= 0 && n_c > evict_to) ? evict_to : n_c;
  if (target > c->cap) return BM_ERR_CAPACITY;
  if (n_c > kMaxCandidates || evict_smem_bytes(n_c, target) > kMaxSmem) return BM_ERR_CAPACITY;
  if ((s = set_device(c)) != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  CacheView view = make_view(c, layer, sample0, nsamples, n_old, pad_active(c, layer, sample0, nsamples, pos0, I));
  BlockArgs a;
  a.q = q; a.k = k; a.v = v; a.out = out;
  // A range's scratch sits at its samples' own place in the workspace when the workspace covers the range there, so
  // that calls on disjoint sample ranges may be in flight on different streams at the same time (stride block_max,
  // whatever I is); micro-batched calls on a smaller workspace, and the static scratch, start at its beginning.
  const bool own_ws = c->ws_lse == c->ws_lse_own;
  const size_t s_off = (own_ws && sample0 + nsamples <= call_samples(&c->cfg)) ? (size_t)sample0 : 0;
  a.lse = c->ws_lse + s_off * c->cfg.n_q_heads * c->cfg.block_max;
  a.new_sum = c->ws_new_sum + s_off * c->cfg.n_kv_heads * c->cfg.block_max;
  a.new_sq = c->ws_new_sq != nullptr ? c->ws_new_sq + s_off * c->cfg.n_kv_heads * c->cfg.block_max : nullptr;
  a.I = I; a.pos0 = pos0; a.scale = c->scale;

  int used_tc = 0;
  if (c->cfg.dtype == BM_BF16 && tc_path_available()) {
    if (cudaError_t e = launch_attn_tc(c->cfg.head_dim, view, a, st, &used_tc); e != cudaSuccess) return cuda_fail(e);
  }
  if (!used_tc)
    if (cudaError_t e = launch_attn_simt(c->cfg.dtype, c->cfg.head_dim, view, a, st); e != cudaSuccess) return cuda_fail(e);
  g_last_prefill_path = used_tc;
  int used_tc_score = 0;
  if (c->cfg.dtype == BM_BF16 && tc_path_available()) {
    if (cudaError_t e = launch_score_tc(c->cfg.head_dim, view, a, st, &used_tc_score); e != cudaSuccess) return cuda_fail(e);
  }
  if (!used_tc_score)
    if (cudaError_t e = launch_score_simt(c->cfg.dtype, c->cfg.head_dim, view, a, st); e != cudaSuccess) return cuda_fail(e);

  int n_new = 0;
  if (target > 0) {
    EvictArgs e;
    e.blk_k = k; e.blk_v = v; e.new_sum = a.new_sum; e.new_sq = a.new_sq;
    e.I = I; e.pos0 = pos0; e.curr_id = pos0 + I - 1; e.target = target;
    if ((s = run_evict(c, view, e, st)) != BM_OK) return s;
    n_new = target;
  }
  set_mirror(c, layer, sample0, nsamples, n_new, pos0 + I - 1);
  pad_update(c, layer, sample0, nsamples, pos0, I, n_c - n_new);
  return BM_OK;
}

bm_status_t bm_decode_step(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, const void* q,
                           const void* k, const void* v, void* out, int32_t evict_to, void* cuda_stream) {
  int n_old = 0, curr = 0;
  bm_status_t s = check_range(c, layer, sample0, nsamples, &n_old, &curr);
  if (s != BM_OK) return s;
  ++c->dev_calls;  // a later host-fed call orders its pipeline after this one
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) return BM_ERR_INVALID;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return BM_ERR_INVALID;
  const int n1 = n_old + 1;
  if (n1 > c->cap) return BM_ERR_CAPACITY;
  const int target = (evict_to >= 0 && n1 > evict_to) ? evict_to : -1;
  const bool mma = c->cfg.dtype == BM_BF16;   // bf16 caches decode on the tensor-core kernel, fp32 caches on the SIMT one
  const size_t smem = mma ? decode_mma_smem_bytes(c->cfg.head_dim, c->g, n1, target)
                          : decode_smem_bytes(c->cfg.head_dim, c->g, n1, target);
  if (n1 > kMaxCandidates || smem > kMaxSmem) return BM_ERR_CAPACITY;
  if ((s = set_device(c)) != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int pos = curr + 1;
  CacheView view = make_view(c, layer, sample0, nsamples, n_old, pad_active(c, layer, sample0, nsamples, pos, 1));
  // target 0: nothing survives -- run the attention and the update, then empty the caches on the host mirror
  const int kernel_target = target == 0 ? -1 : target;
  const cudaError_t err = mma ? launch_decode_mma(c->cfg.head_dim, view, q, k, v, out, pos, c->scale, kernel_target, st)
                              : launch_decode(c->cfg.dtype, c->cfg.head_dim, view, q, k, v, out, pos, c->scale,
                                              kernel_target, st);
  if (err != cudaSuccess) return cuda_fail(err);
  const int n_new = target >= 0 ? target : n1;
  set_mirror(c, layer, sample0, nsamples, n_new, pos);
  pad_update(c, layer, sample0, nsamples, pos, 1, n1 - n_new);
  return BM_OK;
}

static bm_status_t evict_cached(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, int32_t target,
                                bool recent, void* cuda_stream) {
  int n_old = 0, curr = 0;
  bm_status_t s = check_range(c, layer, sample0, nsamples, &n_old, &curr);
  if (s != BM_OK) return s;
  ++c->dev_calls;  // a later host-fed call orders its pipeline after this one
  if (target < 0) return BM_ERR_INVALID;
  if (n_old <= target) return BM_OK;
  if (target == 0) {
    set_mirror(c, layer, sample0, nsamples, 0, curr);
    pad_update(c, layer, sample0, nsamples, 0, 0, n_old);
    if (c->has_pad)                                   // an empty cache holds no padding, whatever was unknown before
      for (int s2 = 0; s2 < nsamples; ++s2) c->npad[(size_t)layer * c->cfg.batch + sample0 + s2] = 0;
    return BM_OK;
  }
  if (n_old > kMaxCandidates) return BM_ERR_CAPACITY;
  if ((s = set_device(c)) != BM_OK) return s;
  CacheView view = make_view(c, layer, sample0, nsamples, n_old, pad_active(c, layer, sample0, nsamples, 0, 0));
  EvictArgs e;
  e.blk_k = nullptr; e.blk_v = nullptr; e.new_sum = nullptr;
  e.I = 0; e.pos0 = 0; e.curr_id = curr; e.target = target; e.recent = recent ? 1 : 0;
  if ((s = run_evict(c, view, e, static_cast<cudaStream_t>(cuda_stream))) != BM_OK) return s;
  set_mirror(c, layer, sample0, nsamples, target, curr);
  pad_update(c, layer, sample0, nsamples, 0, 0, n_old - target);   // both rules remove padding before anything else
  return BM_OK;
}

bm_status_t bm_evict(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, int32_t target,
                     void* cuda_stream) {
  return evict_cached(c, layer, sample0, nsamples, target, false, cuda_stream);
}

bm_status_t bm_keep_most_recent(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, int32_t keep,
                                void* cuda_stream) {
  return evict_cached(c, layer, sample0, nsamples, keep, true, cuda_stream);
}

// ---- host-fed variants ---------------------------------------------------------------------------
static void staging_layout(const bm_config_t* cfg, int nsamples, int I, size_t* oq, size_t* ok, size_t* ov,
                           size_t* oo, size_t* total, size_t* qbytes, size_t* kbytes) {
  const size_t e = elem_size(cfg->dtype);
  *qbytes = (size_t)nsamples * I * cfg->n_q_heads * cfg->head_dim * e;
  *kbytes = (size_t)nsamples * I * cfg->n_kv_heads * cfg->head_dim * e;
  size_t off = 0;
  *oq = off; off = align_up(off + *qbytes, 256);
  *ok = off; off = align_up(off + *kbytes, 256);
  *ov = off; off = align_up(off + *kbytes, 256);
  *oo = off; off = align_up(off + *qbytes, 256);
  *total = off;
}

bm_status_t bm_staging_bytes(const bm_config_t* cfg, int32_t nsamples, int32_t I, size_t* bytes) {
  if (!config_ok(cfg, false) || nsamples < 1 || I < 1 || bytes == nullptr) return BM_ERR_INVALID;
  size_t oq, ok, ov, oo, qb, kb;
  staging_layout(cfg, nsamples, I, &oq, &ok, &ov, &oo, bytes, &qb, &kb);
  return BM_OK;
}

static bm_status_t host_pass(bm_cache_t* c, int layer, int sample0, int nsamples, const void* q, const void* k,
                             const void* v, int I, int pos0, void* out, int evict_to, void* staging,
                             size_t staging_bytes, void* cuda_stream, bool decode) {
  int n_old = 0, curr = 0;
  bm_status_t s = check_range(c, layer, sample0, nsamples, &n_old, &curr);
  if (s != BM_OK) return s;
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr || staging == nullptr) return BM_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(staging) & 255u) return BM_ERR_INVALID;
  if (I < 1 || I > c->cfg.block_max) return BM_ERR_INVALID;
  if ((long long)nsamples * c->cfg.n_kv_heads > 65535) return BM_ERR_CAPACITY;   // caches of a call index grid.y
  size_t oq, ok, ov, oo, total, qb, kb;
  staging_layout(&c->cfg, nsamples, I, &oq, &ok, &ov, &oo, &total, &qb, &kb);
  if (staging_bytes < total) return BM_ERR_OOM;
  // validate the pass itself before any copy is enqueued
  if (decode) {
    if (n_old + 1 > c->cap) return BM_ERR_CAPACITY;
  } else {
    if (pos0 != curr + 1) return BM_ERR_STATE;
    const int n_c = n_old + I;
    const int target = (evict_to >= 0 && n_c > evict_to) ? evict_to : n_c;
    if (target > c->cap || n_c > kMaxCandidates || evict_smem_bytes(n_c, target) > kMaxSmem) return BM_ERR_CAPACITY;
  }
  if ((s = set_device(c)) != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* sp = static_cast<char*>(staging);
  // Inputs go over an internal stream unless cuda_stream is being captured into a graph.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  cudaStreamIsCapturing(st, &cap);
  bm_cache::Slot* slot = nullptr;
  cudaStream_t in = st, work = st, outs = st;
  if (cap == cudaStreamCaptureStatusNone) {
    if (c->in_stream == nullptr) {
      bool ok = cudaStreamCreateWithFlags(&c->in_stream, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&c->work_stream, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking) == cudaSuccess &&
                cudaEventCreateWithFlags(&c->entry_ev, cudaEventDisableTiming) == cudaSuccess;
      for (auto& sl : c->slots)
        ok = ok && cudaEventCreateWithFlags(&sl.in_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&sl.pass_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&sl.call_done, cudaEventDisableTiming) == cudaSuccess;
      if (!ok) return BM_ERR_CUDA;
    }
    for (auto& sl : c->slots)
      if (sl.staging == staging) slot = &sl;
    if (slot == nullptr) { slot = &c->slots[c->next_slot]; c->next_slot = (c->next_slot + 1) % bm_cache::kSlots; }
    in = c->in_stream;
    work = c->work_stream;
    outs = c->out_stream;
    // Device-fed calls (and the creation of the cache) since the last host-fed one are ordered before the
    // pipeline through cuda_stream.  Consecutive host-fed calls skip this, or each pass would wait for the
    // previous call's output copy, which cuda_stream has been made to wait for.
    if (c->dev_calls_seen != c->dev_calls) {
      if (cudaEventRecord(c->entry_ev, st) != cudaSuccess || cudaStreamWaitEvent(work, c->entry_ev, 0) != cudaSuccess)
        return BM_ERR_CUDA;
    }
    // the staging buffer is free again once the previous call that used this slot has finished with it
    if (slot->staging != nullptr && cudaStreamWaitEvent(in, slot->call_done, 0) != cudaSuccess) return BM_ERR_CUDA;
    slot->staging = staging;
  }
  if (cudaMemcpyAsync(sp + oq, q, qb, cudaMemcpyHostToDevice, in) != cudaSuccess) return BM_ERR_CUDA;
  if (cudaMemcpyAsync(sp + ok, k, kb, cudaMemcpyHostToDevice, in) != cudaSuccess) return BM_ERR_CUDA;
  if (cudaMemcpyAsync(sp + ov, v, kb, cudaMemcpyHostToDevice, in) != cudaSuccess) return BM_ERR_CUDA;
  if (slot != nullptr) {
    if (cudaEventRecord(slot->in_done, in) != cudaSuccess) return BM_ERR_CUDA;
    if (cudaStreamWaitEvent(work, slot->in_done, 0) != cudaSuccess) return BM_ERR_CUDA;
  }
  s = decode ? bm_decode_step(c, layer, sample0, nsamples, sp + oq, sp + ok, sp + ov, sp + oo, evict_to, work)
             : bm_prefill_block(c, layer, sample0, nsamples, sp + oq, sp + ok, sp + ov, I, pos0, sp + oo, evict_to,
                                work);
  if (s != BM_OK) return s;
  if (slot != nullptr) {
    c->dev_calls_seen = c->dev_calls;
    if (cudaEventRecord(slot->pass_done, work) != cudaSuccess) return BM_ERR_CUDA;
    if (cudaStreamWaitEvent(outs, slot->pass_done, 0) != cudaSuccess) return BM_ERR_CUDA;
  }
  if (cudaMemcpyAsync(out, sp + oo, qb, cudaMemcpyDeviceToHost, outs) != cudaSuccess) return BM_ERR_CUDA;
  if (slot != nullptr) {
    if (cudaEventRecord(slot->call_done, outs) != cudaSuccess) return BM_ERR_CUDA;
    if (cudaStreamWaitEvent(st, slot->call_done, 0) != cudaSuccess) return BM_ERR_CUDA;
  }
  return BM_OK;
}

bm_status_t bm_prefill_block_host(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, const void* q,
                                  const void* k, const void* v, int32_t I, int32_t pos0, void* out,
                                  int32_t evict_to, void* staging, size_t staging_bytes, void* cuda_stream) {
  return host_pass(c, layer, sample0, nsamples, q, k, v, I, pos0, out, evict_to, staging, staging_bytes,
                   cuda_stream, false);
}

bm_status_t bm_decode_step_host(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples, const void* q,
                                const void* k, const void* v, void* out, int32_t evict_to, void* staging,
                                size_t staging_bytes, void* cuda_stream) {
  return host_pass(c, layer, sample0, nsamples, q, k, v, 1, 0, out, evict_to, staging, staging_bytes, cuda_stream,
                   true);
}

// ---- state access ----------------------------------------------------------------------------------
bm_status_t bm_cache_len(const bm_cache_t* c, int32_t layer, int32_t sample, int32_t* n, int32_t* curr_id) {
  if (c == nullptr || n == nullptr) return BM_ERR_INVALID;
  if (layer < 0 || layer >= c->cfg.n_layers || sample < 0 || sample >= c->cfg.batch) return BM_ERR_INVALID;
  const size_t o = (size_t)layer * c->cfg.batch + sample;
  *n = c->n[o];
  if (curr_id != nullptr) *curr_id = c->curr_id[o];
  return BM_OK;
}

bm_status_t bm_cache_set_left_pad(bm_cache_t* c, const int32_t* pads, void* cuda_stream) {
  if (c == nullptr) return BM_ERR_INVALID;
  for (int v : c->n)
    if (v != 0) return BM_ERR_STATE;
  for (int v : c->curr_id)
    if (v != -1) return BM_ERR_STATE;
  if (c->cfg.rule == BM_RULE_AVERAGE_STD) return BM_ERR_INVALID;   // that rule is defined without padding here
  bool any = false;
  if (pads != nullptr)
    for (int s = 0; s < c->cfg.batch; ++s) {
      if (pads[s] < 0) return BM_ERR_INVALID;
      any = any || pads[s] > 0;
    }
  c->has_pad = any;
  if (!any) return BM_OK;
  c->pad_host.assign(pads, pads + c->cfg.batch);
  c->npad.assign((size_t)c->cfg.n_layers * c->cfg.batch, 0);
  bm_status_t st = set_device(c);
  if (st != BM_OK) return st;
  ++c->dev_calls;
  // the source may be pageable: the runtime stages it before this call returns
  if (cudaMemcpyAsync(c->left_pad, pads, sizeof(int32_t) * (size_t)c->cfg.batch, cudaMemcpyHostToDevice,
                      static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return BM_ERR_CUDA;
  return BM_OK;
}

bm_status_t bm_cache_count_moved_rows(bm_cache_t* c, int32_t on) {
  if (c == nullptr) return BM_ERR_INVALID;
  c->count_moves = on != 0;
  return BM_OK;
}

bm_status_t bm_cache_moved_rows(bm_cache_t* c, uint64_t* rows, int32_t reset, void* cuda_stream) {
  if (c == nullptr || rows == nullptr) return BM_ERR_INVALID;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long part[16];
  void* dev = c->status + 16;
  if (cudaMemcpyAsync(part, dev, sizeof(part), cudaMemcpyDeviceToHost, st) != cudaSuccess) return BM_ERR_CUDA;
  if (reset && cudaMemsetAsync(dev, 0, sizeof(part), st) != cudaSuccess) return BM_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return BM_ERR_CUDA;
  uint64_t tot = 0;
  for (unsigned long long v : part) tot += v;
  *rows = tot;
  return BM_OK;
}

bm_status_t bm_cache_set_len(bm_cache_t* c, int32_t layer, int32_t sample, int32_t n, int32_t curr_id) {
  if (c == nullptr) return BM_ERR_INVALID;
  if (layer < 0 || layer >= c->cfg.n_layers || sample < 0 || sample >= c->cfg.batch) return BM_ERR_INVALID;
  if (n < 0 || n > c->cap || curr_id < -1) return BM_ERR_INVALID;
  const size_t o = (size_t)layer * c->cfg.batch + sample;
  c->n[o] = n;
  c->curr_id[o] = curr_id;
  if (c->has_pad) c->npad[o] = n > 0 ? kNpadUnknown : 0;   // contents come from outside: assume padding may be there
  return BM_OK;
}

static bm_status_t unit_offsets(const bm_cache* c, int layer, int sample, int kv_head, size_t* row0) {
  if (c == nullptr) return BM_ERR_INVALID;
  if (layer < 0 || layer >= c->cfg.n_layers || sample < 0 || sample >= c->cfg.batch) return BM_ERR_INVALID;
  if (kv_head < 0 || kv_head >= c->cfg.n_kv_heads) return BM_ERR_INVALID;
  *row0 = (((size_t)layer * c->cfg.batch + sample) * c->cfg.n_kv_heads + kv_head) * c->cap;
  return BM_OK;
}

bm_status_t bm_cache_export(bm_cache_t* c, int32_t layer, int32_t sample, int32_t kv_head, int32_t* kv_ids,
                            float* sum_weights, void* k_rows, void* v_rows, int32_t* n, void* cuda_stream) {
  size_t row0 = 0;
  bm_status_t s = unit_offsets(c, layer, sample, kv_head, &row0);
  if (s != BM_OK) return s;
  if (n == nullptr) return BM_ERR_INVALID;
  if ((s = set_device(c)) != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int cnt = c->n[(size_t)layer * c->cfg.batch + sample];
  *n = cnt;
  const size_t rb = (size_t)c->cfg.head_dim * c->esz;
  bool ok = true;
  if (cnt > 0) {
    if (kv_ids) ok &= cudaMemcpyAsync(kv_ids, c->kv_ids + row0, 4 * (size_t)cnt, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (sum_weights) ok &= cudaMemcpyAsync(sum_weights, c->sum_weights + row0, 4 * (size_t)cnt, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (k_rows) ok &= cudaMemcpyAsync(k_rows, c->k_slab + row0 * rb, rb * cnt, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (v_rows) ok &= cudaMemcpyAsync(v_rows, c->v_slab + row0 * rb, rb * cnt, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  }
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? BM_OK : BM_ERR_CUDA;
}

bm_status_t bm_cache_import(bm_cache_t* c, int32_t layer, int32_t sample, int32_t kv_head, const int32_t* kv_ids,
                            const float* sum_weights, const void* k_rows, const void* v_rows, int32_t n,
                            void* cuda_stream) {
  size_t row0 = 0;
  bm_status_t s = unit_offsets(c, layer, sample, kv_head, &row0);
  if (s != BM_OK) return s;
  if (kv_ids == nullptr || sum_weights == nullptr || k_rows == nullptr || v_rows == nullptr) return BM_ERR_INVALID;
  if (n != c->n[(size_t)layer * c->cfg.batch + sample]) return BM_ERR_STATE;
  if ((s = set_device(c)) != BM_OK) return s;
  ++c->dev_calls;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t rb = (size_t)c->cfg.head_dim * c->esz;
  bool ok = true;
  if (n > 0) {
    ok &= cudaMemcpyAsync(c->kv_ids + row0, kv_ids, 4 * (size_t)n, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(c->sum_weights + row0, sum_weights, 4 * (size_t)n, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(c->k_slab + row0 * rb, k_rows, rb * n, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(c->v_slab + row0 * rb, v_rows, rb * n, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? BM_OK : BM_ERR_CUDA;
}

bm_status_t bm_cache_export_sum_sq(bm_cache_t* c, int32_t layer, int32_t sample, int32_t kv_head, float* sum_sq,
                                   void* cuda_stream) {
  size_t row0 = 0;
  bm_status_t s = unit_offsets(c, layer, sample, kv_head, &row0);
  if (s != BM_OK) return s;
  if (sum_sq == nullptr || c->sum_sq == nullptr) return BM_ERR_INVALID;
  if ((s = set_device(c)) != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int cnt = c->n[(size_t)layer * c->cfg.batch + sample];
  bool ok = true;
  if (cnt > 0) ok &= cudaMemcpyAsync(sum_sq, c->sum_sq + row0, 4 * (size_t)cnt, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? BM_OK : BM_ERR_CUDA;
}

bm_status_t bm_cache_import_sum_sq(bm_cache_t* c, int32_t layer, int32_t sample, int32_t kv_head, const float* sum_sq,
                                   void* cuda_stream) {
  size_t row0 = 0;
  bm_status_t s = unit_offsets(c, layer, sample, kv_head, &row0);
  if (s != BM_OK) return s;
  if (sum_sq == nullptr || c->sum_sq == nullptr) return BM_ERR_INVALID;
  if ((s = set_device(c)) != BM_OK) return s;
  ++c->dev_calls;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int cnt = c->n[(size_t)layer * c->cfg.batch + sample];
  bool ok = true;
  if (cnt > 0) ok &= cudaMemcpyAsync(c->sum_sq + row0, sum_sq, 4 * (size_t)cnt, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaStreamSynchronize(st) == cudaSuccess;
  return ok ? BM_OK : BM_ERR_CUDA;
}

bm_status_t bm_cache_status(bm_cache_t* c, int32_t* device_status, void* cuda_stream) {
  if (c == nullptr || device_status == nullptr) return BM_ERR_INVALID;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t w = 0;
  if (cudaMemcpyAsync(&w, c->status, sizeof(w), cudaMemcpyDeviceToHost, st) != cudaSuccess) return BM_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return BM_ERR_CUDA;
  *device_status = w;
  return BM_OK;
}

bm_status_t bm_cache_clear_status(bm_cache_t* c, void* cuda_stream) {
  if (c == nullptr) return BM_ERR_INVALID;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  return cudaMemsetAsync(c->status, 0, sizeof(int32_t), static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? BM_OK : BM_ERR_CUDA;
}

bm_status_t bm_selftest_wait_timeout(bm_cache_t* c, void* cuda_stream) {
  if (c == nullptr) return BM_ERR_INVALID;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  return launch_wait_timeout_selftest(c->status, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? BM_OK : BM_ERR_CUDA;
}

int32_t bm_debug_build(void) {
#ifdef BM_DEBUG
  return 1;
#else
  return 0;
#endif
}

bm_status_t bm_cache_check_canaries(bm_cache_t* c, int32_t* damaged, void* cuda_stream) {
  if (c == nullptr || damaged == nullptr) return BM_ERR_INVALID;
  *damaged = 0;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  std::vector<unsigned char> host(256);
  for (char* g : c->canaries) {
    if (cudaMemcpyAsync(host.data(), g, 256, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return BM_ERR_CUDA;
    for (unsigned char b : host)
      if (b != kCanaryByte) { ++*damaged; break; }
  }
  return BM_OK;
}

bm_status_t bm_selftest_row_check(bm_cache_t* c, void* cuda_stream) {
  if (c == nullptr) return BM_ERR_INVALID;
  bm_status_t s = set_device(c);
  if (s != BM_OK) return s;
  const CacheView view = make_view(c, 0, 0, 1, 0, false);
  const cudaError_t e = launch_row_check_selftest(view, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? BM_OK : cuda_fail(e);
}

bm_status_t bm_profile_enable(int32_t on) {
  g_profile_on = on != 0;
  return BM_OK;
}

bm_status_t bm_profile_read(int32_t kernel_class, float* total_ms, int32_t* launches) {
  if (kernel_class < 0 || kernel_class >= kNumKernelClasses || total_ms == nullptr || launches == nullptr)
    return BM_ERR_INVALID;
  float tot = 0.f;
  int cnt = 0;
  bool ok = true;
  for (auto& pr : g_pairs[kernel_class]) {
    float ms = 0.f;
    if (pr.first && pr.second && cudaEventSynchronize(pr.second) == cudaSuccess &&
        cudaEventElapsedTime(&ms, pr.first, pr.second) == cudaSuccess) { tot += ms; ++cnt; }
    else ok = false;
    if (pr.first) g_event_pool.push_back(pr.first);
    if (pr.second) g_event_pool.push_back(pr.second);
  }
  g_pairs[kernel_class].clear();
  *total_ms = tot;
  *launches = cnt;
  return ok ? BM_OK : BM_ERR_CUDA;
}

const char* bm_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

uint64_t bm_kernel_launch_count(void) { return (uint64_t)g_launch_count; }
int32_t bm_last_prefill_path(void) { return g_last_prefill_path; }

const char* bm_status_string(bm_status_t s) {
  switch (s) {
    case BM_OK: return "ok";
    case BM_ERR_INVALID: return "invalid argument";
    case BM_ERR_OOM: return "arena, workspace or budget too small";
    case BM_ERR_CAPACITY: return "cache capacity or candidate limit exceeded";
    case BM_ERR_STATE: return "call out of order for the cache state";
    case BM_ERR_CUDA: return "CUDA call failed";
    case BM_ERR_TIMEOUT: return "bounded device wait expired";
    case BM_ERR_BOUNDS: return "a kernel of the checked build met a row index outside its cache";
    default: return "unknown status";
  }
}

}  // extern "C"

// ---- prefill block with library-resident scratch -------------------------------------------------------
// Some callers cannot hand the library a workspace they allocated: a serving loop that froze its memory
// plan at start-up, a plug-in running under a framework whose caching allocator owns all device memory,
// or a host thread that is not allowed to make allocating CUDA calls at all.  For them the per-call
// scratch of the block forward pass (the log-sum-exp of every query row and the new pairs' column sums)
// lives in a fixed array inside the library image.  Every GPU that loads the library holds these
// kStaticLseFloats + kStaticNewSumFloats floats (5 MiB) until the process exits.
namespace {
constexpr size_t kStaticLseFloats = 1u << 20;     // nsamples * Hq  * I  <= 1,048,576
constexpr size_t kStaticNewSumFloats = 1u << 18;  // nsamples * Hkv * I  <=   262,144
constexpr int kMaxDevices = 64;
static __device__ __align__(256) float g_static_scratch[kStaticLseFloats + kStaticNewSumFloats];
// Device address of g_static_scratch per device ordinal.  In host code the symbol itself is only a
// stand-in, never a device address, so it is resolved once per device with that device current.
float* g_static_scratch_addr[kMaxDevices] = {};
}  // namespace

extern "C" bm_status_t bm_prefill_block_static(bm_cache_t* c, int32_t layer, int32_t sample0, int32_t nsamples,
                                               const void* q, const void* k, const void* v, int32_t I,
                                               int32_t pos0, void* out, int32_t evict_to, void* cuda_stream) {
  if (c == nullptr) return BM_ERR_INVALID;
  if (nsamples < 1 || I < 1) return BM_ERR_INVALID;
  if (c->cfg.rule == BM_RULE_AVERAGE_STD) return BM_ERR_INVALID;   // its second accumulator has no room in the array
  const int dev = c->cfg.device;
  if (dev < 0 || dev >= kMaxDevices) return BM_ERR_INVALID;
  if ((size_t)nsamples * c->cfg.n_q_heads * (size_t)I > kStaticLseFloats ||
      (size_t)nsamples * c->cfg.n_kv_heads * (size_t)I > kStaticNewSumFloats)
    return BM_ERR_CAPACITY;  // the call needs more scratch than the built-in array holds
  if (g_static_scratch_addr[dev] == nullptr) {
    if (cudaSetDevice(dev) != cudaSuccess) return BM_ERR_CUDA;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return BM_ERR_CUDA;
    g_static_scratch_addr[dev] = static_cast<float*>(p);
  }
  // Run the ordinary pass with the handle's scratch pointers redirected for the duration of the call.
  float* const lse_saved = c->ws_lse;
  float* const new_sum_saved = c->ws_new_sum;
  c->ws_lse = g_static_scratch_addr[dev];
  c->ws_new_sum = g_static_scratch_addr[dev] + kStaticLseFloats;
  const bm_status_t s = bm_prefill_block(c, layer, sample0, nsamples, q, k, v, I, pos0, out, evict_to, cuda_stream);
  c->ws_lse = lse_saved;
  c->ws_new_sum = new_sum_saved;
  return s;
}
