// C ABI of the library: argument checks, workspace carving and launches.  No allocation,
// no synchronisation, no host copies.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>
#include <vector>

#include "qp_common.cuh"
#include "qp_mma.cuh"

using namespace qp;

namespace {

// What the last decode call on each (device, stream) wrote through its merge kernel.  On a stream for which the
// caller has enabled it (qp_decode_overlap), the attention kernel of the next call is allowed to start while that
// merge kernel still runs (programmatic dependent launch) if none of its inputs overlaps those outputs; otherwise,
// and on every other stream, it is launched in plain stream order.  The kernels' own protocol (pdl_gate in
// qp_mma.cuh) guarantees that only the previous call can still be running then, so one call of history is enough.
// Host bookkeeping only: a few sorted address ranges per stream.
class PrevOutputs {
 public:
  using Range = std::pair<uintptr_t, uintptr_t>;   // [begin, end)
  struct Decision {
    bool overlap;   // no range of `reads` touches what the previous call on this stream wrote
    int parity;     // workspace half of this call: alternates per (device, stream)
  };
  // decides for this call, then records `writes` as the stream's latest outputs
  // ws_base / half_bytes: this call's partial records go to [ws_base + parity * half_bytes, + half_bytes); if that
  // area meets the one the previous call's merge may still be reading (calls of different sizes place their halves
  // differently), the call must not overlap the previous one either
  // two_halves: the launch is of the kind that alternates between workspace halves and takes part in the
  // overlap; the other kind (the chunked kernels) always writes [ws_base, ws_base + half_bytes), runs in plain
  // stream order, and so does the call after it
  Decision check_and_record(int device, cudaStream_t st, const std::vector<Range>& reads, std::vector<Range>& writes,
                            uintptr_t ws_base, size_t half_bytes, bool two_halves) {
    std::sort(writes.begin(), writes.end());
    // after sorting by begin, writes[i].second becomes the largest end among writes[0..i]: a read [b, e) meets
    // one of the writes that begin before e exactly when that running maximum exceeds b
    for (size_t i = 1; i < writes.size(); ++i) writes[i].second = std::max(writes[i].second, writes[i - 1].second);
    std::lock_guard<std::mutex> lock(mu_);
    const auto key = std::make_pair(device, st);
    auto it = prev_.find(key);
    Decision dec{false, 0};                         // overlap is opt-in per stream
    if (it != prev_.end()) {
      dec.overlap = it->second.allow && !it->second.barrier && two_halves;
      dec.parity = two_halves ? it->second.parity ^ 1 : 0;
      const std::vector<Range>& w = it->second.outs;
      for (const Range& r : reads) {
        if (!dec.overlap) break;
        const auto lo = std::lower_bound(w.begin(), w.end(), r.second,
                                         [](const Range& x, uintptr_t end) { return x.first < end; });
        if (lo != w.begin() && (lo - 1)->second > r.first) { dec.overlap = false; break; }
      }
    } else if (prev_.size() >= kMaxStreams) {       // bounded memory: forget (the opt-ins too: plain order is always safe)
      prev_.clear();
    }
    Entry& e = prev_[key];
    const Range mine{ws_base + (dec.parity ? half_bytes : 0), ws_base + (dec.parity ? half_bytes : 0) + half_bytes};
    if (mine.first < e.scratch.second && e.scratch.first < mine.second) dec.overlap = false;
    e.scratch = mine;
    e.outs.swap(writes);
    e.parity = dec.parity;
    e.barrier = !two_halves;
    return dec;
  }
  // Another kernel of the library has been enqueued on this stream that writes arrays a decode call reads
  // before it waits (a cache being filled or extended): the next decode call on the stream must be launched
  // in plain stream order.
  void barrier(int device, cudaStream_t st) {
    std::lock_guard<std::mutex> lock(mu_);
    if (prev_.size() >= kMaxStreams && prev_.find(std::make_pair(device, st)) == prev_.end()) prev_.clear();
    prev_[std::make_pair(device, st)].barrier = true;
  }
  bool allowed(int device, cudaStream_t st) {
    std::lock_guard<std::mutex> lock(mu_);
    const auto it = prev_.find(std::make_pair(device, st));
    return it != prev_.end() && it->second.allow;
  }
  void allow(int device, cudaStream_t st, bool on) {
    std::lock_guard<std::mutex> lock(mu_);
    if (prev_.size() >= kMaxStreams && prev_.find(std::make_pair(device, st)) == prev_.end()) prev_.clear();
    Entry& e = prev_[std::make_pair(device, st)];
    e.allow = on;
    e.barrier = true;                               // whatever was enqueued before the switch is unknown
  }

 private:
  struct Entry {
    std::vector<Range> outs;
    Range scratch{0, 0};     // where the last call's partial records live
    int parity = 0;
    bool barrier = false;
    bool allow = false;      // the caller's qp_decode_overlap setting for this stream
  };
  static constexpr size_t kMaxStreams = 256;
  std::mutex mu_;
  std::map<std::pair<int, cudaStream_t>, Entry> prev_;
};
PrevOutputs g_prev_outputs;

inline PrevOutputs::Range range_of(const void* p, size_t bytes) {
  const uintptr_t b = reinterpret_cast<uintptr_t>(p);
  return {b, b + bytes};
}

void cache_written(cudaStream_t st) {
  int device = 0;
  if (cudaGetDevice(&device) == cudaSuccess) g_prev_outputs.barrier(device, st);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool pow2_bits(int b) { return b == 2 || b == 4 || b == 8 || b == 16; }
inline bool ok_group(int g) { return g == 32 || g == 64 || g == 128; }

qp_status check_shape(int batch, int Hq, int Hkv, int D) {
  if (batch < 1 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return QP_ERR_INVALID_ARG;
  if ((D != 64 && D != 128) || Hq / Hkv > 8) return QP_ERR_UNSUPPORTED;
  return QP_OK;
}

qp_status check_cache(const qp_cache* c, bool need_ptrs) {
  if (!c) return QP_ERR_INVALID_ARG;
  qp_status s = check_shape(c->batch, c->n_q_heads, c->n_kv_heads, c->head_dim);
  if (s != QP_OK) return s;
  if (!pow2_bits(c->bits) || !ok_group(c->group) || c->head_dim % c->group != 0) return QP_ERR_UNSUPPORTED;
  if (c->n_keep < 1 || c->n_cap < 0) return QP_ERR_INVALID_ARG;
  if (c->bits < 16 && c->n_keep % c->group != 0) return QP_ERR_BUDGET;
  if (c->n_cap != 0 && (c->n_cap < c->n_keep || (c->bits < 16 && c->n_cap % c->group != 0))) return QP_ERR_BUDGET;
  if (need_ptrs) {
    if (!c->k_codes || !c->v_codes) return QP_ERR_INVALID_ARG;
    if (!aligned16(c->k_codes) || !aligned16(c->v_codes)) return QP_ERR_ALIGNMENT;
    if (c->bits < 16) {
      if (!c->k_scale || !c->k_zero || !c->v_scale || !c->v_zero) return QP_ERR_INVALID_ARG;
      if (!aligned16(c->k_scale) || !aligned16(c->k_zero) || !aligned16(c->v_scale) || !aligned16(c->v_zero))
        return QP_ERR_ALIGNMENT;
    }
  }
  return QP_OK;
}

}  // namespace

extern "C" {

const char* qp_status_string(qp_status s) {
  switch (s) {
    case QP_OK: return "ok";
    case QP_ERR_INVALID_ARG: return "invalid argument";
    case QP_ERR_UNSUPPORTED: return "unsupported configuration";
    case QP_ERR_BUDGET: return "budget cannot be met";
    case QP_ERR_WORKSPACE: return "workspace too small";
    case QP_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case QP_ERR_CUDA: return "CUDA launch failed";
  }
  return "unknown status";
}

qp_status qp_n_keep(int64_t budget_bits, int bits, int group, int L, int w, int32_t* n_keep) {
  if (!n_keep || L < 2 || w < 1 || w >= L || budget_bits < 1) return QP_ERR_INVALID_ARG;
  if (!pow2_bits(bits) || !ok_group(group)) return QP_ERR_UNSUPPORTED;
  int64_t n = budget_bits / bits;
  if (n > L) n = L;
  if (n <= w) return QP_ERR_BUDGET;
  if (bits < 16 && n % group != 0) return QP_ERR_BUDGET;
  *n_keep = (int32_t)n;
  return QP_OK;
}

qp_status qp_cache_layout(int batch, int n_q_heads, int n_kv_heads, int head_dim, int bits, int group, int n_keep,
                          qp_cache* out) {
  return qp_cache_layout_cap(batch, n_q_heads, n_kv_heads, head_dim, bits, group, n_keep, 0, out);
}

qp_status qp_cache_layout_cap(int batch, int n_q_heads, int n_kv_heads, int head_dim, int bits, int group, int n_keep,
                              int n_cap, qp_cache* out) {
  if (!out) return QP_ERR_INVALID_ARG;
  qp_cache c;
  std::memset(&c, 0, sizeof(c));
  c.batch = batch; c.n_q_heads = n_q_heads; c.n_kv_heads = n_kv_heads; c.head_dim = head_dim;
  c.bits = bits; c.group = group; c.n_keep = n_keep; c.n_cap = n_cap;
  const qp_status s = check_cache(&c, false);
  if (s != QP_OK) return s;
  const size_t elems = (size_t)batch * n_kv_heads * cache_capacity(c) * head_dim;
  if (bits == 16) {
    c.k_codes_bytes = c.v_codes_bytes = elems * 2;
  } else {
    c.k_codes_bytes = c.v_codes_bytes = elems * bits / 8;
    c.k_meta_bytes = c.v_meta_bytes = elems / group * 2;
  }
  *out = c;
  return QP_OK;
}

size_t qp_compress_workspace_bytes(int batch, int n_q_heads, int n_kv_heads, int head_dim, int L, int w) {
  if (check_shape(batch, n_q_heads, n_kv_heads, head_dim) != QP_OK || w < 1 || w >= L) return 0;
  return score_workspace(batch, n_q_heads, n_kv_heads, L, w).total;
}

size_t qp_decode_workspace_bytes(const qp_cache* cache) {
  if (check_cache(cache, false) != QP_OK) return 0;
  const DecDims d{cache->batch, cache->n_q_heads, cache->n_kv_heads, cache->head_dim, cache->bits, cache->group};
  return decode_workspace_bound(d, cache_capacity(*cache));   // enough for every n_keep the arrays can hold
}

static qp_status check_score_args(const void* Q_win, const void* K, int batch, int Hq, int Hkv, int D, int L, int w,
                                  int pool) {
  if (!Q_win || !K) return QP_ERR_INVALID_ARG;
  qp_status s = check_shape(batch, Hq, Hkv, D);
  if (s != QP_OK) return s;
  if (w < 1 || w >= L || pool < 1 || pool % 2 == 0) return QP_ERR_INVALID_ARG;
  if (w > 64 || pool > 65) return QP_ERR_UNSUPPORTED;
  // the score sweeps address a layer's keys as one matrix of batch * n_kv_heads * L rows with 32-bit row coordinates
  if ((long long)batch * Hkv * L > 0x7fffffffLL - 128) return QP_ERR_UNSUPPORTED;
  if (!aligned16(Q_win) || !aligned16(K)) return QP_ERR_ALIGNMENT;
  return QP_OK;
}

qp_status qp_window_scores(const void* Q_win, const void* K, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                           int L, int w, int pool, float* scores, void* workspace, size_t workspace_bytes,
                           void* stream) {
  qp_status s = check_score_args(Q_win, K, batch, n_q_heads, n_kv_heads, head_dim, L, w, pool);
  if (s != QP_OK) return s;
  if (!scores || !workspace) return QP_ERR_INVALID_ARG;
  if (!aligned16(scores) || !aligned16(workspace)) return QP_ERR_ALIGNMENT;
  if (workspace_bytes < qp_compress_workspace_bytes(batch, n_q_heads, n_kv_heads, head_dim, L, w))
    return QP_ERR_WORKSPACE;
  const ScoreDims d{batch, n_q_heads, n_kv_heads, head_dim, L, w, pool};
  return launch_window_scores(Q_win, K, d, scores, workspace, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? QP_OK : QP_ERR_CUDA;
}

qp_status qp_select_topk(const float* scores, int batch, int n_kv_heads, int L, int w, int n_keep, int32_t* kept_idx,
                         void* stream) {
  if (!scores || !kept_idx || batch < 1 || n_kv_heads < 1 || w < 1 || w >= L) return QP_ERR_INVALID_ARG;
  if (n_keep <= w || n_keep > L) return QP_ERR_BUDGET;
  return launch_select_topk(scores, batch * n_kv_heads, L, w, n_keep, kept_idx,
                            static_cast<cudaStream_t>(stream)) == cudaSuccess ? QP_OK : QP_ERR_CUDA;
}

qp_status qp_gather_quantize(const void* K, const void* V, const int32_t* kept_idx, int L, const qp_cache* cache,
                             void* stream) {
  if (!K || !V || !kept_idx || L < 1) return QP_ERR_INVALID_ARG;
  const qp_status s = check_cache(cache, true);
  if (s != QP_OK) return s;
  if (cache->n_keep > L) return QP_ERR_BUDGET;
  if (!aligned16(K) || !aligned16(V)) return QP_ERR_ALIGNMENT;
  cache_written(static_cast<cudaStream_t>(stream));
  return launch_gather_quantize(K, V, kept_idx, L, *cache, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? QP_OK : QP_ERR_CUDA;
}

qp_status qp_compress_layer(const void* K, const void* V, const void* Q_win, int batch, int n_q_heads, int n_kv_heads,
                            int head_dim, int L, int w, int64_t budget_bits, int bits, int group, int pool,
                            const qp_cache* cache, int32_t* kept_idx, void* workspace, size_t workspace_bytes,
                            void* stream) {
  if (!V || !kept_idx || !workspace) return QP_ERR_INVALID_ARG;
  qp_status s = check_score_args(Q_win, K, batch, n_q_heads, n_kv_heads, head_dim, L, w, pool);
  if (s != QP_OK) return s;
  int32_t n = 0;
  s = qp_n_keep(budget_bits, bits, group, L, w, &n);
  if (s != QP_OK) return s;
  s = check_cache(cache, true);
  if (s != QP_OK) return s;
  if (cache->batch != batch || cache->n_q_heads != n_q_heads || cache->n_kv_heads != n_kv_heads ||
      cache->head_dim != head_dim || cache->bits != bits || cache->group != group)
    return QP_ERR_INVALID_ARG;
  if (cache->n_keep != n) return QP_ERR_BUDGET;
  if (!aligned16(V) || !aligned16(workspace)) return QP_ERR_ALIGNMENT;
  const ScoreWorkspace sw = score_workspace(batch, n_q_heads, n_kv_heads, L, w);
  if (workspace_bytes < sw.total) return QP_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cache_written(st);
  float* pooled = reinterpret_cast<float*>(static_cast<char*>(workspace) + sw.pooled);
  const ScoreDims d{batch, n_q_heads, n_kv_heads, head_dim, L, w, pool};
  if (launch_window_scores(Q_win, K, d, pooled, workspace, st) != cudaSuccess) return QP_ERR_CUDA;
  if (launch_select_topk(pooled, batch * n_kv_heads, L, w, n, kept_idx, st) != cudaSuccess) return QP_ERR_CUDA;
  if (launch_gather_quantize(K, V, kept_idx, L, *cache, st) != cudaSuccess) return QP_ERR_CUDA;
  return QP_OK;
}

qp_status qp_compress_layers(int n_layers, const void* const* K, const void* const* V, const void* const* Q_win,
                             int batch, int n_q_heads, int n_kv_heads, int head_dim, int L, int w,
                             const int64_t* budget_bits, int bits, int group, int pool, const qp_cache* caches,
                             int32_t* const* kept_idx, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_layers < 1 || n_layers > QP_MAX_LAYERS || !K || !V || !Q_win || !budget_bits || !caches || !kept_idx || !workspace)
    return QP_ERR_INVALID_ARG;
  int n_keep[QP_MAX_LAYERS];
  for (int l = 0; l < n_layers; ++l) {
    if (!V[l] || !kept_idx[l]) return QP_ERR_INVALID_ARG;
    qp_status s = check_score_args(Q_win[l], K[l], batch, n_q_heads, n_kv_heads, head_dim, L, w, pool);
    if (s != QP_OK) return s;
    int32_t n = 0;
    s = qp_n_keep(budget_bits[l], bits, group, L, w, &n);
    if (s != QP_OK) return s;
    s = check_cache(&caches[l], true);
    if (s != QP_OK) return s;
    const qp_cache& c = caches[l];
    if (c.batch != batch || c.n_q_heads != n_q_heads || c.n_kv_heads != n_kv_heads || c.head_dim != head_dim ||
        c.bits != bits || c.group != group)
      return QP_ERR_INVALID_ARG;
    if (c.n_keep != n) return QP_ERR_BUDGET;
    if (!aligned16(V[l])) return QP_ERR_ALIGNMENT;
    n_keep[l] = n;
  }
  if (!aligned16(workspace)) return QP_ERR_ALIGNMENT;
  if ((long long)batch * n_layers * n_kv_heads > 65535) return QP_ERR_UNSUPPORTED;   // one grid dimension holds them
  const ScoreWorkspace sw = score_workspace(batch * n_layers, n_q_heads, n_kv_heads, L, w);
  if (workspace_bytes < sw.total) return QP_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cache_written(st);
  float* pooled = reinterpret_cast<float*>(static_cast<char*>(workspace) + sw.pooled);
  const ScoreDims d{batch, n_q_heads, n_kv_heads, head_dim, L, w, pool};
  if (launch_window_scores_layers(n_layers, Q_win, K, d, pooled, workspace, st) != cudaSuccess) return QP_ERR_CUDA;
  if (launch_select_topk_layers(n_layers, pooled, batch * n_kv_heads, L, w, n_keep, kept_idx, st) != cudaSuccess)
    return QP_ERR_CUDA;
  if (launch_gather_quantize_layers(n_layers, K, V, kept_idx, L, caches, st) != cudaSuccess) return QP_ERR_CUDA;
  return QP_OK;
}

}  // extern "C"

namespace {
// Decode attention over layers that agree in bits and group.  check_only: validate everything (workspace size
// included) and return before anything is launched or recorded.
qp_status decode_layers_uniform(int n_layers, const void* const* q, const qp_cache* caches, const qp_tail* tails,
                                void* const* out, void* workspace, size_t workspace_bytes, void* stream,
                                bool check_only) {
  if (n_layers < 1 || n_layers > QP_MAX_LAYERS || !q || !caches || !out || !workspace) return QP_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return QP_ERR_ALIGNMENT;
  const qp_cache& c0 = caches[0];
  DecTable tab;
  tab.n_layers = n_layers;
  for (int l = 0; l < n_layers; ++l) {
    const qp_status s = check_cache(&caches[l], true);
    if (s != QP_OK) return s;
    const qp_cache& c = caches[l];
    if (c.batch != c0.batch || c.n_q_heads != c0.n_q_heads || c.n_kv_heads != c0.n_kv_heads ||
        c.head_dim != c0.head_dim || c.bits != c0.bits || c.group != c0.group)
      return QP_ERR_INVALID_ARG;
    if (!q[l] || !out[l]) return QP_ERR_INVALID_ARG;
    if (!aligned16(q[l]) || !aligned16(out[l])) return QP_ERR_ALIGNMENT;
    tab.l[l] = DecLayer{c.k_codes, c.v_codes,
                        static_cast<const __half*>(c.k_scale), static_cast<const __half*>(c.k_zero),
                        static_cast<const __half*>(c.v_scale), static_cast<const __half*>(c.v_zero),
                        q[l], out[l], c.n_keep, 0, 0, cache_capacity(c)};
  }
  // tails: only when some layer has tokens waiting (B = 16 never has)
  bool any_tail = false;
  if (tails && c0.bits < 16)
    for (int l = 0; l < n_layers; ++l) {
      const qp_tail& t = tails[l];
      if (t.n_tail < 0 || t.n_tail >= c0.group) return QP_ERR_INVALID_ARG;
      if (t.n_tail > 0) {
        if (!t.k_tail || !t.v_tail) return QP_ERR_INVALID_ARG;
        if (!aligned16(t.k_tail) || !aligned16(t.v_tail)) return QP_ERR_ALIGNMENT;
        any_tail = true;
      }
    }
  TailTable ttab;
  if (any_tail)
    for (int l = 0; l < n_layers; ++l) ttab.l[l] = TailLayer{tails[l].k_tail, tails[l].v_tail, tails[l].n_tail, 0};
  const DecDims d{c0.batch, c0.n_q_heads, c0.n_kv_heads, c0.head_dim, c0.bits, c0.group};
  int device = 0;
  const bool have_device = cudaGetDevice(&device) == cudaSuccess;   // (size checks below work without one)
  const size_t need = decode_plan(tab, d, have_device && g_prev_outputs.allowed(device, static_cast<cudaStream_t>(stream)));
  if (workspace_bytes < need) return QP_ERR_WORKSPACE;
  if (check_only) return QP_OK;
  if (!have_device) return QP_ERR_CUDA;
  const bool two_halves = decode_mma_supported(d);
  const size_t half_bytes = two_halves ? decode_workspace_layout(tab, d).record_bytes : need;
  // everything the attention kernel reads before it waits for the stream's previous kernel, and what this
  // call's merge kernel writes
  std::vector<PrevOutputs::Range> reads, writes;
  reads.reserve(7 * (size_t)n_layers);
  writes.reserve((size_t)n_layers);
  const size_t qo_bytes = (size_t)c0.batch * c0.n_q_heads * c0.head_dim * 2;
  for (int l = 0; l < n_layers; ++l) {
    const qp_cache& c = caches[l];
    reads.push_back(range_of(q[l], qo_bytes));
    reads.push_back(range_of(c.k_codes, c.k_codes_bytes));
    reads.push_back(range_of(c.v_codes, c.v_codes_bytes));
    if (c.bits < 16) {
      reads.push_back(range_of(c.k_scale, c.k_meta_bytes));
      reads.push_back(range_of(c.k_zero, c.k_meta_bytes));
      reads.push_back(range_of(c.v_scale, c.v_meta_bytes));
      reads.push_back(range_of(c.v_zero, c.v_meta_bytes));
    }
    writes.push_back(range_of(out[l], qo_bytes));
  }
  const PrevOutputs::Decision dec =
      g_prev_outputs.check_and_record(device, static_cast<cudaStream_t>(stream), reads, writes,
                                      reinterpret_cast<uintptr_t>(workspace), half_bytes, two_halves);
  return launch_decode(tab, d, workspace, dec.parity, static_cast<cudaStream_t>(stream), dec.overlap,
                       any_tail ? &ttab : nullptr) == cudaSuccess
             ? QP_OK : QP_ERR_CUDA;
}

}  // namespace

extern "C" {

qp_status qp_decode_attn_tail_layers(int n_layers, const void* const* q, const qp_cache* caches, const qp_tail* tails,
                                     void* const* out, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_layers < 1 || n_layers > QP_MAX_LAYERS || !q || !caches || !out || !workspace) return QP_ERR_INVALID_ARG;
  bool uniform = true;
  for (int l = 1; l < n_layers; ++l) uniform = uniform && caches[l].bits == caches[0].bits && caches[l].group == caches[0].group;
  if (uniform) return decode_layers_uniform(n_layers, q, caches, tails, out, workspace, workspace_bytes, stream, false);
  // Layers of different precision or group size (a per-layer token/precision mix): one class after the other, each
  // with the kernels of its width.  All classes are validated before the first one is launched.
  std::vector<const void*> cq(n_layers);
  std::vector<void*> co(n_layers);
  std::vector<qp_cache> cc(n_layers);
  std::vector<qp_tail> ct(n_layers);
  std::vector<char> taken(n_layers, 0);
  for (int pass = 0; pass < 2; ++pass) {
    std::fill(taken.begin(), taken.end(), 0);
    for (int first = 0; first < n_layers; ++first) {
      if (taken[first]) continue;
      int m = 0;
      for (int l = first; l < n_layers; ++l)
        if (!taken[l] && caches[l].bits == caches[first].bits && caches[l].group == caches[first].group) {
          taken[l] = 1;
          cq[m] = q[l]; co[m] = out[l]; cc[m] = caches[l];
          if (tails) ct[m] = tails[l];
          ++m;
        }
      const qp_status s = decode_layers_uniform(m, cq.data(), cc.data(), tails ? ct.data() : nullptr, co.data(), workspace,
                                                workspace_bytes, stream, pass == 0);
      if (s != QP_OK) return s;
    }
  }
  return QP_OK;
}

qp_status qp_decode_attn_layers(int n_layers, const void* const* q, const qp_cache* caches, void* const* out,
                                void* workspace, size_t workspace_bytes, void* stream) {
  return qp_decode_attn_tail_layers(n_layers, q, caches, nullptr, out, workspace, workspace_bytes, stream);
}

static qp_status check_strategy(const qp_strategy* s, const qp_cache* c, bool* filter) {
  if (!s) return QP_ERR_INVALID_ARG;
  if (s->k_axis != 0 && s->k_axis != 1) return QP_ERR_INVALID_ARG;
  if (c->bits == 16) return QP_ERR_UNSUPPORTED;                 // nothing is quantized at 16 bit
  *filter = s->outlier_threshold > 0.f && s->outlier_threshold < INFINITY;
  if (*filter)
    for (const qp_side* q : {&s->k_side, &s->v_side}) {
      if (!q->idx || !q->val || !q->cnt || !q->tile_ptr || q->cap < 1) return QP_ERR_INVALID_ARG;
      if ((reinterpret_cast<uintptr_t>(q->idx) | reinterpret_cast<uintptr_t>(q->cnt) |
           reinterpret_cast<uintptr_t>(q->tile_ptr)) & 3u) return QP_ERR_ALIGNMENT;
      if (reinterpret_cast<uintptr_t>(q->val) & 1u) return QP_ERR_ALIGNMENT;
    }
  return QP_OK;
}

qp_status qp_gather_quantize_ex(const void* K, const void* V, const int32_t* kept_idx, int L, const qp_cache* cache,
                                const qp_strategy* strategy, void* stream) {
  if (!K || !V || !kept_idx || L < 1) return QP_ERR_INVALID_ARG;
  qp_status s = check_cache(cache, true);
  if (s != QP_OK) return s;
  bool filter = false;
  s = check_strategy(strategy, cache, &filter);
  if (s != QP_OK) return s;
  if (cache->n_keep > L) return QP_ERR_BUDGET;
  if (!aligned16(K) || !aligned16(V)) return QP_ERR_ALIGNMENT;
  cache_written(static_cast<cudaStream_t>(stream));
  return launch_gather_quantize_ex(K, V, kept_idx, L, *cache, *strategy, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? QP_OK : QP_ERR_CUDA;
}

size_t qp_head_budgets_workspace_bytes(int batch, int n_kv_heads, int L, int w, int n_mean) {
  if (batch < 1 || n_kv_heads < 1 || w < 1 || w >= L || n_mean <= w) return 0;
  const long long P = L - w;
  const long long k_total = std::min<long long>((long long)n_kv_heads * (n_mean - w), (long long)n_kv_heads * P);
  return (size_t)(((size_t)batch * (k_total + 1) * sizeof(int32_t) + 255) & ~(size_t)255);
}

qp_status qp_head_budgets(const float* scores, int batch, int n_kv_heads, int L, int w, int n_mean, int unit,
                          int32_t* n_keep_heads, void* workspace, size_t workspace_bytes, void* stream) {
  if (!scores || !n_keep_heads || !workspace || batch < 1 || n_kv_heads < 1 || w < 1 || w >= L || unit < 1)
    return QP_ERR_INVALID_ARG;
  if (n_mean <= w) return QP_ERR_BUDGET;
  if ((long long)n_kv_heads * (L - w) + 1 > 0x7fffffffLL || n_kv_heads > 8192) return QP_ERR_UNSUPPORTED;
  if (!aligned16(workspace)) return QP_ERR_ALIGNMENT;
  if (workspace_bytes < qp_head_budgets_workspace_bytes(batch, n_kv_heads, L, w, n_mean)) return QP_ERR_WORKSPACE;
  return launch_head_budgets(scores, batch, n_kv_heads, L, w, n_mean, unit, n_keep_heads,
                             static_cast<int32_t*>(workspace), static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? QP_OK : QP_ERR_CUDA;
}

qp_status qp_decode_attn_layers_ex(int n_layers, const void* const* q, const qp_cache* caches, const qp_strategy* strategy,
                                   void* const* out, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_layers < 1 || n_layers > QP_MAX_LAYERS || !q || !caches || !out || !workspace) return QP_ERR_INVALID_ARG;
  if (!aligned16(workspace)) return QP_ERR_ALIGNMENT;
  const qp_cache& c0 = caches[0];
  DecTable tab;
  tab.n_layers = n_layers;
  bool filter = false;
  for (int l = 0; l < n_layers; ++l) {
    const qp_cache& c = caches[l];
    qp_status s = check_cache(&c, true);
    if (s != QP_OK) return s;
    s = check_strategy(strategy, &c, &filter);
    if (s != QP_OK) return s;
    if (c.batch != c0.batch || c.n_q_heads != c0.n_q_heads || c.n_kv_heads != c0.n_kv_heads ||
        c.head_dim != c0.head_dim || c.bits != c0.bits || c.group != c0.group)
      return QP_ERR_INVALID_ARG;
    if (!q[l] || !out[l]) return QP_ERR_INVALID_ARG;
    if (!aligned16(q[l]) || !aligned16(out[l])) return QP_ERR_ALIGNMENT;
    tab.l[l] = DecLayer{c.k_codes, c.v_codes, static_cast<const __half*>(c.k_scale), static_cast<const __half*>(c.k_zero),
                        static_cast<const __half*>(c.v_scale), static_cast<const __half*>(c.v_zero), q[l], out[l], c.n_keep,
                        0, 0, cache_capacity(c)};
  }
  if (filter && n_layers > 1) return QP_ERR_UNSUPPORTED;
  const DecDims d{c0.batch, c0.n_q_heads, c0.n_kv_heads, c0.head_dim, c0.bits, c0.group};
  if (!filter && strategy->k_axis == 1 && decode_mma4t_supported(d)) {
    // per-token keys at 4 bit without side lists: the tensor-core kernel and the flat-range merge, plain stream order
    const size_t need_flat = decode_plan_flat(tab, d, decode_mma4t_workers_per_sm(), 4);
    if (workspace_bytes < need_flat) return QP_ERR_WORKSPACE;
    cache_written(static_cast<cudaStream_t>(stream));
    float* partials = static_cast<float*>(workspace);
    if (launch_decode_mma4t(tab, d, partials, static_cast<cudaStream_t>(stream)) != cudaSuccess) return QP_ERR_CUDA;
    return launch_merge_flat(tab, d, partials, static_cast<cudaStream_t>(stream)) == cudaSuccess ? QP_OK : QP_ERR_CUDA;
  }
  if (workspace_bytes < decode_plan_chunked(tab, d)) return QP_ERR_WORKSPACE;
  DecEx ex{};
  ex.k_axis = strategy->k_axis;
  ex.has_side = filter ? 1 : 0;
  if (filter) {
    const int n_tiles = (c0.n_keep + 31) / 32;
    auto side = [&](const qp_side& x) {
      return SideList{x.idx, static_cast<const uint16_t*>(x.val), x.cnt, x.tile_ptr, x.cap, n_tiles};
    };
    ex.k = side(strategy->k_side);
    ex.v = side(strategy->v_side);
  }
  cache_written(static_cast<cudaStream_t>(stream));           // plain stream order here and for the next decode call
  return launch_decode_ex(tab, d, ex, workspace, static_cast<cudaStream_t>(stream)) == cudaSuccess ? QP_OK : QP_ERR_CUDA;
}

qp_status qp_decode_attn_ex(const void* q, const qp_cache* cache, const qp_strategy* strategy, void* out,
                            void* workspace, size_t workspace_bytes, void* stream) {
  if (!cache) return QP_ERR_INVALID_ARG;
  const void* qs[1] = {q};
  void* os[1] = {out};
  return qp_decode_attn_layers_ex(1, qs, cache, strategy, os, workspace, workspace_bytes, stream);
}

#ifdef QP_CHECKED
}  // extern "C"
namespace qp {
cudaError_t quant_check_read(unsigned int (&out)[4]);
cudaError_t decode_check_read(unsigned int (&out)[4]);
cudaError_t topk_check_read(unsigned int (&out)[4]);
}
extern "C" {
#endif
qp_status qp_debug_check(uint32_t* words4) {
  if (!words4) return QP_ERR_INVALID_ARG;
#ifdef QP_CHECKED
  unsigned int a[4], b[4], c[4];
  if (qp::quant_check_read(a) != cudaSuccess || qp::decode_check_read(b) != cudaSuccess ||
      qp::topk_check_read(c) != cudaSuccess)
    return QP_ERR_CUDA;
  const unsigned int* first = a[0] ? a : b[0] ? b : c;
  words4[0] = first[0]; words4[1] = first[1]; words4[2] = first[2];
  words4[3] = a[3] + b[3] + c[3];
  return QP_OK;
#else
  words4[0] = words4[1] = words4[2] = words4[3] = 0u;
  return QP_ERR_UNSUPPORTED;
#endif
}

qp_status qp_decode_overlap(void* stream, int enable) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return QP_ERR_CUDA;
  g_prev_outputs.allow(device, static_cast<cudaStream_t>(stream), enable != 0);
  return QP_OK;
}

qp_status qp_decode_attn_tail(const void* q, const qp_cache* cache, const qp_tail* tail, void* out, void* workspace,
                              size_t workspace_bytes, void* stream) {
  if (!cache) return QP_ERR_INVALID_ARG;
  const void* qs[1] = {q};
  void* os[1] = {out};
  return qp_decode_attn_tail_layers(1, qs, cache, tail, os, workspace, workspace_bytes, stream);
}

qp_status qp_append_kv_layers(int n_layers, const void* const* k_new, const void* const* v_new, qp_cache* caches,
                              qp_tail* tails, void* stream) {
  if (n_layers < 1 || n_layers > QP_MAX_LAYERS || !k_new || !v_new || !caches) return QP_ERR_INVALID_ARG;
  const qp_cache& c0 = caches[0];
  if (c0.bits < 16 && !tails) return QP_ERR_INVALID_ARG;
  int flush[QP_MAX_LAYERS], n_flush = 0;
  for (int l = 0; l < n_layers; ++l) {
    const qp_cache& c = caches[l];
    const qp_status s = check_cache(&c, true);
    if (s != QP_OK) return s;
    if (c.batch != c0.batch || c.n_q_heads != c0.n_q_heads || c.n_kv_heads != c0.n_kv_heads ||
        c.head_dim != c0.head_dim || c.bits != c0.bits || c.group != c0.group)
      return QP_ERR_INVALID_ARG;
    if (!k_new[l] || !v_new[l]) return QP_ERR_INVALID_ARG;
    if (!aligned16(k_new[l]) || !aligned16(v_new[l])) return QP_ERR_ALIGNMENT;
    if (c.bits == 16) {
      if (c.n_keep + 1 > cache_capacity(c)) return QP_ERR_BUDGET;
      continue;
    }
    const qp_tail& t = tails[l];
    if (t.n_tail < 0 || t.n_tail >= c.group || !t.k_tail || !t.v_tail) return QP_ERR_INVALID_ARG;
    if (!aligned16(t.k_tail) || !aligned16(t.v_tail)) return QP_ERR_ALIGNMENT;
    if (t.n_tail + 1 == c.group) {
      if (c.n_keep + c.group > cache_capacity(c)) return QP_ERR_BUDGET;
      flush[n_flush++] = l;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (c0.bits == 16 || n_flush > 0) cache_written(st);          // arrays the next decode call reads are written
  if (launch_append_rows(n_layers, k_new, v_new, caches, tails, st) != cudaSuccess) return QP_ERR_CUDA;
  if (n_flush > 0 && launch_flush_tails(n_flush, flush, caches, tails, st) != cudaSuccess) return QP_ERR_CUDA;
  for (int l = 0; l < n_layers; ++l) {
    if (c0.bits == 16) {
      caches[l].n_keep += 1;
    } else if (tails[l].n_tail + 1 == c0.group) {
      tails[l].n_tail = 0;
      caches[l].n_keep += c0.group;
    } else {
      tails[l].n_tail += 1;
    }
  }
  return QP_OK;
}

qp_status qp_append_kv(const void* k_new, const void* v_new, qp_cache* cache, qp_tail* tail, void* stream) {
  const void* ks[1] = {k_new};
  const void* vs[1] = {v_new};
  return qp_append_kv_layers(1, ks, vs, cache, tail, stream);
}

qp_status qp_decode_attn(const void* q, const qp_cache* cache, void* out, void* workspace, size_t workspace_bytes,
                         void* stream) {
  if (!cache) return QP_ERR_INVALID_ARG;
  const void* qs[1] = {q};
  void* os[1] = {out};
  return qp_decode_attn_layers(1, qs, cache, os, workspace, workspace_bytes, stream);
}

}  // extern "C"
