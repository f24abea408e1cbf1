// C-ABI of the library (include/lq.h) and the host-side state machine.
//
// The log-based filter of Algorithm 1 is data-independent: which tokens stay at full precision,
// which W leave at each overflow and every store length are functions of the number of appended
// tokens only.  The host therefore mirrors the filter exactly (token ids, age order, physical
// slots) and hands the kernels plain slot lists and lengths; nothing is ever read back.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/lq.h"
#include "lq_kernels.cuh"

using namespace lq;

namespace {

struct LayerState {
  int64_t n_seen = 0, n_events = 0, n_quant = 0;
  int n_fp = 0;
  // n_fp = rows of the fp store in use (always the dense prefix [0, n_fp)) = age_slot.size() + pend_slot.size()
  std::vector<int32_t> age_slot;    // the filter's list A, age order (oldest first) -> physical fp slot
  std::vector<int32_t> pend_slot;   // removed by the filter, waiting for a full key group (only when W % G != 0),
                                    // removal order -> physical fp slot
  std::vector<int32_t> slot_token;  // physical fp slot -> token id; size 3W + G
  std::vector<int32_t> quant_ids;   // token ids in 2-bit store order
};

}  // namespace

struct lq_cache {
  lq_config_t cfg;
  CacheView cv;
  std::vector<LayerState> layers;
  bool dry = false;
  int sm_count = 148;
  int max_splits = 1;
  int64_t bytes_device = 0;
  float* part_o = nullptr;
  float* part_ml = nullptr;
  int* status = nullptr;
  int* ingest_idx = nullptr;  // index lists of the one-launch ingestion (3 max_tokens + 16 W + 3 G ints)
  int* tickets = nullptr;  // per (b, kv) arrival counters of the fused split-K merge
  float* acc = nullptr;    // per (b, kv) sums of the partials added on arrival (DecodeArgs::acc)
  // staging for the host-buffer entry point, one slice per layer
  uint8_t* stage_k = nullptr;
  uint8_t* stage_v = nullptr;
  uint8_t* stage_q = nullptr;
  uint8_t* stage_out = nullptr;
  int64_t n_launches = 0;
  bool stall_next = false;  // lq_debug_stall_next_decode
  // LQ_FLAG_OVERLAP_DECODE: layer and stream of the decode launch that was this cache's last enqueued work (-1: the
  // last work was something else)
  int last_decode_layer = -1;
  cudaStream_t last_decode_stream = nullptr;
  // Rows written by fused append+attention launches that may still be running.  An overlapped launch of the same
  // layer reads that row in its main loop, before its dependency wait, so it may overlap only when the writing
  // launch A is known to be complete.  Known without asking the device: a CTA of these kernels leaves only after
  // the launch before its own has completed, and a launch starts only when every CTA of the one before it has
  // started; so while A is incomplete every launch after A has all of its CTAs resident at once, and their CTA
  // counts cannot add up to more than the device holds.  ctas_since_wait = CTAs of the launches since the last one
  // that took its dependency wait first (which, through the chain of waits, covers everything before it);
  // row_mark[layer] = that count right after the layer's last fused launch, -1 = no row in doubt.  Once the
  // launches after A hold resident_bound CTAs or more, A is complete.
  std::vector<int64_t> row_mark;
  int64_t ctas_since_wait = 0;
  int32_t n_overlapped = 0;  // launches that took the overlapped form (lq_info_t::n_launches_overlapped)
  bool bad_slot_next = false;  // lq_debug_bad_slot_next_append (index-check build only)
  // left padding of a ragged batch (lq_set_padding): pad[b] leading positions of sequence b that attention
  // leaves out.  Device copy per layer: [B][4] row info, [B][fp_words] slot mask, [B][q_words] store mask,
  // rebuilt (mask_dirty) when the layer's stores changed.
  std::vector<int32_t> pad;
  bool has_pad = false;
  std::vector<char> mask_dirty;
  uint32_t* masks = nullptr;
  int fp_words = 0, q_words = 0, map_words = 0;
  int64_t mask_layer_words = 0;
  std::vector<uint32_t> mask_host;
  std::vector<int> pad_grid, pad_stride;  // per layer: CTAs and record stride of the padded tensor-core launch
  std::vector<int> pad_grid_ov, pad_stride_ov;  // the same for a launch that overlaps the one before it
  // optional timing of the split-K attention kernel
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;  // 2 events per timed launch
  size_t ev_used = 0;
  std::string last_error;
  std::vector<std::pair<uint8_t*, int64_t>> blocks;  // device blocks (address, payload bytes): guard bytes follow the payload
};

namespace {

lq_status_t cuda_fail(lq_cache* c, cudaError_t e, const char* what) {
  char buf[256];
  std::snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
  if (c) c->last_error = buf;
  return LQ_ERR_CUDA;
}

constexpr int kGuardBytes = 256;       // after every device block; checked by lq_check_guards
constexpr int kGuardPattern = 0xA5;

// Every device block of a cache -- long-lived or temporary -- comes from here: the caller's allocator when one
// is set, else cudaMalloc.  `bytes` is rounded up to 256 so that the guard starts on an aligned address.
bool dev_alloc(lq_cache* c, void** p, int64_t bytes, bool temporary = false) {
  const int64_t payload = (bytes + 255) / 256 * 256, total = payload + kGuardBytes;
  if (c->cfg.dev_alloc) {  // the caller's allocator
    *p = c->cfg.dev_alloc(static_cast<size_t>(total), c->cfg.alloc_ctx);
    if (*p == nullptr) return false;
  } else if (cudaMalloc(p, static_cast<size_t>(total)) != cudaSuccess) {
    cudaGetLastError();
    *p = nullptr;
    return false;
  }
  if (cudaMemset(static_cast<uint8_t*>(*p) + payload, kGuardPattern, kGuardBytes) != cudaSuccess) cudaGetLastError();
  c->blocks.emplace_back(static_cast<uint8_t*>(*p), payload);
  if (!temporary) c->bytes_device += total;
  return true;
}

void dev_release(lq_cache* c, void* p) {
  if (p == nullptr) return;
  for (size_t i = 0; i < c->blocks.size(); ++i)
    if (c->blocks[i].first == p) { c->blocks.erase(c->blocks.begin() + i); break; }
  if (c->cfg.dev_free) c->cfg.dev_free(p, c->cfg.alloc_ctx);
  else cudaFree(p);
}

// number of blocks whose guard bytes no longer hold the pattern (the device must be idle)
int damaged_guards(const lq_cache* c) {
  int bad = 0;
  uint8_t host[kGuardBytes];
  for (const auto& b : c->blocks) {
    if (cudaMemcpy(host, b.first + b.second, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); ++bad; continue; }
    for (int i = 0; i < kGuardBytes; ++i)
      if (host[i] != kGuardPattern) { ++bad; break; }
  }
  return bad;
}

void free_all(lq_cache* c) {
  if (!c->dry) {
    // the caller's allocator does not wait for work in flight the way cudaFree does
    if (c->cfg.dev_free) cudaDeviceSynchronize();
    dev_release(c, c->cv.quant);
    dev_release(c, c->cv.fp);
    dev_release(c, c->part_o);
    dev_release(c, c->part_ml);
    dev_release(c, c->status);
    dev_release(c, c->tickets);
    dev_release(c, c->acc);
    dev_release(c, c->ingest_idx);
    dev_release(c, c->stage_k);
    dev_release(c, c->stage_v);
    dev_release(c, c->stage_q);
    dev_release(c, c->stage_out);
    dev_release(c, c->masks);
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  }
}

int ratio(const lq_cache* c) { return c->cfg.n_q_heads / c->cfg.n_kv_heads; }

// age position of the e-th token the next overflow removes: A[1], A[3], ..., A[2W-1] (Algorithm 1),
// or A[0], ..., A[W-1] for the recent-window comparator
int evict_pos(const lq_cache* c, int e) { return c->cfg.filter == LQ_FILTER_RECENT ? e : 2 * e + 1; }

// slots and ids of the tokens the next overflow removes, in age order
void next_evicted(const lq_cache* c, const LayerState& L, EvictList* ev, int32_t* ids) {
  const int W = c->cfg.window;
  for (int e = 0; e < W; ++e) {
    const int slot = L.age_slot[evict_pos(c, e)];
    if (ev) {
      ev->slot[e] = static_cast<uint16_t>(slot);
      ev->src[e] = static_cast<uint16_t>(2 * W + e);  // the row of age position 2W + e moves into the hole
    }
    if (ids) ids[e] = L.slot_token[slot];
  }
}

// host bookkeeping of one overflow event (device work is launched separately)
void apply_event(const lq_cache* c, LayerState& L) {
  const int W = c->cfg.window;
  std::vector<int32_t> na;
  na.reserve(3 * W);
  if (c->cfg.filter == LQ_FILTER_RECENT)
    for (int i = W; i < 2 * W; ++i) na.push_back(L.age_slot[i]);
  else
    for (int i = 0; i < 2 * W; i += 2) na.push_back(L.age_slot[i]);
  for (int e = 0; e < W; ++e) {
    const int hole = L.age_slot[evict_pos(c, e)];
    L.quant_ids.push_back(L.slot_token[hole]);
    // the row of slot 2W+e (age position 2W+e) is moved into the hole
    L.slot_token[hole] = L.slot_token[2 * W + e];
    na.push_back(hole);
  }
  L.age_slot.swap(na);
  L.n_fp = 2 * W;
  L.n_quant += W;
  L.n_events++;
}

int kept(const LayerState& L) { return static_cast<int>(L.age_slot.size()); }
bool residual_mode(const lq_cache* c) { return c->cfg.window % c->cfg.group != 0; }

// W not a multiple of G, step 1 of an overflow: the W removed tokens join the waiting list; no row moves.
void apply_event_residual(const lq_cache* c, LayerState& L) {
  const int W = c->cfg.window;
  std::vector<char> gone(3 * W, 0);
  for (int e = 0; e < W; ++e) {
    gone[evict_pos(c, e)] = 1;
    L.pend_slot.push_back(L.age_slot[evict_pos(c, e)]);
  }
  std::vector<int32_t> na;
  na.reserve(3 * W);
  for (int i = 0; i < 3 * W; ++i)
    if (!gone[i]) na.push_back(L.age_slot[i]);
  L.age_slot.swap(na);
  L.n_events++;
}

// W not a multiple of G, step 2: the G oldest waiting tokens form a key group.  Fills the launch
// description (rows to quantise, and which top rows of the dense prefix move into the holes below
// the new end of the prefix) and updates the host maps.  ids: the G token ids, in store order.
void plan_group_residual(const lq_cache* c, LayerState& L, EvictList* ev, int32_t* ids) {
  const int G = c->cfg.group;
  const int live = L.n_fp, new_live = live - G;
  std::vector<char> is_hole(live, 0);
  for (int e = 0; e < G; ++e) is_hole[L.pend_slot[e]] = 1;
  std::vector<int> sources;  // rows above the new end that survive
  for (int s = new_live; s < live; ++s)
    if (!is_hole[s]) sources.push_back(s);
  size_t next = 0;
  std::vector<std::pair<int, int>> moves;  // (src, dst)
  for (int e = 0; e < G; ++e) {
    const int hole = L.pend_slot[e];
    if (ids) ids[e] = L.slot_token[hole];
    L.quant_ids.push_back(L.slot_token[hole]);
    ev->slot[e] = static_cast<uint16_t>(hole);
    if (hole < new_live) {
      ev->src[e] = static_cast<uint16_t>(sources[next]);
      moves.emplace_back(sources[next], hole);
      ++next;
    } else {
      ev->src[e] = kNoMove;
    }
  }
  L.pend_slot.erase(L.pend_slot.begin(), L.pend_slot.begin() + G);
  for (auto& mv : moves) {
    L.slot_token[mv.second] = L.slot_token[mv.first];
    for (auto& s : L.age_slot)
      if (s == mv.first) s = mv.second;
    for (auto& s : L.pend_slot)
      if (s == mv.first) s = mv.second;
  }
  L.n_fp = new_live;
  L.n_quant += G;
}

// overflow of the given layers when W is not a multiple of G (host state and launches): the removed tokens
// join the waiting lists; then, while some layer has G tokens waiting, its G oldest form a key group.  Layers
// whose group comes from the same rows and goes to the same place (layers in lockstep) share one launch.
lq_status_t run_events_residual(lq_cache* c, const std::vector<int>& full_layers, cudaStream_t st) {
  for (int layer : full_layers) apply_event_residual(c, c->layers[layer]);
  struct Plan {
    EvictList ev;
    int64_t tile0;
    int layer;
  };
  for (;;) {
    std::vector<Plan> plans;
    for (int layer : full_layers) {
      LayerState& L = c->layers[layer];
      if (static_cast<int>(L.pend_slot.size()) < c->cfg.group) continue;
      plans.emplace_back();
      Plan& p = plans.back();
      std::memset(&p.ev, 0, sizeof p.ev);
      p.tile0 = L.n_quant / c->cfg.group;
      p.layer = layer;
      plan_group_residual(c, L, &p.ev, nullptr);
    }
    if (plans.empty()) return LQ_OK;
    std::vector<char> done(plans.size(), 0);
    for (size_t i = 0; i < plans.size(); ++i) {
      if (done[i]) continue;
      LayerList ll;
      ll.n = 0;
      for (size_t k = i; k < plans.size() && ll.n < 128; ++k) {
        if (done[k] || plans[k].tile0 != plans[i].tile0 || std::memcmp(&plans[k].ev, &plans[i].ev, sizeof(EvictList)) != 0)
          continue;
        ll.layer[ll.n++] = static_cast<uint8_t>(plans[k].layer);
        done[k] = 1;
      }
      if (!c->dry) {
        cudaError_t e = launch_compress(c->cv, ll, plans[i].ev, plans[i].tile0, 1, st);
        if (e != cudaSuccess) return cuda_fail(c, e, "lq_compress_kernel");
        { c->n_launches++; c->last_decode_layer = -1; }
      }
    }
  }
}

lq_status_t run_events(lq_cache* c, const std::vector<int>& full_layers, cudaStream_t st) {
  if (!c->mask_dirty.empty())
    for (int layer : full_layers) c->mask_dirty[layer] = 1;
  if (residual_mode(c)) return run_events_residual(c, full_layers, st);
  // group layers whose removal lists coincide into one launch
  std::vector<char> done(full_layers.size(), 0);
  for (size_t i = 0; i < full_layers.size(); ++i) {
    if (done[i]) continue;
    LayerState& Li = c->layers[full_layers[i]];
    EvictList ev;
    std::memset(&ev, 0, sizeof ev);
    next_evicted(c, Li, &ev, nullptr);
    LayerList ll;
    ll.n = 0;
    std::vector<int> members;
    for (size_t k = i; k < full_layers.size() && ll.n < 128; ++k) {
      if (done[k]) continue;
      LayerState& Lk = c->layers[full_layers[k]];
      if (Lk.n_quant != Li.n_quant) continue;
      EvictList ek;
      std::memset(&ek, 0, sizeof ek);
      next_evicted(c, Lk, &ek, nullptr);
      if (std::memcmp(&ek, &ev, sizeof ev) != 0) continue;
      ll.layer[ll.n++] = static_cast<uint8_t>(full_layers[k]);
      members.push_back(static_cast<int>(k));
    }
    if (!c->dry) {
      cudaError_t e = launch_compress(c->cv, ll, ev, Li.n_quant / c->cfg.group, c->cfg.window / c->cfg.group, st);
      if (e != cudaSuccess) return cuda_fail(c, e, "lq_compress_kernel");
      { c->n_launches++; c->last_decode_layer = -1; }
    }
    for (int k : members) {
      done[k] = 1;
      apply_event(c, c->layers[full_layers[k]]);
    }
  }
  return LQ_OK;
}

bool use_mma(const lq_cache* c) { return c->cfg.kernel == LQ_KERNEL_AUTO || c->cfg.kernel == LQ_KERNEL_MMA; }
// the tcgen05 kernel serves a call unless the batch is padded (that goes through the plain kernel on the same layout)
bool use_umma(const lq_cache* c) { return c->cfg.kernel == LQ_KERNEL_UMMA && !c->has_pad; }

// Padding masks of one layer from the host mirror of its stores (which token id sits in which fp slot and at
// which place of the quantised store) and upload.  Rows appended later lie beyond the rebuilt prefix of the fp
// store, carry ids above every pad (checked by the caller) and need no bit.
lq_status_t upload_masks(lq_cache* c, int layer, cudaStream_t st) {
  const LayerState& L = c->layers[layer];
  const int B = c->cfg.batch, G = c->cfg.group;
  c->mask_host.assign(static_cast<size_t>(c->mask_layer_words), 0u);
  int32_t* rowinfo = reinterpret_cast<int32_t*>(c->mask_host.data());
  uint32_t* fpm = c->mask_host.data() + 4 * B;
  uint32_t* qm = fpm + static_cast<size_t>(c->fp_words) * B;
  const int64_t tiles = L.n_quant / G;
  for (int b = 0; b < B; ++b) {
    const int pad = c->pad[b];
    bool any_fp = false;
    for (int s = 0; s < L.n_fp; ++s)
      if (L.slot_token[s] < pad) {
        fpm[static_cast<size_t>(b) * c->fp_words + s / 32] |= 1u << (s % 32);
        any_fp = true;
      }
    int64_t skip = 0, last = 0;  // leading tiles that are padding entirely; one past the last tile with padding
    bool leading = true;
    for (int64_t t = 0; t < tiles; ++t) {
      int n_masked = 0;
      for (int i = 0; i < G; ++i) {
        const int64_t qi = t * G + i;
        if (L.quant_ids[qi] < pad) {
          qm[static_cast<size_t>(b) * c->q_words + qi / 32] |= 1u << (qi % 32);
          ++n_masked;
        }
      }
      if (leading && n_masked == G) skip = t + 1;
      else leading = false;
      if (n_masked) last = t + 1;
    }
    rowinfo[4 * b + 0] = static_cast<int32_t>(skip);
    rowinfo[4 * b + 1] = static_cast<int32_t>(last);
    rowinfo[4 * b + 2] = any_fp ? 1 : 0;
  }
  if (use_mma(c)) {
    // the CTAs of the tensor-core launch, shared out by the work each sequence has left
    int32_t* pair_ctas = reinterpret_cast<int32_t*>(qm + static_cast<size_t>(c->q_words) * B);
    int32_t* cta_map = pair_ctas + B * c->cfg.n_kv_heads;
    DecodeArgs a;
    a.cv = c->cv;
    a.n_fp = L.n_fp;
    a.n_quant = L.n_quant;
    c->pad_grid[layer] = plan_decode_mma_padded(a, c->sm_count, c->max_splits, rowinfo, cta_map, pair_ctas,
                                                &c->pad_stride[layer]);
    // second plan, behind the first: a third of the wave for launches that overlap (LQ_FLAG_OVERLAP_DECODE)
    int32_t* pair_ctas_ov = cta_map + c->map_words;
    c->pad_grid_ov[layer] = plan_decode_mma_padded(a, c->sm_count, c->max_splits, rowinfo, pair_ctas_ov + B * c->cfg.n_kv_heads,
                                                   pair_ctas_ov, &c->pad_stride_ov[layer], true);
  }
  // pageable source: staged by the runtime before the call returns
  c->last_decode_layer = -1;
  cudaError_t e = cudaMemcpyAsync(c->masks + layer * c->mask_layer_words, c->mask_host.data(),
                                  c->mask_host.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(c, e, "padding mask upload");
  c->mask_dirty[layer] = 0;
  return LQ_OK;
}

int choose_splits(const lq_cache* c, const LayerState& L) {
  if (c->cfg.n_splits > 0) return std::min(c->cfg.n_splits, c->max_splits);
  const int pairs = c->cfg.batch * c->cfg.n_kv_heads;
  const int64_t T = L.n_fp + L.n_quant;
  int64_t s = (4LL * c->sm_count + pairs - 1) / pairs;
  s = std::min<int64_t>(s, (T + 127) / 128);
  s = std::max<int64_t>(1, std::min<int64_t>(s, c->max_splits));
  return static_cast<int>(s);
}


}  // namespace

extern "C" {

const char* lq_status_str(lq_status_t s) {
  switch (s) {
    case LQ_OK: return "ok";
    case LQ_ERR_INVALID_ARG: return "invalid argument";
    case LQ_ERR_UNSUPPORTED: return "unsupported configuration";
    case LQ_ERR_OOM: return "out of device memory";
    case LQ_ERR_WINDOW_FULL: return "full-precision window is full";
    case LQ_ERR_NOT_FULL: return "full-precision window is not full";
    case LQ_ERR_CAPACITY: return "capacity exceeded (max_tokens of the cache, or the fixed scratch of the static entry point)";
    case LQ_ERR_CUDA: return "CUDA error";
  }
  return "unknown status";
}

const char* lq_last_error(const lq_cache_t* c) { return c ? c->last_error.c_str() : ""; }

lq_status_t lq_cache_create(const lq_config_t* cfg, lq_cache_t** out) {
  if (!cfg || !out) return LQ_ERR_INVALID_ARG;
  if (cfg->n_layers < 1 || cfg->batch < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 ||
      cfg->window < 1 || cfg->group < 1 || cfg->max_tokens < 1 || cfg->n_splits < 0)
    return LQ_ERR_INVALID_ARG;
  if (cfg->n_q_heads % cfg->n_kv_heads) return LQ_ERR_INVALID_ARG;
  if ((cfg->dev_alloc == nullptr) != (cfg->dev_free == nullptr)) return LQ_ERR_INVALID_ARG;
  if (cfg->head_dim != kD || (cfg->bits != 2 && cfg->bits != 4)) return LQ_ERR_UNSUPPORTED;
  if (cfg->group != 32 && cfg->group != 64) return LQ_ERR_UNSUPPORTED;
  if (cfg->window > kMaxW) return LQ_ERR_UNSUPPORTED;
  if (cfg->n_q_heads / cfg->n_kv_heads > kMaxRatio || cfg->n_layers > 128) return LQ_ERR_UNSUPPORTED;
  if (cfg->kernel < LQ_KERNEL_AUTO || cfg->kernel > LQ_KERNEL_UMMA) return LQ_ERR_INVALID_ARG;
  if (cfg->kernel == LQ_KERNEL_UMMA && cfg->bits != 2) return LQ_ERR_UNSUPPORTED;
  if (cfg->filter != LQ_FILTER_LOG && cfg->filter != LQ_FILTER_RECENT) return LQ_ERR_INVALID_ARG;

  lq_cache* c = new (std::nothrow) lq_cache;
  if (!c) return LQ_ERR_OOM;
  c->cfg = *cfg;
  c->dry = cfg->device == LQ_DEVICE_NONE;
  const int W = cfg->window, G = cfg->group;
  const int64_t pairs = static_cast<int64_t>(cfg->batch) * cfg->n_kv_heads;
  CacheView& cv = c->cv;
  std::memset(&cv, 0, sizeof cv);
  cv.B = cfg->batch; cv.Hq = cfg->n_q_heads; cv.Hkv = cfg->n_kv_heads; cv.G = G; cv.W = W;
  cv.planes = cfg->bits / 2;
  cv.layout = cfg->kernel == LQ_KERNEL_UMMA ? kLayoutRow : kLayoutFragment;
  cv.quant_tiles_cap = (cfg->max_tokens + G - 1) / G;
  cv.quant_head_stride = cv.quant_tiles_cap * quant_tile_bytes(G, cv.planes);
  cv.quant_layer_stride = cv.quant_head_stride * pairs;
  // W % G != 0: up to G - 1 removed tokens wait in the fp store for a full key group
  const int fp_slots = 3 * W + (W % G ? G : 0);
  cv.fp_head_stride = fp_store_bytes(cv.layout, fp_slots);
  cv.fp_layer_stride = cv.fp_head_stride * pairs;
  c->layers.resize(cfg->n_layers);
  for (auto& L : c->layers) L.slot_token.assign(3 * W + G, -1);

  if (!c->dry) {
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) { delete c; cudaGetLastError(); return LQ_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) == cudaSuccess) c->sm_count = prop.multiProcessorCount;
    // split-K partial records reserved per (b, kv) (one more than the CTAs per pair: some pairs get an extra CTA)
    c->max_splits = 1 + (cfg->n_splits > 0
                        ? cfg->n_splits
                        : static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(256, (8LL * c->sm_count + pairs - 1) / pairs))));
    if (cfg->kernel == LQ_KERNEL_UMMA)  // the tcgen05 kernel cuts one cost line over all pairs: a few more slots per pair
      c->max_splits = std::max(c->max_splits, static_cast<int>(std::min<int64_t>(128, (2LL * c->sm_count + pairs - 1) / pairs + 3)));
    const int r = ratio(c);
    bool ok = dev_alloc(c, reinterpret_cast<void**>(&cv.quant), cv.quant_layer_stride * cfg->n_layers) &&
              dev_alloc(c, reinterpret_cast<void**>(&cv.fp), cv.fp_layer_stride * cfg->n_layers) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->part_o), pairs * c->max_splits * r * kD * 4) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->part_ml), pairs * c->max_splits * r * 2 * 4) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->status), 256) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->tickets), pairs * 128) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->acc), static_cast<int64_t>(pairs) * kAccStride * 4) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->ingest_idx), (3 * cfg->max_tokens + 16 * cfg->window + 3 * cfg->group) * 4) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->stage_k), cfg->n_layers * pairs * kD * 2) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->stage_v), cfg->n_layers * pairs * kD * 2) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->stage_q),
                        static_cast<int64_t>(cfg->n_layers) * cfg->batch * cfg->n_q_heads * kD * 2) &&
              dev_alloc(c, reinterpret_cast<void**>(&c->stage_out),
                        static_cast<int64_t>(cfg->n_layers) * cfg->batch * cfg->n_q_heads * kD * 4);
    if (ok) ok = cudaMemset(c->status, 0, 256) == cudaSuccess;
    cv.status = c->status;
    if (ok) ok = cudaMemset(c->tickets, 0, pairs * 128) == cudaSuccess;
    if (ok) ok = cudaMemset(c->acc, 0, static_cast<size_t>(pairs) * kAccStride * 4) == cudaSuccess;
    // the fp store must never hold non-finite garbage in unused slots of a partly filled tile
    if (ok) ok = cudaMemset(cv.fp, 0, static_cast<size_t>(cv.fp_layer_stride) * cfg->n_layers) == cudaSuccess;
    if (!ok) {
      free_all(c);
      delete c;
      cudaGetLastError();
      return LQ_ERR_OOM;
    }
  } else {
    c->max_splits = std::max(1, cfg->n_splits);
  }
  *out = c;
  return LQ_OK;
}

lq_status_t lq_destroy(lq_cache_t* c) {
  if (!c) return LQ_OK;
  free_all(c);
  delete c;
  return LQ_OK;
}

namespace {

// A prompt (or a chunk of one) appended in one launch: the host plays Algorithm 1 token by token on its mirror
// of the filter (which never looks at the data), collects the removed token ids of every overflow
// step and the final slot map, and one kernel writes both stores.
// host bookkeeping of one overflow of layer L (no device work); idx, when given, collects the ids of the tokens that
// enter the 2-bit store, in store order
void host_event(const lq_cache* c, LayerState& L, std::vector<int32_t>* idx) {
  const int W = c->cfg.window, G = c->cfg.group;
  std::vector<int32_t> ids(std::max(W, G));
  if (residual_mode(c)) {
    apply_event_residual(c, L);
    while (static_cast<int>(L.pend_slot.size()) >= G) {
      EvictList unused;
      plan_group_residual(c, L, &unused, ids.data());
      if (idx) idx->insert(idx->end(), ids.begin(), ids.begin() + G);
    }
  } else {
    next_evicted(c, L, nullptr, ids.data());
    if (idx) idx->insert(idx->end(), ids.begin(), ids.end());
    apply_event(c, L);
  }
}

// host bookkeeping of n tokens appended one by one with the overflow step run whenever the window is full
void replay_appends(const lq_cache* c, LayerState& L, int64_t n, std::vector<int32_t>* idx) {
  const int W = c->cfg.window;
  int64_t done = 0;
  while (done < n) {
    if (kept(L) == 3 * W) host_event(c, L, idx);
    const int take = static_cast<int>(std::min<int64_t>(n - done, 3 * W - kept(L)));
    for (int t = 0; t < take; ++t) {
      L.age_slot.push_back(L.n_fp + t);
      L.slot_token[L.n_fp + t] = static_cast<int32_t>(L.n_seen + t);
    }
    L.n_fp += take;
    L.n_seen += take;
    done += take;
  }
}

// Plays an ingestion plan on token ids instead of rows (host only, no device work) and checks what the kernel
// relies on: every key group gathers its tokens in store order; no fp slot is written twice or read twice; a slot
// that is both read and written has its reader and its writer in the same list entry (one thread of one CTA, the read
// first); copied slots held nothing before; the store ends as the host maps say; and (top_in_place: W a multiple of
// G) age positions from 2W on sit in the slot of the same number, as the overflow step expects.  old_tok: slot ->
// token before the call.  Used by the device-less mode, so that the CPU tests cover the planner.
bool ingest_plan_is_sound(const LayerState& L, int W, bool top_in_place, const std::vector<int32_t>& old_tok, int64_t seen_old,
                          const std::vector<int32_t>& ids, const std::vector<int32_t>& idx, bool has_fill, int n_copy) {
  const int NQ = static_cast<int>(ids.size()), n_old = static_cast<int>(old_tok.size());
  const int cap = static_cast<int>(L.slot_token.size());
  std::vector<int32_t> content(cap, -1), reader(cap, -1), writer(cap, -1);
  for (int s = 0; s < n_old; ++s) content[s] = old_tok[s];
  std::vector<int32_t> final_tok(content);
  auto read = [&](int slot, int who) {
    if (slot < 0 || slot >= n_old || reader[slot] != -1) return false;
    reader[slot] = who;
    return true;
  };
  auto write = [&](int slot, int who, int32_t tok) {
    if (slot < 0 || slot >= cap || writer[slot] != -1) return false;
    writer[slot] = who;
    final_tok[slot] = tok;
    return true;
  };
  for (int i = 0; i < NQ; ++i) {
    const int32_t src = idx[i];
    if (src == -1) return false;
    if (src >= 0) {
      if (seen_old + src != ids[i]) return false;
      if (has_fill && (idx[NQ + i] != -1 || idx[2 * NQ + i] != -1)) return false;
      continue;
    }
    const int s = -2 - src;
    if (!has_fill || !read(s, i) || content[s] != ids[i]) return false;
    const int32_t f1 = idx[NQ + i], f2 = idx[2 * NQ + i];
    if (f1 >= 0) {
      if (!write(s, i, static_cast<int32_t>(seen_old + f1)) || f2 != -1) return false;
    } else if (f1 <= -2) {
      const int m = -2 - f1;
      if (!read(m, i) || !write(s, i, content[m])) return false;
      if (f2 >= 0 && !write(m, i, static_cast<int32_t>(seen_old + f2))) return false;
    } else if (f2 != -1) {
      return false;
    }
  }
  const size_t copy0 = static_cast<size_t>(has_fill ? 3 : 1) * NQ;
  for (int j = 0; j < n_copy; ++j) {
    const int slot = idx[copy0 + 2 * j];
    if (slot < n_old || idx[copy0 + 2 * j + 1] < 0) return false;
    if (!write(slot, -2, static_cast<int32_t>(seen_old + idx[copy0 + 2 * j + 1]))) return false;
  }
  for (int s = 0; s < cap; ++s)
    if (reader[s] != -1 && writer[s] != -1 && reader[s] != writer[s]) return false;
  for (int s = 0; s < L.n_fp; ++s)
    if (final_tok[s] != L.slot_token[s]) return false;
  std::vector<char> used(cap, 0);
  for (size_t a = 0; a < L.age_slot.size(); ++a) {
    const int s = L.age_slot[a];
    if (s < 0 || s >= L.n_fp || used[s]) return false;
    used[s] = 1;
    if (top_in_place && static_cast<int>(a) >= 2 * W && s != static_cast<int>(a)) return false;
  }
  for (int s : L.pend_slot) {
    if (s < 0 || s >= L.n_fp || used[s]) return false;
    used[s] = 1;
  }
  return L.pend_slot.size() + L.age_slot.size() == static_cast<size_t>(L.n_fp);
}

lq_status_t ingest_prompt(lq_cache* c, int layer, const void* k, const void* v, int n, cudaStream_t st) {
  LayerState& L = c->layers[layer];
  if (!c->mask_dirty.empty()) c->mask_dirty[layer] = 1;
  const int W = c->cfg.window, G = c->cfg.group;
  // the layer as it is now: token -> slot of its full-precision rows
  const int n_fp_old = L.n_fp;
  const int64_t seen_old = L.n_seen, tile0 = L.n_quant / G;
  const std::vector<int32_t> old_tok(L.slot_token.begin(), L.slot_token.begin() + n_fp_old);
  std::vector<std::pair<int32_t, int32_t>> old_slots(n_fp_old);  // (token, slot), sorted by token
  for (int s = 0; s < n_fp_old; ++s) old_slots[s] = {old_tok[s], s};
  std::sort(old_slots.begin(), old_slots.end());
  auto old_slot_of = [&](int32_t tok) {
    auto it = std::lower_bound(old_slots.begin(), old_slots.end(), std::make_pair(tok, static_cast<int32_t>(-1)));
    return it != old_slots.end() && it->first == tok ? it->second : -1;
  };
  std::vector<int32_t> ids;  // tokens that enter the 2-bit store, in store order
  ids.reserve(static_cast<size_t>(n) + 3 * W);
  replay_appends(c, L, n, &ids);
  const int n_tiles = static_cast<int>(ids.size()) / G, NQ = n_tiles * G;
  const bool has_fill = n_fp_old > 0;
  std::vector<int32_t> idx(static_cast<size_t>(has_fill ? 3 : 1) * NQ, -1);
  std::vector<int32_t> copy;  // (slot, new-tensor row)
  if (!has_fill) {
    for (int i = 0; i < NQ; ++i) idx[i] = ids[i];
    for (int s = 0; s < L.n_fp; ++s) {
      copy.push_back(s);
      copy.push_back(L.slot_token[s]);
    }
  } else {
    // The replay above moved rows the way the token-by-token path does; the slots are private, so this launch is
    // free to place them otherwise, and it places them so that no slot is read by one thread and written by another.
    // W a multiple of G: old rows that stay below 2W keep their slot; age positions >= 2W (new tokens all: an
    // overflow step has run) sit in the slot of the same number, as the overflow step expects; the slots below 2W
    // that lost their token take first the old rows that sat at 2W or above, then new tokens.  Otherwise (removed
    // tokens may wait in the store, and the step path expects nothing but a dense prefix): the same with the end of
    // the store in place of 2W.
    const bool residual = residual_mode(c);
    const int kept_now = kept(L), n_pend = static_cast<int>(L.pend_slot.size()), n_fp_new = L.n_fp;
    const int n_live = kept_now + n_pend;  // survivors: list A in age order, then the waiting tokens
    const int limit = residual ? n_fp_new : 2 * W;
    std::vector<int32_t> tok_of(n_live), new_slot(n_live, -1);
    for (int a = 0; a < kept_now; ++a) tok_of[a] = L.slot_token[L.age_slot[a]];
    for (int p = 0; p < n_pend; ++p) tok_of[kept_now + p] = L.slot_token[L.pend_slot[p]];
    const int low = std::min(limit, n_fp_old);
    std::vector<char> stays(std::max(low, 1), 0);
    std::vector<int> movers, fresh_tokens;  // survivors that still need a slot below `limit`
    for (int a = 0; a < n_live; ++a) {
      if (a >= limit) {  // (only when W is a multiple of G: there is no waiting list then)
        new_slot[a] = a;
        continue;
      }
      const int so = tok_of[a] < seen_old ? old_slot_of(tok_of[a]) : -1;
      if (so >= 0 && so < limit) {
        new_slot[a] = so;
        stays[so] = 1;
      } else if (so >= 0) {
        movers.push_back(a);
      } else {
        fresh_tokens.push_back(a);
      }
    }
    std::vector<int32_t> fill1_of(std::max(n_fp_old, 1), -1), fill2_of(std::max(n_fp_old, 1), -1);
    std::vector<int> free_slots;  // below `limit`: first the slots that lost their token, then those never used
    for (int s = 0; s < low; ++s)
      if (!stays[s]) free_slots.push_back(s);
    for (int s = n_fp_old; s < limit; ++s) free_slots.push_back(s);
    size_t next = 0;
    for (int a : movers) {
      const int s = free_slots[next++], m = old_slot_of(tok_of[a]);
      new_slot[a] = s;
      fill1_of[s] = -2 - m;
      // slot m itself goes to the new token of age position m, if the store reaches that far
      if (m < n_fp_new) fill2_of[m] = static_cast<int32_t>(tok_of[m] - seen_old);
    }
    for (int a : fresh_tokens) {
      const int s = free_slots[next++];
      new_slot[a] = s;
      const int32_t row = static_cast<int32_t>(tok_of[a] - seen_old);
      if (s < n_fp_old) {
        fill1_of[s] = row;
      } else {
        copy.push_back(s);
        copy.push_back(row);
      }
    }
    for (int a = limit; a < n_fp_new; ++a) {
      const int32_t row = static_cast<int32_t>(tok_of[a] - seen_old);
      if (a >= n_fp_old) {
        copy.push_back(a);
        copy.push_back(row);
      } else if (fill2_of[a] == -1) {
        fill1_of[a] = row;  // its old token leaves through a key group (or it would be a mover with fill2 set)
      }
    }
    for (int i = 0; i < NQ; ++i) {
      if (ids[i] >= seen_old) {
        idx[i] = static_cast<int32_t>(ids[i] - seen_old);
        continue;
      }
      const int s = old_slot_of(ids[i]);
      idx[i] = -2 - s;
      idx[NQ + i] = fill1_of[s];
      if (fill1_of[s] <= -2) idx[2 * NQ + i] = fill2_of[-2 - fill1_of[s]];
    }
    for (int a = 0; a < n_live; ++a) {
      (a < kept_now ? L.age_slot[a] : L.pend_slot[a - kept_now]) = new_slot[a];
      L.slot_token[new_slot[a]] = tok_of[a];
    }
  }
  const int n_copy = static_cast<int>(copy.size()) / 2;
  idx.insert(idx.end(), copy.begin(), copy.end());
  if (c->dry) {
    if (ingest_plan_is_sound(L, W, !residual_mode(c), old_tok, seen_old, ids, idx, has_fill, n_copy)) return LQ_OK;
    c->last_error = "ingestion plan failed its self-check";
    return LQ_ERR_CUDA;
  }
  // pageable source: the runtime stages it before the call returns, so `idx` may die here
  cudaError_t e = cudaMemcpyAsync(c->ingest_idx, idx.data(), idx.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(c, e, "prompt index upload");
  e = launch_ingest(c->cv, layer, k, v, n, c->ingest_idx, n_tiles, has_fill, n_copy, tile0, st);
  if (e != cudaSuccess) return cuda_fail(c, e, "lq_ingest_kernel");
  { c->n_launches++; c->last_decode_layer = -1; }
  return LQ_OK;
}

}  // namespace

namespace {
lq_status_t append_impl(lq_cache_t* c, int32_t layer, const void* k, const void* v, int32_t n, void* stream,
                        const void* extra_src, void* extra_dst, int extra_bytes);
}

lq_status_t lq_append(lq_cache_t* c, int32_t layer, const void* k, const void* v, int32_t n, void* stream) {
  return append_impl(c, layer, k, v, n, stream, nullptr, nullptr, 0);
}

namespace {
// lq_append; the last launch also copies extra_bytes from extra_src to extra_dst (device-addressable)
lq_status_t append_impl(lq_cache_t* c, int32_t layer, const void* k, const void* v, int32_t n, void* stream,
                        const void* extra_src, void* extra_dst, int extra_bytes) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || n < 0) return LQ_ERR_INVALID_ARG;
  if (!c->dry && (!k || !v)) return LQ_ERR_INVALID_ARG;
  if (!c->dry && ((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v)) & 15)) return LQ_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  const int W = c->cfg.window;
  if (L.n_seen + n > c->cfg.max_tokens) return LQ_ERR_CAPACITY;
  if (!c->cfg.auto_compress && kept(L) + n > 3 * W) return LQ_ERR_WINDOW_FULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // more than one launch's worth of work: a prompt for an empty layer, or a chunk of at least two windows that makes
  // a layer already in use overflow.  Below two windows the index upload of the one-launch path costs more than the
  // launches it saves.
  if (c->cfg.auto_compress && extra_bytes == 0 &&
      (L.n_seen == 0 ? n > 3 * W : (n >= 2 * W && kept(L) + n > 3 * W)))
    return ingest_prompt(c, layer, k, v, n, st);
  int done = 0;
  while (done < n) {
    if (kept(L) == 3 * W) {
      lq_status_t s = run_events(c, std::vector<int>{layer}, st);
      if (s != LQ_OK) return s;
    }
    const int take = std::min(n - done, 3 * W - kept(L));
    if (!c->dry) {
      const bool last = done + take == n;
      // (test hook of the index-check build: a first slot beyond the store, which the kernel's check must refuse)
      const int slot0 = L.n_fp + (c->bad_slot_next ? static_cast<int>(fp_slots_cap(c->cv)) : 0);
      c->bad_slot_next = false;
      cudaError_t e = launch_append(c->cv, layer, k, v, n, done, take, slot0, st, last ? extra_src : nullptr,
                                    last ? extra_dst : nullptr, last ? extra_bytes : 0);
      if (e != cudaSuccess) return cuda_fail(c, e, "lq_append_kernel");
      { c->n_launches++; c->last_decode_layer = -1; }
    }
    for (int t = 0; t < take; ++t) {
      L.age_slot.push_back(L.n_fp + t);
      L.slot_token[L.n_fp + t] = static_cast<int32_t>(L.n_seen + t);
    }
    L.n_fp += take;
    L.n_seen += take;
    done += take;
  }
  return LQ_OK;
}
}  // namespace

lq_status_t lq_compress(lq_cache_t* c, int32_t layer, void* stream) {
  if (!c || layer < -1 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  const int W = c->cfg.window;
  std::vector<int> full;
  if (layer >= 0) {
    if (kept(c->layers[layer]) != 3 * W) return LQ_ERR_NOT_FULL;
    full.push_back(layer);
  } else {
    for (int i = 0; i < c->cfg.n_layers; ++i)
      if (kept(c->layers[i]) == 3 * W) full.push_back(i);
  }
  if (full.empty()) return LQ_OK;
  return run_events(c, full, static_cast<cudaStream_t>(stream));
}

namespace {
lq_status_t decode_impl(lq_cache_t* c, int32_t layer, const void* q, float sm_scale, void* out, int32_t out_dtype,
                        void* stream, const void* new_k, const void* new_v, int new_slot, bool fp_only = false);
}

lq_status_t lq_decode_attn(lq_cache_t* c, int32_t layer, const void* q, float sm_scale, void* out,
                           int32_t out_dtype, void* stream) {
  return decode_impl(c, layer, q, sm_scale, out, out_dtype, stream, nullptr, nullptr, 0);
}

lq_status_t lq_decode_attn_fp_only(lq_cache_t* c, int32_t layer, const void* q, float sm_scale, void* out,
                                   int32_t out_dtype, void* stream) {
  return decode_impl(c, layer, q, sm_scale, out, out_dtype, stream, nullptr, nullptr, 0, true);
}

lq_status_t lq_set_padding(lq_cache_t* c, const int32_t* pad_host) {
  if (!c) return LQ_ERR_INVALID_ARG;
  if (!pad_host) {
    c->has_pad = false;
    return LQ_OK;
  }
  const int B = c->cfg.batch;
  for (int b = 0; b < B; ++b)
    if (pad_host[b] < 0) return LQ_ERR_INVALID_ARG;
  if (B * c->cfg.n_kv_heads > 0xFFFF) return LQ_ERR_UNSUPPORTED;  // the CTA map packs the pair into 16 bits
  if (!c->dry && !c->masks) {
    const int slots = 3 * c->cfg.window + c->cfg.group;
    c->fp_words = (slots + 31) / 32;
    c->q_words = static_cast<int>((c->cfg.max_tokens + 31) / 32);
    c->map_words = std::max(max_ctas_decode_mma(c->sm_count), B * c->cfg.n_kv_heads);  // at least one CTA per pair
    c->mask_layer_words = static_cast<int64_t>(B) * (4 + c->fp_words + c->q_words) + 2 * (B * c->cfg.n_kv_heads + c->map_words);
    if (!dev_alloc(c, reinterpret_cast<void**>(&c->masks), c->mask_layer_words * c->cfg.n_layers * 4)) return LQ_ERR_OOM;
  }
  c->pad.assign(pad_host, pad_host + B);
  c->has_pad = false;
  for (int b = 0; b < B; ++b) c->has_pad |= pad_host[b] > 0;
  c->mask_dirty.assign(c->cfg.n_layers, 1);
  c->pad_grid.assign(c->cfg.n_layers, 0);
  c->pad_stride.assign(c->cfg.n_layers, 1);
  c->pad_grid_ov.assign(c->cfg.n_layers, 0);
  c->pad_stride_ov.assign(c->cfg.n_layers, 1);
  return LQ_OK;
}

lq_status_t lq_append_decode_attn(lq_cache_t* c, int32_t layer, const void* k, const void* v, const void* q,
                                  float sm_scale, void* out, int32_t out_dtype, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || (out_dtype != 0 && out_dtype != 1)) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  if (!k || !v || !q || !out || ((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
                                  reinterpret_cast<uintptr_t>(q)) & 15))
    return LQ_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  const int W = c->cfg.window;
  if (L.n_seen + 1 > c->cfg.max_tokens) return LQ_ERR_CAPACITY;
  // The fused instantiation of the kernel runs its main loop about 2 % slower than the plain one
  // and saves a 2 us launch: it pays below roughly 200 MB per launch -- unless launches overlap
  // (LQ_FLAG_OVERLAP_DECODE): a separate append kernel between two attention launches would make the second one
  // wait for the first, which costs far more than 2 %.
  const int64_t step_bytes = static_cast<int64_t>(c->cfg.batch) * c->cfg.n_kv_heads *
                             (L.n_quant * (quant_tile_bytes(c->cfg.group, c->cfg.bits / 2) / c->cfg.group) +
                              static_cast<int64_t>(L.n_fp) * 4 * kD);
  const bool overlap = (c->cfg.flags & LQ_FLAG_OVERLAP_DECODE) != 0;
  if (kept(L) == 3 * W || !use_mma(c) || (!overlap && step_bytes > (192LL << 20))) {
    // the window is full (the overflow step has to run between the two), the plain kernel is
    // selected, or the launch is long: the two separate calls
    lq_status_t s = lq_append(c, layer, k, v, 1, stream);
    if (s != LQ_OK) return s;
    return lq_decode_attn(c, layer, q, sm_scale, out, out_dtype, stream);
  }
  // host side of the append; the row itself is written by the attention kernel
  const int slot = L.n_fp;
  L.age_slot.push_back(slot);
  L.slot_token[slot] = static_cast<int32_t>(L.n_seen);
  L.n_fp += 1;
  L.n_seen += 1;
  lq_status_t s = decode_impl(c, layer, q, sm_scale, out, out_dtype, stream, k, v, slot);
  if (s != LQ_OK) {  // nothing was launched: take the token back
    L.age_slot.pop_back();
    L.slot_token[slot] = -1;
    L.n_fp -= 1;
    L.n_seen -= 1;
  }
  return s;
}

namespace {
lq_status_t decode_impl(lq_cache_t* c, int32_t layer, const void* q, float sm_scale, void* out, int32_t out_dtype,
                        void* stream, const void* new_k, const void* new_v, int new_slot, bool fp_only) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || (out_dtype != 0 && out_dtype != 1)) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  if (!q || !out || (reinterpret_cast<uintptr_t>(q) & 15)) return LQ_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  if (L.n_fp + L.n_quant == 0) return LQ_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DecodeArgs a;
  a.cv = c->cv;
  a.layer = layer;
  a.n_fp = L.n_fp;
  a.n_quant = fp_only ? 0 : L.n_quant;
  a.rowinfo = nullptr;
  a.qmask = a.fpmask = nullptr;
  a.qmask_words = a.fpmask_words = 0;
  a.cta_map = a.pair_ctas = nullptr;
  a.n_ctas = 0;
  if (c->has_pad) {
    // every sequence keeps at least its newest token
    for (int b = 0; b < c->cfg.batch; ++b)
      if (c->pad[b] >= L.n_seen) return LQ_ERR_INVALID_ARG;
    if (c->mask_dirty[layer]) {
      lq_status_t ms = upload_masks(c, layer, st);
      if (ms != LQ_OK) return ms;
    }
    const uint32_t* base = c->masks + layer * c->mask_layer_words;
    a.rowinfo = reinterpret_cast<const int32_t*>(base);
    a.fpmask = base + 4 * c->cfg.batch;
    a.qmask = a.fpmask + static_cast<int64_t>(c->fp_words) * c->cfg.batch;
    a.fpmask_words = c->fp_words;
    a.qmask_words = c->q_words;
    a.pair_ctas = reinterpret_cast<const int32_t*>(a.qmask + static_cast<int64_t>(c->q_words) * c->cfg.batch);
    a.cta_map = a.pair_ctas + c->cfg.batch * c->cfg.n_kv_heads;
  }
  if (!(sm_scale > 0.f)) sm_scale = 1.0f / std::sqrt(static_cast<float>(kD));
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.q = q;
  a.part_o = c->part_o;
  a.part_ml = c->part_ml;
  a.out = out;
  a.out_bf16 = out_dtype;
  a.status = c->status;
  a.new_k = new_k;
  a.new_v = new_v;
  a.new_slot = new_slot;
  a.tickets = nullptr;
  a.acc = nullptr;
  a.debug_stall = c->stall_next ? 1 : 0;
  c->stall_next = false;
  cudaError_t e;
  const bool timed = c->profiling && c->ev_used + 2 <= c->ev_pool.size();
  if (timed) cudaEventRecord(c->ev_pool[c->ev_used], st);
  a.tiles_fp = a.tiles_quant = 0;
  a.zero = 0;
  a.n_extra = 0;
  a.early = 0;
  if (use_mma(c)) {
    if (c->row_mark.empty()) c->row_mark.assign(c->cfg.n_layers, -1);
    // twice the CTAs of these kernels the device can hold (51 KB of shared memory each: at most four per SM)
    const int64_t resident_bound = 2LL * max_ctas_decode_mma(c->sm_count);
    const bool row_safe = c->row_mark[layer] < 0 || c->ctas_since_wait - c->row_mark[layer] >= resident_bound;
    a.early = (c->cfg.flags & LQ_FLAG_OVERLAP_DECODE) && !timed && c->last_decode_layer >= 0 &&
              c->last_decode_layer != layer && c->last_decode_stream == st && row_safe;
    if (!a.early) {
      std::fill(c->row_mark.begin(), c->row_mark.end(), -1);
      c->ctas_since_wait = 0;
    }
    plan_decode_mma(a, c->sm_count, c->max_splits, c->cfg.n_splits);
    if (a.rowinfo) {
      a.S = a.early ? c->pad_stride_ov[layer] : c->pad_stride[layer];
      a.n_ctas = a.early ? c->pad_grid_ov[layer] : c->pad_grid[layer];
      if (a.early) {  // the second plan lies behind the first in the mask block
        a.pair_ctas = a.cta_map + c->map_words;
        a.cta_map = a.pair_ctas + c->cfg.batch * c->cfg.n_kv_heads;
      }
      a.n_extra = 0;
    }
    c->ctas_since_wait += a.rowinfo ? a.n_ctas : c->cfg.batch * c->cfg.n_kv_heads * (a.S - 1) + a.n_extra;  // the grid
    if (a.early) c->n_overlapped++;
    c->row_mark[layer] = new_k != nullptr ? c->ctas_since_wait : -1;
    a.tickets = c->tickets;  // the CTA that completes a (b, kv) pair merges it: no second launch
    a.acc = c->acc;
    e = launch_decode_mma(a, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "lq_decode_mma_kernel");
  } else if (use_umma(c)) {
    plan_decode_umma(a, c->sm_count, c->max_splits, c->cfg.n_splits);
    a.tickets = c->tickets;
    e = launch_decode_umma(a, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "lq_decode_umma_kernel");
  } else {
    a.S = choose_splits(c, L);
    e = launch_decode_scalar(a, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "lq_decode_scalar_kernel");
  }
  if (timed) {
    cudaEventRecord(c->ev_pool[c->ev_used + 1], st);
    c->ev_used += 2;
  }
  if (a.tickets == nullptr) {
    e = launch_merge(a, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "lq_merge_kernel");
    c->n_launches++;
  }
  c->n_launches++;
  c->last_decode_layer = use_mma(c) && !timed ? layer : -1;
  c->last_decode_stream = st;
  return LQ_OK;
}
}  // namespace

lq_status_t lq_decode_step_host(lq_cache_t* c, int32_t layer, const void* k_host, const void* v_host,
                                const void* q_host, float sm_scale, float* out_host, int32_t sync, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  if (!k_host || !v_host || !q_host || !out_host) return LQ_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  if (L.n_seen + 1 > c->cfg.max_tokens) return LQ_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t kvb = static_cast<size_t>(c->cfg.batch) * c->cfg.n_kv_heads * kD * 2;
  const size_t qb = static_cast<size_t>(c->cfg.batch) * c->cfg.n_q_heads * kD * 2;
  uint8_t* sk = c->stage_k + layer * kvb;
  uint8_t* sv = c->stage_v + layer * kvb;
  uint8_t* sq = c->stage_q + layer * qb;
  uint8_t* so = c->stage_out + layer * qb * 2;
  cudaError_t e;
  // Page-locked host buffers that the device can address are used in place, by the same single launch as the
  // device-buffer step (lq_append_decode_attn): the attention kernel takes the new k and v rows and the query
  // rows straight from host memory (the query once per CTA: about 1 KB each) and writes its result straight into
  // out_host; consecutive layers overlap like device-resident steps.  No separate copy is left.  Anything else
  // goes through the staging buffers with one copy each.
  auto mapped = [](const void* p) -> void* {
    cudaPointerAttributes at;
    if ((reinterpret_cast<uintptr_t>(p) & 15) != 0) return nullptr;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
  };
  void* dk = mapped(k_host);
  void* dv = mapped(v_host);
  void* dq = mapped(q_host);
  void* dout = mapped(out_host);
  const bool direct = dk && dv && dq && dout;
  if (!direct) {
    if ((e = cudaMemcpyAsync(sk, k_host, kvb, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(sv, v_host, kvb, cudaMemcpyHostToDevice, st)) != cudaSuccess)
      return cuda_fail(c, e, "host-to-device copy");
    if ((e = cudaMemcpyAsync(sq, q_host, qb, cudaMemcpyHostToDevice, st)) != cudaSuccess)
      return cuda_fail(c, e, "host-to-device copy");
  }
  lq_status_t s;
  if (kept(L) == 3 * c->cfg.window) {  // the overflow step of this layer is due
    s = run_events(c, std::vector<int>{layer}, st);
    if (s != LQ_OK) return s;
  }
  if (direct) {
    s = lq_append_decode_attn(c, layer, dk, dv, dq, sm_scale, dout, 0, stream);
    if (s != LQ_OK) return s;
  } else {
    s = lq_append(c, layer, sk, sv, 1, stream);
    if (s != LQ_OK) return s;
    s = lq_decode_attn(c, layer, sq, sm_scale, so, 0, stream);
    if (s != LQ_OK) return s;
  }
  if (!direct && (e = cudaMemcpyAsync(out_host, so, qb * 2, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
    return cuda_fail(c, e, "device-to-host copy");
  if (sync && (e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(c, e, "cudaStreamSynchronize");
  return LQ_OK;
}

lq_status_t lq_profile_enable(lq_cache_t* c, int32_t on) {
  if (!c) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  if (on && c->ev_pool.empty()) {
    c->ev_pool.resize(2 * 8192);
    for (auto& ev : c->ev_pool)
      if (cudaEventCreate(&ev) != cudaSuccess) return cuda_fail(c, cudaGetLastError(), "cudaEventCreate");
  }
  c->profiling = on != 0;
  c->ev_used = 0;
  return LQ_OK;
}

lq_status_t lq_profile_read(lq_cache_t* c, double* total_ms, int64_t* n_launches) {
  if (!c || !total_ms || !n_launches) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaDeviceSynchronize");
  double sum = 0.0;
  for (size_t i = 0; i + 1 < c->ev_used; i += 2) {
    float ms = 0.f;
    if ((e = cudaEventElapsedTime(&ms, c->ev_pool[i], c->ev_pool[i + 1])) != cudaSuccess)
      return cuda_fail(c, e, "cudaEventElapsedTime");
    sum += ms;
  }
  *total_ms = sum;
  *n_launches = static_cast<int64_t>(c->ev_used / 2);
  return LQ_OK;
}



lq_status_t lq_kernel_status(lq_cache_t* c, int32_t* word) {
  if (!c || !word) return LQ_ERR_INVALID_ARG;
  *word = 0;
  if (c->dry) return LQ_OK;
  cudaError_t e = cudaMemcpy(word, c->status, sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(c, e, "status read");
  return LQ_OK;
}

lq_status_t lq_reset_kernel_status(lq_cache_t* c) {
  if (!c) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(int32_t));
  if (e != cudaSuccess) return cuda_fail(c, e, "status reset");
  return LQ_OK;
}

lq_status_t lq_debug_bad_slot_next_append(lq_cache_t* c) {
  if (!c) return LQ_ERR_INVALID_ARG;
#ifdef LQ_DEBUG_BOUNDS
  c->bad_slot_next = true;
  return LQ_OK;
#else
  return LQ_ERR_UNSUPPORTED;  // without the checks the rows would really be written out of range
#endif
}

lq_status_t lq_debug_stall_next_decode(lq_cache_t* c) {
  if (!c) return LQ_ERR_INVALID_ARG;
  c->stall_next = true;
  return LQ_OK;
}

lq_status_t lq_cache_info(const lq_cache_t* c, int32_t layer, lq_info_t* info) {
  if (!c || !info || layer < 0 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  std::memset(info, 0, sizeof *info);
  info->n_seen = L.n_seen;
  info->n_fp = L.n_fp;
  info->n_quant = L.n_quant;
  info->n_events = L.n_events;
  info->bytes_device = c->bytes_device;
  info->n_kernel_launches = c->n_launches;
  info->n_launches_overlapped = c->n_overlapped;
  info->bytes_quant_per_token = quant_tile_bytes(c->cfg.group, c->cfg.bits / 2) / c->cfg.group;
  info->bytes_decode_step = static_cast<int64_t>(c->cfg.batch) * c->cfg.n_kv_heads *
                            (L.n_quant * info->bytes_quant_per_token + static_cast<int64_t>(L.n_fp) * 4 * kD);
  if (c->dry || L.n_fp + L.n_quant == 0)
    info->n_splits = 0;
  else if (use_mma(c)) {
    DecodeArgs a;
    a.cv = c->cv;
    a.n_fp = L.n_fp;
    a.n_quant = L.n_quant;
    a.early = 0;  // the plan of a launch that does not overlap (an overlapped one uses a third of these CTAs)
    plan_decode_mma(a, c->sm_count, c->max_splits, c->cfg.n_splits);
    info->n_splits = a.S - 1;
    info->n_ctas = (a.S - 1) * c->cfg.batch * c->cfg.n_kv_heads + a.n_extra;
    if ((c->cfg.flags & LQ_FLAG_OVERLAP_DECODE) && !c->has_pad) {
      a.early = 1;
      plan_decode_mma(a, c->sm_count, c->max_splits, c->cfg.n_splits);
      info->n_ctas_overlapped = (a.S - 1) * c->cfg.batch * c->cfg.n_kv_heads + a.n_extra;
    }
  } else if (use_umma(c)) {
    DecodeArgs a;
    a.cv = c->cv;
    a.n_fp = L.n_fp;
    a.n_quant = L.n_quant;
    plan_decode_umma(a, c->sm_count, c->max_splits, c->cfg.n_splits);
    info->n_splits = a.S;
    info->n_ctas = a.n_ctas;
  } else
    info->n_splits = choose_splits(c, L);
  return LQ_OK;
}

lq_status_t lq_next_evicted_ids(const lq_cache_t* c, int32_t layer, int32_t* ids) {
  if (!c || !ids || layer < 0 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  if (kept(L) != 3 * c->cfg.window) return LQ_ERR_NOT_FULL;
  next_evicted(c, L, nullptr, ids);
  return LQ_OK;
}

lq_status_t lq_export(const lq_cache_t* cc, int32_t layer, lq_image_t* img) {
  lq_cache* c = const_cast<lq_cache*>(cc);
  if (!c || !img || layer < 0 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  // kept ids ascending, with the slot each lives in
  // (tokens still waiting for a full key group are at full precision too)
  std::vector<std::pair<int32_t, int32_t>> rows;  // (token id, slot)
  for (int slot : L.age_slot) rows.emplace_back(L.slot_token[slot], slot);
  for (int slot : L.pend_slot) rows.emplace_back(L.slot_token[slot], slot);
  std::sort(rows.begin(), rows.end());
  if (img->kept_ids) for (int i = 0; i < L.n_fp; ++i) img->kept_ids[i] = rows[i].first;
  if (img->quant_ids) std::copy(L.quant_ids.begin(), L.quant_ids.end(), img->quant_ids);
  const bool want_dev = img->k_codes || img->v_codes || img->k_scale || img->k_zero || img->v_scale ||
                        img->v_zero || img->fp_k || img->fp_v;
  if (!want_dev) return LQ_OK;
  if (c->dry) return LQ_ERR_UNSUPPORTED;

  const int64_t pairs = static_cast<int64_t>(c->cfg.batch) * c->cfg.n_kv_heads;
  const int G = c->cfg.group;
  const int64_t nq = L.n_quant, nf = L.n_fp;
  const int64_t sz_codes = pairs * nq * (kD * c->cfg.bits / 8);
  const int64_t sz_kp = pairs * (nq / G) * kD * 2;
  const int64_t sz_vp = pairs * nq * (kD / G) * 2;
  const int64_t sz_fp = pairs * nf * kD * 2;
  struct Buf { void* host; int64_t bytes; void* dev; };
  Buf bufs[8] = {{img->k_codes, sz_codes, nullptr}, {img->v_codes, sz_codes, nullptr},
                 {img->k_scale, sz_kp, nullptr},    {img->k_zero, sz_kp, nullptr},
                 {img->v_scale, sz_vp, nullptr},    {img->v_zero, sz_vp, nullptr},
                 {img->fp_k, sz_fp, nullptr},       {img->fp_v, sz_fp, nullptr}};
  int* slots_dev = nullptr;
  lq_status_t status = LQ_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaDeviceSynchronize");
  for (auto& b : bufs)
    if (b.host && b.bytes > 0 && !dev_alloc(c, &b.dev, b.bytes, true)) status = LQ_ERR_OOM;
  if (status == LQ_OK && nf > 0) {
    std::vector<int> slots(nf);
    for (int i = 0; i < nf; ++i) slots[i] = rows[i].second;
    if (!dev_alloc(c, reinterpret_cast<void**>(&slots_dev), nf * sizeof(int), true)) status = LQ_ERR_OOM;
    else cudaMemcpy(slots_dev, slots.data(), nf * sizeof(int), cudaMemcpyHostToDevice);
  }
  if (status == LQ_OK) {
    e = launch_export(c->cv, layer, static_cast<int>(nf), nq, slots_dev,
                      static_cast<uint8_t*>(bufs[0].dev), static_cast<uint8_t*>(bufs[1].dev),
                      static_cast<uint16_t*>(bufs[2].dev), static_cast<uint16_t*>(bufs[3].dev),
                      static_cast<uint16_t*>(bufs[4].dev), static_cast<uint16_t*>(bufs[5].dev),
                      static_cast<uint16_t*>(bufs[6].dev), static_cast<uint16_t*>(bufs[7].dev), nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) status = cuda_fail(c, e, "export kernels");
  }
  if (status == LQ_OK)
    for (auto& b : bufs)
      if (b.dev) {
        e = cudaMemcpy(b.host, b.dev, static_cast<size_t>(b.bytes), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) { status = cuda_fail(c, e, "export copy"); break; }
      }
  // (the device is idle here: a caller's allocator may hand the blocks out again at once)
  for (auto& b : bufs) dev_release(c, b.dev);
  dev_release(c, slots_dev);
  if (status == LQ_ERR_OOM) cudaGetLastError();
  return status;
}

lq_status_t lq_import(lq_cache_t* c, int32_t layer, const lq_image_t* img, int64_t n_seen, int64_t n_fp, int64_t n_quant) {
  if (!c || !img || layer < 0 || layer >= c->cfg.n_layers) return LQ_ERR_INVALID_ARG;
  if (c->dry) return LQ_ERR_UNSUPPORTED;
  LayerState& L = c->layers[layer];
  if (L.n_seen != 0 || n_seen <= 0 || n_fp < 0 || n_quant < 0) return LQ_ERR_INVALID_ARG;
  if (n_seen > c->cfg.max_tokens) return LQ_ERR_CAPACITY;
  const bool have_q = img->k_codes && img->v_codes && img->k_scale && img->k_zero && img->v_scale && img->v_zero;
  if ((n_quant > 0 && !have_q) || (n_fp > 0 && (!img->fp_k || !img->fp_v))) return LQ_ERR_INVALID_ARG;
  // The filter never looks at the data: the layer's bookkeeping is that of n_seen single appends.  A layer that was
  // full when it was exported may or may not have had its overflow step run (lq_compress with auto_compress = 0):
  // the sizes tell.
  const LayerState saved = L;
  replay_appends(c, L, n_seen, nullptr);
  if ((L.n_fp != n_fp || L.n_quant != n_quant) && kept(L) == 3 * c->cfg.window) host_event(c, L, nullptr);
  std::vector<std::pair<int32_t, int32_t>> rows;  // (token id, slot), ascending ids as in the image
  for (int slot : L.age_slot) rows.emplace_back(L.slot_token[slot], slot);
  for (int slot : L.pend_slot) rows.emplace_back(L.slot_token[slot], slot);
  std::sort(rows.begin(), rows.end());
  bool match = L.n_fp == n_fp && L.n_quant == n_quant;
  if (match && img->kept_ids)
    for (int64_t i = 0; i < n_fp && match; ++i) match = img->kept_ids[i] == rows[i].first;
  if (match && img->quant_ids)
    for (int64_t i = 0; i < n_quant && match; ++i) match = img->quant_ids[i] == L.quant_ids[i];
  if (!match) {  // not an image of this configuration after n_seen tokens
    L = saved;
    return LQ_ERR_INVALID_ARG;
  }
  const int64_t pairs = static_cast<int64_t>(c->cfg.batch) * c->cfg.n_kv_heads;
  const int G = c->cfg.group;
  const int64_t sz_codes = pairs * n_quant * (kD * c->cfg.bits / 8), sz_kp = pairs * (n_quant / G) * kD * 2,
                sz_vp = pairs * n_quant * (kD / G) * 2, sz_fp = pairs * n_fp * kD * 2;
  struct Buf { const void* host; int64_t bytes; void* dev; };
  Buf bufs[8] = {{img->k_codes, sz_codes, nullptr}, {img->v_codes, sz_codes, nullptr},
                 {img->k_scale, sz_kp, nullptr},    {img->k_zero, sz_kp, nullptr},
                 {img->v_scale, sz_vp, nullptr},    {img->v_zero, sz_vp, nullptr},
                 {img->fp_k, sz_fp, nullptr},       {img->fp_v, sz_fp, nullptr}};
  int* slots_dev = nullptr;
  lq_status_t status = LQ_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) status = cuda_fail(c, e, "cudaDeviceSynchronize");
  for (auto& b : bufs) {
    if (status != LQ_OK || b.bytes == 0) continue;
    if (!dev_alloc(c, &b.dev, b.bytes, true)) status = LQ_ERR_OOM;
    else if ((e = cudaMemcpy(b.dev, b.host, static_cast<size_t>(b.bytes), cudaMemcpyHostToDevice)) != cudaSuccess)
      status = cuda_fail(c, e, "import copy");
  }
  if (status == LQ_OK && n_fp > 0) {
    std::vector<int> slots(n_fp);
    for (int64_t i = 0; i < n_fp; ++i) slots[i] = rows[i].second;
    if (!dev_alloc(c, reinterpret_cast<void**>(&slots_dev), n_fp * sizeof(int), true)) status = LQ_ERR_OOM;
    else cudaMemcpy(slots_dev, slots.data(), n_fp * sizeof(int), cudaMemcpyHostToDevice);
  }
  if (status == LQ_OK) {
    e = launch_import(c->cv, layer, static_cast<int>(n_fp), n_quant, slots_dev,
                      static_cast<const uint8_t*>(bufs[0].dev), static_cast<const uint8_t*>(bufs[1].dev),
                      static_cast<const uint16_t*>(bufs[2].dev), static_cast<const uint16_t*>(bufs[3].dev),
                      static_cast<const uint16_t*>(bufs[4].dev), static_cast<const uint16_t*>(bufs[5].dev),
                      static_cast<const uint16_t*>(bufs[6].dev), static_cast<const uint16_t*>(bufs[7].dev), nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) status = cuda_fail(c, e, "import kernels");
    c->n_launches += (n_quant > 0) + (n_fp > 0);
    c->last_decode_layer = -1;
  }
  for (auto& b : bufs) dev_release(c, b.dev);
  dev_release(c, slots_dev);
  if (status == LQ_ERR_OOM) cudaGetLastError();
  if (status != LQ_OK) L = saved;
  else if (!c->mask_dirty.empty()) c->mask_dirty[layer] = 1;
  return status;
}

lq_status_t lq_check_guards(lq_cache_t* c, int32_t* n_damaged) {
  if (!c || !n_damaged) return LQ_ERR_INVALID_ARG;
  *n_damaged = 0;
  if (c->dry) return LQ_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(c, e, "cudaDeviceSynchronize");
  *n_damaged = damaged_guards(c);
  return LQ_OK;
}

}  // extern "C"
