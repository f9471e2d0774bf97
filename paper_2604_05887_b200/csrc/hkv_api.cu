// Host side of libhkv: argument checks, the planner (every size, offset and work list follows from
// host inputs, so nothing here waits for the device) and the C ABI.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <initializer_list>
#include <mutex>
#include <cstring>
#include <new>
#include <vector>

#include "hkv_internal.h"

using namespace hkv;

namespace {

inline int64_t align_up(int64_t x, int64_t a = kAlign) { return (x + a - 1) / a * a; }

hkv_status check_config(const hkv_config* cfg) {
  if (!cfg) return HKV_ERR_INVALID_ARG;
  if (cfg->batch < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->max_seq_len < 1) return HKV_ERR_SHAPE;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return HKV_ERR_SHAPE;
  if (cfg->head_dim != kHeadDim) return HKV_ERR_UNSUPPORTED;
  if (cfg->n_q_heads / cfg->n_kv_heads > kMaxGroup) return HKV_ERR_UNSUPPORTED;
  if (cfg->chunk_size < 1 || cfg->obs_window < 1) return HKV_ERR_SHAPE;
  if (cfg->flags & ~(HKV_CAUSAL_WINDOW | HKV_OUT_F32 | HKV_GROUP_MAX | HKV_OFFLOAD_DYNAMIC)) return HKV_ERR_INVALID_ARG;
  if (!(cfg->softmax_scale >= 0.f) || std::isinf(cfg->softmax_scale)) return HKV_ERR_INVALID_ARG;
  if (static_cast<int64_t>(cfg->batch) * cfg->n_kv_heads > 60000) return HKV_ERR_UNSUPPORTED;
  if (cfg->append_capacity < 0 || cfg->append_capacity > (1 << 24)) return HKV_ERR_SHAPE;
  return HKV_OK;
}

// Fills every host-side field of `c` (units, splits, header with offsets, sizes).
hkv_status build_plan(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type, const int32_t* budgets,
                      hkv_cache& c, int64_t* ws_rowstat_off, int* n_col_tiles_max, bool offload = false) {
  hkv_status st = check_config(cfg);
  if (st != HKV_OK) return st;
  // the flag and the entry point go together: the dynamic planes need a second buffer
  if (((cfg->flags & HKV_OFFLOAD_DYNAMIC) != 0) != offload) return HKV_ERR_INVALID_ARG;
  if (!seq_lens || !head_type || !budgets) return HKV_ERR_INVALID_ARG;
  const int B = cfg->batch, Hkv = cfg->n_kv_heads, G = cfg->n_q_heads / Hkv, cs = cfg->chunk_size, w = cfg->obs_window;
  for (int b = 0; b < B; ++b) {
    if (seq_lens[b] < 1 || seq_lens[b] > cfg->max_seq_len) return HKV_ERR_SHAPE;
    if (w > seq_lens[b]) return HKV_ERR_SHAPE;
    for (int h = 0; h < Hkv; ++h) {
      if (head_type[b * Hkv + h] > 1) return HKV_ERR_INVALID_ARG;
      if (budgets[b * Hkv + h] < 1) return HKV_ERR_BUDGET;
    }
  }
  c.cfg = *cfg;
  c.units.clear();
  Header& H = c.hdr;
  std::memset(&H, 0, sizeof(H));
  H.batch = B; H.n_q_heads = cfg->n_q_heads; H.n_kv_heads = Hkv; H.group = G;
  H.chunk_size = cs; H.obs_window = w; H.max_seq_len = cfg->max_seq_len; H.flags = cfg->flags;
  H.scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(static_cast<float>(cfg->head_dim));
  H.n_units = B * Hkv;

  int max_C = 0;
  c.max_static_rows = c.max_dyn_rows = c.max_chunks = 0;
  c.retained = c.kv_bytes = c.summary_bytes = c.algo_bytes = 0;
  for (int b = 0; b < B; ++b) {
    for (int h = 0; h < Hkv; ++h) {
      Unit u;
      std::memset(&u, 0, sizeof(u));
      u.type = head_type[b * Hkv + h];
      u.b = b; u.h = h; u.C = seq_lens[b];
      u.budget = std::min(budgets[b * Hkv + h], u.C);
      u.budget_raw = budgets[b * Hkv + h];
      const int cap = cfg->append_capacity;
      if (u.type == 0) {
        u.n_tok = u.budget;
        u.plane_rows = u.n_tok + cap;
        u.cap_sel = u.n_tok + cap;
        c.max_static_rows = std::max(c.max_static_rows, u.plane_rows);
        max_C = std::max(max_C, u.C);
        H.n_static++;
        c.algo_bytes += 2ll * kRowBytes * u.n_tok;
      } else {
        u.n_chunks = (u.C + cs - 1) / cs;
        u.k_sel = std::min(u.n_chunks, (u.budget + cs - 1) / cs);
        const int64_t nt = static_cast<int64_t>(u.k_sel) * cs;
        u.cap_chunks = static_cast<int32_t>((static_cast<int64_t>(u.C) + cap + cs - 1) / cs);
        u.cap_sel = static_cast<int32_t>(std::min<int64_t>(u.cap_chunks, (static_cast<int64_t>(std::min<int64_t>(u.budget_raw, static_cast<int64_t>(u.C) + cap)) + cs - 1) / cs));
        const int64_t pr = static_cast<int64_t>(u.cap_chunks) * cs;
        if (pr > 0x7FFFFFF0ll) return HKV_ERR_UNSUPPORTED;
        u.n_tok = static_cast<int32_t>(nt);
        u.plane_rows = static_cast<int32_t>(pr);
        c.max_dyn_rows = std::max(c.max_dyn_rows, u.plane_rows);
        c.max_chunks = std::max(c.max_chunks, u.cap_chunks);
        H.n_dynamic++;
        c.algo_bytes += 2ll * kRowBytes * std::min<int64_t>(nt, u.C) + static_cast<int64_t>(kRowBytes) * u.n_chunks;
        c.summary_bytes += static_cast<int64_t>(kRowBytes) * u.n_chunks;
      }
      c.retained += std::min(u.n_tok, u.C);
      c.kv_bytes += 2ll * kRowBytes * u.plane_rows;
      c.units.push_back(u);
    }
  }

  c.max_tiles = 1;
  for (auto& u : c.units) c.max_tiles = std::max(c.max_tiles, (u.n_tok + kTile - 1) / kTile);

  // ---- cache_mem layout ----
  int64_t off = kUnitsOff;
  off = align_up(off + sizeof(Unit) * H.n_units);
  H.dyn_list_off = off;  off = align_up(off + 4ll * std::max(1, H.n_dynamic));
  H.sta_list_off = off;  off = align_up(off + 4ll * std::max(1, H.n_static));
  H.n_valid_off = off;   off = align_up(off + 4ll * H.n_units);   // tables end here; the rest starts at zero
  H.err_off = off;       off = align_up(off + 8);
  for (auto& u : c.units) {
    u.idx_off = off;
    off = align_up(off + 4ll * std::max(1, u.cap_sel));
    if (u.type == 1) {
      u.scores_off = off;    off = align_up(off + 4ll * u.cap_chunks);
      u.summ_off = off;      off = align_up(off + static_cast<int64_t>(kRowBytes) * u.cap_chunks);
      u.tail_sum_off = off;  off = align_up(off + 4ll * kHeadDim);
    }
  }
  // K and V planes; with HKV_OFFLOAD_DYNAMIC those of the dynamic units are laid out in the host buffer
  // (their offsets stay relative to that buffer until hkv_compress_offload knows both addresses)
  int64_t hoff = 0;
  for (auto& u : c.units) {
    int64_t& o = (offload && u.type == 1) ? hoff : off;
    u.k_off = o;  o = align_up(o + static_cast<int64_t>(kRowBytes) * u.plane_rows);
    u.v_off = o;  o = align_up(o + static_cast<int64_t>(kRowBytes) * u.plane_rows);
  }
  c.cache_bytes = static_cast<size_t>(off);
  c.host_bytes = static_cast<size_t>(hoff);

  // ---- workspace layout: s_w per static unit, then the row statistics of the window softmax ----
  int64_t woff = 0;
  for (auto& u : c.units) {
    if (u.type == 0) { u.ws_scores_off = woff; woff = align_up(woff + 4ll * u.C); }
  }
  const int R = w * G, Rpad = (R + 15) / 16 * 16;
  const int tiles_max = 2 * ((max_C + 127) / 128);   // two partial row statistics per 128-key tile at most
  if (ws_rowstat_off) *ws_rowstat_off = woff;
  if (n_col_tiles_max) *n_col_tiles_max = tiles_max;
  woff = align_up(woff + 8ll * H.n_static * tiles_max * Rpad + 8ll * H.n_static * Rpad);
  c.workspace_bytes = static_cast<size_t>(std::max<int64_t>(woff, kAlign));
  return HKV_OK;
}

bool bad_unit(const hkv_cache* c, int b, int h) {
  return !c || b < 0 || h < 0 || b >= c->cfg.batch || h >= c->cfg.n_kv_heads;
}

hkv_status d2h(void* dst, const void* src, size_t bytes, cudaStream_t s) {
  if (cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return HKV_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return HKV_ERR_CUDA;
  return HKV_OK;
}

}  // namespace

extern "C" {

namespace {
// A second stream and a few events per device, created on first use and never destroyed.
// hkv_decode_step_host: the queries of the layers after the first travel to the device while the
// first layer runs, and the outputs of all but the last group of layers travel back while later
// layers run.  hkv_compress: the dynamic heads' planes and chunk means are built beside the static
// heads' window scores, selection and gather (independent work on disjoint memory).
constexpr int kStepGroups = 4;
struct StepSide {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, q_done = nullptr, q_done2 = nullptr, join = nullptr, out[kStepGroups] = {};
  bool ready = false;
  std::mutex enqueue;   // held while a call records and waits on these events, so that host threads do not interleave
};
StepSide g_step_side[64];
std::mutex g_step_mutex;

StepSide* step_side() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_step_mutex);
  StepSide& s = g_step_side[dev];
  if (!s.ready) {
    bool ok = cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s.q_done, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s.q_done2, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kStepGroups; ++i)
      ok = cudaEventCreateWithFlags(&s.out[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return nullptr; }
    s.ready = true;
  }
  return &s;
}
}  // namespace

static hkv_status plan_common(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type,
                              const int32_t* budgets, size_t* cache_bytes, size_t* workspace_bytes, size_t* host_bytes) {
  if (!cache_bytes || !workspace_bytes) return HKV_ERR_INVALID_ARG;
  try {
    hkv_cache tmp;
    hkv_status st = build_plan(cfg, seq_lens, head_type, budgets, tmp, nullptr, nullptr, host_bytes != nullptr);
    if (st != HKV_OK) return st;
    *cache_bytes = tmp.cache_bytes;
    *workspace_bytes = tmp.workspace_bytes;
    if (host_bytes) *host_bytes = tmp.host_bytes;
    return HKV_OK;
  } catch (...) {
    return HKV_ERR_INVALID_ARG;
  }
}

hkv_status hkv_plan(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type, const int32_t* budgets,
                    size_t* cache_bytes, size_t* workspace_bytes) {
  return plan_common(cfg, seq_lens, head_type, budgets, cache_bytes, workspace_bytes, nullptr);
}

hkv_status hkv_plan_offload(const hkv_config* cfg, const int32_t* seq_lens, const uint8_t* head_type,
                            const int32_t* budgets, size_t* cache_bytes, size_t* workspace_bytes, size_t* host_bytes) {
  if (!host_bytes) return HKV_ERR_INVALID_ARG;
  return plan_common(cfg, seq_lens, head_type, budgets, cache_bytes, workspace_bytes, host_bytes);
}

static hkv_status compress_common(const hkv_config* cfg, const void* k, const void* v, const void* q_obs,
                                  const float* token_scores, const uint8_t* is_text, const int32_t* seq_lens,
                                  const uint8_t* head_type, const int32_t* budgets, void* cache_mem, size_t cache_bytes,
                                  void* host_mem, size_t host_bytes, bool offload, void* workspace,
                                  size_t workspace_bytes, void* stream, hkv_cache** out) {
  if (!out) return HKV_ERR_INVALID_ARG;
  *out = nullptr;
  if (!k || !v || !is_text || !cache_mem || !workspace) return HKV_ERR_INVALID_ARG;
  hkv_cache* c = nullptr;
  try {
    c = new hkv_cache();
    int64_t ws_rowstat_off = 0;
    int tiles_max = 0;
    hkv_status st = build_plan(cfg, seq_lens, head_type, budgets, *c, &ws_rowstat_off, &tiles_max, offload);
    if (st == HKV_OK && offload) {
      if (c->host_bytes > 0 && !host_mem) st = HKV_ERR_INVALID_ARG;
      else if (host_bytes < c->host_bytes || (reinterpret_cast<uintptr_t>(host_mem) & (kAlign - 1))) st = HKV_ERR_WORKSPACE;
      if (st == HKV_OK && c->host_bytes > 0) {
        // the device must reach the whole buffer at the very pointer values given: pinned host memory under
        // unified addressing.  Anything else is refused here rather than found out by a kernel.
        for (const char* p : {static_cast<const char*>(host_mem), static_cast<const char*>(host_mem) + c->host_bytes - 1}) {
          cudaPointerAttributes attr;
          if (cudaPointerGetAttributes(&attr, p) != cudaSuccess || attr.type != cudaMemoryTypeHost ||
              attr.devicePointer != static_cast<const void*>(p)) {
            cudaGetLastError();
            st = HKV_ERR_INVALID_ARG;
          }
        }
      }
      if (st == HKV_OK) {
        // the kernels address every plane as cache_mem + offset: the dynamic planes' offsets now span the
        // distance to the host buffer, which the device reaches at the same (unified) address
        const int64_t delta = static_cast<int64_t>(reinterpret_cast<intptr_t>(host_mem) -
                                                   reinterpret_cast<intptr_t>(cache_mem));
        for (auto& u : c->units)
          if (u.type == 1) { u.k_off += delta; u.v_off += delta; }
      }
    }
    if (st == HKV_OK && c->hdr.n_static > 0 && !q_obs && !token_scores) st = HKV_ERR_INVALID_ARG;
    if (st == HKV_OK && (cache_bytes < c->cache_bytes || workspace_bytes < c->workspace_bytes)) st = HKV_ERR_WORKSPACE;
    if (st == HKV_OK && ((reinterpret_cast<uintptr_t>(cache_mem) | reinterpret_cast<uintptr_t>(workspace)) & (kAlign - 1)))
      st = HKV_ERR_WORKSPACE;
    if (st != HKV_OK) { delete c; return st; }
    c->dev_base = static_cast<char*>(cache_mem);
    c->fresh = true;
    c->appended = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const Header& H = c->hdr;

    // tables: one host image, one copy
    const size_t tables = static_cast<size_t>(H.n_valid_off);
    std::vector<char> img(tables, 0);
    std::memcpy(img.data(), &H, sizeof(H));
    std::memcpy(img.data() + kUnitsOff, c->units.data(), sizeof(Unit) * c->units.size());
    int32_t* dl = reinterpret_cast<int32_t*>(img.data() + H.dyn_list_off);
    int32_t* sl = reinterpret_cast<int32_t*>(img.data() + H.sta_list_off);
    for (int i = 0; i < H.n_units; ++i) {
      if (c->units[i].type) *dl++ = i; else *sl++ = i;
    }
    bool ok = cudaMemcpyAsync(c->dev_base, img.data(), tables, cudaMemcpyHostToDevice, s) == cudaSuccess;
    // n_valid and the error word start at zero
    ok = ok && cudaMemsetAsync(c->dev_base + H.n_valid_off, 0, static_cast<size_t>(H.err_off + 8 - H.n_valid_off), s) ==
                   cudaSuccess;
    // dynamic heads beside the static ones, on the library's second stream (forked from and joined to `s`)
    StepSide* side = (H.n_static > 0 && H.n_dynamic > 0) ? step_side() : nullptr;
    std::unique_lock<std::mutex> side_lock;
    if (side) side_lock = std::unique_lock<std::mutex>(side->enqueue);
    if (ok && side) {
      ok = cudaEventRecord(side->fork, s) == cudaSuccess && cudaStreamWaitEvent(side->stream, side->fork, 0) == cudaSuccess;
      ok = ok && launch_build_dynamic(c->dev_base, k, v, H, c->max_dyn_rows, c->max_chunks, side->stream) == cudaSuccess;
      ok = ok && cudaEventRecord(side->join, side->stream) == cudaSuccess;
    }
    if (ok && H.n_static > 0) {
      if (!token_scores)
        ok = launch_window_scores(c->dev_base, static_cast<char*>(workspace), k, q_obs, H, c->units, ws_rowstat_off,
                                  tiles_max, s) == cudaSuccess;
      ok = ok && launch_static_select(c->dev_base, static_cast<char*>(workspace), token_scores, is_text, H, s) == cudaSuccess;
      ok = ok && launch_gather_static(c->dev_base, k, v, H, c->max_static_rows, s) == cudaSuccess;
    }
    if (ok && H.n_dynamic > 0 && !side)
      ok = launch_build_dynamic(c->dev_base, k, v, H, c->max_dyn_rows, c->max_chunks, s) == cudaSuccess;
    if (ok && side) ok = cudaStreamWaitEvent(s, side->join, 0) == cudaSuccess;
    if (!ok) { cudaGetLastError(); delete c; return HKV_ERR_CUDA; }
    *out = c;
    return HKV_OK;
  } catch (...) {
    delete c;
    return HKV_ERR_INVALID_ARG;
  }
}

hkv_status hkv_compress(const hkv_config* cfg, const void* k, const void* v, const void* q_obs,
                        const float* token_scores, const uint8_t* is_text, const int32_t* seq_lens,
                        const uint8_t* head_type, const int32_t* budgets, void* cache_mem, size_t cache_bytes,
                        void* workspace, size_t workspace_bytes, void* stream, hkv_cache** out) {
  return compress_common(cfg, k, v, q_obs, token_scores, is_text, seq_lens, head_type, budgets, cache_mem, cache_bytes,
                         nullptr, 0, false, workspace, workspace_bytes, stream, out);
}

hkv_status hkv_compress_offload(const hkv_config* cfg, const void* k, const void* v, const void* q_obs,
                                const float* token_scores, const uint8_t* is_text, const int32_t* seq_lens,
                                const uint8_t* head_type, const int32_t* budgets, void* cache_mem, size_t cache_bytes,
                                void* host_mem, size_t host_bytes, void* workspace, size_t workspace_bytes,
                                void* stream, hkv_cache** out) {
  return compress_common(cfg, k, v, q_obs, token_scores, is_text, seq_lens, head_type, budgets, cache_mem, cache_bytes,
                         host_mem, host_bytes, true, workspace, workspace_bytes, stream, out);
}

#ifdef HKV_CHECKED
hkv_status hkv_selftest_wait_timeout(hkv_cache* c, void* stream) {
  if (!c) return HKV_ERR_INVALID_ARG;
  if (launch_selftest_wait(reinterpret_cast<int32_t*>(c->dev_base + c->hdr.err_off), static_cast<cudaStream_t>(stream)) !=
      cudaSuccess) {
    cudaGetLastError();
    return HKV_ERR_CUDA;
  }
  return HKV_OK;
}
hkv_status hkv_clear_device_error(hkv_cache* c, void* stream) {
  if (!c) return HKV_ERR_INVALID_ARG;
  if (cudaMemsetAsync(c->dev_base + c->hdr.err_off, 0, 8, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return HKV_ERR_CUDA;
  }
  return HKV_OK;
}
#endif

#ifdef HKV_PROFILE
static unsigned long long* g_prof = nullptr;
static long long g_prof_ctas = 0, g_prof_cursor = 0;
// Profiling build only: device buffer of kProfSlots x 8 bytes per CTA; successive decode launches
// take successive regions of it (a launch that no longer fits is not recorded).
int hkv_profile_attach(void* dev_buffer, long long n_ctas) {
  g_prof = static_cast<unsigned long long*>(dev_buffer);
  g_prof_ctas = n_ctas;
  g_prof_cursor = 0;
  return 0;
}
#endif

static hkv_status decode_stages(hkv_cache* const* caches, const void* const* q, void* const* out, int32_t n,
                                void* stream, bool do_select, bool do_attend) {
  if (!caches || !q || n < 1 || n > kMaxMulti || (do_attend && !out)) return HKV_ERR_INVALID_ARG;
  DecodeParams P;
  std::memset(&P, 0, sizeof(P));
  P.n = n;
  int max_tiles = 1, n_dynamic = 0;
  for (int i = 0; i < n; ++i) {
    const hkv_cache* c = caches[i];
    if (!c || !q[i] || (do_attend && !out[i])) return HKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q[i]) & 3) || (do_attend && (reinterpret_cast<uintptr_t>(out[i]) & 15)))
      return HKV_ERR_INVALID_ARG;
    const Header& H = c->hdr;
    const Header& H0 = caches[0]->hdr;
    if (H.group != H0.group || H.n_q_heads != H0.n_q_heads || H.n_kv_heads != H0.n_kv_heads ||
        H.chunk_size != H0.chunk_size || H.scale != H0.scale || ((H.flags ^ H0.flags) & (HKV_OUT_F32 | HKV_GROUP_MAX | HKV_OFFLOAD_DYNAMIC)))
      return HKV_ERR_SHAPE;
    P.cache[i] = c->dev_base;
    P.q[i] = q[i];
    P.out[i] = do_attend ? out[i] : nullptr;
    P.n_valid_off[i] = H.n_valid_off;
    P.err_off[i] = H.err_off;
    P.dyn_list_off[i] = H.dyn_list_off;
    P.sta_list_off[i] = H.sta_list_off;
    P.n_dynamic[i] = H.n_dynamic;
    P.unit_prefix[i + 1] = P.unit_prefix[i] + H.n_units;
    max_tiles = std::max(max_tiles, c->max_tiles);
    n_dynamic += H.n_dynamic;
  }
  if (!do_attend && n_dynamic == 0) return HKV_OK;   // nothing to select
  const Header& H0 = caches[0]->hdr;
  P.group = H0.group; P.n_q_heads = H0.n_q_heads; P.n_kv_heads = H0.n_kv_heads; P.chunk_size = H0.chunk_size;
  P.scale_log2e = H0.scale * 1.4426950408889634f;
  P.phase = (do_select ? kPhaseSelect : 0u) | (do_attend ? kPhaseAttend : 0u);
  P.out_f32 = (H0.flags & HKV_OUT_F32) ? 1u : 0u;
  P.group_max = (H0.flags & HKV_GROUP_MAX) ? 1u : 0u;
  P.offload = (H0.flags & HKV_OFFLOAD_DYNAMIC) ? 1u : 0u;
  const int* max_active = nullptr;
  if (decode_cluster_caps(P.group, &max_active) != cudaSuccess) { cudaGetLastError(); return HKV_ERR_CUDA; }
  const int total_units = P.unit_prefix[n];
  P.cluster = choose_cluster(total_units, max_tiles, max_active);
  // A launch that follows another decode launch starts, in block order, as many blocks as the device has room
  // for beside its predecessor's.  When that is not all of them, the static units go first if they all fit:
  // they use the head start to stage their first K/V tiles, which is worth most.  Otherwise (everything fits,
  // or not even the static units do) the dynamic units go first: their chain of dependent stages is the
  // longer one and must not also wait for a slot.
  {
    const long long slots = static_cast<long long>(max_active[P.cluster]) * P.cluster;
    const long long all = static_cast<long long>(total_units) * P.cluster;
    const long long sta = static_cast<long long>(total_units - n_dynamic) * P.cluster;
    P.static_first = (2 * all > slots && sta <= slots - all) ? 1u : 0u;
  }
  // The launch may overlap the tail of a preceding decode launch (it touches nothing that depends on
  // earlier work before its dependency wait).  Right after hkv_compress the cache itself is what
  // the preceding kernels are still writing, so that first launch is fully serialised.
  bool fresh = false;
  for (int i = 0; i < n; ++i) fresh = fresh || caches[i]->fresh;
  P.pdl = fresh ? 0u : 1u;
#ifdef HKV_PROFILE
  {
    const long long ctas = static_cast<long long>(total_units) * P.cluster;
    P.prof = nullptr;
    if (g_prof && g_prof_cursor + ctas <= g_prof_ctas) {
      P.prof = g_prof + g_prof_cursor * kProfSlots;
      g_prof_cursor += ctas;
    }
  }
#endif
  if (launch_decode(P, total_units, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return HKV_ERR_CUDA;
  }
  for (int i = 0; i < n; ++i) caches[i]->fresh = false;
  return HKV_OK;
}

hkv_status hkv_decode_attn_multi(hkv_cache* const* caches, const void* const* q, void* const* out, int32_t n,
                                 void* stream) {
  return decode_stages(caches, q, out, n, stream, true, true);
}

hkv_status hkv_decode_attn(hkv_cache* cache, const void* q, void* out, void* stream) {
  if (!cache) return HKV_ERR_INVALID_ARG;
  hkv_cache* one[1] = {cache};
  const void* qs[1] = {q};
  void* os[1] = {out};
  return decode_stages(one, qs, os, 1, stream, true, true);
}

hkv_status hkv_select_chunks(hkv_cache* cache, const void* q, void* stream) {
  if (!cache) return HKV_ERR_INVALID_ARG;
  hkv_cache* one[1] = {cache};
  const void* qs[1] = {q};
  return decode_stages(one, qs, nullptr, 1, stream, true, false);
}

hkv_status hkv_attend(hkv_cache* cache, const void* q, void* out, void* stream) {
  if (!cache) return HKV_ERR_INVALID_ARG;
  hkv_cache* one[1] = {cache};
  const void* qs[1] = {q};
  void* os[1] = {out};
  return decode_stages(one, qs, os, 1, stream, false, true);
}

hkv_status hkv_decode_attn_host(hkv_cache* cache, const void* q_host, void* out_host, void* q_dev, void* out_dev,
                                void* stream) {
  if (!cache || !q_host || !out_host || !q_dev || !out_dev) return HKV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t n = static_cast<size_t>(cache->cfg.batch) * cache->cfg.n_q_heads * cache->cfg.head_dim;
  const size_t out_elt = (cache->hdr.flags & HKV_OUT_F32) ? 4 : 2;
  if (cudaMemcpyAsync(q_dev, q_host, n * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) { cudaGetLastError(); return HKV_ERR_CUDA; }
  hkv_status st = hkv_decode_attn(cache, q_dev, out_dev, stream);
  if (st != HKV_OK) return st;
  if (cudaMemcpyAsync(out_host, out_dev, n * out_elt, cudaMemcpyDeviceToHost, s) != cudaSuccess) { cudaGetLastError(); return HKV_ERR_CUDA; }
  return HKV_OK;
}

hkv_status hkv_decode_step_host(hkv_cache* const* caches, int32_t n, const void* q_host, void* out_host, void* q_dev,
                                void* out_dev, void* stream) {
  if (!caches || n < 1 || !q_host || !out_host || !q_dev || !out_dev) return HKV_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!caches[i]) return HKV_ERR_INVALID_ARG;
    const hkv_config &a = caches[i]->cfg, &b = caches[0]->cfg;
    if (a.batch != b.batch || a.n_q_heads != b.n_q_heads || a.head_dim != b.head_dim ||
        ((a.flags ^ b.flags) & (HKV_OUT_F32 | HKV_GROUP_MAX)))
      return HKV_ERR_SHAPE;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t per = static_cast<size_t>(caches[0]->cfg.batch) * caches[0]->cfg.n_q_heads * caches[0]->cfg.head_dim;
  const size_t out_elt = (caches[0]->hdr.flags & HKV_OUT_F32) ? 4 : 2;
  const char* qh = static_cast<const char*>(q_host);
  char* qd = static_cast<char*>(q_dev);
  char* oh = static_cast<char*>(out_host);
  char* od = static_cast<char*>(out_dev);
  StepSide* side = n >= 2 ? step_side() : nullptr;
  std::unique_lock<std::mutex> side_lock;
  if (side) side_lock = std::unique_lock<std::mutex>(side->enqueue);
  const int q_split = std::min(n, 4);   // layers 1 .. q_split - 1 get their queries in a first, short transfer
  bool ok = true;
  auto cu = [&](cudaError_t e) { ok = ok && e == cudaSuccess; };

  // queries: the first layer's on the caller's stream, the rest beside it
  cu(cudaMemcpyAsync(qd, qh, per * 2 * (side ? 1 : n), cudaMemcpyHostToDevice, s));
  if (side) {
    cu(cudaEventRecord(side->fork, s));
    cu(cudaStreamWaitEvent(side->stream, side->fork, 0));
    // a short piece first, so that the second layer is not held up by the whole transfer
    cu(cudaMemcpyAsync(qd + per * 2, qh + per * 2, per * 2 * (q_split - 1), cudaMemcpyHostToDevice, side->stream));
    cu(cudaEventRecord(side->q_done, side->stream));
    if (q_split < n) {
      cu(cudaMemcpyAsync(qd + per * 2 * q_split, qh + per * 2 * q_split, per * 2 * (n - q_split), cudaMemcpyHostToDevice,
                         side->stream));
      cu(cudaEventRecord(side->q_done2, side->stream));
    }
  }
  if (!ok) { cudaGetLastError(); return HKV_ERR_CUDA; }
  // layers in order; after each group of layers but the last, its outputs start their way back
  const int groups = side ? std::min(kStepGroups, n) : 1;
  int done_out = 0;   // layers whose outputs have been sent
  for (int i = 0; i < n; ++i) {
    if (side && i == 1) cu(cudaStreamWaitEvent(s, side->q_done, 0));
    if (side && i == q_split && q_split < n) cu(cudaStreamWaitEvent(s, side->q_done2, 0));
    hkv_status st = hkv_decode_attn(caches[i], qd + per * 2 * i, od + per * out_elt * i, stream);
    if (st != HKV_OK) return st;
    const int g = static_cast<int>((static_cast<long long>(i + 1) * groups) / n);   // groups complete after layer i
    const int g_prev = static_cast<int>((static_cast<long long>(i) * groups) / n);
    if (side && g > g_prev && g < groups) {
      cu(cudaEventRecord(side->out[g - 1], s));
      cu(cudaStreamWaitEvent(side->stream, side->out[g - 1], 0));
      cu(cudaMemcpyAsync(oh + per * out_elt * done_out, od + per * out_elt * done_out,
                         per * out_elt * (i + 1 - done_out), cudaMemcpyDeviceToHost, side->stream));
      done_out = i + 1;
    }
  }
  cu(cudaMemcpyAsync(oh + per * out_elt * done_out, od + per * out_elt * done_out, per * out_elt * (n - done_out),
                     cudaMemcpyDeviceToHost, s));
  if (side) {   // the caller's stream ends the step only when the side copies have ended
    cu(cudaEventRecord(side->join, side->stream));
    cu(cudaStreamWaitEvent(s, side->join, 0));
  }
  if (!ok) { cudaGetLastError(); return HKV_ERR_CUDA; }
  return HKV_OK;
}

hkv_status hkv_append(hkv_cache* c, const void* k_new, const void* v_new, void* stream) {
  if (!c || !k_new || !v_new) return HKV_ERR_INVALID_ARG;
  if (c->appended >= c->cfg.append_capacity) return HKV_ERR_WORKSPACE;
  if (launch_append(c->dev_base, k_new, v_new, c->hdr, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    cudaGetLastError();
    return HKV_ERR_CUDA;
  }
  // the host mirror follows the same rule as the kernel, so that no call has to wait for the device
  const int cs = c->cfg.chunk_size;
  c->retained = c->algo_bytes = c->summary_bytes = 0;
  c->max_tiles = 1;
  for (auto& u : c->units) {
    u.C += 1;
    if (u.type == 0) {
      u.n_tok += 1;
      c->algo_bytes += 2ll * kRowBytes * u.n_tok;
    } else {
      u.n_chunks = (u.C + cs - 1) / cs;
      u.k_sel = std::min(u.n_chunks, (std::min(u.budget_raw, u.C) + cs - 1) / cs);
      u.n_tok = u.k_sel * cs;
      c->algo_bytes += 2ll * kRowBytes * std::min(u.n_tok, u.C) + static_cast<int64_t>(kRowBytes) * u.n_chunks;
      c->summary_bytes += static_cast<int64_t>(kRowBytes) * u.n_chunks;
    }
    c->retained += std::min(u.n_tok, u.C);
    c->max_tiles = std::max(c->max_tiles, (u.n_tok + kTile - 1) / kTile);
  }
  c->appended += 1;
  c->fresh = true;   // the next decode launch must not start before this kernel has finished
  return HKV_OK;
}

hkv_status hkv_cache_destroy(hkv_cache* cache) {
  delete cache;
  return HKV_OK;
}

hkv_status hkv_get_static_indices(hkv_cache* c, int32_t b, int32_t h, int32_t* host_out, int32_t capacity, int32_t* n,
                                  void* stream) {
  if (bad_unit(c, b, h) || !host_out || !n) return HKV_ERR_INVALID_ARG;
  const Unit& u = c->units[b * c->cfg.n_kv_heads + h];
  if (u.type != 0) return HKV_ERR_INVALID_ARG;
  *n = u.n_tok;
  if (capacity < u.n_tok) return HKV_ERR_WORKSPACE;
  return d2h(host_out, c->dev_base + u.idx_off, 4ull * u.n_tok, static_cast<cudaStream_t>(stream));
}

hkv_status hkv_get_selected_chunks(hkv_cache* c, int32_t b, int32_t h, int32_t* host_out, int32_t capacity, int32_t* n,
                                   void* stream) {
  if (bad_unit(c, b, h) || !host_out || !n) return HKV_ERR_INVALID_ARG;
  const Unit& u = c->units[b * c->cfg.n_kv_heads + h];
  if (u.type != 1) return HKV_ERR_INVALID_ARG;
  *n = u.k_sel;
  if (capacity < u.k_sel) return HKV_ERR_WORKSPACE;
  return d2h(host_out, c->dev_base + u.idx_off, 4ull * u.k_sel, static_cast<cudaStream_t>(stream));
}

hkv_status hkv_get_chunk_scores(hkv_cache* c, int32_t b, int32_t h, float* host_out, int32_t capacity, int32_t* n,
                                void* stream) {
  if (bad_unit(c, b, h) || !host_out || !n) return HKV_ERR_INVALID_ARG;
  const Unit& u = c->units[b * c->cfg.n_kv_heads + h];
  if (u.type != 1) return HKV_ERR_INVALID_ARG;
  *n = u.n_chunks;
  if (capacity < u.n_chunks) return HKV_ERR_WORKSPACE;
  return d2h(host_out, c->dev_base + u.scores_off, 4ull * u.n_chunks, static_cast<cudaStream_t>(stream));
}

hkv_status hkv_get_summaries(hkv_cache* c, int32_t b, int32_t h, uint16_t* host_out, int32_t capacity_rows,
                             int32_t* n_chunks, void* stream) {
  if (bad_unit(c, b, h) || !host_out || !n_chunks) return HKV_ERR_INVALID_ARG;
  const Unit& u = c->units[b * c->cfg.n_kv_heads + h];
  if (u.type != 1) return HKV_ERR_INVALID_ARG;
  *n_chunks = u.n_chunks;
  if (capacity_rows < u.n_chunks) return HKV_ERR_WORKSPACE;
  hkv_status st = d2h(host_out, c->dev_base + u.summ_off, static_cast<size_t>(kRowBytes) * u.n_chunks,
                      static_cast<cudaStream_t>(stream));
  if (st != HKV_OK) return st;
  // rows are held with their 16-byte pieces permuted by (row & 7): put them back in order
  for (int r = 0; r < u.n_chunks; ++r) {
    uint16_t* row = host_out + static_cast<size_t>(r) * kHeadDim;
    uint16_t tmp[kHeadDim];
    std::memcpy(tmp, row, sizeof(tmp));
    for (int p = 0; p < 16; ++p) std::memcpy(row + p * 8, tmp + ((p ^ (r & 7)) * 8), 16);
  }
  return HKV_OK;
}

hkv_status hkv_window_scores_offset(const hkv_cache* c, int32_t b, int32_t h, size_t* offset) {
  if (bad_unit(c, b, h) || !offset) return HKV_ERR_INVALID_ARG;
  const Unit& u = c->units[b * c->cfg.n_kv_heads + h];
  if (u.type != 0) return HKV_ERR_INVALID_ARG;
  *offset = static_cast<size_t>(u.ws_scores_off);
  return HKV_OK;
}

hkv_status hkv_decode_cluster_capacity(int32_t group, int32_t* max_active_clusters) {
  if (!max_active_clusters || group < 1 || group > kMaxGroup) return HKV_ERR_INVALID_ARG;
  const int* caps = nullptr;
  if (decode_cluster_caps(group, &caps) != cudaSuccess) { cudaGetLastError(); return HKV_ERR_CUDA; }
  for (int c = 1; c <= kMaxCluster; ++c) max_active_clusters[c - 1] = caps[c];
  return HKV_OK;
}

hkv_status hkv_cache_stats(const hkv_cache* c, hkv_stats* st) {
  if (!c || !st) return HKV_ERR_INVALID_ARG;
  std::memset(st, 0, sizeof(*st));
  st->retained_tokens = c->retained;
  st->kv_bytes_resident = c->kv_bytes;
  st->summary_bytes = c->summary_bytes;
  st->algorithmic_bytes_per_step = c->algo_bytes;
  st->cache_bytes = static_cast<int64_t>(c->cache_bytes);
  st->workspace_bytes = static_cast<int64_t>(c->workspace_bytes);
  st->n_static = c->hdr.n_static;
  st->n_dynamic = c->hdr.n_dynamic;
  {
    // CTAs of a decode launch on this cache alone; without a device, the capacities of a B200
    const int* max_active = nullptr;
    int assumed[kMaxCluster + 1] = {};
    if (decode_cluster_caps(c->hdr.group, &max_active) != cudaSuccess) {
      cudaGetLastError();
      static const int b200[kMaxCluster + 1] = {0, 296, 148, 93, 71, 56, 45, 37, 33, 30, 26, 21, 21, 17, 14, 14, 14};
      for (int k = 1; k <= kMaxCluster; ++k) assumed[k] = b200[k];   // as measured on a B200 (148 SMs, two CTAs each)
      max_active = assumed;
    }
    st->n_splits = c->hdr.n_units * choose_cluster(c->hdr.n_units, c->max_tiles, max_active);
  }
  st->launches_per_decode = 1;
  return HKV_OK;
}

hkv_status hkv_last_device_error(hkv_cache* c, int32_t* code, int32_t* detail, void* stream) {
  if (!c || !code || !detail) return HKV_ERR_INVALID_ARG;
  int32_t w[2] = {0, 0};
  hkv_status st = d2h(w, c->dev_base + c->hdr.err_off, sizeof(w), static_cast<cudaStream_t>(stream));
  if (st != HKV_OK) return st;
  *code = w[0];
  *detail = w[1];
  return HKV_OK;
}

const char* hkv_status_string(hkv_status s) {
  switch (s) {
    case HKV_OK: return "ok";
    case HKV_ERR_INVALID_ARG: return "invalid argument";
    case HKV_ERR_SHAPE: return "inconsistent shape";
    case HKV_ERR_BUDGET: return "budget below one token";
    case HKV_ERR_WORKSPACE: return "buffer too small or misaligned";
    case HKV_ERR_UNSUPPORTED: return "unsupported geometry";
    case HKV_ERR_CUDA: return "CUDA runtime error";
    case HKV_ERR_TIMEOUT: return "device-side wait ran out";
    case HKV_ERR_INDEX: return "device-side index check failed";
  }
  return "unknown status";
}

}  // extern "C"
