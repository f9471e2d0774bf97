// Compression kernels (run once per prompt and layer): observation-window scores s_w for static
// heads, the text-prior keep-set, the gather into the compacted static cache, and for dynamic heads
// the chunk means plus the copy of K/V into the cache.  K/V rows are written with their sixteen
// 16-byte pieces XOR-permuted by (row & 7), the layout the flash-decode kernel stages with plain
// bulk copies and reads with bank-conflict-free ldmatrix.
#include <algorithm>

#include "hkv_device.cuh"
#include "hkv_internal.h"
#include "hkv_tc.cuh"

namespace hkv {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ const Unit* unit_of(const char* cache, const Header* hdr, bool dynamic, int ordinal,
                                               int* uid_out) {
  const int32_t* list = reinterpret_cast<const int32_t*>(cache + (dynamic ? hdr->dyn_list_off : hdr->sta_list_off));
  const int uid = list[ordinal];
  if (uid_out) *uid_out = uid;
  return reinterpret_cast<const Unit*>(cache + kUnitsOff) + uid;
}

// ---------------------------------------------------------------------------------------------
// Window scores.  S_w = softmax over ALL tokens of the w*G window rows' logits, s_w = mean of rows
// (row r = window position r / G, query head r % G of the group).  The logits run on the tcgen05
// tensor cores: one CTA = one static unit x one range of 128-key tiles x one block of up to 256
// rows; the row block stays in shared memory, the key tiles stream; logits in base 2.
// MODE 0: accumulator rows = window rows; a draining thread owns one row and keeps its running
//         (max, exp-sum) over its half of the CTA's keys; stats: float2 [n_static][2 ranges][Rpad].
// MODE 1: with the rows' final (max, sum) known, accumulator rows = keys; a draining thread owns
//         one key and sums the normalised probabilities of its quarter of the rows, the four
//         quarters meet in shared memory, and s_w[key] (+)= sum / R (written by the first row block, added
//         to by later ones).
// grid (key ranges, n_static).
// ---------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(tc::kThreads, 1)
    window_scores_tc_kernel(char* cache, char* workspace, const __nv_bfloat16* kin, const __nv_bfloat16* q_obs,
                            float2* stats, const float2* final_stats, int n_ranges_max, int Rpad,
                            int tiles_per_cta, int row_block) {
  extern __shared__ __align__(16) uint8_t tc_smem[];
  __shared__ float4 rowinfo[tc::kQRows];   // MODE 1: (max, 1 / sum, last visible key, -) of each resident row

  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, false, blockIdx.y, nullptr);
  const int C = u->C, G = hdr->group, w = hdr->obs_window, Hq = hdr->n_q_heads, Hkv = hdr->n_kv_heads;
  const int R = w * G, row0 = row_block * tc::kQRows;
  const int n_tiles = (C + tc::kKeysPerTile - 1) / tc::kKeysPerTile;
  const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(n_tiles, tile_begin + tiles_per_cta);
  if (tile_begin >= tile_end) return;
  const bool causal = (hdr->flags & HKV_CAUSAL_WINDOW) != 0;
  const float sc = hdr->scale * kLog2e;
  const int ub = u->b, uh = u->h;

  auto q_row = [&](int row) -> const __nv_bfloat16* {
    const int r = row0 + row;
    if (r >= R) return nullptr;
    const int i = r / G;
    return q_obs + ((static_cast<size_t>(ub) * w + i) * Hq + uh * G + (r - i * G)) * kHeadDim;
  };
  const __nv_bfloat16* keys =
      kin + (static_cast<size_t>(ub) * Hkv + uh) * static_cast<size_t>(hdr->max_seq_len) * kHeadDim;
  int32_t* err = reinterpret_cast<int32_t*>(cache + hdr->err_off);

  if (MODE == 0) {
    float m_run = -INFINITY, z_run = 0.f;
    int my_row = -1;
    int my_half = 0;
    auto epilogue = [&](int tile, int lane_row, int part, auto groups, float*, auto, uint64_t*) {
      // accumulator columns 64 part .. + 63 = keys 64 (part & 1) .. + 63 of the tile for the rows of block part >> 1
      const int r = row0 + 128 * (part >> 1) + lane_row;
      my_row = r;
      my_half = part & 1;
      if (row0 + 128 * (part >> 1) + (lane_row & ~31) >= R) return;   // the warp's rows are all padding
      const int lim = causal ? (C - w + r / G) : (C - 1);      // last key the row sees
      const int j0 = tile * tc::kKeysPerTile;
      const bool all_visible = j0 + tc::kKeysPerTile - 1 <= (causal ? C - w : C - 1);   // to every row
      groups([&](int g, float (&v)[32]) {
        const int jg = j0 + 64 * (part & 1) + g * 32;
        float gmax = -INFINITY;
        if (all_visible) {
          float g0 = v[0], g1 = v[1], g2 = v[2], g3 = v[3];   // four short chains instead of one long one
#pragma unroll
          for (int c = 4; c < 32; c += 4) {
            g0 = fmaxf(g0, v[c]);
            g1 = fmaxf(g1, v[c + 1]);
            g2 = fmaxf(g2, v[c + 2]);
            g3 = fmaxf(g3, v[c + 3]);
          }
          gmax = fmaxf(fmaxf(g0, g1), fmaxf(g2, g3)) * sc;   // the scale is positive
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            v[c] = (jg + c <= lim && jg + c < C) ? v[c] : -INFINITY;
            gmax = fmaxf(gmax, v[c] * sc);
          }
        }
        if (gmax > -INFINITY) {
          const float m_new = fmaxf(m_run, gmax);
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            a0 += fast_exp2(fmaf(v[c], sc, -m_new));
            a1 += fast_exp2(fmaf(v[c + 1], sc, -m_new));
            a2 += fast_exp2(fmaf(v[c + 2], sc, -m_new));
            a3 += fast_exp2(fmaf(v[c + 3], sc, -m_new));
          }
          z_run = z_run * fast_exp2(m_run - m_new) + ((a0 + a1) + (a2 + a3));   // 2^(-inf) = 0 on the first visible group
          m_run = m_new;
        }
      });
    };
    const bool ok = tc::scores_cta<false>(tc_smem, q_row, keys, C, tile_begin, tile_end, epilogue);
    // two threads share a row (one per half of every tile): two partial statistics per key range
    if (threadIdx.x >= 64 && my_row >= 0 && my_row < R)
      stats[(static_cast<size_t>(blockIdx.y) * n_ranges_max + 2 * blockIdx.x + my_half) * Rpad + my_row] =
          make_float2(m_run, z_run);
    if (!ok && threadIdx.x == 0) { atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT); err[1] = kErrScoreWait; }
  } else {
    for (int i = threadIdx.x; i < tc::kQRows; i += tc::kThreads) {
      const int r = row0 + i;
      float4 info = make_float4(0.f, 0.f, -1.f, 0.f);   // a padding row sees no key
      if (r < R) {
        const float2 f = final_stats[static_cast<size_t>(blockIdx.y) * Rpad + r];
        info = make_float4(f.x, 1.f / f.y, static_cast<float>(causal ? (C - w + r / G) : (C - 1)), 0.f);
      }
      rowinfo[i] = info;
    }
    // (scores_cta synchronises the CTA before any tile is drained)
    float* sw = reinterpret_cast<float*>(workspace + u->ws_scores_off);
    const float inv_R = 1.f / static_cast<float>(R);
    int n_done = 0;
    bool pair_ok = true;
    auto epilogue = [&](int tile, int lane_row, int part, auto groups, float* scratch, auto siblings,
                        uint64_t* pair_bar) {
      // accumulator columns 64 part .. + 63 = window rows row0 + 64 part + (0..63) for the key of this lane
      const int j0 = tile * tc::kKeysPerTile, j = j0 + lane_row;
      const float jf = static_cast<float>(j);
      const bool all_visible = j0 + tc::kKeysPerTile - 1 <= (causal ? C - w : C - 1);   // to every row
      float acc = 0.f, acc2 = 0.f, acc3 = 0.f, acc4 = 0.f;
      if (row0 + 64 * part < R) {                      // same for the whole warp
        groups([&](int g, float (&v)[32]) {
          if (row0 + 64 * part + 32 * g >= R) return;   // 32 padding rows: nothing to add (same for the whole warp)
          const float4* info = rowinfo + 64 * part + 32 * g;
          if (all_visible) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              const float4 r0 = info[c], r1 = info[c + 1], r2 = info[c + 2], r3 = info[c + 3];   // padding rows: 1 / sum = 0
              acc = fmaf(fast_exp2(fmaf(v[c], sc, -r0.x)), r0.y, acc);
              acc2 = fmaf(fast_exp2(fmaf(v[c + 1], sc, -r1.x)), r1.y, acc2);
              acc3 = fmaf(fast_exp2(fmaf(v[c + 2], sc, -r2.x)), r2.y, acc3);
              acc4 = fmaf(fast_exp2(fmaf(v[c + 3], sc, -r3.x)), r3.y, acc4);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const float4 ri = info[c];
              const float p = fast_exp2(fmaf(v[c], sc, -ri.x)) * ri.y;
              acc += (jf <= ri.z) ? p : 0.f;
            }
          }
        });
      }
      acc = (acc + acc2) + (acc3 + acc4);
      // the warps of parts 1..3 hand their sums over (two buffers, by tile parity); the part-0 warp adds them in
      // a fixed order and stores.  pair_bar is the barrier of this tile's parity: its (n_done / 2)-th use.
      const int slot = (n_done & 1) * 32 + (lane_row & 31);
      if (part != 0) {
        scratch[slot] = acc;
        tc::mbar_arrive(pair_bar);
      } else {
        if (pair_ok) pair_ok = mbar_wait_bounded(pair_bar, (n_done >> 1) & 1);
        if (pair_ok && j < C) {
          const float tot = ((acc + siblings(1)[slot]) + (siblings(2)[slot] + siblings(3)[slot])) * inv_R;
          sw[j] = row_block == 0 ? tot : sw[j] + tot;
        }
      }
      ++n_done;
    };
    const bool ok = tc::scores_cta<true>(tc_smem, q_row, keys, C, tile_begin, tile_end, epilogue);
    const bool pairs = __syncthreads_and(pair_ok);
    if (!(ok && pairs) && threadIdx.x == 0) {
      atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT);
      err[1] = kErrScoreWait;
    }
  }
}

// Combines the per-range (max, sum) of every window row into the row's final (max, sum): one warp per
// row, lanes stride the key ranges.
constexpr int kRowReduceWarps = 8;
__global__ void __launch_bounds__(kRowReduceWarps * 32)
    window_rowreduce_kernel(const char* cache, const float2* stats, float2* final_stats, int n_tiles_max, int Rpad,
                            int tiles_per_cta) {
  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, false, blockIdx.y, nullptr);
  const int R = hdr->obs_window * hdr->group;
  // two partial statistics (one per half of the key tiles) for every key range of the unit
  const int n_tiles = 2 * (((u->C + tc::kKeysPerTile - 1) / tc::kKeysPerTile + tiles_per_cta - 1) / tiles_per_cta);
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * kRowReduceWarps + (threadIdx.x >> 5);
  if (r >= R) return;
  const float2* st = stats + static_cast<size_t>(blockIdx.y) * n_tiles_max * Rpad + r;
  float M = -INFINITY;
  for (int jt = lane; jt < n_tiles; jt += 32) M = fmaxf(M, st[static_cast<size_t>(jt) * Rpad].x);
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
  float Z = 0.f;
  for (int jt = lane; jt < n_tiles; jt += 32) {
    const float2 v = st[static_cast<size_t>(jt) * Rpad];
    if (v.x > -INFINITY) Z += v.y * exp2f(v.x - M);
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, off);
  if (lane == 0) final_stats[static_cast<size_t>(blockIdx.y) * Rpad + r] = make_float2(M, Z);
}

// ---------------------------------------------------------------------------------------------
// Static keep-set: window U text-before-window U Top-M visual-before-window by score (ties to the
// lower position); when window + text exceed the budget, text is ranked instead; when the budget
// does not exceed the window, the last `budget` tokens.  One CTA per static unit, ascending output.
// The selection makes several passes over the tokens; each token's role (kept regardless / out of the
// ranking / ranked by this key) is therefore computed once into shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int kKeepThreads = 1024;
constexpr int kKeepScratchInts = keyed_scratch_ints(kKeepThreads);

constexpr uint32_t kKeepAlways = 0xFFFFFFFFu;   // no float's key (it would be a NaN's)

__global__ void __launch_bounds__(kKeepThreads)
    static_select_kernel(char* cache, const char* workspace, const float* token_scores, const uint8_t* is_text,
                         int key_slots, int skip_done) {
  __shared__ __align__(16) int scratch[kKeepScratchInts];
  __shared__ int s_ntext;
  extern __shared__ __align__(16) uint32_t skey[];   // key_slots entries: every token's role, computed once

  const Header* hdr = reinterpret_cast<const Header*>(cache);
  int uid;
  const Unit* u = unit_of(cache, hdr, false, blockIdx.x, &uid);
  const int C = u->C, w = hdr->obs_window, budget = u->n_tok;
  const int tid = threadIdx.x;
  const uint8_t* txt = is_text + static_cast<size_t>(u->b) * hdr->max_seq_len;
  const float* scores = token_scores
                            ? token_scores + (static_cast<size_t>(u->b) * hdr->n_kv_heads + u->h) * hdr->max_seq_len
                            : reinterpret_cast<const float*>(workspace + u->ws_scores_off);
  int32_t* out = reinterpret_cast<int32_t*>(cache + u->idx_off);
  const int hist_end = C - w;   // tokens before the window
  const bool cached = C <= key_slots;
  // after the cluster kernel: only the units it left (their count of kept tokens is still zero)
  if (skip_done && reinterpret_cast<const int32_t*>(cache + hdr->n_valid_off)[uid] != 0) return;

  if (tid == 0) s_ntext = 0;
  __syncthreads();
  // four tokens per thread and step when the rows of is_text and of the scores start on 4-token boundaries
  const bool vec = cached && (hdr->max_seq_len & 3) == 0 && (reinterpret_cast<uintptr_t>(is_text) & 3) == 0 &&
                   (reinterpret_cast<uintptr_t>(scores) & 15) == 0;
  int cnt = 0;
  if (vec) {
#pragma unroll 8
    for (int i = 4 * tid; i < hist_end; i += 4 * kKeepThreads) {
      const uchar4 t4 = *reinterpret_cast<const uchar4*>(txt + i);
      uint4 f = make_uint4(t4.x != 0, t4.y != 0, t4.z != 0, t4.w != 0);
      if (i + 1 >= hist_end) f.y = 0u;   // the tokens of the window are not counted
      if (i + 2 >= hist_end) f.z = 0u;
      if (i + 3 >= hist_end) f.w = 0u;
      cnt += static_cast<int>(f.x + f.y + f.z + f.w);
      *reinterpret_cast<uint4*>(skey + i) = f;
    }
  } else {
#pragma unroll 16
    for (int i = tid; i < hist_end; i += kKeepThreads) {
      const int t = txt[i] != 0;
      cnt += t;
      if (cached) skey[i] = static_cast<uint32_t>(t);
    }
  }
  for (int off = 16; off >= 1; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
  if ((tid & 31) == 0 && cnt) atomicAdd(&s_ntext, cnt);
  __syncthreads();
  const int n_text = s_ntext;

  int emitted;
  if (budget <= w) {
    const int start = C - budget;
    emitted = block_topk_keyed<kKeepThreads>(
        C, 0, [](int) { return 0u; }, [&](int i) { return i >= start; }, [&](int pos, int i) { out[pos] = i; }, scratch);
  } else {
    const int room = budget - w;
    const bool rank_text = n_text >= room;       // window + text do not fit: rank the text tokens
    const int k = rank_text ? room : room - n_text;
    if (cached) {
      // each token's role once: kKeepAlways = kept regardless, 0 = out of the ranking, else its score's key
      // (a thread rewrites only the entries it flagged above)
      auto role = [&](int i, uint32_t flag, float score) {
        if (i >= hist_end) return kKeepAlways;
        const bool is_t = flag != 0u;
        return (is_t == rank_text) ? float_key(score) : (is_t ? kKeepAlways : 0u);
      };
      if (vec) {
        // (the rows are max_seq_len floats long, so a whole float4 is readable wherever its first token is)
#pragma unroll 8
        for (int i = 4 * tid; i < C; i += 4 * kKeepThreads) {
          const float4 sc4 = *reinterpret_cast<const float4*>(scores + i);
          const uint4 f = i < hist_end ? *reinterpret_cast<const uint4*>(skey + i) : make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(skey + i) =
              make_uint4(role(i, f.x, sc4.x), role(i + 1, f.y, sc4.y), role(i + 2, f.z, sc4.z), role(i + 3, f.w, sc4.w));
        }
      } else {
#pragma unroll 16
        for (int i = tid; i < C; i += kKeepThreads) skey[i] = role(i, i < hist_end ? skey[i] : 0u, i < hist_end ? scores[i] : 0.f);
      }
      __syncthreads();
      emitted = block_topk_keyed<kKeepThreads>(
          C, k, [&](int i) { const uint32_t v = skey[i]; return v == kKeepAlways ? 0u : v; },
          [&](int i) { return skey[i] == kKeepAlways; }, [&](int pos, int i) { out[pos] = i; }, scratch);
    } else {
      emitted = block_topk_keyed<kKeepThreads>(
          C, k,
          [&](int i) {
            if (i >= hist_end) return 0u;
            const bool is_t = txt[i] != 0;
            return (is_t == rank_text) ? float_key(scores[i]) : 0u;
          },
          [&](int i) { return i >= hist_end || (!rank_text && txt[i] != 0); }, [&](int pos, int i) { out[pos] = i; },
          scratch);
    }
  }
  if (tid == 0) {
    reinterpret_cast<int32_t*>(cache + hdr->n_valid_off)[uid] = emitted;
    if (emitted != budget) {
      int32_t* err = reinterpret_cast<int32_t*>(cache + hdr->err_off);
      atomicCAS(&err[0], 0, HKV_ERR_INDEX);
      err[1] = kErrIndex;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same keep-set with one thread-block CLUSTER per static unit: the unit's tokens are cut into kSelCluster
// contiguous slices, one per CTA, so that no SM walks a whole 32 K-token sequence alone.  Four cluster barriers:
//   1. every CTA publishes its slice's statistics (text tokens before the window; smallest / largest score key
//      among the text and among the visual tokens) -> all know which class is ranked, k, and the key range;
//   2. local 1024-bin histograms of the ranked keys are complete -> every CTA adds up all eight (thread b reads
//      bin b of every peer through distributed shared memory) and finds the threshold bin on its own copy;
//   3. the threshold bin's items, (key, index), have been stored into every CTA's candidate list at slots that
//      follow from the peers' counts of that bin -> every CTA ranks them exactly and knows the threshold element;
//   4. the per-CTA numbers of selected tokens are known -> each CTA emits its ascending run at its offset.
// Units this path does not take (a threshold bin with more than 1024 items, which needs the radix selection)
// are left untouched: the single-CTA kernel, launched afterwards, does every unit whose count is still zero.
// ---------------------------------------------------------------------------------------------
constexpr int kSelCluster = 8;
struct __align__(16) SelStats { int n_text; uint32_t tmin, tmax, vmin, vmax; int pad[3]; };

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kKeepThreads)
    static_select_cluster_kernel(char* cache, const char* workspace, const float* token_scores, const uint8_t* is_text,
                                 int slice_slots) {
  __shared__ __align__(16) int hist[kKeyedBins];
  __shared__ __align__(16) uint2 cand[kKeepThreads];
  __shared__ SelStats stats[kSelCluster];
  __shared__ int counts[kSelCluster];
  __shared__ int cnt_by_rank[kSelCluster];
  __shared__ int ctl[8];
  __shared__ int wtot[32];
  extern __shared__ __align__(16) uint32_t skey[];          // slice_slots keys, then slice_slots text flags (bytes)
  uint8_t* stxt = reinterpret_cast<uint8_t*>(skey + slice_slots);

  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const uint32_t rank = cluster_ctarank();
  int uid;
  const Unit* u = unit_of(cache, hdr, false, blockIdx.x / kSelCluster, &uid);
  const int C = u->C, w = hdr->obs_window, budget = u->n_tok;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint8_t* txt = is_text + static_cast<size_t>(u->b) * hdr->max_seq_len;
  const float* scores = token_scores
                            ? token_scores + (static_cast<size_t>(u->b) * hdr->n_kv_heads + u->h) * hdr->max_seq_len
                            : reinterpret_cast<const float*>(workspace + u->ws_scores_off);
  int32_t* out = reinterpret_cast<int32_t*>(cache + u->idx_off);
  int32_t* n_valid = reinterpret_cast<int32_t*>(cache + hdr->n_valid_off) + uid;
  const int hist_end = C - w;
  const int per = (((C + kSelCluster - 1) / kSelCluster) + 3) & ~3;
  const int lo = min(C, static_cast<int>(rank) * per), hi = min(C, lo + per), n = hi - lo;

  if (budget <= w) {   // the last `budget` tokens, whatever their scores (uniform over the cluster)
    const int start = C - budget;
    for (int i = max(lo, start) + tid; i < hi; i += kKeepThreads) out[i - start] = i;
    if (rank == 0 && tid == 0) *n_valid = budget;
    return;
  }

  // ---- slice statistics ----
  for (int i = tid; i < kKeyedBins; i += kKeepThreads) hist[i] = 0;
  if (tid == 0) { ctl[0] = 0; ctl[1] = 0; ctl[4] = 0; ctl[5] = 0; }
  int nt = 0;
  uint32_t tmin = 0xFFFFFFFFu, tmax = 0u, vmin = 0xFFFFFFFFu, vmax = 0u;
  for (int i = lo + tid; i < hi; i += kKeepThreads) {
    const uint32_t kv = float_key(scores[i]);
    const bool is_t = txt[i] != 0;
    skey[i - lo] = kv;
    stxt[i - lo] = is_t;
    if (i < hist_end) {
      if (is_t) { ++nt; tmin = min(tmin, kv); tmax = max(tmax, kv); }
      else { vmin = min(vmin, kv); vmax = max(vmax, kv); }
    }
  }
  nt = __reduce_add_sync(0xffffffffu, nt);
  tmin = __reduce_min_sync(0xffffffffu, tmin); tmax = __reduce_max_sync(0xffffffffu, tmax);
  vmin = __reduce_min_sync(0xffffffffu, vmin); vmax = __reduce_max_sync(0xffffffffu, vmax);
  __shared__ SelStats mine;
  if (tid == 0) mine = SelStats{0, 0xFFFFFFFFu, 0u, 0xFFFFFFFFu, 0u, {0, 0, 0}};
  __syncthreads();
  if (lane == 0) {
    atomicAdd(&mine.n_text, nt);
    atomicMin(&mine.tmin, tmin); atomicMax(&mine.tmax, tmax);
    atomicMin(&mine.vmin, vmin); atomicMax(&mine.vmax, vmax);
  }
  __syncthreads();
  if (tid < kSelCluster) {   // my statistics into slot `rank` of every CTA
    const uint32_t dst = mapa(smem_u32(&stats[rank]), tid);
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(static_cast<uint32_t>(mine.n_text)),
                 "r"(mine.tmin), "r"(mine.tmax), "r"(mine.vmin)
                 : "memory");
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(dst + 16), "r"(mine.vmax) : "memory");
  }
  cluster_arrive(); cluster_wait();   // 1

  int n_text = 0;
  uint32_t kmin_t = 0xFFFFFFFFu, kmax_t = 0u, kmin_v = 0xFFFFFFFFu, kmax_v = 0u;
#pragma unroll
  for (int r = 0; r < kSelCluster; ++r) {
    n_text += stats[r].n_text;
    kmin_t = min(kmin_t, stats[r].tmin); kmax_t = max(kmax_t, stats[r].tmax);
    kmin_v = min(kmin_v, stats[r].vmin); kmax_v = max(kmax_v, stats[r].vmax);
  }
  const int room = budget - w;
  const bool rank_text = n_text >= room;       // window + text do not fit: rank the text tokens
  const int k = rank_text ? room : room - n_text;
  const uint32_t kmin = rank_text ? kmin_t : kmin_v, kmax = rank_text ? kmax_t : kmax_v;
  const int shift = max(0, 32 - __clz((kmax - kmin) | 1u) - 10);
  // roles of a token of my slice: ranked candidate / kept regardless / out
  auto is_cand = [&](int j) { return lo + j < hist_end && (stxt[j] != 0) == rank_text; };
  auto is_always = [&](int j) { return lo + j >= hist_end || (!rank_text && stxt[j] != 0); };

  uint32_t tkey = 0xFFFFFFFFu;   // nothing ranked is taken unless the selection below says so
  int tidx = -1;
  if (k > 0) {
    // ---- histograms ----
    for (int j = tid; j < n; j += kKeepThreads)
      if (is_cand(j)) atomicAdd(&hist[(skey[j] - kmin) >> shift], 1);
    __syncthreads();
    cluster_arrive(); cluster_wait();   // 2
    int hr[kSelCluster], mine_tot = 0;
    {
      const uint32_t a = smem_u32(&hist[tid]);
#pragma unroll
      for (int r = 0; r < kSelCluster; ++r) {
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(hr[r]) : "r"(mapa(a, r)) : "memory");
        mine_tot += hr[r];
      }
    }
    // the highest bin b with count(bins > b) < k <= count(bins >= b): thread t owns bin t
    {
      int run = mine_tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, run, off);
        if (lane + off < 32) run += v;
      }
      if (lane == 0) wtot[warp] = run;
      __syncthreads();
      const int wt = wtot[lane];
      int wrun = wt;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, wrun, off);
        if (lane + off < 32) wrun += v;
      }
      const int above = __shfl_sync(0xffffffffu, wrun - wt, warp) + run - mine_tot;
      if (above < k && k <= above + mine_tot) {
        ctl[1] = tid; ctl[2] = k - above; ctl[3] = mine_tot;
#pragma unroll
        for (int r = 0; r < kSelCluster; ++r) cnt_by_rank[r] = hr[r];
      }
      __syncthreads();
    }
    const int tbin = ctl[1], need = ctl[2], cnt = ctl[3];
    if (cnt > kKeepThreads) {   // too many near-equal scores for the direct ranking: leave the unit to the general kernel
      cluster_arrive(); cluster_wait();   // peers may still be reading my histogram
      return;
    }
    // ---- the threshold bin's items into every CTA's candidate list ----
    int base = 0;
    for (int r = 0; r < static_cast<int>(rank); ++r) base += cnt_by_rank[r];
    for (int j = tid; j < n; j += kKeepThreads) {
      if (is_cand(j) && static_cast<int>((skey[j] - kmin) >> shift) == tbin) {
        const int slot = base + atomicAdd(&ctl[0], 1);
        const uint32_t a = smem_u32(&cand[slot]);
#pragma unroll
        for (int r = 0; r < kSelCluster; ++r)
          asm volatile("st.shared::cluster.v2.u32 [%0], {%1, %2};" ::"r"(mapa(a, r)), "r"(skey[j]), "r"(static_cast<uint32_t>(lo + j))
                       : "memory");
      }
    }
    cluster_arrive(); cluster_wait();   // 3
    if (tid < cnt) {
      const uint2 me = cand[tid];
      int rk = 0;
      for (int j = 0; j < cnt; ++j) {
        const uint2 o = cand[j];
        rk += (o.x > me.x) || (o.x == me.x && o.y < me.y);
      }
      if (rk == need - 1) { ctl[4] = static_cast<int>(me.x); ctl[5] = static_cast<int>(me.y); }
    }
    __syncthreads();
    tkey = static_cast<uint32_t>(ctl[4]);
    tidx = ctl[5];
  }

  // ---- ordered emission: warp w owns a contiguous run of the slice ----
  auto taken = [&](int j) {
    if (is_always(j)) return true;
    if (!is_cand(j)) return false;
    const uint32_t kv = skey[j];
    return kv > tkey || (kv == tkey && lo + j <= tidx);
  };
  constexpr int kWarps = kKeepThreads / 32;
  const int wper = ((n + kWarps - 1) / kWarps + 31) & ~31;
  const int beg = min(n, warp * wper), end = min(n, beg + wper);
  int mine_n = 0;
  for (int j0 = beg; j0 < end; j0 += 32) {
    const int j = j0 + lane;
    mine_n += __popc(__ballot_sync(0xffffffffu, j < end && taken(j)));
  }
  __syncthreads();   // wtot is free again
  if (lane == 0) wtot[warp] = mine_n;
  __syncthreads();
  int before = 0, total = 0;
  {
    const int wt = wtot[lane];
    int incl = wt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += v;
    }
    before = __shfl_sync(0xffffffffu, incl - wt, warp);
    total = __shfl_sync(0xffffffffu, incl, 31);
  }
  if (tid < kSelCluster)
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa(smem_u32(&counts[rank]), tid)), "r"(total) : "memory");
  cluster_arrive(); cluster_wait();   // 4
  int off0 = 0, all = 0;
#pragma unroll
  for (int r = 0; r < kSelCluster; ++r) {
    if (r < static_cast<int>(rank)) off0 += counts[r];
    all += counts[r];
  }
  before += off0;
  const uint32_t below = (1u << lane) - 1u;
  for (int j0 = beg; j0 < end; j0 += 32) {
    const int j = j0 + lane;
    const bool sel = j < end && taken(j);
    const uint32_t b = __ballot_sync(0xffffffffu, sel);
    if (sel) out[before + __popc(b & below)] = lo + j;
    before += __popc(b);
  }
  if (rank == 0 && tid == 0) {
    *n_valid = all;
    if (all != budget) {
      int32_t* err = reinterpret_cast<int32_t*>(cache + hdr->err_off);
      atomicCAS(&err[0], 0, HKV_ERR_INDEX);
      err[1] = kErrIndex;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Row movers.  One half-warp per row: 16 lanes x 16 bytes; lanes 0-15 move the K row, 16-31 the V
// row.  Destination piece c of plane row i goes to position c ^ (i & 7).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    gather_rows_kernel(char* cache, const uint4* kin, const uint4* vin, int dynamic) {
  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, dynamic != 0, blockIdx.y, nullptr);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = lane & 15;
  const bool is_v = lane >= 16;
  const int rows = dynamic ? u->plane_rows : u->n_tok;   // (rows kept for appended tokens are written by the append kernel)
  const int32_t* idx = reinterpret_cast<const int32_t*>(cache + u->idx_off);
  const size_t plane_in = (static_cast<size_t>(u->b) * hdr->n_kv_heads + u->h) * static_cast<size_t>(hdr->max_seq_len);
  uint4* dst_plane = reinterpret_cast<uint4*>(cache + (is_v ? u->v_off : u->k_off));
  const uint4* src = is_v ? vin : kin;
  for (int rr = 0; rr < 8; ++rr) {
    const int i = blockIdx.x * 64 + warp * 8 + rr;
    if (i >= rows) break;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (dynamic) {
      if (i < u->C) val = src[(plane_in + i) * 16 + c];
    } else {
      val = src[(plane_in + idx[i]) * 16 + c];
    }
    dst_plane[static_cast<size_t>(i) * 16 + (c ^ (i & 7))] = val;
  }
}

// Chunk means: half a warp per chunk, lane = eight channels (one 16-byte piece of a key row); every
// channel keeps its own float32 running sum over the chunk's tokens IN ORDER, then a float32 division
// by the chunk's own length and round-to-nearest-even to bf16 — the arithmetic the method's metadata
// is defined with, so the result is bit-exact whatever the launch shape.  Rows of consecutive tokens
// are independent loads, so four are kept in flight.
constexpr int kMeanWarps = 8;
__global__ void __launch_bounds__(kMeanWarps * 32) chunk_means_kernel(char* cache, const uint4* kin) {
  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, true, blockIdx.y, nullptr);
  const int cs = hdr->chunk_size, C = u->C;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, sub = lane & 15;
  const int c = (blockIdx.x * kMeanWarps + warp) * 2 + (lane >> 4);
  if (c >= u->n_chunks) return;
  const uint4* kp = kin + (static_cast<size_t>(u->b) * hdr->n_kv_heads + u->h) * static_cast<size_t>(hdr->max_seq_len) * 16;
  const int t0 = c * cs, t1 = min(t0 + cs, C);
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.f;
  auto add_row = [&](const uint4& r) {
    acc[0] = __fadd_rn(acc[0], bf16_lo(r.x)); acc[1] = __fadd_rn(acc[1], bf16_hi(r.x));
    acc[2] = __fadd_rn(acc[2], bf16_lo(r.y)); acc[3] = __fadd_rn(acc[3], bf16_hi(r.y));
    acc[4] = __fadd_rn(acc[4], bf16_lo(r.z)); acc[5] = __fadd_rn(acc[5], bf16_hi(r.z));
    acc[6] = __fadd_rn(acc[6], bf16_lo(r.w)); acc[7] = __fadd_rn(acc[7], bf16_hi(r.w));
  };
  int tk = t0;
  for (; tk + 4 <= t1; tk += 4) {
    const uint4 r0 = kp[static_cast<size_t>(tk) * 16 + sub], r1 = kp[static_cast<size_t>(tk + 1) * 16 + sub];
    const uint4 r2 = kp[static_cast<size_t>(tk + 2) * 16 + sub], r3 = kp[static_cast<size_t>(tk + 3) * 16 + sub];
    add_row(r0); add_row(r1); add_row(r2); add_row(r3);
  }
  for (; tk < t1; ++tk) add_row(kp[static_cast<size_t>(tk) * 16 + sub]);
  const float len = static_cast<float>(t1 - t0);
  uint4 o;
  o.x = pack_bf16(__fdiv_rn(acc[0], len), __fdiv_rn(acc[1], len));
  o.y = pack_bf16(__fdiv_rn(acc[2], len), __fdiv_rn(acc[3], len));
  o.z = pack_bf16(__fdiv_rn(acc[4], len), __fdiv_rn(acc[5], len));
  o.w = pack_bf16(__fdiv_rn(acc[6], len), __fdiv_rn(acc[7], len));
  // 16-byte piece p of chunk c is stored at position p ^ (c & 7), like K/V rows
  reinterpret_cast<uint4*>(cache + u->summ_off)[static_cast<size_t>(c) * 16 + (sub ^ (c & 7))] = o;
  if (c == u->n_chunks - 1) {
    // running sum of the open last chunk, continued by appended tokens (a full chunk leaves nothing open)
    float* tail = reinterpret_cast<float*>(cache + u->tail_sum_off) + sub * 8;
    const bool open = (t1 - t0) < cs;
#pragma unroll
    for (int j = 0; j < 8; ++j) tail[j] = open ? acc[j] : 0.f;
  }
}

// Adds one token to every unit: the key / value rows go to the end of the unit's planes (static: the
// condensed cache, position recorded in the kept list; dynamic: row C of the chunk-major store), a
// dynamic unit's open chunk gets its running sum and mean updated (or a new chunk is opened), and the
// unit's record is advanced.  One CTA of 128 threads per unit; thread = channel.
__global__ void __launch_bounds__(kHeadDim)
    append_kernel(char* cache, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new) {
  const Header* hdr = reinterpret_cast<const Header*>(cache);
  Unit* u = reinterpret_cast<Unit*>(cache + kUnitsOff) + blockIdx.x;
  const int d = threadIdx.x, cs = hdr->chunk_size;
  const int C = u->C;
  const bool dynamic = u->type != 0;
  const int row = dynamic ? C : u->n_tok;
  if (row >= u->plane_rows) {   // no room left (the host refuses this before launching)
    if (d == 0) {
      int32_t* err = reinterpret_cast<int32_t*>(cache + hdr->err_off);
      if (atomicCAS(&err[0], 0, HKV_ERR_INDEX) == 0) err[1] = kErrIndex;
    }
    return;
  }
  const size_t in = (static_cast<size_t>(u->b) * hdr->n_kv_heads + u->h) * kHeadDim + d;
  const __nv_bfloat16 kv = k_new[in], vv = v_new[in];
  const size_t out = static_cast<size_t>(row) * kHeadDim + ((((d >> 3) ^ (row & 7)) << 3) | (d & 7));
  reinterpret_cast<__nv_bfloat16*>(cache + u->k_off)[out] = kv;
  reinterpret_cast<__nv_bfloat16*>(cache + u->v_off)[out] = vv;
  int n_chunks = u->n_chunks;
  if (dynamic) {
    const int c = C / cs;                       // chunk the new token falls into
    const int len = C - c * cs + 1;
    float* tail = reinterpret_cast<float*>(cache + u->tail_sum_off);
    const float sum = __fadd_rn(len == 1 ? 0.f : tail[d], __bfloat162float(kv));
    tail[d] = (len == cs) ? 0.f : sum;          // a chunk that just filled up leaves nothing open
    reinterpret_cast<__nv_bfloat16*>(cache + u->summ_off)[static_cast<size_t>(c) * kHeadDim + ((((d >> 3) ^ (c & 7)) << 3) | (d & 7))] =
        __float2bfloat16_rn(__fdiv_rn(sum, static_cast<float>(len)));
    n_chunks = c + 1;
  }
  __syncthreads();   // every thread has read the record
  if (d == 0) {
    u->C = C + 1;
    if (dynamic) {
      u->n_chunks = n_chunks;
      const int k_sel = min(n_chunks, (min(u->budget_raw, C + 1) + cs - 1) / cs);
      u->k_sel = k_sel;
      u->n_tok = k_sel * cs;
    } else {
      reinterpret_cast<int32_t*>(cache + u->idx_off)[u->n_tok] = C;   // position of the new token
      u->n_tok = u->n_tok + 1;
    }
  }
}

}  // namespace

cudaError_t launch_window_scores(char* cache, char* workspace, const void* k, const void* q_obs, const Header& hdr,
                                 const std::vector<Unit>&, int64_t ws_rowstat_off, int n_col_tiles_max,
                                 cudaStream_t stream) {
  if (hdr.n_static == 0) return cudaSuccess;
  const int R = hdr.obs_window * hdr.group;
  const int Rpad = (R + 15) / 16 * 16;
  float2* stats = reinterpret_cast<float2*>(workspace + ws_rowstat_off);
  float2* fin = stats + static_cast<size_t>(hdr.n_static) * n_col_tiles_max * Rpad;
  int dev = 0, n_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(window_scores_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(window_scores_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
  if (e != cudaSuccess) return e;
  // key ranges sized so that one launch is at most one wave of CTAs; n_col_tiles_max counts 64-key tiles
  const int n_tiles = (n_col_tiles_max + 1) / 2;
  const int splits = std::max(1, std::min(n_tiles, n_sm / hdr.n_static));
  const int tiles_per_cta = (n_tiles + splits - 1) / splits;
  const int n_ranges = (n_tiles + tiles_per_cta - 1) / tiles_per_cta;
  const int n_row_blocks = (R + tc::kQRows - 1) / tc::kQRows;
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q_obs);
  const dim3 grid(n_ranges, hdr.n_static);
  for (int rb = 0; rb < n_row_blocks; ++rb)
    window_scores_tc_kernel<0><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(cache, workspace, kb, qb, stats, fin,
                                                                              n_col_tiles_max, Rpad, tiles_per_cta, rb);
  window_rowreduce_kernel<<<dim3((R + kRowReduceWarps - 1) / kRowReduceWarps, hdr.n_static), kRowReduceWarps * 32, 0,
                            stream>>>(cache, stats, fin, n_col_tiles_max, Rpad, tiles_per_cta);
  for (int rb = 0; rb < n_row_blocks; ++rb)
    window_scores_tc_kernel<1><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(cache, workspace, kb, qb, stats, fin,
                                                                              n_col_tiles_max, Rpad, tiles_per_cta, rb);
  return cudaGetLastError();
}

cudaError_t launch_static_select(char* cache, char* workspace, const float* token_scores, const uint8_t* is_text,
                                 const Header& hdr, cudaStream_t stream) {
  if (hdr.n_static == 0) return cudaSuccess;
  // A cluster of kSelCluster CTAs per unit when a slice of the longest sequence (keys + text flags) fits one
  // CTA's shared memory; the single-CTA kernel follows for the units the cluster kernel leaves (crowded threshold
  // bin) and does everything for longer sequences.
  const int slice = ((hdr.max_seq_len + kSelCluster - 1) / kSelCluster + 3) & ~3;
  const size_t slice_smem = static_cast<size_t>(slice) * 5 + 16;
  const bool clustered = slice_smem <= 160 * 1024;
  if (clustered) {
    cudaError_t e = cudaFuncSetAttribute(static_select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(slice_smem));
    if (e != cudaSuccess) return e;
    static_select_cluster_kernel<<<hdr.n_static * kSelCluster, kKeepThreads, slice_smem, stream>>>(
        cache, workspace, token_scores, is_text, slice);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  // every token's role is kept in shared memory when the longest sequence fits (else it is recomputed per pass)
  const int key_slots = std::min(hdr.max_seq_len, 49152);
  const size_t smem = static_cast<size_t>(key_slots) * sizeof(uint32_t);
  cudaError_t e =
      cudaFuncSetAttribute(static_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  static_select_kernel<<<hdr.n_static, kKeepThreads, smem, stream>>>(cache, workspace, token_scores, is_text,
                                                                     key_slots, clustered ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_gather_static(char* cache, const void* k, const void* v, const Header& hdr, int max_rows,
                                 cudaStream_t stream) {
  if (hdr.n_static == 0 || max_rows <= 0) return cudaSuccess;
  dim3 grid((max_rows + 63) / 64, hdr.n_static);
  gather_rows_kernel<<<grid, 256, 0, stream>>>(cache, static_cast<const uint4*>(k), static_cast<const uint4*>(v), 0);
  return cudaGetLastError();
}

cudaError_t launch_build_dynamic(char* cache, const void* k, const void* v, const Header& hdr, int max_rows,
                                 int max_chunks, cudaStream_t stream) {
  if (hdr.n_dynamic == 0) return cudaSuccess;
  dim3 grid((max_rows + 63) / 64, hdr.n_dynamic);
  gather_rows_kernel<<<grid, 256, 0, stream>>>(cache, static_cast<const uint4*>(k), static_cast<const uint4*>(v), 1);
  dim3 grid2((max_chunks + kMeanWarps * 2 - 1) / (kMeanWarps * 2), hdr.n_dynamic);
  chunk_means_kernel<<<grid2, kMeanWarps * 32, 0, stream>>>(cache, static_cast<const uint4*>(k));
  return cudaGetLastError();
}

cudaError_t launch_append(char* cache, const void* k_new, const void* v_new, const Header& hdr, cudaStream_t stream) {
  append_kernel<<<hdr.n_units, kHeadDim, 0, stream>>>(cache, static_cast<const __nv_bfloat16*>(k_new),
                                                      static_cast<const __nv_bfloat16*>(v_new));
  return cudaGetLastError();
}

}  // namespace hkv
