// Internal layout shared by the host planner and the kernels of libhkv.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "hkv.h"

namespace hkv {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;   // one bf16 K or V row (or one chunk mean)
constexpr int kTile = 32;                 // tokens a warp stages and consumes at a time
constexpr int kMaxGroup = 16;             // query heads per kv head the mma tiles can hold
constexpr int kMaxMulti = 32;             // caches one hkv_decode_attn_multi launch can take
constexpr int kAlign = 256;
constexpr int kMaxCluster = 16;           // CTAs that may share one (sequence, kv head) unit

// decode kernel launch shape
constexpr int kDecStages = 6;             // staging ring of a CTA (tiles in flight); two CTAs fit one SM
constexpr int kStageBytes = kTile * kRowBytes * 2 + 256;   // K tile + V tile + row keys; a multiple of the row size, so that every staged row starts on a 256-byte boundary
constexpr int kScoreTile = 2 * kTile;     // most chunk means one stage holds while chunks are scored
constexpr int kSelSmemChunks = 2048;      // chunk scores / selected ids a CTA keeps in shared memory

// One (sequence b, kv head h) pair of a layer; unit id = b * n_kv_heads + h.
struct Unit {
  int32_t type;        // 0 static, 1 dynamic
  int32_t b, h;
  int32_t C;           // tokens of the sequence
  int32_t budget;      // tokens, clamped to C
  int32_t n_tok;       // static: kept tokens; dynamic: k_sel * cs (upper bound of attended tokens)
  int32_t n_chunks;    // dynamic: ceil(C / cs)
  int32_t k_sel;       // dynamic: chunks loaded per step
  int32_t plane_rows;  // rows of the K (and V) plane held in the cache (capacity, including room for appended tokens)
  int32_t budget_raw;  // the caller's budget before clamping to the sequence length
  int32_t cap_chunks;  // dynamic: chunk means / scores the cache has room for
  int32_t cap_sel;     // entries the index list has room for
  int64_t k_off, v_off;    // byte offsets (from the cache base) of the K / V planes
  int64_t summ_off;        // dynamic: bf16 chunk means [n_chunks, d], 16-byte pieces permuted like K/V rows
  int64_t idx_off;         // static: int32 kept positions [n_tok]; dynamic: int32 chunk ids [k_sel]
  int64_t scores_off;      // dynamic: float32 chunk scores [n_chunks] (decode scratch)
  int64_t ws_scores_off;   // static: float32 s_w [C] inside the compress workspace
  int64_t tail_sum_off;    // dynamic: float32 [d] running key sum of the open last chunk (zero when it is full)
};
static_assert(sizeof(Unit) == 104, "Unit layout");

// Device-side table of contents, at offset 0 of cache_mem.  Unit[n_units] follows at kUnitsOff.
struct Header {
  int32_t n_units, n_static, n_dynamic, pad1;
  int32_t batch, n_q_heads, n_kv_heads, group;
  int32_t chunk_size, obs_window, max_seq_len;
  uint32_t flags;
  float scale;
  int32_t pad[3];
  int64_t dyn_list_off;  // int32[n_dynamic] unit ids of dynamic units
  int64_t sta_list_off;  // int32[n_static]
  int64_t n_valid_off;   // int32[n_units] attended tokens (dynamic: written by every selection)
  int64_t err_off;       // int32[2] device error word: code, detail
};
constexpr int64_t kUnitsOff = 256;
static_assert(sizeof(Header) <= kUnitsOff, "Header layout");

// Arguments of the decode kernel: up to kMaxMulti caches side by side.  A cluster of `cluster`
// CTAs works on one unit; clusters [unit_prefix[i], unit_prefix[i+1]) belong to cache i.
enum DecodePhase : uint32_t { kPhaseSelect = 1u, kPhaseAttend = 2u };
struct DecodeParams {
  int32_t n;
  int32_t cluster;
  int32_t group, n_q_heads, n_kv_heads, chunk_size;
  float scale_log2e;
  uint32_t phase;      // kPhaseSelect | kPhaseAttend
  uint32_t out_f32;
  uint32_t pdl;        // launched with programmatic stream serialization
  uint32_t group_max;  // chunk score = max over the group's heads instead of their sum
  uint32_t offload;    // the dynamic units' K/V planes live in host memory: no L2 prefetch requests for them
  int32_t unit_prefix[kMaxMulti + 1];
  char* cache[kMaxMulti];
  const void* q[kMaxMulti];
  void* out[kMaxMulti];
  int64_t n_valid_off[kMaxMulti];
  int64_t err_off[kMaxMulti];
  int64_t dyn_list_off[kMaxMulti];   // unit ids of each cache's dynamic / static units: a cache's clusters take one
  int64_t sta_list_off[kMaxMulti];   // type first, then the other (static_first)
  int32_t n_dynamic[kMaxMulti];
  uint32_t static_first;
#ifdef HKV_PROFILE
  unsigned long long* prof;   // kProfSlots time stamps (ns) per CTA, or null
#endif
};
constexpr int kProfSlots = 32;

// device error word helpers
enum ErrPlace : int32_t { kErrDecodeWait = 1, kErrIndex = 2, kErrScoreWait = 3, kErrExchangeWait = 4, kErrMergeWait = 5, kErrSelfTest = 6 };

// Upper bound on resident CTAs per SM the decode kernel is built for.
constexpr int kDecCtasPerSm = 2;

// ---- kernel launchers (definitions in the .cu files) ----
// Picks the cluster size for `total_units` units whose longest token list has `max_tiles` tiles;
// max_active[c] = clusters of c CTAs the device holds at once (index 1 .. kMaxCluster).
int choose_cluster(int total_units, int max_tiles, const int* max_active);
// Cluster capacities of the decode kernel for this group size (also performs the kernel's one-time
// set-up; call before the first launch_decode).
cudaError_t decode_cluster_caps(int group, const int** max_active);
cudaError_t launch_decode(const DecodeParams& params, int total_units, cudaStream_t stream);
cudaError_t launch_window_scores(char* cache, char* workspace, const void* k, const void* q_obs,
                                 const Header& hdr, const std::vector<Unit>& units, int64_t ws_rowstat_off,
                                 int n_col_tiles_max, cudaStream_t stream);
cudaError_t launch_static_select(char* cache, char* workspace, const float* token_scores,
                                 const uint8_t* is_text, const Header& hdr, cudaStream_t stream);
cudaError_t launch_gather_static(char* cache, const void* k, const void* v, const Header& hdr,
                                 int max_rows, cudaStream_t stream);
cudaError_t launch_build_dynamic(char* cache, const void* k, const void* v, const Header& hdr,
                                 int max_rows, int max_chunks, cudaStream_t stream);
cudaError_t launch_append(char* cache, const void* k_new, const void* v_new, const Header& hdr, cudaStream_t stream);
size_t decode_smem_bytes();
#ifdef HKV_CHECKED
cudaError_t launch_selftest_wait(int32_t* err_word, cudaStream_t stream);
#endif

}  // namespace hkv

struct hkv_cache {
  hkv_config cfg;
  hkv::Header hdr;
  std::vector<hkv::Unit> units;
  char* dev_base;
  size_t cache_bytes, workspace_bytes, host_bytes;
  int64_t kv_bytes, summary_bytes, algo_bytes, retained;
  int max_static_rows, max_dyn_rows, max_chunks, max_tiles;
  bool fresh;   // no decode launch has followed the last compression / append yet
  int appended; // tokens added by hkv_append so far
};
