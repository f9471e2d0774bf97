// Internal layout shared by the host planner and the kernels of libhkv.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "hkv.h"

namespace hkv {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;   // one bf16 K or V row
constexpr int kTile = 32;                 // tokens a warp stages and consumes at a time
constexpr int kMaxGroup = 16;             // query heads per kv head the mma tile can hold
constexpr int kMaxMulti = 32;             // caches one hkv_decode_attn_multi launch can take
constexpr int kAlign = 256;

// flash-decode launch shape
constexpr int kDecWarps = 4;              // warps per CTA, each with its own staging ring
constexpr int kDecStages = 3;             // ring depth per warp (tiles in flight)
constexpr int kStageBytes = kTile * kRowBytes * 2 + 128;   // K tile + V tile + row keys

// One (sequence b, kv head h) pair of a layer.
struct Unit {
  int32_t type;        // 0 static, 1 dynamic
  int32_t b, h;
  int32_t C;           // tokens of the sequence
  int32_t budget;      // tokens, clamped to C
  int32_t n_tok;       // static: kept tokens; dynamic: k_sel * cs (upper bound of attended tokens)
  int32_t n_chunks;    // dynamic: ceil(C / cs)
  int32_t k_sel;       // dynamic: chunks loaded per step
  int32_t n_splits;    // CTAs of the flash-decode launch working on this unit
  int32_t split_base;  // first partial slot of this unit
  int32_t plane_rows;  // rows of the K (and V) plane held in the cache
  int32_t pad0;
  int64_t k_off, v_off;    // byte offsets (from the cache base) of the K / V planes
  int64_t summ_off;        // dynamic: bf16 chunk means [n_chunks, d]
  int64_t idx_off;         // static: int32 kept positions [n_tok]; dynamic: int32 chunk ids [k_sel]
  int64_t scores_off;      // dynamic: float32 chunk scores [n_chunks] (decode scratch)
  int64_t ws_scores_off;   // static: float32 s_w [C] inside the compress workspace
};

// One CTA of the flash-decode launch: tiles [tile_begin, tile_end) of a unit's token list.
struct Split {
  int32_t unit;
  int32_t tile_begin, tile_end;
  int32_t slot;        // index of this split among the unit's splits
};

// Device-side table of contents, at offset 0 of cache_mem.
struct Header {
  int32_t n_units, n_static, n_dynamic, n_splits;
  int32_t batch, n_q_heads, n_kv_heads, group;
  int32_t chunk_size, obs_window, max_seq_len;
  uint32_t flags;
  float scale;
  int32_t pad[3];
  int64_t units_off;     // Unit[n_units]
  int64_t splits_off;    // Split[n_splits]
  int64_t dyn_list_off;  // int32[n_dynamic] unit ids of dynamic units
  int64_t sta_list_off;  // int32[n_static]
  int64_t counters_off;  // int32[n_units] arrival counters of the split merge (zero between calls)
  int64_t n_valid_off;   // int32[n_units] attended tokens (dynamic: written by every selection)
  int64_t err_off;       // int32[2] device error word: code, detail
  int64_t partials_off;  // float32 [n_splits_total][group][d + 2]
};

// Arguments of the decode kernels: up to kMaxMulti caches side by side.
struct DecodeBatch {
  int32_t n;
  int32_t split_prefix[kMaxMulti + 1];   // CTA ranges of the flash-decode grid
  int32_t dyn_prefix[kMaxMulti + 1];     // CTA ranges of the selection grid
  char* cache[kMaxMulti];
  const void* q[kMaxMulti];
  void* out[kMaxMulti];
};

// device error word helpers
enum ErrPlace : int32_t { kErrDecodeWait = 1, kErrIndex = 2 };

// ---- kernel launchers (definitions in the .cu files) ----
cudaError_t launch_select_chunks(const DecodeBatch& batch, int total_dyn, cudaStream_t stream);
cudaError_t launch_flash_decode(const DecodeBatch& batch, int total_splits, int group, bool out_f32,
                                cudaStream_t stream);
cudaError_t launch_window_scores(char* cache, char* workspace, const void* k, const void* q_obs,
                                 const Header& hdr, const std::vector<Unit>& units, int64_t ws_rowstat_off,
                                 int n_col_tiles_max, cudaStream_t stream);
cudaError_t launch_static_select(char* cache, char* workspace, const float* token_scores,
                                 const uint8_t* is_text, const Header& hdr, cudaStream_t stream);
cudaError_t launch_gather_static(char* cache, const void* k, const void* v, const Header& hdr,
                                 int max_rows, cudaStream_t stream);
cudaError_t launch_build_dynamic(char* cache, const void* k, const void* v, const Header& hdr,
                                 int max_rows, int max_chunks, cudaStream_t stream);
size_t flash_decode_smem_bytes();

}  // namespace hkv

struct hkv_cache {
  hkv_config cfg;
  hkv::Header hdr;
  std::vector<hkv::Unit> units;
  std::vector<hkv::Split> splits;
  char* dev_base;
  size_t cache_bytes, workspace_bytes;
  int64_t kv_bytes, summary_bytes, algo_bytes, retained;
  int max_static_rows, max_dyn_rows, max_chunks;
};
