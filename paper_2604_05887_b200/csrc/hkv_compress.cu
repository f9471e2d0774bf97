// Compression kernels (run once per prompt and layer): observation-window scores s_w for static
// heads, the text-prior keep-set, the gather into the compacted static cache, and for dynamic heads
// the chunk means plus the copy of K/V into the cache.  K/V rows are written with their sixteen
// 16-byte pieces XOR-permuted by (row & 7), the layout the flash-decode kernel stages with plain
// bulk copies and reads with bank-conflict-free ldmatrix.
#include "hkv_device.cuh"
#include "hkv_internal.h"

namespace hkv {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kWsTile = 64;      // key columns per CTA of the window-score kernels
constexpr int kWsWarps = 8;

__device__ __forceinline__ const Unit* unit_of(const char* cache, const Header* hdr, bool dynamic, int ordinal,
                                               int* uid_out) {
  const int32_t* list = reinterpret_cast<const int32_t*>(cache + (dynamic ? hdr->dyn_list_off : hdr->sta_list_off));
  const int uid = list[ordinal];
  if (uid_out) *uid_out = uid;
  return reinterpret_cast<const Unit*>(cache + kUnitsOff) + uid;
}

// ---------------------------------------------------------------------------------------------
// Window scores.  S_w = softmax over ALL tokens of the w*G window rows' logits, s_w = mean of rows.
// MODE 0: per (row, column tile) running max and exp-sum.  MODE 1: with the rows' final (max, sum)
// known, column sums of the normalised probabilities -> s_w.
// One CTA = one 64-token column tile of one static unit; warps loop over 16-row tiles of the
// R = w*G rows; logits on tensor cores.
// stats: float2 [n_static][n_tiles_max][Rpad], final: float2 [n_static][Rpad]
// ---------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(kWsWarps * 32)
    window_scores_kernel(const char* cache, char* workspace, const __nv_bfloat16* kin, const __nv_bfloat16* q_obs,
                         float2* stats, const float2* final_stats, int n_tiles_max, int Rpad) {
  __shared__ __align__(128) uint8_t ktile[kWsTile * kRowBytes];
  __shared__ float colsum[kWsWarps][kWsTile];

  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, false, blockIdx.y, nullptr);
  const int C = u->C, j0 = blockIdx.x * kWsTile;
  if (j0 >= C) return;
  const int G = hdr->group, w = hdr->obs_window, Hq = hdr->n_q_heads, Hkv = hdr->n_kv_heads;
  const int R = w * G;
  const bool causal = (hdr->flags & HKV_CAUSAL_WINDOW) != 0;
  const float sc = hdr->scale * kLog2e;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;

  // stage the key tile (rows past C are zero), 16-byte pieces permuted by row & 7
  const uint4* ksrc = reinterpret_cast<const uint4*>(
      kin + (static_cast<size_t>(u->b) * Hkv + u->h) * static_cast<size_t>(hdr->max_seq_len) * kHeadDim);
  for (int idx = tid; idx < kWsTile * 16; idx += kWsWarps * 32) {
    const int row = idx >> 4, c = idx & 15;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (j0 + row < C) v = ksrc[static_cast<size_t>(j0 + row) * 16 + c];
    *reinterpret_cast<uint4*>(ktile + row * kRowBytes + ((c ^ (row & 7)) << 4)) = v;
  }
  __syncthreads();

  const uint32_t kbase = smem_u32(ktile);
  const int mj = lane >> 3, mi = lane & 7;
  const int krow = mi + ((mj >> 1) << 3), kcsel = mj & 1;
  float cacc[8][2];
#pragma unroll
  for (int n = 0; n < 8; ++n) cacc[n][0] = cacc[n][1] = 0.f;

  const int n_mt = (R + 15) / 16;
  for (int mt = warp; mt < n_mt; mt += kWsWarps) {
    const int r0 = mt * 16 + g, r1 = r0 + 8;
    const int i0 = r0 / G, i1 = r1 / G;   // window row index of each mma row
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(
        q_obs + ((static_cast<size_t>(u->b) * w + i0) * Hq + u->h * G + (r0 - i0 * G)) * kHeadDim);
    const uint32_t* q1 = reinterpret_cast<const uint32_t*>(
        q_obs + ((static_cast<size_t>(u->b) * w + i1) * Hq + u->h * G + (r1 - i1 * G)) * kHeadDim);
    uint32_t qa[8][4];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      qa[kk][0] = (r0 < R) ? q0[kk * 8 + t] : 0u;
      qa[kk][2] = (r0 < R) ? q0[kk * 8 + 4 + t] : 0u;
      qa[kk][1] = (r1 < R) ? q1[kk * 8 + t] : 0u;
      qa[kk][3] = (r1 < R) ? q1[kk * 8 + 4 + t] : 0u;
    }
    float s[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
    for (int sl = 0; sl < 4; ++sl) {
      const int r = sl * 16 + krow;
      const uint32_t rowaddr = kbase + r * kRowBytes;
      const uint32_t key = r & 7;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(b0, b1, b2, b3, rowaddr + (((2 * kk + kcsel) ^ key) << 4));
        mma_bf16(s[2 * sl], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
        mma_bf16(s[2 * sl + 1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b2, b3);
      }
    }
    // scale (base-2 logits) and mask: columns past C, and keys after the row's own position if causal
    const int lim0 = causal ? (C - w + i0) : (C - 1), lim1 = causal ? (C - w + i1) : (C - 1);
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int j = j0 + n * 8 + 2 * t + e;
        s[n][e] = (j < C && j <= lim0) ? s[n][e] * sc : -INFINITY;
        s[n][2 + e] = (j < C && j <= lim1) ? s[n][2 + e] * sc : -INFINITY;
      }
    }
    if (MODE == 0) {
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
        mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      float z0 = 0.f, z1 = 0.f;
      if (mx0 > -INFINITY) {
#pragma unroll
        for (int n = 0; n < 8; ++n) z0 += exp2f(s[n][0] - mx0) + exp2f(s[n][1] - mx0);
      }
      if (mx1 > -INFINITY) {
#pragma unroll
        for (int n = 0; n < 8; ++n) z1 += exp2f(s[n][2] - mx1) + exp2f(s[n][3] - mx1);
      }
      z0 += __shfl_xor_sync(0xffffffffu, z0, 1);
      z0 += __shfl_xor_sync(0xffffffffu, z0, 2);
      z1 += __shfl_xor_sync(0xffffffffu, z1, 1);
      z1 += __shfl_xor_sync(0xffffffffu, z1, 2);
      if (t == 0) {
        float2* dst = stats + (static_cast<size_t>(blockIdx.y) * n_tiles_max + blockIdx.x) * Rpad;
        if (r0 < R) dst[r0] = make_float2(mx0, z0);
        if (r1 < R) dst[r1] = make_float2(mx1, z1);
      }
    } else {
      const float2* fin = final_stats + static_cast<size_t>(blockIdx.y) * Rpad;
      const float2 f0 = (r0 < R) ? fin[r0] : make_float2(0.f, 1.f);
      const float2 f1 = (r1 < R) ? fin[r1] : make_float2(0.f, 1.f);
      const float inv0 = (r0 < R) ? 1.f / f0.y : 0.f, inv1 = (r1 < R) ? 1.f / f1.y : 0.f;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int e = 0; e < 2; ++e)
          cacc[n][e] += exp2f(s[n][e] - f0.x) * inv0 + exp2f(s[n][2 + e] - f1.x) * inv1;
      }
    }
  }
  if (MODE == 1) {
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float v = cacc[n][e];
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (g == 0) colsum[warp][n * 8 + 2 * t + e] = v;
      }
    }
    __syncthreads();
    if (tid < kWsTile && j0 + tid < C) {
      float tot = 0.f;
#pragma unroll
      for (int w2 = 0; w2 < kWsWarps; ++w2) tot += colsum[w2][tid];
      float* sw = reinterpret_cast<float*>(workspace + u->ws_scores_off);
      sw[j0 + tid] = tot / static_cast<float>(R);
    }
  }
}

// Combines the per-tile (max, sum) of every window row into the row's final (max, sum): one warp per
// row, lanes stride the column tiles.
constexpr int kRowReduceWarps = 8;
__global__ void __launch_bounds__(kRowReduceWarps * 32)
    window_rowreduce_kernel(const char* cache, const float2* stats, float2* final_stats, int n_tiles_max, int Rpad) {
  const Header* hdr = reinterpret_cast<const Header*>(cache);
  const Unit* u = unit_of(cache, hdr, false, blockIdx.y, nullptr);
  const int R = hdr->obs_window * hdr->group;
  const int n_tiles = (u->C + kWsTile - 1) / kWsTile;
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
// ---------------------------------------------------------------------------------------------
constexpr int kKeepThreads = 1024;
constexpr int kKeepScratchInts = keyed_scratch_ints(kKeepThreads);

__global__ void __launch_bounds__(kKeepThreads)
    static_select_kernel(char* cache, const char* workspace, const float* token_scores, const uint8_t* is_text) {
  __shared__ __align__(16) int scratch[kKeepScratchInts];
  __shared__ int s_ntext;

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

  if (tid == 0) s_ntext = 0;
  __syncthreads();
  int cnt = 0;
  for (int i = tid; i < hist_end; i += kKeepThreads) cnt += txt[i] != 0;
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
  dim3 grid(n_col_tiles_max, hdr.n_static);
  window_scores_kernel<0><<<grid, kWsWarps * 32, 0, stream>>>(
      cache, workspace, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(q_obs), stats, fin,
      n_col_tiles_max, Rpad);
  window_rowreduce_kernel<<<dim3((R + kRowReduceWarps - 1) / kRowReduceWarps, hdr.n_static), kRowReduceWarps * 32, 0, stream>>>(
      cache, stats, fin, n_col_tiles_max, Rpad);
  window_scores_kernel<1><<<grid, kWsWarps * 32, 0, stream>>>(
      cache, workspace, static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(q_obs), stats, fin,
      n_col_tiles_max, Rpad);
  return cudaGetLastError();
}

cudaError_t launch_static_select(char* cache, char* workspace, const float* token_scores, const uint8_t* is_text,
                                 const Header& hdr, cudaStream_t stream) {
  if (hdr.n_static == 0) return cudaSuccess;
  static_select_kernel<<<hdr.n_static, kKeepThreads, 0, stream>>>(cache, workspace, token_scores, is_text);
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
