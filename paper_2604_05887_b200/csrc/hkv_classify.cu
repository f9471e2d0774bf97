// Text-centric head classification (paper Section 3.1): for every (sequence, kv head) the rows of
// S_text = softmax(Q_text K^T / sqrt(d)) over the whole context, the sum of each row's k largest
// entries, their mean over the rows (the text-centric sparsity score) and the comparison with the
// threshold theta.  Runs once per prompt and layer, before the budgets and the compression.
//
// Three kernels per pass over a block of rows:
//   cls_logits_tc_kernel  base-2 logits of 256 rows x a range of 128-key tiles, tcgen05 tensor cores,
//                      float32 into the workspace (rows padded to a multiple of 128 floats);
//   cls_row_kernel     one CTA per row: the row in shared memory, max, p = 2^(l - max), normaliser,
//                      the exact k-th largest p (histogram over the float bits, then exact ranking
//                      of the threshold bin), the sum of the entries above it plus the tied share
//                      (cls_row_regs_kernel when no row of the group is longer than 32768 entries:
//                      the row in registers, the next row's copy in flight meanwhile);
//   cls_finish_kernel  (after the last pass) mean of the rows' sums in double, fixed order, and
//                      the label.
#include <algorithm>
#include <cmath>

#include "hkv_device.cuh"
#include "hkv_internal.h"
#include "hkv_tc.cuh"

namespace hkv {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kClsBatch = 64;          // sequences one group of launches takes
constexpr int kClsRowThreads = 1024;
constexpr int kClsSmemCols = 49152;    // longest row the row kernel keeps in shared memory
constexpr int kClsRank = 256;          // largest threshold bin that is sorted directly
constexpr int kClsBins = 4096;          // bits 30..18 of a float in [0, 1]: 32 bins per octave
constexpr int kClsShift = 18;
constexpr int kClsLoadParts = 4;       // pieces a row arrives in, so that the maximum overlaps the copy
constexpr int kClsRegVecs = 8;         // float4s of a row a thread keeps in registers (rows up to 32768 floats)
constexpr int kClsRowScratch = (kClsBins + kClsRank + 32 + 8 + 32) * 4 + kClsLoadParts * 8;   // histogram, candidates, reduction slots, control words, warp sums, mbarriers

struct ClsParams {
  int32_t C[kClsBatch];   // context length of each sequence
  int32_t T[kClsBatch];   // text tokens (query rows / group) of each sequence
  int32_t k[kClsBatch];   // entries summed per row
  int32_t n_kv_heads, n_q_heads, group, max_seq_len, t_stride;
  int32_t row_begin, row_block;   // this pass covers rows [row_begin, row_begin + row_block) of every unit
  int32_t c_stride;               // floats between two rows of the logits workspace (multiple of 128)
  int32_t r_stride;               // floats between two units of the row-sum array
  int32_t smem_cols;              // rows up to this length are staged in shared memory
  float scale_log2e;
};

// ---------------------------------------------------------------------------------------------
// Logits (tcgen05 tensor cores, accumulators in tensor memory).  One CTA = 256 rows of one unit x a range of
// 128-key tiles; the tile's keys are the accumulator's rows (lanes) and the 256 query rows its columns, so a
// draining warp owns 32 consecutive keys and 64 rows and writes, per row, one 128-byte line.
// grid (key ranges, 256-row blocks of the pass, units).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(tc::kThreads, 1)
    cls_logits_tc_kernel(const ClsParams P, const __nv_bfloat16* kin, const __nv_bfloat16* q_text, float* logits,
                         int tiles_per_cta, int32_t* err) {
  extern __shared__ __align__(16) uint8_t tc_smem[];
  const int unit = blockIdx.z, b = unit / P.n_kv_heads, h = unit - b * P.n_kv_heads;
  const int C = P.C[b], G = P.group, R = P.T[b] * G;
  const int r_end = min(R, P.row_begin + P.row_block);
  const int row0 = P.row_begin + blockIdx.y * tc::kQRows;
  const int n_tiles = (C + tc::kKeysPerTile - 1) / tc::kKeysPerTile;
  const int tile_begin = blockIdx.x * tiles_per_cta, tile_end = min(n_tiles, tile_begin + tiles_per_cta);
  if (row0 >= r_end || tile_begin >= tile_end) return;

  auto q_row = [&](int row) -> const __nv_bfloat16* {
    const int r = row0 + row;
    if (r >= r_end) return nullptr;
    const int i = r / G;
    return q_text + ((static_cast<size_t>(b) * P.t_stride + i) * P.n_q_heads + h * G + (r - i * G)) * kHeadDim;
  };
  const __nv_bfloat16* keys =
      kin + (static_cast<size_t>(b) * P.n_kv_heads + h) * static_cast<size_t>(P.max_seq_len) * kHeadDim;
  float* out = logits + static_cast<size_t>(unit) * P.row_block * P.c_stride;
  const float sc = P.scale_log2e;
  auto epilogue = [&](int tile, int lane_row, int part, auto groups, float*, auto, uint64_t*) {
    // accumulator lane = key lane_row of the tile, columns 64 part .. + 63 = rows row0 + 64 part + (0..63): for one
    // row the 32 lanes of a warp hold 32 consecutive keys, so every store instruction writes one 128-byte line of
    // that row and nothing has to be transposed
    const int rb = row0 + 64 * part;   // the warp's first row (the same in every lane)
    if (rb >= r_end) return;           // 64 padding rows
    float* dst = out + static_cast<size_t>(rb - P.row_begin) * P.c_stride + static_cast<size_t>(tile) * tc::kKeysPerTile +
                 lane_row;
    const size_t stride = static_cast<size_t>(P.c_stride);
    groups([&](int g, float (&v)[32]) {
      const int nv = r_end - (rb + 32 * g);   // rows of this group that exist (the same in every lane)
      float* p = dst + static_cast<size_t>(32 * g) * stride;
      if (nv >= 32) {
#pragma unroll
        for (int i = 0; i < 32; ++i) { *p = v[i] * sc; p += stride; }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i < nv) *p = v[i] * sc;
          p += stride;
        }
      }
    });
  };
  if (!tc::scores_cta<true>(tc_smem, q_row, keys, C, tile_begin, tile_end, epilogue) && threadIdx.x == 0)
    atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT);
}

// Whole block (kClsRowThreads threads, every one calls): the highest bin b of hist[0, nbins) with
// count(bins > b) < need <= count(bins >= b).  ctl[0] = b, ctl[1] = need - count(bins > b),
// ctl[2] = count(b); visible after the caller's next barrier.  nbins is 4096, 1024 or 256; wsum is
// scratch for 32 ints.
__device__ __forceinline__ void cls_find_bin(const int* hist, int nbins, int need, int* ctl, int* wsum) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int loc[4] = {0, 0, 0, 0};
  const int per = nbins == 4096 ? 4 : 1;
  if (per == 4) {
    const int4 v = reinterpret_cast<const int4*>(hist)[tid];
    loc[0] = v.x; loc[1] = v.y; loc[2] = v.z; loc[3] = v.w;
  } else if (tid < nbins) {
    loc[0] = hist[tid];
  }
  const int tot = (loc[0] + loc[1]) + (loc[2] + loc[3]);
  int run = tot;   // becomes the sum over this and the higher lanes of the warp
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_down_sync(0xffffffffu, run, off);
    if (lane + off < 32) run += v;
  }
  if (lane == 0) wsum[warp] = run;
  __syncthreads();
  const int wt = wsum[lane];
  int wrun = wt;   // sum over warps >= lane
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_down_sync(0xffffffffu, wrun, off);
    if (lane + off < 32) wrun += v;
  }
  int acc = __shfl_sync(0xffffffffu, wrun - wt, warp) + run - tot;   // items in the bins above this thread's
  if (acc < need && need <= acc + tot) {
#pragma unroll
    for (int j = 3; j >= 0; --j) {
      if (j < per && acc < need && need <= acc + loc[j]) {
        ctl[0] = tid * per + j;
        ctl[1] = need - acc;
        ctl[2] = loc[j];
      }
      if (j < per) acc += loc[j];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Sum of the k largest softmax entries of every row; a persistent CTA takes one row at a time.
// The row's logits arrive in shared memory by bulk copy (the next row is meanwhile prefetched into
// L2) and are replaced by p = 2^(l - max) in [0, 1], whose float bits order like the values.  The
// k-th largest p is found exactly: a histogram over bits 30..18 of p (32 bins per octave, so the
// lanes of a warp rarely meet in a bin), then the threshold bin's entries are sorted outright (four
// threads per entry) and the first `need` of them join the sum of everything above the bin; a
// crowded bin is first narrowed by histograms over bits 17..8 and 7..0.  Sums run in a fixed
// order, so the result is deterministic.
// rowsum: float [unit][r_stride]
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kClsRowThreads)
    cls_row_kernel(const ClsParams P, float* logits, float* rowsum, int rows_pass, int total_rows) {
  extern __shared__ __align__(16) uint8_t cls_smem[];
  int* hist = reinterpret_cast<int*>(cls_smem);                   // [kClsBins]
  uint32_t* cand = reinterpret_cast<uint32_t*>(hist + kClsBins);  // [kClsRank]
  float* red = reinterpret_cast<float*>(cand + kClsRank);         // [32]
  int* ctl = reinterpret_cast<int*>(red + 32);                    // [8]
  int* wsum = ctl + 8;                                            // [32]
  uint64_t* bar = reinterpret_cast<uint64_t*>(wsum + 32);         // [kClsLoadParts]
  float* srow = reinterpret_cast<float*>(cls_smem + kClsRowScratch);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < kClsLoadParts; ++i) mbar_init(bar + i, 1);
    mbar_fence_init();
  }
  uint32_t phases = 0;   // bit i: parity the next wait on barrier i looks for

  // block-wide reductions in a fixed order; every thread gets the result
  auto block_sum = [&](float v) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    v = red[lane];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
  };
  auto block_max = [&](float v) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    v = red[lane];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    return v;
  };
  // row `idx` of the pass: its unit, length and place; false for the rows a short sequence does not have
  auto locate = [&](int idx, int* unit, int* C, int* r, size_t* off) {
    if (idx >= total_rows) return false;
    *unit = idx / rows_pass;
    const int rr = idx - *unit * rows_pass, b = *unit / P.n_kv_heads;
    *C = P.C[b];
    *r = P.row_begin + rr;
    *off = (static_cast<size_t>(*unit) * P.row_block + rr) * P.c_stride;
    return *r < P.T[b] * P.group;
  };

  for (int idx = blockIdx.x; idx < total_rows; idx += gridDim.x) {
    int unit, C, r;
    size_t row_off;
    if (!locate(idx, &unit, &C, &r, &row_off)) continue;
    const int k = P.k[unit / P.n_kv_heads];
    const bool staged = C <= P.smem_cols;
    // p overwrites the logits: in shared memory, or for longer rows in place in the workspace
    float* row = staged ? srow : logits + row_off;
    float4* row4 = reinterpret_cast<float4*>(row);
    const int n4 = (C + 3) >> 2;
    // the row arrives in kClsLoadParts pieces of part4 float4s (a multiple of the block size), each on its own barrier
    const int part4 = ((n4 + kClsLoadParts - 1) / kClsLoadParts + kClsRowThreads - 1) / kClsRowThreads * kClsRowThreads;

    __syncthreads();   // the previous row's readers are done with the buffers
    if (tid == 0 && staged) {
      // whole 16-byte pieces: rows start 256-byte aligned and are padded to a multiple of 128 floats
      fence_proxy_async();
      for (int part = 0; part < kClsLoadParts; ++part) {
        const int beg = part * part4, end = min(n4, beg + part4);
        if (beg >= end) break;
        mbar_arrive_expect_tx(bar + part, static_cast<uint32_t>(end - beg) * 16u);
        for (int o = beg; o < end; o += 2048)
          bulk_g2s(row4 + o, reinterpret_cast<const float4*>(logits + row_off) + o,
                   static_cast<uint32_t>(min(2048, end - o)) * 16u, bar + part);
      }
      // start the next row's trip from HBM to L2 meanwhile
      int u2, C2, r2;
      size_t off2;
      if (locate(idx + gridDim.x, &u2, &C2, &r2, &off2) && C2 <= P.smem_cols) {
        const uint32_t b2 = static_cast<uint32_t>((C2 + 3) / 4 * 16);
        for (uint32_t o = 0; o < b2; o += 32768u)
          bulk_prefetch_l2(reinterpret_cast<const char*>(logits + off2) + o, min(32768u, b2 - o));
      }
    }
    for (int i = tid; i < kClsBins; i += kClsRowThreads) hist[i] = 0;
    if (tid == 0) ctl[3] = 0;

    // Rows of up to kClsRegItems floats per thread stay in REGISTERS from the moment they land: the maximum, the
    // probabilities, the histogram and the final sum are then computed without another trip through shared memory.
    // Longer rows keep p in the row buffer (shared memory, or the workspace) and are walked again per pass.
    const bool regs = staged && n4 <= kClsRegVecs * kClsRowThreads;
    float4 rv[kClsRegVecs];
    // visits every float4 this thread owns (p once the probabilities exist)
    auto each4 = [&](auto fn) {
      if (regs) {
#pragma unroll
        for (int q = 0; q < kClsRegVecs; ++q) {
          if (q * kClsRowThreads + tid < n4) fn(rv[q]);
        }
      } else {
#pragma unroll 4
        for (int i = tid; i < n4; i += kClsRowThreads) fn(row4[i]);
      }
    };
    auto each = [&](auto fn) {
      each4([&](const float4& v) { fn(v.x); fn(v.y); fn(v.z); fn(v.w); });
    };
    // top += every entry whose bit pattern is at least `from` (the bits of a float in [0, 1] order like its value);
    // four independent partial sums, added in a fixed order
    auto add_from = [&](uint32_t from) {
      float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
      each4([&](const float4& v) {
        t0 += __float_as_uint(v.x) >= from ? v.x : 0.f;
        t1 += __float_as_uint(v.y) >= from ? v.y : 0.f;
        t2 += __float_as_uint(v.z) >= from ? v.z : 0.f;
        t3 += __float_as_uint(v.w) >= from ? v.w : 0.f;
      });
      return (t0 + t1) + (t2 + t3);
    };

    // maximum, piece by piece as the row lands; the up to three floats between C and the next
    // multiple of four become -inf, that is p = 0: zeros below every real entry, which no top-k
    // sum can feel
    float mx = -INFINITY;
    bool landed = true;
    auto tail_fix = [&](float4& v, int i) {
      if (i == n4 - 1 && (C & 3)) {
        if ((C & 3) < 2) v.y = -INFINITY;
        if ((C & 3) < 3) v.z = -INFINITY;
        v.w = -INFINITY;
      }
    };
    if (regs) {
      static_assert(kClsLoadParts == 4, "piece index by three comparisons");
      const int m4 = part4 / kClsRowThreads;   // blocks of kClsRowThreads vectors per piece
      uint32_t waited = 0u;
#pragma unroll
      for (int q = 0; q < kClsRegVecs; ++q) {
        rv[q] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (q * kClsRowThreads < n4) {                       // the whole block of 1024 vectors lies in one piece
          const int part = (q >= m4) + (q >= 2 * m4) + (q >= 3 * m4);   // = q * kClsRowThreads / part4
          if (landed && !((waited >> part) & 1u)) {
            landed = mbar_wait_bounded(bar + part, (phases >> part) & 1u);
            phases ^= 1u << part;
            waited |= 1u << part;
          }
          const int i = q * kClsRowThreads + tid;
          if (landed && i < n4) {
            float4 v = row4[i];
            tail_fix(v, i);
            rv[q] = v;
            mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
          }
        }
      }
      // pieces past the row's end were never armed; pieces armed but not visited cannot exist (every armed piece
      // holds at least one block of vectors)
    } else {
      for (int part = 0; part < kClsLoadParts; ++part) {
        const int beg = part * part4, end = min(n4, beg + part4);
        if (beg >= end) break;
        if (staged && landed) {
          landed = mbar_wait_bounded(bar + part, (phases >> part) & 1u);
          phases ^= 1u << part;
        }
        if (!landed) continue;
        for (int i = beg + tid; i < end; i += kClsRowThreads) {
          float4 v = row4[i];
          if (i == n4 - 1 && (C & 3)) {
            tail_fix(v, i);
            row4[i] = v;
          }
          mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
        }
      }
    }
    if (__syncthreads_or(!landed)) {   // never seen; the whole CTA leaves, the row's sum and the score become NaN
      if (tid == 0) rowsum[static_cast<size_t>(unit) * P.r_stride + r] = __int_as_float(0x7FC00000);
      return;
    }
    const float M = block_max(mx);

    // p, normaliser, histogram
    auto prob = [&](float l) {
      // a NaN logit counts as no attention (fmaxf returns its other operand); every bit pattern stays in [0, bits(1)]
      return fminf(fmaxf(fast_exp2(l - M), 0.f), 1.f);
    };
    float z = 0.f;
    if (regs) {
#pragma unroll
      for (int q = 0; q < kClsRegVecs; ++q) {
        if (q * kClsRowThreads + tid < n4) {
          const float4 pq = make_float4(prob(rv[q].x), prob(rv[q].y), prob(rv[q].z), prob(rv[q].w));
          rv[q] = pq;
          z += (pq.x + pq.y) + (pq.z + pq.w);
          atomicAdd(&hist[__float_as_uint(pq.x) >> kClsShift], 1);
          atomicAdd(&hist[__float_as_uint(pq.y) >> kClsShift], 1);
          atomicAdd(&hist[__float_as_uint(pq.z) >> kClsShift], 1);
          atomicAdd(&hist[__float_as_uint(pq.w) >> kClsShift], 1);
        }
      }
    } else {
#pragma unroll 4
      for (int i = tid; i < n4; i += kClsRowThreads) {
        const float4 v = row4[i];
        const float4 q = make_float4(prob(v.x), prob(v.y), prob(v.z), prob(v.w));
        row4[i] = q;
        z += (q.x + q.y) + (q.z + q.w);
        atomicAdd(&hist[__float_as_uint(q.x) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(q.y) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(q.z) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(q.w) >> kClsShift], 1);
      }
    }
    const float Z = block_sum(z);   // its barriers also publish the histogram
    cls_find_bin(hist, kClsBins, k, ctl, wsum);
    __syncthreads();
    uint32_t prefix = static_cast<uint32_t>(ctl[0]);
    int shift = kClsShift, need = ctl[1], cnt = ctl[2];
    float top = 0.f;
    for (;;) {
      const uint32_t bin_lo = prefix << shift, bin_span = 1u << shift;   // the bin = bit patterns [bin_lo, bin_lo + bin_span)
      if (need == cnt) {                      // the whole bin is inside the top k
        top = add_from(bin_lo);
        break;
      }
      // A sharply peaked row: the k-th largest probability is so small that all `need` entries taken from its bin
      // add up to less than 2^-26, while the sum holds the row's maximum p = 1 — they cannot move a float32 sum
      // that is at least 1 by half a unit in the last place, so which of them count does not matter.
      if (static_cast<float>(need) * __uint_as_float((prefix + 1u) << shift) < 1.4901161e-8f) {
        top = add_from(bin_lo + bin_span);
        break;
      }
      if (cnt <= kClsRank) {
        // sum what lies above the bin, collect the bin's entries (each reserves its slot with one atomic; there
        // are at most kClsRank of them in the whole row) and sort them exactly (descending; equal values in an
        // arbitrary but complete order): the first `need` join the sum
        top = add_from(bin_lo + bin_span);
        each4([&](const float4& v) {
          const uint32_t a = __float_as_uint(v.x) - bin_lo, b = __float_as_uint(v.y) - bin_lo,
                         c = __float_as_uint(v.z) - bin_lo, d = __float_as_uint(v.w) - bin_lo;
          if (min(min(a, b), min(c, d)) < bin_span) {   // rare: at most kClsRank entries of the row pass
            if (a < bin_span) cand[atomicAdd(&ctl[3], 1)] = a + bin_lo;
            if (b < bin_span) cand[atomicAdd(&ctl[3], 1)] = b + bin_lo;
            if (c < bin_span) cand[atomicAdd(&ctl[3], 1)] = c + bin_lo;
            if (d < bin_span) cand[atomicAdd(&ctl[3], 1)] = d + bin_lo;
          }
        });
        __syncthreads();
        float* sorted = reinterpret_cast<float*>(hist);
        const int c = tid >> 2, part = tid & 3;          // four threads rank one entry
        int above = 0, before = 0;
        const uint32_t mk = c < cnt ? cand[c] : 0u;
        if (c < cnt) {
          for (int j = part; j < cnt; j += 4) {
            const uint32_t o = cand[j];
            above += o > mk;
            before += (o == mk) && (j < c);
          }
        }
        above += __shfl_xor_sync(0xffffffffu, above, 1);
        above += __shfl_xor_sync(0xffffffffu, above, 2);
        before += __shfl_xor_sync(0xffffffffu, before, 1);
        before += __shfl_xor_sync(0xffffffffu, before, 2);
        if (c < cnt && part == 0) sorted[above + before] = __uint_as_float(mk);
        __syncthreads();
        if (tid < need) top += sorted[tid];
        break;
      }
      if (shift == 0) {                       // more than kClsRank copies of one value: `need` of them count
        top = add_from(prefix + 1u);
        if (tid == 0) top += static_cast<float>(need) * __uint_as_float(prefix);
        break;
      }
      // a crowded bin: histogram of the next bits of its entries (17..8, then 7..0)
      const int width = shift == kClsShift ? 10 : 8;
      const int nshift = shift - width;
      const uint32_t mask = (1u << width) - 1u;
      for (int i = tid; i < (1 << width); i += kClsRowThreads) hist[i] = 0;
      __syncthreads();
      each([&](float e) {
        const uint32_t u = __float_as_uint(e);
        if ((u >> shift) == prefix) atomicAdd(&hist[(u >> nshift) & mask], 1);
      });
      __syncthreads();
      cls_find_bin(hist, 1 << width, need, ctl, wsum);
      __syncthreads();
      prefix = (prefix << width) | static_cast<uint32_t>(ctl[0]);
      shift = nshift;
      need = ctl[1];
      cnt = ctl[2];
    }
    top = block_sum(top);
    if (tid == 0) rowsum[static_cast<size_t>(unit) * P.r_stride + r] = top / Z;
  }
}

// ---------------------------------------------------------------------------------------------
// The same row sums for rows of up to kClsRegCols entries, every entry in a register of the CTA
// (kClsRegThreads threads x 32 entries), as a two-row pipeline: a row lands in shared memory in
// pieces of one vector per thread, each on its own mbarrier; once every thread has taken its
// entries into registers (the first block barrier of the row) one thread starts the NEXT row's
// copies into the same buffer, so they travel while this row's probabilities, histogram,
// threshold and sums are computed.  That thread also works out where the next row lies and hands
// it over through a two-slot descriptor in shared memory.  Arithmetic as in cls_row_kernel; sums in
// a fixed order.  (Measured and dropped: 512 threads of 64 entries -- a sixth fewer instructions,
// but a quarter slower with half the warps to hide latency; the threshold bin ranked by one warp
// after the last barrier -- slower than ranking it with the whole block between two barriers.)
// ---------------------------------------------------------------------------------------------
constexpr int kClsRegCols = 32768;
constexpr int kClsRegThreads = 1024;   // 512 threads x 128 entries issue a sixth fewer instructions but hide less latency: slower
constexpr int kClsRegWarps = kClsRegThreads / 32;
constexpr int kClsRegVecsT = kClsRegCols / 4 / kClsRegThreads;   // float4s per thread: 16
// histogram, candidates, their sorted copy, three reduction slots, control words, warp sums, two row descriptors,
// piece barriers
constexpr int kClsRegScratch = (kClsBins + 2 * kClsRank + 3 * 32 + 8 + 32 + 2 * 8) * 4 + kClsRegVecsT * 8;
static_assert(kClsRegScratch % 16 == 0, "the row buffer is 16-byte aligned");
constexpr int kClsRegBinsPer = kClsBins / kClsRegThreads;   // bins a thread sums in the threshold search
static_assert((kClsRegBinsPer == 4 || kClsRegBinsPer == 8) && kClsRegVecsT <= 32, "whole int4s of bins per thread; one phase bit per piece");

// cls_find_bin for a block of kClsRegThreads threads (nbins 4096, 1024 or 256).
__device__ __forceinline__ void cls_find_bin_regs(const int* hist, int nbins, int need, int* ctl, int* wsum) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = nbins == kClsBins ? kClsRegBinsPer : nbins > kClsRegThreads ? nbins / kClsRegThreads : 1;   // 4 or 8; 2 or 1; 1
  int loc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (nbins == kClsBins) {
    const int4 u = reinterpret_cast<const int4*>(hist)[tid * (kClsRegBinsPer / 4)];
    loc[0] = u.x; loc[1] = u.y; loc[2] = u.z; loc[3] = u.w;
    if (kClsRegBinsPer == 8) {
      const int4 v = reinterpret_cast<const int4*>(hist)[tid * 2 + 1];
      loc[4] = v.x; loc[5] = v.y; loc[6] = v.z; loc[7] = v.w;
    }
  } else if (per == 2) {
    const int2 u = reinterpret_cast<const int2*>(hist)[tid];
    loc[0] = u.x; loc[1] = u.y;
  } else if (tid < nbins) {
    loc[0] = hist[tid];
  }
  const int tot = ((loc[0] + loc[1]) + (loc[2] + loc[3])) + ((loc[4] + loc[5]) + (loc[6] + loc[7]));
  int run = tot;   // becomes the sum over this and the higher lanes of the warp
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_down_sync(0xffffffffu, run, off);
    if (lane + off < 32) run += v;
  }
  if (lane == 0) wsum[warp] = run;
  __syncthreads();
  const int wt = lane < kClsRegWarps ? wsum[lane] : 0;
  int wrun = wt;   // sum over warps >= lane
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_down_sync(0xffffffffu, wrun, off);
    if (lane + off < 32) wrun += v;
  }
  int acc = __shfl_sync(0xffffffffu, wrun - wt, warp) + run - tot;   // items in the bins above this thread's
  if (acc < need && need <= acc + tot) {
#pragma unroll
    for (int j = 7; j >= 0; --j) {
      if (j < per && acc < need && need <= acc + loc[j]) {
        ctl[0] = tid * per + j;
        ctl[1] = need - acc;
        ctl[2] = loc[j];
      }
      if (j < per) acc += loc[j];
    }
  }
}

__global__ void __launch_bounds__(kClsRegThreads)
    cls_row_regs_kernel(const ClsParams P, const float* logits, float* rowsum, int rows_pass, int total_rows) {
  extern __shared__ __align__(16) uint8_t cls_smem[];
  int* hist = reinterpret_cast<int*>(cls_smem);                   // [kClsBins]
  uint32_t* cand = reinterpret_cast<uint32_t*>(hist + kClsBins);  // [kClsRank]
  float* sorted = reinterpret_cast<float*>(cand + kClsRank);      // [kClsRank]: the threshold bin in descending order
  float* red = sorted + kClsRank;                                 // [3][32]: one slot per reduction of a row
  int* ctl = reinterpret_cast<int*>(red + 3 * 32);                // [8]
  int* wsum = ctl + 8;                                            // [32]
  int* desc = wsum + 32;                                          // [2][8]: idx (-1: none), unit, C, r, k, offset lo, hi
  uint64_t* bar = reinterpret_cast<uint64_t*>(desc + 16);         // [kClsRegVecsT]
  float4* srow4 = reinterpret_cast<float4*>(cls_smem + kClsRegScratch);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // thread 0 only: the first row at or after `idx` (stride gridDim.x) that exists -> descriptor slot, and its copies
  auto post_row = [&](int idx, int slot) {
    int* d = desc + slot * 8;
    for (; idx < total_rows; idx += gridDim.x) {
      const int unit = idx / rows_pass, rr = idx - unit * rows_pass, b = unit / P.n_kv_heads;
      const int r = P.row_begin + rr;
      if (r >= P.T[b] * P.group) continue;      // a short sequence does not have this row
      const int C = P.C[b];
      const size_t off = (static_cast<size_t>(unit) * P.row_block + rr) * P.c_stride;
      d[0] = idx; d[1] = unit; d[2] = C; d[3] = r; d[4] = P.k[b];
      const int n4 = (C + 3) >> 2;
      // whole 16-byte pieces: rows start 256-byte aligned and are padded to a multiple of 128 floats
      fence_proxy_async();
      const float4* src = reinterpret_cast<const float4*>(logits + off);
      for (int q = 0; q * kClsRegThreads < n4; ++q) {
        const uint32_t bytes = static_cast<uint32_t>(min(kClsRegThreads, n4 - q * kClsRegThreads)) * 16u;
        mbar_arrive_expect_tx(bar + q, bytes);
        bulk_g2s(srow4 + q * kClsRegThreads, src + q * kClsRegThreads, bytes, bar + q);
      }
      return;
    }
    d[0] = -1;
  };

  if (tid == 0) {
    for (int i = 0; i < kClsRegVecsT; ++i) mbar_init(bar + i, 1);
    mbar_fence_init();
    ctl[3] = 0;
    post_row(blockIdx.x, 0);
  }
  for (int i = tid; i < kClsBins; i += kClsRegThreads) hist[i] = 0;
  __syncthreads();
  uint32_t phases = 0;   // bit q: parity the next wait on barrier q looks for

  for (int it = 0;; ++it) {
    const int* d = desc + (it & 1) * 8;
    const int idx = d[0];
    if (idx < 0) break;
    const int unit = d[1], C = d[2], r = d[3], k = d[4];
    const int n4 = (C + 3) >> 2;

    // the row's entries into registers, piece by piece as they land, with the running maximum; the up to three
    // floats between C and the next multiple of four become -inf, that is p = 0: zeros below every real entry,
    // which no top-k sum can feel
    float4 rv[kClsRegVecsT];   // rv[q] is used only where q * kClsRegThreads + tid < n4
    float mx = -INFINITY;
    bool landed = true;
    const int i_fix = (C & 3) ? n4 - 1 : -1;   // the vector with floats past the row's end
#pragma unroll
    for (int q = 0; q < kClsRegVecsT; ++q) {
      if (q * kClsRegThreads < n4) {
        if (landed) landed = mbar_wait_bounded(bar + q, (phases >> q) & 1u);
        phases ^= 1u << q;
        const int i = q * kClsRegThreads + tid;
        if (landed && i < n4) {
          float4 v = srow4[i];
          if (i == i_fix) {
            if ((C & 3) < 2) v.y = -INFINITY;
            if ((C & 3) < 3) v.z = -INFINITY;
            v.w = -INFINITY;
          }
          rv[q] = v;
          mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
        }
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0) red[warp] = mx;
    // every thread holds its entries: the buffer is free.  A wait that ran out (never seen): the whole CTA
    // leaves, the row's sum and with it the unit's score become NaN
    if (__syncthreads_or(!landed)) {
      if (tid == 0) rowsum[static_cast<size_t>(unit) * P.r_stride + r] = __int_as_float(0x7FC00000);
      return;
    }
    if (tid == 0) post_row(idx + gridDim.x, (it + 1) & 1);   // the next row travels during the rest of this one
    float M = lane < kClsRegWarps ? red[lane] : -INFINITY;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));

    // p = 2^(l - max) in [0, 1] (a NaN logit counts as no attention: fmaxf returns its other operand), the
    // normaliser, and the histogram over bits 30..18 of p
    float z = 0.f;
#pragma unroll
    for (int q = 0; q < kClsRegVecsT; ++q) {
      if (q * kClsRegThreads + tid < n4) {
        float4 pq;
        pq.x = fminf(fmaxf(fast_exp2(rv[q].x - M), 0.f), 1.f);
        pq.y = fminf(fmaxf(fast_exp2(rv[q].y - M), 0.f), 1.f);
        pq.z = fminf(fmaxf(fast_exp2(rv[q].z - M), 0.f), 1.f);
        pq.w = fminf(fmaxf(fast_exp2(rv[q].w - M), 0.f), 1.f);
        rv[q] = pq;
        z += (pq.x + pq.y) + (pq.z + pq.w);
        atomicAdd(&hist[__float_as_uint(pq.x) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(pq.y) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(pq.z) >> kClsShift], 1);
        atomicAdd(&hist[__float_as_uint(pq.w) >> kClsShift], 1);
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
    if (lane == 0) red[32 + warp] = z;
    __syncthreads();   // publishes the warp sums and the histogram
    float Z = lane < kClsRegWarps ? red[32 + lane] : 0.f;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, off);
    cls_find_bin_regs(hist, kClsBins, k, ctl, wsum);
    __syncthreads();
    auto each4 = [&](auto fn) {
#pragma unroll
      for (int q = 0; q < kClsRegVecsT; ++q) {
        if (q * kClsRegThreads + tid < n4) fn(rv[q]);
      }
    };
    // the sum of every entry whose bit pattern is at least `from`; four partial sums added in a fixed order
    auto add_from = [&](uint32_t from) {
      float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
      each4([&](const float4& v) {
        t0 += __float_as_uint(v.x) >= from ? v.x : 0.f;
        t1 += __float_as_uint(v.y) >= from ? v.y : 0.f;
        t2 += __float_as_uint(v.z) >= from ? v.z : 0.f;
        t3 += __float_as_uint(v.w) >= from ? v.w : 0.f;
      });
      return (t0 + t1) + (t2 + t3);
    };
    // the entries with bit patterns in [lo, lo + span) each reserve a slot of cand[] (the caller knows their number)
    auto collect = [&](uint32_t lo, uint32_t span) {
      each4([&](const float4& v) {
        const uint32_t a = __float_as_uint(v.x) - lo, b = __float_as_uint(v.y) - lo, c = __float_as_uint(v.z) - lo,
                       e = __float_as_uint(v.w) - lo;
        if (min(min(a, b), min(c, e)) < span) {
          if (a < span) cand[atomicAdd(&ctl[3], 1)] = a + lo;
          if (b < span) cand[atomicAdd(&ctl[3], 1)] = b + lo;
          if (c < span) cand[atomicAdd(&ctl[3], 1)] = c + lo;
          if (e < span) cand[atomicAdd(&ctl[3], 1)] = e + lo;
        }
      });
    };
    uint32_t prefix = static_cast<uint32_t>(ctl[0]);
    int shift = kClsShift, need = ctl[1], cnt = ctl[2];
    float top = 0.f;
    int n_sorted = 0;   // entries of sorted[] that belong to the sum
    for (;;) {
      const uint32_t bin_lo = prefix << shift, bin_span = 1u << shift;   // the bin = bit patterns [bin_lo, bin_lo + bin_span)
      if (need == cnt) {                      // the whole bin is inside the top k
        top = add_from(bin_lo);
        break;
      }
      // A sharply peaked row: all `need` entries taken from the bin add up to less than 2^-26 while the sum holds
      // the row's maximum p = 1, so they cannot move it by half a unit in the last place
      if (static_cast<float>(need) * __uint_as_float(bin_lo + bin_span) < 1.4901161e-8f) {
        top = add_from(bin_lo + bin_span);
        break;
      }
      if (cnt <= kClsRank) {
        // up to kClsRank entries: ranked exactly (descending; equal values in an arbitrary but complete order) by
        // several threads per entry; warp 0 adds the first `need` in that order after the row's last barrier
        top = add_from(bin_lo + bin_span);
        collect(bin_lo, bin_span);
        __syncthreads();
        constexpr int kSh = kClsRegThreads == 1024 ? 2 : 1;   // log2 of threads per entry when all kClsRank slots are in use
        const int sh = cnt <= kClsRank / 2 ? kSh + 1 : kSh;
        const int c = tid >> sh, part = tid & ((1 << sh) - 1);
        const uint32_t mk = c < cnt ? cand[c] : 0u;
        int rank = 0;   // entries that come before this one
        if (c < cnt) {
          for (int j = part; j < cnt; j += 1 << sh) {
            const uint32_t o = cand[j];
            rank += (o > mk) || (o == mk && j < c);
          }
        }
        for (int off = 1; off < (1 << sh); off <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, off);
        if (c < cnt && part == 0) sorted[rank] = __uint_as_float(mk);
        n_sorted = need;
        break;
      }
      if (shift == 0) {                       // more than kClsRank copies of one value: `need` of them count
        top = add_from(prefix + 1u);
        if (tid == 0) top += static_cast<float>(need) * __uint_as_float(prefix);
        break;
      }
      // a crowded bin: histogram of the next bits of its entries (17..8, then 7..0)
      const int width = shift == kClsShift ? 10 : 8;
      const int nshift = shift - width;
      const uint32_t mask = (1u << width) - 1u;
      for (int i = tid; i < (1 << width); i += kClsRegThreads) hist[i] = 0;
      __syncthreads();
      each4([&](const float4& v) {
        const uint32_t u[4] = {__float_as_uint(v.x), __float_as_uint(v.y), __float_as_uint(v.z), __float_as_uint(v.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if ((u[e] >> shift) == prefix) atomicAdd(&hist[(u[e] >> nshift) & mask], 1);
      });
      __syncthreads();
      cls_find_bin_regs(hist, 1 << width, need, ctl, wsum);
      __syncthreads();
      prefix = (prefix << width) | static_cast<uint32_t>(ctl[0]);
      shift = nshift;
      need = ctl[1];
      cnt = ctl[2];
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) top += __shfl_xor_sync(0xffffffffu, top, off);
    if (lane == 0) red[64 + warp] = top;
    __syncthreads();   // every reader of the histogram area and of the control words is done
    if (warp == 0) {
      float t = lane < kClsRegWarps ? red[64 + lane] : 0.f;
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
      if (n_sorted > 0) {   // the threshold bin's share, largest first, in a fixed order
        float s = 0.f;
        for (int j = lane; j < n_sorted; j += 32) s += sorted[j];
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        t += s;
      }
      if (lane == 0) {
        rowsum[static_cast<size_t>(unit) * P.r_stride + r] = t / Z;
        ctl[3] = 0;
      }
    }
    for (int i = tid; i < kClsBins; i += kClsRegThreads) hist[i] = 0;   // for the next row; its first barrier orders it
  }
}

// Mean of a unit's row sums (double, fixed order) and its label: 0 static if score >= theta, else 1.
__global__ void __launch_bounds__(256)
    cls_finish_kernel(const ClsParams P, const float* rowsum, const int32_t* err, double theta, double* scores_out,
                      uint8_t* type_out, int unit0) {
  __shared__ double part[256];
  const int unit = blockIdx.x, b = unit / P.n_kv_heads;
  const int R = P.T[b] * P.group;
  const float* rs = rowsum + static_cast<size_t>(unit) * P.r_stride;
  double acc = 0.0;
  for (int i = threadIdx.x; i < R; i += 256) acc += static_cast<double>(rs[i]);
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int s = 128; s >= 1; s >>= 1) {
    if (threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    // a device-side wait that ran out (never seen) turns every score into NaN
    const double score = err[0] == 0 ? part[0] / static_cast<double>(R) : __longlong_as_double(0x7FF8000000000000ll);
    scores_out[unit0 + unit] = score;
    type_out[unit0 + unit] = score >= theta ? 0 : 1;
  }
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

hkv_status cls_check(const hkv_config* cfg, int32_t n_text_max) {
  if (!cfg) return HKV_ERR_INVALID_ARG;
  if (cfg->batch < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->max_seq_len < 1 || n_text_max < 1)
    return HKV_ERR_SHAPE;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return HKV_ERR_SHAPE;
  if (cfg->head_dim != kHeadDim || cfg->n_kv_heads > 60000 || cfg->max_seq_len > (1 << 23)) return HKV_ERR_UNSUPPORTED;
  if (!(cfg->softmax_scale >= 0.f) || std::isinf(cfg->softmax_scale)) return HKV_ERR_INVALID_ARG;
  if (static_cast<int64_t>(n_text_max) * (cfg->n_q_heads / cfg->n_kv_heads) > (1 << 24)) return HKV_ERR_UNSUPPORTED;
  return HKV_OK;
}

// sequences per group of launches, units of a group, bytes of the row-sum array in front of the logits
struct ClsShape {
  int group_batch, group_units, r_max;
  size_t head_bytes;   // error word (kAlign bytes) + row sums
};
ClsShape cls_shape(const hkv_config* cfg, int32_t n_text_max) {
  ClsShape s;
  s.group_batch = std::min(std::min(cfg->batch, kClsBatch), 60000 / cfg->n_kv_heads);
  s.group_units = s.group_batch * cfg->n_kv_heads;
  s.r_max = n_text_max * (cfg->n_q_heads / cfg->n_kv_heads);
  s.head_bytes = kAlign + round_up(static_cast<size_t>(s.group_units) * s.r_max * sizeof(float), kAlign);
  return s;
}

}  // namespace

}  // namespace hkv

using namespace hkv;

extern "C" hkv_status hkv_classify_workspace(const hkv_config* cfg, int32_t n_text_max, size_t* min_bytes,
                                             size_t* preferred_bytes) {
  const hkv_status st = cls_check(cfg, n_text_max);
  if (st != HKV_OK) return st;
  if (!min_bytes && !preferred_bytes) return HKV_ERR_INVALID_ARG;
  const ClsShape s = cls_shape(cfg, n_text_max);
  const size_t row_bytes = round_up(cfg->max_seq_len, tc::kKeysPerTile) * sizeof(float) * s.group_units;
  if (min_bytes) *min_bytes = s.head_bytes + 16 * row_bytes;
  if (preferred_bytes) {
    // every row at once, up to half a gigabyte of logits
    size_t rows = round_up(s.r_max, 16);
    const size_t cap = std::max<size_t>(16, (static_cast<size_t>(512) << 20) / row_bytes / 16 * 16);
    rows = std::min(rows, cap);
    *preferred_bytes = s.head_bytes + rows * row_bytes;
  }
  return HKV_OK;
}

extern "C" hkv_status hkv_classify_heads(const hkv_config* cfg, const void* k, const void* q_text,
                                         int32_t n_text_max, const int32_t* seq_lens, const int32_t* n_text,
                                         double topk_fraction, double theta, void* workspace,
                                         size_t workspace_bytes, double* scores_out, uint8_t* head_type_out,
                                         void* stream) {
  const hkv_status st = cls_check(cfg, n_text_max);
  if (st != HKV_OK) return st;
  if (!k || !q_text || !seq_lens || !n_text || !workspace || !scores_out || !head_type_out)
    return HKV_ERR_INVALID_ARG;
  if (!(topk_fraction > 0.0 && topk_fraction <= 1.0) || !std::isfinite(theta)) return HKV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return HKV_ERR_WORKSPACE;
  int c_max = 0;
  for (int b = 0; b < cfg->batch; ++b) {
    if (seq_lens[b] < 1 || seq_lens[b] > cfg->max_seq_len) return HKV_ERR_SHAPE;
    if (n_text[b] < 1 || n_text[b] > n_text_max) return HKV_ERR_SHAPE;
    c_max = std::max(c_max, seq_lens[b]);
  }
  const ClsShape s = cls_shape(cfg, n_text_max);
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  const size_t c_stride = round_up(c_max, tc::kKeysPerTile);
  const size_t row_bytes = c_stride * sizeof(float) * s.group_units;
  if (workspace_bytes < s.head_bytes + 16 * row_bytes) return HKV_ERR_WORKSPACE;
  const int row_block = static_cast<int>(
      std::min<size_t>(round_up(s.r_max, 16), (workspace_bytes - s.head_bytes) / row_bytes / 16 * 16));

  const int smem_cols = static_cast<int>(round_up(std::min(c_max, kClsSmemCols), 64));
  const size_t row_smem = kClsRowScratch + static_cast<size_t>(smem_cols) * sizeof(float);
  if (cudaFuncSetAttribute(cls_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(row_smem)) != cudaSuccess)
    return HKV_ERR_CUDA;
  const size_t regs_smem = kClsRegScratch + static_cast<size_t>(kClsRegCols) * sizeof(float);
  if (cudaFuncSetAttribute(cls_row_regs_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(regs_smem)) != cudaSuccess)
    return HKV_ERR_CUDA;

  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1)
    return HKV_ERR_CUDA;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int32_t* err = static_cast<int32_t*>(workspace);
  float* rowsum = reinterpret_cast<float*>(static_cast<char*>(workspace) + kAlign);
  if (cudaMemsetAsync(err, 0, kAlign, cs) != cudaSuccess) return HKV_ERR_CUDA;
  if (cudaFuncSetAttribute(cls_logits_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes) !=
      cudaSuccess)
    return HKV_ERR_CUDA;
  float* logits = reinterpret_cast<float*>(static_cast<char*>(workspace) + s.head_bytes);
  const float scale =
      cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(static_cast<float>(cfg->head_dim));
  for (int b0 = 0; b0 < cfg->batch; b0 += s.group_batch) {
    const int nb = std::min(s.group_batch, cfg->batch - b0);
    ClsParams P{};
    int r_max = 0, cg_max = 0;
    for (int i = 0; i < nb; ++i) {
      const int C = seq_lens[b0 + i];
      P.C[i] = C;
      P.T[i] = n_text[b0 + i];
      const double kk = std::ceil(topk_fraction * static_cast<double>(C) - 1e-9);
      P.k[i] = static_cast<int32_t>(std::max(1.0, std::min(static_cast<double>(C), kk)));
      r_max = std::max(r_max, P.T[i] * G);
      cg_max = std::max(cg_max, C);
    }
    P.n_kv_heads = cfg->n_kv_heads;
    P.n_q_heads = cfg->n_q_heads;
    P.group = G;
    P.max_seq_len = cfg->max_seq_len;
    P.t_stride = n_text_max;
    P.row_block = row_block;
    P.c_stride = static_cast<int32_t>(c_stride);
    P.r_stride = s.r_max;
    P.smem_cols = smem_cols;
    P.scale_log2e = scale * kLog2e;
    const __nv_bfloat16* kg = static_cast<const __nv_bfloat16*>(k) +
                              static_cast<size_t>(b0) * cfg->n_kv_heads * cfg->max_seq_len * kHeadDim;
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(q_text) +
                              static_cast<size_t>(b0) * n_text_max * cfg->n_q_heads * kHeadDim;
    const int units = nb * cfg->n_kv_heads;
    for (int rb = 0; rb < r_max; rb += row_block) {
      P.row_begin = rb;
      const int rows = std::min(row_block, r_max - rb);
      // key ranges sized so that the launch is about one wave of CTAs
      const int row_blocks = (rows + tc::kQRows - 1) / tc::kQRows;
      const int n_tiles = (cg_max + tc::kKeysPerTile - 1) / tc::kKeysPerTile;
      const int splits = std::max(1, std::min(n_tiles, n_sm / std::max(1, units * row_blocks)));
      const int tiles_per_cta = (n_tiles + splits - 1) / splits;
      cls_logits_tc_kernel<<<dim3((n_tiles + tiles_per_cta - 1) / tiles_per_cta, row_blocks, units), tc::kThreads,
                             tc::kSmemBytes, cs>>>(P, kg, qg, logits, tiles_per_cta, err);
      const int total_rows = rows * units;
      if (cg_max <= kClsRegCols)   // every row of the group fits the threads' registers: the pipelined kernel
        cls_row_regs_kernel<<<std::min(total_rows, n_sm), kClsRegThreads, regs_smem, cs>>>(P, logits, rowsum, rows,
                                                                                           total_rows);
      else
        cls_row_kernel<<<std::min(total_rows, n_sm), kClsRowThreads, row_smem, cs>>>(P, logits, rowsum, rows, total_rows);
    }
    cls_finish_kernel<<<units, 256, 0, cs>>>(P, rowsum, err, theta, scores_out, head_type_out, b0 * cfg->n_kv_heads);
    if (cudaGetLastError() != cudaSuccess) return HKV_ERR_CUDA;
  }
  return HKV_OK;
}
