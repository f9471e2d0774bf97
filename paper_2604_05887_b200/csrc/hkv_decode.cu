// Decode-step kernels: chunk scoring + exact top-k chunk selection for dynamic heads, and the
// split-K flash-decode over each head's retained token list with the split merge fused in.
#include "hkv_device.cuh"
#include "hkv_internal.h"

namespace hkv {

namespace {

__device__ __forceinline__ int find_slot(const int32_t* prefix, int n, int x) {
  int i = 0;
  while (i + 1 < n && x >= prefix[i + 1]) ++i;
  return i;
}

// ---------------------------------------------------------------------------------------------
// Chunk score + top-k (one CTA per dynamic unit).
// score_c = <sum_g q_g, mean_c> in float32; the k_sel best chunks, ties to the lower id, are written
// in ascending id order; n_valid = tokens those chunks hold (the last chunk of a sequence may be
// short, and being the highest id it is always last in the list).
// ---------------------------------------------------------------------------------------------
constexpr int kSelThreads = 256;
constexpr int kSelSmemScores = 8192;

__global__ void __launch_bounds__(kSelThreads) select_chunks_kernel(const __grid_constant__ DecodeBatch batch) {
  __shared__ float qsum[kHeadDim];
  __shared__ float sc_smem[kSelSmemScores];
  __shared__ int hist[256];
  __shared__ int wsum[96];
  __shared__ int bc[4];

  const int li = find_slot(batch.dyn_prefix, batch.n, blockIdx.x);
  char* base = batch.cache[li];
  const Header* hdr = reinterpret_cast<const Header*>(base);
  const int uid = reinterpret_cast<const int32_t*>(base + hdr->dyn_list_off)[blockIdx.x - batch.dyn_prefix[li]];
  const Unit* u = reinterpret_cast<const Unit*>(base + hdr->units_off) + uid;
  const int G = hdr->group, cs = hdr->chunk_size;
  const int n_chunks = u->n_chunks, k_sel = u->k_sel, C = u->C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid < kHeadDim) {
    const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(batch.q[li]) +
                             (static_cast<size_t>(u->b) * hdr->n_q_heads + static_cast<size_t>(u->h) * G) * kHeadDim;
    float s = 0.f;
    for (int g = 0; g < G; ++g) s += __bfloat162float(q[g * kHeadDim + tid]);
    qsum[tid] = s;
  }
  __syncthreads();

  float* scores = reinterpret_cast<float*>(base + u->scores_off);
  const uint4* summ = reinterpret_cast<const uint4*>(base + u->summ_off);   // 16 uint4 per chunk mean
  const bool in_smem = n_chunks <= kSelSmemScores;
  {
    // 16 lanes per chunk mean (16 B each), two chunks per warp pass
    const int sub = lane & 15, half = lane >> 4;
    float qv[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) qv[j] = qsum[sub * 8 + j];
    for (int c0 = warp * 2; c0 < n_chunks; c0 += (kSelThreads / 32) * 2) {
      const int c = c0 + half;
      float acc = 0.f;
      if (c < n_chunks) {
        const uint4 m = summ[static_cast<size_t>(c) * 16 + sub];
        acc = fmaf(bf16_lo(m.x), qv[0], acc); acc = fmaf(bf16_hi(m.x), qv[1], acc);
        acc = fmaf(bf16_lo(m.y), qv[2], acc); acc = fmaf(bf16_hi(m.y), qv[3], acc);
        acc = fmaf(bf16_lo(m.z), qv[4], acc); acc = fmaf(bf16_hi(m.z), qv[5], acc);
        acc = fmaf(bf16_lo(m.w), qv[6], acc); acc = fmaf(bf16_hi(m.w), qv[7], acc);
      }
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
      if (c < n_chunks && sub == 0) {
        scores[c] = acc;
        if (in_smem) sc_smem[c] = acc;
      }
    }
  }
  __syncthreads();

  int32_t* sel = reinterpret_cast<int32_t*>(base + u->idx_off);
  const float* src = in_smem ? sc_smem : scores;
  int emitted;
  if (k_sel >= n_chunks) {
    for (int i = tid; i < n_chunks; i += kSelThreads) sel[i] = i;
    emitted = n_chunks;
  } else {
    emitted = block_select_emit(
        n_chunks, k_sel, [&](int i) { return float_key(src[i]); }, [](int) { return false; }, sel, hist, wsum, bc);
  }
  __syncthreads();
  if (tid == 0) {
    int32_t* n_valid = reinterpret_cast<int32_t*>(base + hdr->n_valid_off);
    int nv = emitted * cs;
    if (emitted > 0 && sel[emitted - 1] == n_chunks - 1) nv -= n_chunks * cs - C;
    n_valid[uid] = nv;
  }
}

// ---------------------------------------------------------------------------------------------
// Split-K flash-decode.
//
// One CTA per split (a contiguous range of 32-token tiles of one unit's retained token list).  Each
// of the CTA's warps is an independent consumer with its own ring of kDecStages staging buffers and
// its own mbarriers: it takes every kDecWarps-th tile of the split, has the TMA engine copy the
// tile's K and V rows (1-D bulk copies, one pair per chunk piece) into the ring, and runs
//   S = Q K^T  (rows = the group's query heads padded to 16, cols = 32 tokens)  on tensor cores,
//   online softmax in float32 (base-2 exponent),  O += P V  on tensor cores,
// so that every loaded KV tile is shared by all query heads of the group.  K/V rows live in HBM
// with their eight... sixteen 16-byte pieces XOR-permuted by (row & 7) (see swz()), which makes the
// ldmatrix reads of the staged tile bank-conflict free without any copy in shared memory.
// At the end the warps of a CTA are merged in shared memory, the CTA writes one partial
// (m, l, O) — or the final output when the unit has a single split — and the last CTA of a unit to
// arrive merges the unit's partials in split order (deterministic) and writes the output.
// ---------------------------------------------------------------------------------------------
constexpr float kLog2e = 1.4426950408889634f;

struct WarpState {
  float m0, m1, l0, l1;
};

template <bool HI>
__global__ void __launch_bounds__(kDecWarps * 32, 1)
    flash_decode_kernel(const __grid_constant__ DecodeBatch batch, int out_f32) {
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ int s_is_last;

  const int li = find_slot(batch.split_prefix, batch.n, blockIdx.x);
  char* base = batch.cache[li];
  const Header* hdr = reinterpret_cast<const Header*>(base);
  const Split sp = reinterpret_cast<const Split*>(base + hdr->splits_off)[blockIdx.x - batch.split_prefix[li]];
  const Unit* up = reinterpret_cast<const Unit*>(base + hdr->units_off) + sp.unit;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int G = hdr->group, Hq = hdr->n_q_heads;
  const int cs = hdr->chunk_size;
  const bool dynamic = up->type != 0;
  const int ub = up->b, uh = up->h, n_splits = up->n_splits;
  const int n_valid = dynamic ? reinterpret_cast<const int32_t*>(base + hdr->n_valid_off)[sp.unit] : up->n_tok;
  const uint8_t* kplane = reinterpret_cast<const uint8_t*>(base + up->k_off);
  const uint8_t* vplane = reinterpret_cast<const uint8_t*>(base + up->v_off);
  const int32_t* sel = reinterpret_cast<const int32_t*>(base + up->idx_off);
  int32_t* err = reinterpret_cast<int32_t*>(base + hdr->err_off);
  const float sc = hdr->scale * kLog2e;

  uint8_t* ring = smem + warp * (kDecStages * kStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kDecWarps * kDecStages * kStageBytes) + warp * kDecStages;
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kDecStages; ++s) mbar_init(&bars[s], 1);
    mbar_fence_init();
  }
  __syncwarp();

  // tiles of this warp: first, first + kDecWarps, ... below tile_end (clipped to the valid tokens)
  const int tile_end = min(sp.tile_end, (n_valid + kTile - 1) / kTile);
  const int first = sp.tile_begin + warp;
  const int n_my = first < tile_end ? (tile_end - first + kDecWarps - 1) / kDecWarps : 0;

  auto issue = [&](int it) {
    const int stage = it % kDecStages;
    uint8_t* st = ring + stage * kStageBytes;
    const int v0 = (first + it * kDecWarps) * kTile;
    const int v1 = min(v0 + kTile, n_valid);
    uint32_t* keys = reinterpret_cast<uint32_t*>(st + 2 * kTile * kRowBytes);
    fence_proxy_async();
    if (lane == 0) mbar_arrive_expect_tx(&bars[stage], static_cast<uint32_t>(v1 - v0) * 2u * kRowBytes);
    __syncwarp();
    if (dynamic) {
      const int ci = v0 / cs + lane;                       // lane-th chunk touching this tile
      const int p0 = max(v0, ci * cs), p1 = min(v1, (ci + 1) * cs);
      if (p0 < p1) {
        const size_t row = static_cast<size_t>(sel[ci]) * cs + (p0 - ci * cs);
        const uint32_t bytes = static_cast<uint32_t>(p1 - p0) * kRowBytes;
        bulk_g2s(st + (p0 - v0) * kRowBytes, kplane + row * kRowBytes, bytes, &bars[stage]);
        bulk_g2s(st + kTile * kRowBytes + (p0 - v0) * kRowBytes, vplane + row * kRowBytes, bytes, &bars[stage]);
      }
      const int v = v0 + lane;
      uint32_t key = lane & 7;
      if (v < v1) {
        const int cj = v / cs;
        key = static_cast<uint32_t>(sel[cj] * cs + (v - cj * cs)) & 7u;
      }
      keys[lane] = key;
    } else {
      if (lane == 0) {
        const uint32_t bytes = static_cast<uint32_t>(v1 - v0) * kRowBytes;
        bulk_g2s(st, kplane + static_cast<size_t>(v0) * kRowBytes, bytes, &bars[stage]);
        bulk_g2s(st + kTile * kRowBytes, vplane + static_cast<size_t>(v0) * kRowBytes, bytes, &bars[stage]);
      }
      keys[lane] = lane & 7;
    }
  };

  // prologue: fill the ring, then fetch this group's queries as A fragments (rows >= G are zero)
  for (int it = 0; it < min(n_my, kDecStages); ++it) issue(it);

  uint32_t qa[8][4];
  {
    const uint32_t* q = reinterpret_cast<const uint32_t*>(batch.q[li]) +
                        (static_cast<size_t>(ub) * Hq + static_cast<size_t>(uh) * G) * (kHeadDim / 2);
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      qa[kk][0] = (g < G) ? q[g * 64 + kk * 8 + t] : 0u;
      qa[kk][2] = (g < G) ? q[g * 64 + kk * 8 + 4 + t] : 0u;
      if (HI) {
        qa[kk][1] = (g + 8 < G) ? q[(g + 8) * 64 + kk * 8 + t] : 0u;
        qa[kk][3] = (g + 8 < G) ? q[(g + 8) * 64 + kk * 8 + 4 + t] : 0u;
      } else {
        qa[kk][1] = 0u;
        qa[kk][3] = 0u;
      }
    }
  }

  float o[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  bool dead = false;

  // per-lane row roles for the two ldmatrix patterns
  const int mj = lane >> 3, mi = lane & 7;
  const int krow = mi + ((mj >> 1) << 3), kcsel = mj & 1;     // K (B of S = Q K^T): tokens x d-pieces
  const int vrow = mi + ((mj & 1) << 3), vcsel = mj >> 1;     // V (B of O = P V), transposed load

  for (int it = 0; it < n_my; ++it) {
    const int stage = it % kDecStages;
    uint8_t* st = ring + stage * kStageBytes;
    const int v0 = (first + it * kDecWarps) * kTile;
    const int nrow = min(kTile, n_valid - v0);
    if (!mbar_wait_bounded(&bars[stage], (it / kDecStages) & 1)) {
      if (lane == 0) { atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT); err[1] = kErrDecodeWait; }
      dead = true;
      break;
    }
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(st + 2 * kTile * kRowBytes);
    if (nrow < kTile) {
      // rows past the end were not copied: clear them so that stale bits cannot poison P*V
      for (int r = nrow; r < kTile; ++r) {
        reinterpret_cast<uint2*>(st + r * kRowBytes)[lane] = make_uint2(0u, 0u);
        reinterpret_cast<uint2*>(st + kTile * kRowBytes + r * kRowBytes)[lane] = make_uint2(0u, 0u);
      }
      __syncwarp();
    }
    const uint32_t kbase = smem_u32(st), vbase = kbase + kTile * kRowBytes;

    float s[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
      const int r = sl * 16 + krow;
      const uint32_t key = keys[r];
      const uint32_t rowaddr = kbase + r * kRowBytes;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(b0, b1, b2, b3, rowaddr + (((2 * kk + kcsel) ^ key) << 4));
        mma_bf16(s[2 * sl], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
        mma_bf16(s[2 * sl + 1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b2, b3);
      }
    }

    // online softmax over the tile (rows g and, for large groups, g + 8)
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const bool ok = (j * 8 + 2 * t + e) < nrow;
        s[j][e] = ok ? s[j][e] * sc : -INFINITY;
        mx0 = fmaxf(mx0, s[j][e]);
        if (HI) {
          s[j][2 + e] = ok ? s[j][2 + e] * sc : -INFINITY;
          mx1 = fmaxf(mx1, s[j][2 + e]);
        }
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    const float mn0 = fmaxf(m0, mx0);
    const float c0 = exp2f(m0 - mn0);
    m0 = mn0;
    float c1 = 1.f;
    if (HI) {
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn1 = fmaxf(m1, mx1);
      c1 = exp2f(m1 - mn1);
      m1 = mn1;
    }
    float ps0 = 0.f, ps1 = 0.f;
    uint32_t pa[2][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float p0 = exp2f(s[j][0] - m0), p1 = exp2f(s[j][1] - m0);
      ps0 += p0 + p1;
      pa[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
      if (HI) {
        const float p2 = exp2f(s[j][2] - m1), p3 = exp2f(s[j][3] - m1);
        ps1 += p2 + p3;
        pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
      } else {
        pa[j >> 1][(j & 1) * 2 + 1] = 0u;
      }
    }
    l0 = l0 * c0 + ps0;
    if (HI) l1 = l1 * c1 + ps1;
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      o[n][0] *= c0;
      o[n][1] *= c0;
      if (HI) { o[n][2] *= c1; o[n][3] *= c1; }
    }

#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
      const int r = sl * 16 + vrow;
      const uint32_t key = keys[r];
      const uint32_t rowaddr = vbase + r * kRowBytes;
#pragma unroll
      for (int np = 0; np < 8; ++np) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_trans(b0, b1, b2, b3, rowaddr + (((2 * np + vcsel) ^ key) << 4));
        mma_bf16(o[2 * np], pa[sl][0], pa[sl][1], pa[sl][2], pa[sl][3], b0, b1);
        mma_bf16(o[2 * np + 1], pa[sl][0], pa[sl][1], pa[sl][2], pa[sl][3], b2, b3);
      }
    }
    __syncwarp();
    if (it + kDecStages < n_my) issue(it + kDecStages);
  }

  if (dead) {
    // leave only after our own copies in flight had another bounded chance to land
    for (int s2 = 0; s2 < kDecStages; ++s2) {
      for (int it = 0; it < 1024 && !mbar_try_wait(&bars[s2], 0) && !mbar_try_wait(&bars[s2], 1); ++it) {}
    }
  }

  // ---- merge the warps of this CTA ----
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  if (HI) {
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }
  // each warp parks (m, l, O) in its own (now idle) ring: [16][128] floats, then m[16], l[16]
  float* wo = reinterpret_cast<float*>(ring);
  float* wm = wo + 16 * kHeadDim;
  float* wl = wm + 16;
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    *reinterpret_cast<float2*>(&wo[g * kHeadDim + n * 8 + 2 * t]) = make_float2(o[n][0], o[n][1]);
    if (HI) *reinterpret_cast<float2*>(&wo[(g + 8) * kHeadDim + n * 8 + 2 * t]) = make_float2(o[n][2], o[n][3]);
  }
  if (t == 0) {
    wm[g] = m0; wl[g] = l0;
    wm[g + 8] = HI ? m1 : -INFINITY;
    wl[g + 8] = HI ? l1 : 0.f;
  }
  __syncthreads();

  const int d = threadIdx.x;   // blockDim.x == kHeadDim
  const size_t pstride = static_cast<size_t>(G) * (kHeadDim + 2);
  float* partials = reinterpret_cast<float*>(base + hdr->partials_off);
  float* mypart = partials + (static_cast<size_t>(up->split_base) + sp.slot) * pstride;
  const size_t out_row0 = static_cast<size_t>(ub) * Hq + static_cast<size_t>(uh) * G;
  for (int row = 0; row < G; ++row) {
    float M = -INFINITY;
#pragma unroll
    for (int w2 = 0; w2 < kDecWarps; ++w2)
      M = fmaxf(M, reinterpret_cast<const float*>(smem + w2 * (kDecStages * kStageBytes))[16 * kHeadDim + row]);
    float acc = 0.f, L = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w2 = 0; w2 < kDecWarps; ++w2) {
        const float* po = reinterpret_cast<const float*>(smem + w2 * (kDecStages * kStageBytes));
        const float f = exp2f(po[16 * kHeadDim + row] - M);
        acc += po[row * kHeadDim + d] * f;
        L += po[16 * kHeadDim + 16 + row] * f;
      }
    }
    if (n_splits == 1) {
      const float r = (L > 0.f && !dead) ? acc / L : 0.f;
      if (out_f32) reinterpret_cast<float*>(batch.out[li])[(out_row0 + row) * kHeadDim + d] = r;
      else reinterpret_cast<__nv_bfloat16*>(batch.out[li])[(out_row0 + row) * kHeadDim + d] = __float2bfloat16_rn(r);
    } else {
      mypart[row * kHeadDim + d] = acc;
      if (d == 0) { mypart[G * kHeadDim + row] = M; mypart[G * kHeadDim + G + row] = L; }
    }
  }
  if (n_splits == 1) return;

  // ---- the last split of the unit to arrive merges all of them, in split order ----
  int32_t* counter = reinterpret_cast<int32_t*>(base + hdr->counters_off) + sp.unit;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(counter, 1);
    s_is_last = (prev == n_splits - 1);
  }
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();
  const float* up_part = partials + static_cast<size_t>(up->split_base) * pstride;
  for (int row = 0; row < G; ++row) {
    float M = -INFINITY;
    for (int s2 = 0; s2 < n_splits; ++s2) M = fmaxf(M, __ldcg(&up_part[s2 * pstride + G * kHeadDim + row]));
    float acc = 0.f, L = 0.f;
    if (M > -INFINITY) {
      for (int s2 = 0; s2 < n_splits; ++s2) {
        const float* p = up_part + s2 * pstride;
        const float f = exp2f(__ldcg(&p[G * kHeadDim + row]) - M);
        acc += __ldcg(&p[row * kHeadDim + d]) * f;
        L += __ldcg(&p[G * kHeadDim + G + row]) * f;
      }
    }
    const float r = L > 0.f ? acc / L : 0.f;
    if (out_f32) reinterpret_cast<float*>(batch.out[li])[(out_row0 + row) * kHeadDim + d] = r;
    else reinterpret_cast<__nv_bfloat16*>(batch.out[li])[(out_row0 + row) * kHeadDim + d] = __float2bfloat16_rn(r);
  }
  if (threadIdx.x == 0) *counter = 0;   // ready for the next step
}

}  // namespace

size_t flash_decode_smem_bytes() {
  return static_cast<size_t>(kDecWarps) * kDecStages * kStageBytes + kDecWarps * kDecStages * sizeof(uint64_t);
}

cudaError_t launch_select_chunks(const DecodeBatch& batch, int total_dyn, cudaStream_t stream) {
  if (total_dyn <= 0) return cudaSuccess;
  select_chunks_kernel<<<total_dyn, kSelThreads, 0, stream>>>(batch);
  return cudaGetLastError();
}

cudaError_t launch_flash_decode(const DecodeBatch& batch, int total_splits, int group, bool out_f32,
                                cudaStream_t stream) {
  if (total_splits <= 0) return cudaSuccess;
  const size_t smem = flash_decode_smem_bytes();
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(flash_decode_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(flash_decode_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  if (group > 8)
    flash_decode_kernel<true><<<total_splits, kDecWarps * 32, smem, stream>>>(batch, out_f32 ? 1 : 0);
  else
    flash_decode_kernel<false><<<total_splits, kDecWarps * 32, smem, stream>>>(batch, out_f32 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace hkv
