// Device-side helpers shared by the kernels of libhkv: PTX wrappers (mbarrier, bulk copy, ldmatrix,
// mma), the order-preserving float key, and a block-wide exact top-k selection that emits ascending
// indices.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace hkv {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier + bulk async copy (TMA engine, 1-D, no multicast) ----
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Limit of every device-side wait, in SM clocks (about a second at full clock).
#ifndef HKV_WAIT_CYCLES
#define HKV_WAIT_CYCLES 2000000000ll
#endif
// Bounded wait: returns false when the limit ran out; the caller records an error and leaves
// instead of spinning for ever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0u && clock64() - start > HKV_WAIT_CYCLES) return false;
  }
}
// The same wait with acquire semantics at cluster scope: for barriers whose bytes are delivered by
// other CTAs of the cluster (st.async below).
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long start = clock64();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((it & 255u) == 0u && clock64() - start > HKV_WAIT_CYCLES) return false;
  }
}
// global -> shared bulk copy; src, dst 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// asks the L2 cache to fetch [src, src + bytes) from HBM; nothing is written to shared memory and
// nothing has to be waited for.  src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// ---- tensor-core tile ops (warp-level mma on 16x8x16 bf16 tiles, fp32 accumulate) ----
__device__ __forceinline__ void ldsm_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                              uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// transposes an 8x8 matrix of 16-bit elements held in the usual fragment layout (thread 4g+t owns
// row g, columns 2t and 2t+1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// ---- thread-block cluster: rank, barrier, distributed shared memory ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
// arrival that orders no memory operations (a pure "I got here" signal: no fence, no stall on stores in flight)
__device__ __forceinline__ void cluster_arrive_relaxed() {
  asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// address of the same shared-memory location in the CTA of rank `rank` of this cluster
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x2(uint32_t addr, float x, float y) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ void st_cluster_f32x4(uint32_t addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}
// Asynchronous stores into the shared memory of a CTA of the cluster (addr, bar: shared::cluster addresses
// of the SAME destination CTA, from mapa): the value is written and its byte count is credited to the
// destination's mbarrier, whose waiters then see the data.  No cluster barrier is involved.
__device__ __forceinline__ void st_async_f32x4(uint32_t addr, float4 v, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void st_async_f32x2(uint32_t addr, float x, float y, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(addr),
               "f"(x), "f"(y), "r"(bar)
               : "memory");
}
// asks L2 for the 128-byte line holding p (nothing is read into the SM, nothing to wait for)
__device__ __forceinline__ void prefetch_l2_line(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p) : "memory");
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f32x2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}

// ---- division by a divisor that is fixed for the whole kernel (chunk size, cluster size): the multiplier is
// computed once, off the critical path, and x / d becomes one multiply-high.  Exact while x * d < 2^32, d > 1.
__device__ __forceinline__ uint32_t fastdiv_magic(uint32_t d) { return 0xFFFFFFFFu / d + 1u; }
__device__ __forceinline__ int fastdiv(int x, uint32_t magic) { return static_cast<int>(__umulhi(static_cast<uint32_t>(x), magic)); }

// ---- order-preserving key of a finite float: larger float <=> larger key; every key > 0 ----
__device__ __forceinline__ uint32_t float_key(float f) {
  f = f + 0.0f;   // -0 -> +0 so that equal floats have equal keys
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---------------------------------------------------------------------------------------------
// Block-wide exact selection.  Among the n items, every item with always(i) is emitted, and of the
// items with key(i) != 0 ("candidates") the k with the largest keys are emitted, equal keys going
// to the lower index.  Emission is in ascending index order: emit(position, index) is called once
// per selected item; returns the number emitted (valid in every thread).  Requires k <= number of
// candidates, blockDim.x a multiple of 32 and at most 1024.  hist: 256 ints, wsum: 3*32 ints,
// bc: 4 ints of shared memory.
// ---------------------------------------------------------------------------------------------
template <class KeyFn, class AlwaysFn, class EmitFn>
__device__ int block_select_emit(int n, int k, KeyFn key, AlwaysFn always, EmitFn emit, int* hist, int* wsum,
                                 int* bc) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
  uint32_t prefix = 0, mask = 0;
  int need = k;   // how many still to take among the keys matching the prefix
  if (k > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = tid; i < 256; i += nthr) hist[i] = 0;
      __syncthreads();
      for (int i = tid; i < n; i += nthr) {
        uint32_t kv = key(i);
        if (kv != 0 && (kv & mask) == prefix) atomicAdd(&hist[(kv >> shift) & 255], 1);
      }
      __syncthreads();
      if (warp == 0) {
        // lane L owns bins [8L, 8L+8); find the highest bin b with count(bins > b) < need <= count(bins >= b)
        int loc[8], tot = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { loc[j] = hist[lane * 8 + j]; tot += loc[j]; }
        int above = 0;   // total of lanes above this one
        int run = tot;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          int v = __shfl_down_sync(0xffffffffu, run, off);
          if (lane + off < 32) run += v;
        }
        above = run - tot;   // sum over lanes > lane
        if (above < need && need <= above + tot) {
          int acc = above;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (acc < need && need <= acc + loc[j]) { bc[0] = lane * 8 + j; bc[1] = need - acc; }
            acc += loc[j];
          }
        }
      }
      __syncthreads();
      prefix |= static_cast<uint32_t>(bc[0]) << shift;
      mask |= 0xFFu << shift;
      need = bc[1];
      __syncthreads();
    }
  }
  const uint32_t T = (k > 0) ? prefix : 0xFFFFFFFFu;
  if (k <= 0) need = 0;
  // ordered emission
  int emitted = 0, eq_seen = 0;
  for (int base = 0; base < n; base += nthr) {
    const int i = base + tid;
    bool gt = false, eq = false, alw = false;
    if (i < n) {
      uint32_t kv = key(i);
      alw = always(i);
      gt = (kv != 0) && (kv > T);
      eq = (kv != 0) && (kv == T);
    }
    const uint32_t beq = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) wsum[warp] = __popc(beq);
    __syncthreads();
    int eq_before = eq_seen, eq_total = 0;
    for (int w2 = 0; w2 < nwarp; ++w2) {
      int c = wsum[w2];
      if (w2 < warp) eq_before += c;
      eq_total += c;
    }
    const int my_eq_rank = eq_before + __popc(beq & ((1u << lane) - 1u));
    const bool sel = alw || gt || (eq && my_eq_rank < need);
    const uint32_t bsel = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) wsum[32 + warp] = __popc(bsel);
    __syncthreads();
    int sel_before = emitted, sel_total = 0;
    for (int w2 = 0; w2 < nwarp; ++w2) {
      int c = wsum[32 + w2];
      if (w2 < warp) sel_before += c;
      sel_total += c;
    }
    if (sel) emit(sel_before + __popc(bsel & ((1u << lane) - 1u)), i);
    emitted += sel_total;
    eq_seen += eq_total;
    __syncthreads();
  }
  return emitted;
}

// 2^x by the hardware approximation (relative error about 2^-22; -inf -> 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------------------------------------
// Block-wide exact top-k over finite float scores held in shared memory (the decode step's chunk
// selection).  Selects the k largest of scores[0..n), equal scores going to the lower index, and
// calls emit(position, index) in ascending index order; returns the number selected (= k).
// Requires 1 <= k < n, blockDim.x = 32 * NWARPS.  scratch: kTopkScratchInts ints of shared memory.
// Contains block barriers: every thread of the block must call it.
//
// One histogram pass over 256 equal-width value bins between the block's min and max score (the
// map score -> bin is monotone, so every score in a higher bin is larger); the few scores that
// share the bin of the k-th are then ranked exactly against each other (key, then index), which
// yields the exact threshold element; one ordered compaction emits the result.  When that bin
// holds more scores than the block has threads (many equal scores), the byte-wise radix
// selection above takes over.
// ---------------------------------------------------------------------------------------------
constexpr int kTopkScratchInts = 256 + 2 * 256 + 16 + 64 + 96 + 4;
template <int NWARPS, class EmitFn>
__device__ int block_topk_smem(const float* scores, int n, int k, EmitFn emit, int* scratch) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NTHR = NWARPS * 32;
  int* hist = scratch;                               // [256]
  uint32_t* cand = reinterpret_cast<uint32_t*>(scratch + 256);   // [NTHR][2]: key, index
  int* misc = scratch + 256 + 2 * 256;               // [0] candidates gathered, [1..2] threshold key / index
  float* red = reinterpret_cast<float*>(misc + 16);  // [NWARPS][2] min / max per warp, then [NWARPS][2] counts
  int* wsum = misc + 16 + 64;
  int* bc = wsum + 96;

  float lo = INFINITY, hi = -INFINITY;
  for (int i = tid; i < n; i += NTHR) { const float v = scores[i]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
  }
  if (lane == 0) { red[2 * warp] = lo; red[2 * warp + 1] = hi; }
  for (int i = tid; i < 256; i += NTHR) hist[i] = 0;
  if (tid == 0) misc[0] = 0;
  __syncthreads();
#pragma unroll
  for (int w2 = 0; w2 < NWARPS; ++w2) { lo = fminf(lo, red[2 * w2]); hi = fmaxf(hi, red[2 * w2 + 1]); }
  const float width = hi - lo;
  const float scale = (width > 0.f && width < INFINITY) ? 255.0f / width : 0.f;
  auto bin_of = [&](float v) { return max(0, min(255, __float2int_rd((v - lo) * scale))); };
  for (int i = tid; i < n; i += NTHR) atomicAdd(&hist[bin_of(scores[i])], 1);
  __syncthreads();

  // every warp: the highest bin b with count(bins > b) < k <= count(bins >= b)
  int tbin, need, cnt;
  {
    const int4 v0 = reinterpret_cast<const int4*>(hist)[lane * 2], v1 = reinterpret_cast<const int4*>(hist)[lane * 2 + 1];
    const int loc[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    int tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) tot += loc[j];
    int run = tot;   // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, run, off);
      if (lane + off < 32) run += v;
    }
    const int above = run - tot;
    const bool mine = above < k && k <= above + tot;
    int my_bin = 0, my_need = 0, my_cnt = 0;
    if (mine) {
      int acc = above;
#pragma unroll
      for (int j = 7; j >= 0; --j) {
        if (acc < k && k <= acc + loc[j]) { my_bin = lane * 8 + j; my_need = k - acc; my_cnt = loc[j]; }
        acc += loc[j];
      }
    }
    const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
    tbin = __shfl_sync(0xffffffffu, my_bin, src);
    need = __shfl_sync(0xffffffffu, my_need, src);
    cnt = __shfl_sync(0xffffffffu, my_cnt, src);
  }
  if (cnt > NTHR) {
    return block_select_emit(
        n, k, [&](int i) { return float_key(scores[i]); }, [](int) { return false; }, emit, hist, wsum, bc);
  }
  // the scores of the threshold bin, ranked exactly: key descending, index ascending
  for (int i = tid; i < n; i += NTHR) {
    const float v = scores[i];
    if (bin_of(v) == tbin) {
      const int slot = atomicAdd(&misc[0], 1);
      cand[2 * slot] = float_key(v);
      cand[2 * slot + 1] = static_cast<uint32_t>(i);
    }
  }
  __syncthreads();
  if (tid < cnt) {
    const uint32_t mk = cand[2 * tid], mi = cand[2 * tid + 1];
    int rank = 0;
    for (int j = 0; j < cnt; ++j) {
      const uint32_t ok = cand[2 * j], oi = cand[2 * j + 1];
      rank += (ok > mk) || (ok == mk && oi < mi);
    }
    if (rank == need - 1) { misc[1] = static_cast<int>(mk); misc[2] = static_cast<int>(mi); }
  }
  __syncthreads();
  const uint32_t tkey = static_cast<uint32_t>(misc[1]);
  const int tidx = misc[2];
  auto taken = [&](int i) {
    const uint32_t kv = float_key(scores[i]);
    return kv > tkey || (kv == tkey && i <= tidx);
  };
  // ordered emission: warp w owns items [w * per, (w + 1) * per), per a multiple of 32
  const int per = ((n + NWARPS - 1) / NWARPS + 31) & ~31;
  const int beg = warp * per, end = min(n, beg + per);
  int mine_n = 0;
  for (int i0 = beg; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    mine_n += __popc(__ballot_sync(0xffffffffu, i < end && taken(i)));
  }
  int* wtot = reinterpret_cast<int*>(red) + 2 * NWARPS;
  if (lane == 0) wtot[warp] = mine_n;
  __syncthreads();
  int before = 0, total = 0;
#pragma unroll
  for (int w2 = 0; w2 < NWARPS; ++w2) {
    const int a = wtot[w2];
    if (w2 < warp) before += a;
    total += a;
  }
  const uint32_t below = (1u << lane) - 1u;
  for (int i0 = beg; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    const bool sel = i < end && taken(i);
    const uint32_t b = __ballot_sync(0xffffffffu, sel);
    if (sel) emit(before + __popc(b & below), i);
    before += __popc(b);
  }
  return total;
}

// ---------------------------------------------------------------------------------------------
// The decode step's fast path of the same selection: exact top-k over at most 256 * IPT finite float
// scores in shared memory, three block barriers in all.  Thread t owns the IPT consecutive scores
// [t * IPT, (t + 1) * IPT) in registers, so that the ascending output order is the thread order.
//   1. every thread bins its scores into NB (256 or 512) equal-width value bins between lo and hi (lower and
//      upper bound of the scores, known to the caller) with shared-memory atomics        -> barrier
//   2. every warp finds, redundantly, the bin of the k-th largest score; the scores of that bin are
//      gathered as (key, index) candidates, and each warp publishes how many of its scores lie in
//      higher bins                                                                          -> barrier
//   3. every warp ranks the candidates (at most 32) exactly by (key, index), which gives the
//      threshold element and, for every warp, how many selected items precede its own; one warp scan
//      places each selected index                                                           -> barrier
// early(i) is called, by the thread that owns score i, for every score above the threshold bin as soon
// as that bin is known (most of the selection, well before the list exists).  stamp(0..3) is called
// after the first barrier, the bin search, the second barrier and the ranking (profiling builds).
// Returns k, or -1 without having written anything when the threshold bin holds more than 32 scores
// (many near-equal scores): the caller then runs block_topk_smem.  The decision is the same in
// every thread.  Requires 1 <= k < n <= 256 * IPT, n_pad = n rounded up to a multiple of 16 readable
// floats, blockDim.x = 32 * NWARPS with 256 * IPT >= n.  hist: NB ints ZEROED by the caller, cand: 32 x (key, index), misc: 1 + NWARPS
// ints with misc[0] ZEROED by the caller.
// ---------------------------------------------------------------------------------------------
template <int NWARPS, int IPT, int NB, class EarlyFn, class StampFn>
__device__ int block_topk_blocked(const float* scores, int n, int n_pad, int k, float lo, float hi, uint16_t* out,
                                  int* hist, uint2* cand, int* misc, EarlyFn early, StampFn stamp) {
  static_assert(IPT == 1 || IPT == 2 || IPT == 4 || IPT == 8, "items per thread");
  static_assert(NB == 256 || NB == 512, "value bins");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int i0 = tid * IPT;
  float v[IPT];
  if (i0 < n_pad) {
    if constexpr (IPT == 1) {
      v[0] = scores[i0];
    } else if constexpr (IPT == 2) {
      const float2 x = *reinterpret_cast<const float2*>(scores + i0);
      v[0] = x.x; v[1] = x.y;
    } else {
#pragma unroll
      for (int q = 0; q < IPT / 4; ++q) {
        const float4 x = *reinterpret_cast<const float4*>(scores + i0 + 4 * q);
        v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
      }
    }
  } else {
#pragma unroll
    for (int e = 0; e < IPT; ++e) v[e] = 0.f;
  }
  const float width = hi - lo;
  // the map score -> bin only has to be monotone, so an approximate quotient will do
  const float scale = (width > 0.f && width < INFINITY) ? __fdividef(static_cast<float>(NB - 1), width) : 0.f;
  int bin[IPT];
#pragma unroll
  for (int e = 0; e < IPT; ++e) {
    bin[e] = -1;   // not an item
    if (i0 + e < n) {
      bin[e] = max(0, min(NB - 1, __float2int_rd((v[e] - lo) * scale)));
      atomicAdd(&hist[bin[e]], 1);
    }
  }
  __syncthreads();
  stamp(0);

  // every warp: the highest bin b with count(bins > b) < k <= count(bins >= b)
  int tbin, need, cnt;
  {
    constexpr int PER = NB / 32;   // bins per lane
    int loc[PER];
#pragma unroll
    for (int q = 0; q < PER / 4; ++q) {
      const int4 h = reinterpret_cast<const int4*>(hist)[lane * (PER / 4) + q];
      loc[4 * q] = h.x; loc[4 * q + 1] = h.y; loc[4 * q + 2] = h.z; loc[4 * q + 3] = h.w;
    }
    int tot = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) tot += loc[j];
    int run = tot;   // becomes the sum over lanes >= this one
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int x = __shfl_down_sync(0xffffffffu, run, off);
      if (lane + off < 32) run += x;
    }
    const int above = run - tot;
    const bool mine = above < k && k <= above + tot;
    int my_bin = 0, my_need = 0, my_cnt = 0;
    if (mine) {
      int acc = above;
#pragma unroll
      for (int j = PER - 1; j >= 0; --j) {
        if (acc < k && k <= acc + loc[j]) { my_bin = lane * PER + j; my_need = k - acc; my_cnt = loc[j]; }
        acc += loc[j];
      }
    }
    const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
    tbin = __shfl_sync(0xffffffffu, my_bin, src);
    need = __shfl_sync(0xffffffffu, my_need, src);
    cnt = __shfl_sync(0xffffffffu, my_cnt, src);
  }
  stamp(1);
  if (cnt > 32) return -1;

  int gt = 0;
#pragma unroll
  for (int e = 0; e < IPT; ++e) {
    if (bin[e] > tbin) early(i0 + e);   // selected whatever the ranking below says: the caller may start on it
    gt += bin[e] > tbin;
    if (bin[e] == tbin) {
      const int slot = atomicAdd(&misc[0], 1);
      cand[slot] = make_uint2(float_key(v[e]), static_cast<uint32_t>(i0 + e));
    }
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  if (lane == 0) misc[1 + warp] = gt;
  __syncthreads();
  stamp(2);

  // every warp: exact rank of the candidates, lane j holding candidate j
  const uint2 mine = lane < cnt ? cand[lane] : make_uint2(0u, 0xFFFFFFFFu);
  int rank = 0;
  if (cnt <= 4) {   // the usual case: a handful of scores share the threshold bin
    for (int j = 0; j < cnt; ++j) {
      const uint32_t ok = __shfl_sync(0xffffffffu, mine.x, j), oi = __shfl_sync(0xffffffffu, mine.y, j);
      rank += (ok > mine.x) || (ok == mine.x && oi < mine.y);
    }
  } else {
    for (int j0 = 0; j0 < cnt; j0 += 8) {   // every lane reads the same candidate: broadcast loads, eight in flight
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint2 o = cand[(j0 + j) & 31];
        rank += (j0 + j < cnt) && ((o.x > mine.x) || (o.x == mine.x && o.y < mine.y));
      }
    }
  }
  const bool c_taken = lane < cnt && rank < need;
  const int tsrc = __ffs(__ballot_sync(0xffffffffu, lane < cnt && rank == need - 1)) - 1;
  const uint32_t tkey = __shfl_sync(0xffffffffu, mine.x, tsrc), tidx = __shfl_sync(0xffffffffu, mine.y, tsrc);
  // selected items that precede this warp's: those of higher bins in lower warps, and taken candidates there
  const int owner = static_cast<int>(mine.y / (32u * IPT));
  int before = __popc(__ballot_sync(0xffffffffu, c_taken && owner < warp));
  {
    const int g = (lane < NWARPS && lane < warp) ? misc[1 + lane] : 0;
    before += __reduce_add_sync(0xffffffffu, g);
  }
  stamp(3);
  uint32_t taken = 0u;
#pragma unroll
  for (int e = 0; e < IPT; ++e) {
    bool tk = bin[e] > tbin;
    if (bin[e] == tbin) {
      const uint32_t kv = float_key(v[e]);
      tk = kv > tkey || (kv == tkey && static_cast<uint32_t>(i0 + e) <= tidx);
    }
    taken |= (tk ? 1u : 0u) << e;
  }
  const int c = __popc(taken);
  int incl = c;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += x;
  }
  int pos = before + incl - c;
#pragma unroll
  for (int e = 0; e < IPT; ++e) {
    if ((taken >> e) & 1u) out[pos++] = static_cast<uint16_t>(i0 + e);
  }
  __syncthreads();
  return k;
}

// ---------------------------------------------------------------------------------------------
// Block-wide exact selection over keyed items that need not sit in shared memory (the static
// heads' Top-M visual tokens: tens of thousands of candidates with a heavy-tailed score).  Same
// contract as block_select_emit: items with always(i) are emitted, and of the items with
// key(i) != 0 the k with the largest keys, equal keys going to the lower index; emission in
// ascending index order; returns the number emitted.  Requires k <= number of candidates.
//
// One 1024-bin histogram over (key - min key) >> shift (order-preserving keys of floats are close to
// log-spaced, which suits a heavy tail), exact ranking of the threshold bin's items by (key, index),
// one ordered compaction.  Falls back to the byte-wise radix selection when the threshold bin
// holds more items than the block has threads or when k = 0.
// scratch: kKeyedScratchInts(NTHR) ints of shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int kKeyedBins = 1024;
constexpr int keyed_scratch_ints(int nthr) { return kKeyedBins + 2 * nthr + 8 + 64 + 256 + 96 + 4; }
template <int NTHR, class KeyFn, class AlwaysFn, class EmitFn>
__device__ int block_topk_keyed(int n, int k, KeyFn key, AlwaysFn always, EmitFn emit, int* scratch) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NWARPS = NTHR / 32;
  int* hist = scratch;                                                   // [1024]
  uint32_t* cand = reinterpret_cast<uint32_t*>(scratch + kKeyedBins);   // [NTHR][2]
  int* misc = scratch + kKeyedBins + 2 * NTHR;                           // [0] candidates, [1..2] threshold, [4] min, [5] max
  int* wtot = misc + 8;                                                  // [NWARPS]
  int* fb_hist = wtot + 64;                                              // fallback's scratch
  int* fb_wsum = fb_hist + 256;
  int* fb_bc = fb_wsum + 96;
  if (k <= 0) return block_select_emit(n, k, key, always, emit, fb_hist, fb_wsum, fb_bc);

  for (int i = tid; i < kKeyedBins; i += NTHR) hist[i] = 0;
  if (tid == 0) { misc[0] = 0; misc[4] = -1; misc[5] = 0; }   // min as unsigned: 0xFFFFFFFF
  __syncthreads();
  uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
  for (int i = tid; i < n; i += NTHR) {
    const uint32_t kv = key(i);
    if (kv != 0u) { kmin = min(kmin, kv); kmax = max(kmax, kv); }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) {
    atomicMin(reinterpret_cast<unsigned int*>(&misc[4]), kmin);
    atomicMax(reinterpret_cast<unsigned int*>(&misc[5]), kmax);
  }
  __syncthreads();
  kmin = static_cast<uint32_t>(misc[4]);
  kmax = static_cast<uint32_t>(misc[5]);
  const uint32_t range = kmax - kmin;
  const int shift = max(0, 32 - __clz(range | 1u) - 10);      // (range >> shift) < 1024
  auto bin_of = [&](uint32_t kv) { return static_cast<int>((kv - kmin) >> shift); };
  for (int i = tid; i < n; i += NTHR) {
    const uint32_t kv = key(i);
    if (kv != 0u) atomicAdd(&hist[bin_of(kv)], 1);
  }
  __syncthreads();
  // the highest bin b with count(bins > b) < k <= count(bins >= b): thread t owns bin t, suffix sums by
  // warp shuffles and one exchange of warp totals
  int tbin, need, cnt;
  {
    static_assert(NTHR == kKeyedBins, "one bin per thread");
    const int mine = hist[tid];
    int run = mine;   // becomes the sum over this and the higher lanes of the warp
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, run, off);
      if (lane + off < 32) run += v;
    }
    if (lane == 0) wtot[warp] = run;
    __syncthreads();
    const int wt = wtot[lane];
    int wrun = wt;    // sum over warps >= lane
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, wrun, off);
      if (lane + off < 32) wrun += v;
    }
    const int above = __shfl_sync(0xffffffffu, wrun - wt, warp) + run - mine;
    if (above < k && k <= above + mine) { misc[1] = tid; misc[2] = k - above; misc[3] = mine; }
    __syncthreads();
    tbin = misc[1];
    need = misc[2];
    cnt = misc[3];
    __syncthreads();   // misc[1..2] are reused for the threshold below, wtot for the emission
  }
  if (cnt > NTHR) return block_select_emit(n, k, key, always, emit, fb_hist, fb_wsum, fb_bc);
  for (int i = tid; i < n; i += NTHR) {
    const uint32_t kv = key(i);
    if (kv != 0u && bin_of(kv) == tbin) {
      const int slot = atomicAdd(&misc[0], 1);
      cand[2 * slot] = kv;
      cand[2 * slot + 1] = static_cast<uint32_t>(i);
    }
  }
  __syncthreads();
  if (tid < cnt) {
    const uint32_t mk = cand[2 * tid], mi = cand[2 * tid + 1];
    int rank = 0;
    for (int j = 0; j < cnt; ++j) {
      const uint32_t ok = cand[2 * j], oi = cand[2 * j + 1];
      rank += (ok > mk) || (ok == mk && oi < mi);
    }
    if (rank == need - 1) { misc[1] = static_cast<int>(mk); misc[2] = static_cast<int>(mi); }
  }
  __syncthreads();
  const uint32_t tkey = static_cast<uint32_t>(misc[1]);
  const int tidx = misc[2];
  auto taken = [&](int i) {
    if (always(i)) return true;
    const uint32_t kv = key(i);
    return kv != 0u && (kv > tkey || (kv == tkey && i <= tidx));
  };
  // ordered emission: warp w owns items [w * per, (w + 1) * per), per a multiple of 32.  With at most 32
  // chunks of 32 items per warp, lane c keeps chunk c's ballot from the counting pass for the emitting pass.
  const int per = ((n + NWARPS - 1) / NWARPS + 31) & ~31;
  const int beg = warp * per, end = min(n, beg + per);
  const bool keep = per <= 1024;
  int mine_n = 0;
  uint32_t kept = 0u;
  for (int i0 = beg, c = 0; i0 < end; i0 += 32, ++c) {
    const int i = i0 + lane;
    const uint32_t b = __ballot_sync(0xffffffffu, i < end && taken(i));
    if (lane == c) kept = b;
    mine_n += __popc(b);
  }
  if (lane == 0) wtot[warp] = mine_n;
  __syncthreads();
  int before = 0, total = 0;
  {
    static_assert(NWARPS <= 32, "one lane per warp total");
    const int wt = lane < NWARPS ? wtot[lane] : 0;
    int incl = wt;   // inclusive prefix over warps
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += v;
    }
    before = __shfl_sync(0xffffffffu, incl - wt, warp);
    total = __shfl_sync(0xffffffffu, incl, 31);
  }
  const uint32_t below = (1u << lane) - 1u;
  for (int i0 = beg, c = 0; i0 < end; i0 += 32, ++c) {
    const int i = i0 + lane;
    const uint32_t b = keep ? __shfl_sync(0xffffffffu, kept, c & 31)
                            : __ballot_sync(0xffffffffu, i < end && taken(i));
    if ((b >> lane) & 1u) emit(before + __popc(b & below), i);
    before += __popc(b);
  }
  return total;
}

}  // namespace hkv
