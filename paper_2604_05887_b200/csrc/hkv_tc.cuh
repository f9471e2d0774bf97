// Fifth-generation tensor-core path (tcgen05, accumulators in tensor memory) for the two dense
// contractions of the library: the observation-window scores S_w of the static heads and the
// text-centric attention rows of the head classification.  Both are "queries x keys^T" with
// head_dim 128: a block of up to 256 query rows stays in shared memory, 128-key tiles stream through
// a ring of stages, every tile is one complete accumulation (K = 128 = 8 instructions of K = 16).
//
// Operands are bf16, K-major, in the 128-byte-swizzled canonical layout of the matrix descriptors:
// a row's 128 elements are split into two halves of 64 (128 bytes); each half-plane is
// [row][128 B] with the eight 16-byte pieces of a row XOR-permuted by (row & 7); planes are 1024-byte
// aligned.  Shared-memory descriptor: start address >> 4 in bits 0..13, leading byte offset (unused
// for swizzled K-major, set to 1) in bits 16..29, stride byte offset (1024 B between 8-row groups)
// >> 4 in bits 32..45, descriptor version 1 in bits 46..47, layout type 2 (128-byte swizzle) in
// bits 61..63.  Instruction descriptor (kind::f16): D format f32 (1) in bits 4..5, A and B format
// bf16 (1) in bits 7..9 and 10..12, both K-major (bits 15, 16 clear), N >> 3 in bits 17..22, M >> 4
// in bits 24..28.  An M = 128 accumulator puts row i in tensor-memory lane i and column j in column
// base + j; warp w of the CTA may read lanes 32 * (w % 4) .. + 31.
#pragma once
#include "hkv_device.cuh"

namespace hkv {
namespace tc {

constexpr int kKeysPerTile = 128;                   // keys of one streamed tile
constexpr int kQRows = 256;                         // query rows resident per CTA (two M = 128 blocks)
constexpr int kPlaneBytesK = kKeysPerTile * 128;    // one 64-element half of a key tile
constexpr int kPlaneBytesQ = kQRows * 128;
constexpr int kStageBytes = 2 * kPlaneBytesK;       // 32 KB
constexpr int kQBytes = 2 * kPlaneBytesQ;           // 64 KB
constexpr int kStages = 3;
constexpr int kLoadLag = 2;                         // key tiles in flight per CTA
constexpr int kTmemCols = 512;                      // two accumulator buffers of 256 columns
constexpr int kDrainWarps = 16;                     // four per lane quarter, 64 accumulator columns each
constexpr int kThreads = (2 + kDrainWarps) * 32;    // warp 0 loads, warp 1 issues, warps 2..17 drain
constexpr int kBarBytes = 256;
constexpr int kScratchPerWarp = 2048;               // 32 x 16 floats a draining warp may use to reorder its output
constexpr int kSmemBytes =
    kQBytes + kStages * kStageBytes + kDrainWarps * kScratchPerWarp + kBarBytes + 1024;   // + slack to align to 1024

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async16_addr(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, one thread issues
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the barrier gets one arrival once every tensor-core instruction issued so far by this thread is done
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 lanes x 32 consecutive columns: thread i of the warp gets lane (base lane + i), r[j] = column base + j.
// The registers hold the values only after tmem_ld_wait(r), which also ties them to the wait for the compiler.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]),
                 "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]),
                 "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// The two 32-column groups of a draining thread's 64 columns, the read of the second in flight while
// fn(0, v) works on the first.  Whole warps call it.
template <class Fn>
__device__ __forceinline__ void drain_groups(uint32_t taddr, Fn fn) {
  uint32_t ra[32], rb[32];
  float v[32];
  tmem_ld32_issue(taddr, ra);
  tmem_ld_wait(ra);
  tmem_ld32_issue(taddr + 32u, rb);
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(ra[i]);
  fn(0, v);
  tmem_ld_wait(rb);
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(rb[i]);
  fn(1, v);
}

__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
template <int M, int N>
struct InstrDesc {
  static constexpr uint32_t value = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
                                    (static_cast<uint32_t>(M >> 4) << 24);
};

// One 16-byte piece of row `row` (piece 0..15 of its 256 bytes) inside a two-plane operand block.
__device__ __forceinline__ uint32_t piece_offset(int row, int piece, int plane_bytes) {
  return static_cast<uint32_t>((piece >> 3) * plane_bytes + row * 128 + (((piece & 7) ^ (row & 7)) << 4));
}

// ---------------------------------------------------------------------------------------------
// The CTA-wide engine.  All kThreads threads call it with the same arguments.
//   smem_raw    dynamic shared memory (kSmemBytes)
//   q_row       functor: row 0..kQRows-1 -> pointer to the row's 128 bf16, or nullptr for a zero row
//   keys        bf16 [C][128] of the head; tiles [tile_begin, tile_end) of 128 keys are processed
//   kKeysAsRows false: accumulator rows = query rows (two M = 128 blocks side by side, block t in
//               columns 128 t .. 128 t + 127 = the tile's keys); true: accumulator rows = the tile's keys,
//               columns = the 256 query rows
//   epilogue    functor called by each of the 512 draining threads for every tile:
//               epilogue(tile, lane 0..127, part 0..3, groups, scratch, siblings, pair_bar): the thread owns
//               accumulator lane `lane`, columns 64 part .. 64 part + 63; groups(fn) calls fn(g, v) for
//               g = 0, 1 with its columns 64 part + 32 g .. + 31 in float v[32] and must be called by whole
//               warps (or not at all); scratch is the warp's 2 KB of shared memory; siblings(p) is the
//               scratch of the warp that owns part p of the same lanes; pair_bar is a barrier (96 arrivals per
//               phase; one for the even and one for the odd tiles of the CTA, so its k-th use has parity
//               k & 1) the warps of parts 1..3 may use to hand data to the part-0 warp: the two accumulator
//               buffers keep the warps within one tile of each other, so a phase is never met twice
// Returns false if a bounded wait ran out (the caller reports it); tensor memory is freed either way.
// ---------------------------------------------------------------------------------------------
template <bool kKeysAsRows, class QRowFn, class Epilogue>
__device__ bool scores_cta(uint8_t* smem_raw, QRowFn q_row, const __nv_bfloat16* keys, int C, int tile_begin,
                           int tile_end, Epilogue epilogue) {
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // operand planes are 1024-byte aligned
  uint8_t* qs = smem;
  uint8_t* ks = smem + kQBytes;
  uint8_t* scratch = ks + kStages * kStageBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(scratch + kDrainWarps * kScratchPerWarp);
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* pair_bar = acc_empty + 2;   // [4][2]: per lane quarter, one for even and one for odd tiles
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pair_bar + 8);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_tiles = tile_end - tile_begin;

  // query block -> shared memory (plain loads, four in flight per thread, and stores), barriers, tensor memory
  for (int base = tid; base < kQRows * 16; base += 4 * kThreads) {
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = base + u * kThreads;
      v[u] = make_uint4(0u, 0u, 0u, 0u);
      if (idx < kQRows * 16) {
        const __nv_bfloat16* src = q_row(idx >> 4);
        if (src) v[u] = __ldg(reinterpret_cast<const uint4*>(src) + (idx & 15));
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = base + u * kThreads;
      if (idx < kQRows * 16) *reinterpret_cast<uint4*>(qs + piece_offset(idx >> 4, idx & 15, kPlaneBytesQ)) = v[u];
    }
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full + s, 32);
      mbar_init(empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full + b, 1);
      mbar_init(acc_empty + b, kDrainWarps * 32);
    }
    for (int q = 0; q < 8; ++q) mbar_init(pair_bar + q, 96);
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  fence_proxy_async();   // the query block was written by ordinary stores, the tensor core reads it
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  bool ok = true;

  if (warp == 0) {
    // ---- loader: 16-byte asynchronous copies, kLoadLag tiles ahead of the tile handed over ----
    uint32_t ld_dst[4];
    int ld_src[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int row = 2 * u + (lane >> 4), piece = lane & 15;
      ld_dst[u] = piece_offset(row, piece, kPlaneBytesK);
      ld_src[u] = row * 256 + piece * 16;
    }
    for (int i = 0; i < n_tiles + kLoadLag; ++i) {
      if (i < n_tiles) {
        const int s = i % kStages;
        if (i >= kStages && !mbar_wait_bounded(empty + s, ((i / kStages) - 1) & 1)) { ok = false; break; }
        uint8_t* dst = ks + s * kStageBytes;
        const int j0 = (tile_begin + i) * kKeysPerTile;
        if (j0 + kKeysPerTile <= C) {
          // a whole tile: lane = (row parity r0, piece); rows 8 it + 2 u + r0, so the swizzle depends on u only
          const uint32_t dbase = smem_u32(dst);
          const char* sbase = reinterpret_cast<const char*>(keys + static_cast<size_t>(j0) * 128);
#pragma unroll 4
          for (int it = 0; it < kKeysPerTile / 8; ++it) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
              cp_async16_addr(dbase + ld_dst[u] + static_cast<uint32_t>(it * 1024), sbase + ld_src[u] + it * 2048);
          }
        } else {
#pragma unroll 4
          for (int it = 0; it < kKeysPerTile * 16 / 32; ++it) {
            const int p = it * 32 + lane, row = p >> 4, piece = p & 15;
            const bool in = j0 + row < C;
            const __nv_bfloat16* src = keys + static_cast<size_t>(in ? j0 + row : 0) * 128 + piece * 8;
            cp_async16(dst + piece_offset(row, piece, kPlaneBytesK), src, in ? 16u : 0u);
          }
        }
      }
      cp_async_commit();
      if (i >= kLoadLag) {
        cp_async_wait<kLoadLag>();
        fence_proxy_async();
        mbar_arrive(full + (i - kLoadLag) % kStages);
      }
    }
    cp_async_wait<0>();
    // the last instructions' arrivals on the `empty` barriers must land before the CTA may leave
    for (int i = max(0, n_tiles - kStages); ok && i < n_tiles; ++i)
      if (!mbar_wait_bounded(empty + i % kStages, (i / kStages) & 1)) ok = false;
  } else if (warp == 1) {
    // ---- issuer: one thread feeds the tensor core ----
    constexpr uint32_t idesc = kKeysAsRows ? InstrDesc<128, 256>::value : InstrDesc<128, 128>::value;
    const uint32_t q_addr = smem_u32(qs);
    for (int i = 0; i < n_tiles; ++i) {
      const int s = i % kStages, buf = i & 1;
      if (i >= 2 && !mbar_wait_bounded(acc_empty + buf, ((i >> 1) - 1) & 1)) { ok = false; break; }
      if (!mbar_wait_bounded(full + s, (i / kStages) & 1)) { ok = false; break; }
      fence_after_sync();
      if (lane == 0) {
        const uint32_t k_addr = smem_u32(ks + s * kStageBytes);
        const uint32_t d = tmem_base + static_cast<uint32_t>(buf * 256);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {   // K = 16 elements = 32 bytes per instruction; 4 per half-plane
          const uint32_t koff = static_cast<uint32_t>((kk >> 2) * kPlaneBytesK + (kk & 3) * 32);
          const uint32_t qoff = static_cast<uint32_t>((kk >> 2) * kPlaneBytesQ + (kk & 3) * 32);
          if (kKeysAsRows) {
            umma_bf16(d, smem_desc(k_addr + koff), smem_desc(q_addr + qoff), idesc, kk != 0);
          } else {
            umma_bf16(d, smem_desc(q_addr + qoff), smem_desc(k_addr + koff), idesc, kk != 0);
            umma_bf16(d + 128u, smem_desc(q_addr + qoff + 128u * 128u), smem_desc(k_addr + koff), idesc, kk != 0);
          }
        }
        umma_commit(empty + s);        // the stage may be refilled once these instructions have read it
        umma_commit(acc_full + buf);   // and the accumulator is complete
      }
      __syncwarp();
    }
  } else {
    // ---- drain: warp w owns lane quarter w % 4 (the hardware's rule) and column part (w - 2) / 4 ----
    const int quarter = warp & 3, part = (warp - 2) >> 2, slot = (warp - 2) & 3;
    const int row = quarter * 32 + lane;
    for (int i = 0; i < n_tiles; ++i) {
      const int buf = i & 1;
      if (!mbar_wait_bounded(acc_full + buf, (i >> 1) & 1)) { ok = false; break; }
      fence_after_sync();
      const uint32_t taddr =
          tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * 256 + part * 64);
      epilogue(tile_begin + i, row, part, [&](auto fn) { drain_groups(taddr, fn); },
               reinterpret_cast<float*>(scratch + (warp - 2) * kScratchPerWarp),
               [&](int p) { return reinterpret_cast<float*>(scratch + (p * 4 + slot) * kScratchPerWarp); },
               pair_bar + 2 * quarter + (i & 1));
      fence_before_sync();
      mbar_arrive(acc_empty + buf);
    }
  }
  // a failed wait leaves copies or instructions possibly in flight: give them the time of one more bounded wait
  const bool all_ok = !__syncthreads_or(!ok);
  fence_after_sync();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
  return all_ok;
}

}  // namespace tc
}  // namespace hkv
