// The decode-step kernel: for every (sequence, kv head) unit, chunk scoring and exact top-k chunk
// selection (dynamic heads), flash-decoding over the unit's retained token list, and the merge of
// the partial results — one launch per layer.
//
// Work decomposition.  A thread-block CLUSTER of `cluster` CTAs owns one unit.  A CTA has a ring of
// kDecStages staging buffers filled by the TMA engine with 1-D bulk copies (no multicast), each
// completing on its own mbarrier; tile j of the CTA lives in stage j % kDecStages and is consumed by
// one of the CTA's W warps (j % W), which then re-arms the stage with tile j + kDecStages.  Because the warp that
// arms a stage is not the warp that consumes it, a consumer first checks the stage's "armed with
// tile" counter and only then waits on the mbarrier's phase parity (parity alone cannot tell a
// phase from the one two later, and a fast warp may get that far ahead).  The footprint is kept
// under half an SM's shared memory so that two CTAs — of this launch or of two consecutive
// launches — are resident per SM.
//
// A decode step is a chain of dependent stages (query -> chunk scores -> selection -> fetch -> attention
// -> merge) and at small batch its latency, not the bytes, sets the time; the cross-CTA hand-overs
// therefore use asynchronous remote stores that complete on the RECEIVER's mbarrier (st.async): the
// receiver waits for exactly the bytes it needs and no cluster-wide barrier sits on the chain.
//
//   dynamic unit, selection:  the cluster's CTAs split the unit's chunk means between them; a warp
//     takes up to 64 staged means and computes  S^T = M Q^T  (rows = chunks, columns = the group's
//     query heads) on tensor cores; the chunk score is the float32 sum over the group's heads.
//     Every score is sent to every CTA of the cluster (16-byte st.async, together with each warp's
//     lower / upper bound of its scores); a CTA whose score barrier has received all bytes runs the
//     same exact selection on its own copy (block_topk_blocked: one value histogram, exact ranking
//     of the threshold bin, three block barriers), so that every CTA knows the ascending list of
//     selected chunks without a round trip through global memory.  Chunks above the threshold bin
//     are requested from HBM into L2 as soon as that bin is known (short lists only).  The lists later calls may ask
//     for (scores, ids, token count) are written to global memory only after the attention's first
//     copies have been issued.
//   every unit, attention:  the unit's token list (static: the compacted rows; dynamic: the rows of
//     the selected chunks) is cut into 32-token tiles, dealt to the cluster's CTAs as contiguous
//     ranges.  Per tile:  S^T = K Q^T  (rows = tokens, columns = query heads, so the group shares
//     every loaded KV tile and no tensor-core row is padding), online softmax in float32 (base-2
//     exponent, accumulators rescaled only when a running maximum moves), P^T moved into operand
//     layout with movmatrix,  O^T += V^T P^T.
//   merge:  the warps of a CTA are combined in shared memory.  Groups up to 8: every CTA then sends
//     each owner CTA its share of (m, l, O) into the owner's idle score area (st.async crediting the
//     owner's merge barrier), and each owner, once its bytes are in, reduces its slice of the output
//     from its own shared memory in CTA-rank order.  Wider groups: the CTAs read each other's
//     partials after a cluster barrier and a second barrier keeps them alive.  Fixed order, no
//     atomics: deterministic.
//
// Programmatic dependent launch.  Nothing the kernel does before griddepcontrol.wait depends on the
// step's query or on an earlier decode launch: it reads the unit table, arms the barriers, has
// the first ring-full of K/V rows (or chunk means) copied in and asks L2 for the query's lines.  A
// launch that follows another decode launch on the stream may therefore start while its predecessor
// is still running; it reads q and writes anything only after the wait.
//
// K/V rows and chunk means live in HBM with their sixteen 16-byte pieces XOR-permuted by (row & 7),
// which makes the ldmatrix reads of a staged tile bank-conflict free without any copy in shared
// memory.
#include <cstring>
#include <mutex>
#include <type_traits>

#include "hkv_device.cuh"
#include "hkv_internal.h"

namespace hkv {

namespace {

// ---- shared memory map of the decode kernel ----
constexpr int kRingBytes = kDecStages * kStageBytes;                 // staging ring
constexpr int kParkStride = kHeadDim + 4;                            // floats per parked output row
constexpr int kParkBytes = 16 * kParkStride * 4 + 128;               // one warp's (O, m, l)
constexpr int kRecvMlOff = 6144;   // inside the score area: (m, l) of every sender and row, after the O slices
static_assert(kMaxCluster * 8 * 8 + kRecvMlOff <= kSelSmemChunks * 4 && 8 * kHeadDim * 4 + 4 * 4 * kMaxCluster <= kRecvMlOff,
              "push-merge receive area fits the score area for groups up to 8");
// A dynamic unit whose CTAs get at most this many tiles each (a short, latency-bound list) asks L2 for the chunks
// it is certain to select while the list is still being built; longer lists are bandwidth-bound and do better
// without the extra requests.
constexpr int kPrefetchMaxTiles = 2 * kDecStages + 2;

constexpr int kMaxWarps = 8;                                         // consumer warps per CTA (8 for groups up to 8, 4 above)
constexpr int part_off(int warps) { return warps * kParkBytes; }    // CTA partial: acc[16][128] f32, (m, l)[16]
constexpr int kPartBytes = kMaxGroup * kHeadDim * 4 + kMaxGroup * 8;
constexpr int kSelOff = kRingBytes;                                  // uint16 ids of the selected chunks
constexpr int kScoresOff = kSelOff + kSelSmemChunks * 2;             // float32 chunk scores; later the merge's receive area
constexpr int kBarsOff = kScoresOff + kSelSmemChunks * 4;            // mbarriers: ring stages, then scores, then merge
constexpr int kScoreBar = kDecStages, kMergeBar = kDecStages + 1;
constexpr int kArmedOff = kBarsOff + (kDecStages + 2) * 8;           // per stage: sequence number of the tile it was last armed with
constexpr int kHistBins = 512;                                       // value bins of the selection (256 used for up to 512 chunks)
constexpr int kHistOff = kArmedOff + kDecStages * 4 + 8;             // selection: histogram
constexpr int kBoundsOff = kHistOff + kHistBins * 4;                       // selection: (lower, upper) score bound of every warp of the cluster
constexpr int kCandOff = kBoundsOff;                                 // selection: 32 candidates (key, index); the bounds are dead by then
constexpr int kMiscOff = kBoundsOff + kMaxCluster * kMaxWarps * 8;   // selection: counters
constexpr int kSmemBytes = kMiscOff + 96;
// the slower selections (crowded threshold bin, more chunks than shared memory holds) keep their scratch in
// the ring, which is idle between the scoring and the attention of a dynamic unit
static_assert(kTopkScratchInts * 4 <= kStageBytes, "fallback selection scratch fits one ring stage");
static_assert(kStageBytes % kRowBytes == 0, "staged rows start on 256-byte boundaries (the ldmatrix addresses rely on it)");
static_assert(kDecCtasPerSm * (kSmemBytes + 1024) <= 233472, "two CTAs per SM");
static_assert(part_off(kMaxWarps) + kPartBytes <= kRingBytes, "parking and the CTA partial reuse the idle ring");
static_assert(part_off(1) % 16 == 0 && kSelOff % 16 == 0 && kScoresOff % 16 == 0 && kBarsOff % 8 == 0 && kHistOff % 16 == 0 &&
                  kBoundsOff % 8 == 0 && kCandOff % 8 == 0,
              "alignment");

__device__ __forceinline__ int find_slot(const int32_t* prefix, int n, int x) {
  int i = 0;
  while (i + 1 < n && x >= prefix[i + 1]) ++i;
  return i;
}

// Checked build (-DHKV_CHECKED): every index that feeds an address is validated first; a violation is
// recorded in the cache's error word (HKV_ERR_INDEX, detail = place) and the access is skipped.
#ifdef HKV_CHECKED
#define HKV_CHECK(cond, place)                                             \
  if (!(cond)) {                                                           \
    if (atomicCAS(&err[0], 0, HKV_ERR_INDEX) == 0) err[1] = (place);       \
    dead = true;                                                           \
  }
#else
#define HKV_CHECK(cond, place)
#endif

// Profiling build (-DHKV_PROFILE): thread 0 of every CTA stamps the phase boundaries of the kernel into a
// buffer attached with hkv_profile_attach.  A stamp holds the low 32 bits of the global nanosecond timer
// (coarse ticks, but one clock for all SMs) and, above them, the low 32 bits of the SM's cycle counter
// (exact durations within a CTA).
#ifdef HKV_PROFILE
__device__ __forceinline__ unsigned long long phase_stamp() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return (static_cast<unsigned long long>(static_cast<uint32_t>(clock64())) << 32) | (t & 0xFFFFFFFFull);
}
#define HKV_STAMP(k) \
  if (P.prof && threadIdx.x == 0) P.prof[static_cast<size_t>(blockIdx.x) * kProfSlots + (k)] = phase_stamp();
#else
#define HKV_STAMP(k)
#endif

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <int NT, int W>   // NT: 8-wide column tiles of query heads (1 for groups up to 8, 2 up to 16); W: warps
__global__ void __launch_bounds__(W * 32, kDecCtasPerSm) decode_kernel(const __grid_constant__ DecodeParams P) {
  extern __shared__ __align__(1024) uint8_t smem[];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int csize = P.cluster;
  const bool clustered = csize > 1;
  const uint32_t crank = clustered ? cluster_ctarank() : 0u;
  HKV_STAMP(0)
  pdl_launch_dependents();

  const int cid = blockIdx.x / csize;
  const int li = find_slot(P.unit_prefix, P.n, cid);
  char* base = P.cache[li];
  int uid;
  {
    // Blocks start in index order, and a launch that follows another decode launch starts as many of them as the
    // device has room for while its predecessor still runs: the unit type that gains most from that early
    // start (see decode_stages) takes the cache's first clusters.
    const int c = cid - P.unit_prefix[li], nd = P.n_dynamic[li], ns = P.unit_prefix[li + 1] - P.unit_prefix[li] - nd;
    const int32_t* dl = reinterpret_cast<const int32_t*>(base + P.dyn_list_off[li]);
    const int32_t* sl = reinterpret_cast<const int32_t*>(base + P.sta_list_off[li]);
    if (P.static_first) uid = c < ns ? sl[c] : dl[c - ns];
    else uid = c < nd ? dl[c] : sl[c - nd];
  }
  const Unit* up = reinterpret_cast<const Unit*>(base + kUnitsOff) + uid;
  const int G = P.group, Hq = P.n_q_heads, cs = P.chunk_size;
  const int ub = uid / P.n_kv_heads, uh = uid - ub * P.n_kv_heads;
  const bool do_select = (P.phase & kPhaseSelect) != 0, do_attend = (P.phase & kPhaseAttend) != 0;
  constexpr bool kPushMerge = NT == 1;   // wider groups do not fit the receive area and use the pull merge

  // the unit's record (uniform loads, issued together)
  const int utype = up->type, C = up->C, n_tok = up->n_tok, n_chunks = up->n_chunks, k_sel = up->k_sel;
#ifdef HKV_CHECKED
  const int plane_rows = up->plane_rows;
#endif
  const uint8_t* kplane = reinterpret_cast<const uint8_t*>(base + up->k_off);
  const uint8_t* vplane = reinterpret_cast<const uint8_t*>(base + up->v_off);
  const uint8_t* summ = reinterpret_cast<const uint8_t*>(base + up->summ_off);
  int32_t* gsel = reinterpret_cast<int32_t*>(base + up->idx_off);
  float* gscores = reinterpret_cast<float*>(base + up->scores_off);
  int32_t* n_valid_g = reinterpret_cast<int32_t*>(base + P.n_valid_off[li]) + uid;
  int32_t* err = reinterpret_cast<int32_t*>(base + P.err_off[li]);
  const bool dynamic = utype != 0;

  // merge geometry (push merge): the output's G*128 elements are dealt to the cluster's CTAs in slices of
  // `per`; CTA r owns elements [r * per, r * per + own_cnt(r))
  const int total = G * kHeadDim;
  const int per = (((total + csize - 1) / csize) + 3) & ~3;
  // divisions by the cluster size, the slice length and the chunk size sit on the step's critical path
  // further down: their multipliers are worked out here, before the dependency wait
  const uint32_t csize_magic = clustered ? fastdiv_magic(static_cast<uint32_t>(csize)) : 0u;
  const uint32_t per_magic = fastdiv_magic(static_cast<uint32_t>(per));
  const bool cs_fast = cs > 1 && static_cast<uint64_t>(n_tok) * static_cast<uint64_t>(cs) < (1ull << 32);
  const uint32_t cs_magic = cs > 1 ? fastdiv_magic(static_cast<uint32_t>(cs)) : 0u;
  auto div_cs = [&](int x) { return cs_fast ? fastdiv(x, cs_magic) : x / cs; };
  auto own_cnt = [&](int r) { return max(0, min(total, (r + 1) * per) - r * per); };

  const bool identity = dynamic && k_sel >= n_chunks;          // every chunk is loaded: no list needed
  const bool fits = n_chunks <= kSelSmemChunks;                // scores and ids fit shared memory
  const bool scoring = dynamic && do_select;
  // scores travel through shared memory (and the exchange between the cluster's CTAs) only when a selection
  // needs them there; otherwise they go straight to global memory
  const bool exchange = scoring && fits && !identity;
  const int n_mt = (n_chunks + 15) >> 4;                       // 16-chunk groups, the unit of the exchange

  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kBarsOff);
  volatile uint32_t* armed = reinterpret_cast<volatile uint32_t*>(smem + kArmedOff);
  int* hist = reinterpret_cast<int*>(smem + kHistOff);
  float2* bounds = reinterpret_cast<float2*>(smem + kBoundsOff);
  int* misc = reinterpret_cast<int*>(smem + kMiscOff);
  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kDecStages; ++s) { mbar_init(&bars[s], 1); armed[s] = 0u; }
    mbar_init(&bars[kScoreBar], 1);
    mbar_init(&bars[kMergeBar], 1);
    mbar_fence_init();
    // what this CTA will receive from the cluster (itself included): every score of the unit plus one
    // (lower, upper) bound per warp; later one slice of every CTA's partial output plus its (m, l) rows
    if (clustered) {
      if (exchange) mbar_arrive_expect_tx(&bars[kScoreBar], static_cast<uint32_t>(n_mt * 64 + csize * W * 8));
      if (kPushMerge && do_attend) {
        const int mine = own_cnt(static_cast<int>(crank));
        mbar_arrive_expect_tx(&bars[kMergeBar], mine > 0 ? static_cast<uint32_t>(csize * (mine * 4 + G * 8)) : 0u);
      }
    }
    misc[0] = 0;
  }
  if (exchange) { for (int i = tid; i < kHistBins; i += W * 32) hist[i] = 0; }
  // "this CTA is running and its barriers exist": has to be known before anybody touches its shared memory remotely
  if (clustered) cluster_arrive();
  bool bar_pending = clustered;   // an arrival on the cluster barrier that has not been waited for yet

  if (!dynamic && !do_attend) {   // nothing to select for a static unit
    if (clustered) cluster_wait();
    return;
  }
  __syncthreads();

  // Waits until stage `stage` holds the tile with ring sequence number `q` (0-based over both
  // phases): first until it has been armed with that tile, then until the copies have landed.
  // Both waits are bounded; false = gave up.
  auto wait_tile = [&](int stage, uint32_t q) -> bool {
    if (armed[stage] != q + 1u) {
      const long long start = clock64();
      for (uint32_t it = 1; armed[stage] != q + 1u; ++it) {
        if ((it & 255u) == 0u && clock64() - start > HKV_WAIT_CYCLES) return false;
      }
    }
    return mbar_wait_bounded(&bars[stage], (q / kDecStages) & 1u);
  };

  bool dead = false;    // a bounded wait ran out: stop issuing, keep every hand-over
  // ldmatrix lane roles: matrix index mi = lane >> 3
  const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8, a_piece = lane >> 4;      // non-transposed A tile
  const int v_row = (lane & 7) + (lane >> 4) * 8, v_piece = (lane >> 3) & 1;      // transposed A tile

  float* sc_smem = reinterpret_cast<float*>(smem + kScoresOff);
  uint16_t* sel16 = reinterpret_cast<uint16_t*>(smem + kSelOff);
  const bool contiguous = !dynamic || identity;
  bool sel_in_smem = false;
  uint32_t seq0 = 0;    // tiles the CTA's ring has carried in earlier phases

  // ---- attention phase: tiles [at_tile0, at_tile0 + at_n) of the unit's token list ----
  int n_valid = 0, at_tile0 = 0, at_n = 0;
  auto setup_attn = [&](int nv) {
    n_valid = nv;
    const int n_tiles = (nv + kTile - 1) / kTile;
    const int t_per = clustered ? fastdiv(n_tiles + csize - 1, csize_magic) : n_tiles;
    at_tile0 = static_cast<int>(crank) * t_per;
    at_n = max(0, min(n_tiles, at_tile0 + t_per) - at_tile0);
  };
  auto sel_at = [&](int i) -> int { return sel_in_smem ? static_cast<int>(sel16[i]) : gsel[i]; };
  // How a tile of a dynamic unit maps onto chunks: a chunk size that is a multiple of the tile holds
  // every tile inside one chunk (one copy pair, issued by lane 0); any other size lets up to 32
  // chunks touch a tile (one lane per chunk).  Row keys differ from (row & 7) only when the chunk
  // size is not a multiple of 8.
  const bool one_chunk = !contiguous && (cs % kTile) == 0;
  const bool need_keys = !contiguous && (cs & 7) != 0;
  auto issue_attn = [&](int j) {   // whole warp; arms stage (seq0 + j) % stages with CTA tile j
    const int stage = (seq0 + j) % kDecStages;
    uint8_t* st = smem + stage * kStageBytes;
    const int v0 = (at_tile0 + j) * kTile;
    const int v1 = min(v0 + kTile, n_valid);
    HKV_CHECK(v0 >= 0 && v0 < v1 && v1 - v0 <= kTile, 100);
    if (contiguous || one_chunk) {
      if (lane == 0) {
        size_t row = static_cast<size_t>(v0);
        if (one_chunk) {
          const int ci = div_cs(v0);
          const int sid = sel_at(ci);
          HKV_CHECK(sid >= 0 && sid < n_chunks, 102);
          row = static_cast<size_t>(sid) * cs + (v0 - ci * cs);
        }
        HKV_CHECK(static_cast<int64_t>(row) + (v1 - v0) <= plane_rows, 103);
#ifdef HKV_CHECKED
        if (dead) return;
#endif
        const uint32_t bytes = static_cast<uint32_t>(v1 - v0) * kRowBytes;
        armed[stage] = seq0 + static_cast<uint32_t>(j) + 1u;
        mbar_arrive_expect_tx(&bars[stage], 2u * bytes);
        bulk_g2s(st, kplane + row * kRowBytes, bytes, &bars[stage]);
        bulk_g2s(st + kTile * kRowBytes, vplane + row * kRowBytes, bytes, &bars[stage]);
      }
      return;
    }
    uint32_t* keys = reinterpret_cast<uint32_t*>(st + 2 * kTile * kRowBytes);
    const int ci = div_cs(v0) + lane;                      // lane-th chunk touching this tile
    const int p0 = max(v0, ci * cs), p1 = min(v1, (ci + 1) * cs);
    if (need_keys) {
      const int v = v0 + lane;
      uint32_t key = lane & 7;
      if (v < v1) {
        const int cj = div_cs(v);
        key = static_cast<uint32_t>(sel_at(cj) * cs + (v - cj * cs)) & 7u;
      }
      keys[lane] = key;
    }
    size_t row = 0;
    if (p0 < p1) {
      const int sid = sel_at(ci);
      HKV_CHECK(sid >= 0 && sid < n_chunks, 102);
      row = static_cast<size_t>(sid) * cs + (p0 - ci * cs);
      HKV_CHECK(static_cast<int64_t>(row) + (p1 - p0) <= plane_rows, 103);
      HKV_CHECK(p0 - v0 >= 0 && p1 - v0 <= kTile, 104);
    }
#ifdef HKV_CHECKED
    dead = __any_sync(0xffffffffu, dead);
    if (dead) return;
#endif
    __syncwarp();
    if (lane == 0) {
      armed[stage] = seq0 + static_cast<uint32_t>(j) + 1u;
      mbar_arrive_expect_tx(&bars[stage], static_cast<uint32_t>(v1 - v0) * 2u * kRowBytes);
    }
    __syncwarp();
    if (p0 < p1) {
      const uint32_t bytes = static_cast<uint32_t>(p1 - p0) * kRowBytes;
      bulk_g2s(st + (p0 - v0) * kRowBytes, kplane + row * kRowBytes, bytes, &bars[stage]);
      bulk_g2s(st + kTile * kRowBytes + (p0 - v0) * kRowBytes, vplane + row * kRowBytes, bytes, &bars[stage]);
    }
  };

  // ---- scoring phase: this CTA's chunk means are rows [sc_row0, sc_row1) of the unit's table, staged as
  // sc_n pieces of up to kScoreTile rows (one ring stage, one copy, one barrier each).  The unit of work is a
  // group of 16 rows (one tensor-core tile): when all pieces fit the ring at once, the groups are dealt to
  // the warps one by one (several warps share a staged piece); otherwise a warp takes whole pieces and
  // re-arms their stages.
  int sc_row0 = 0, sc_row1 = 0, sc_n = 0;
  int wb_lo = 0, wb_hi = 0;   // this CTA's share of the score write-back
  bool sc_fine = true;
  if (scoring) {
    const int mt_per = (n_mt + csize - 1) / csize;
    sc_row0 = min(n_chunks, static_cast<int>(crank) * mt_per * 16);
    sc_row1 = min(n_chunks, sc_row0 + mt_per * 16);
    sc_n = (sc_row1 - sc_row0 + kScoreTile - 1) / kScoreTile;
    sc_fine = sc_n <= kDecStages;
    wb_lo = sc_row0;
    wb_hi = sc_row1;
  }
  auto issue_score = [&](int j) {   // piece j of this CTA's chunk means into stage j % stages
    if (lane == 0) {
      const int stage = j % kDecStages;
      const int r0 = sc_row0 + j * kScoreTile;
      const uint32_t bytes = static_cast<uint32_t>(min(r0 + kScoreTile, sc_row1) - r0) * kRowBytes;
      HKV_CHECK(r0 >= 0 && r0 < sc_row1 && sc_row1 <= n_chunks && bytes <= 2u * kTile * kRowBytes, 120);
#ifdef HKV_CHECKED
      if (dead) return;
#endif
      armed[stage] = static_cast<uint32_t>(j) + 1u;
      mbar_arrive_expect_tx(&bars[stage], bytes);
      bulk_g2s(smem + stage * kStageBytes, summ + static_cast<size_t>(r0) * kRowBytes, bytes, &bars[stage]);
    }
  };

  // Short token lists are latency-bound: a chunk that is known to be selected while the list is still being
  // built is requested from HBM into L2 at once, by one CTA of the cluster (nothing is requested that the step
  // does not read).  Who asks for what is settled here, off the critical path.
  bool early_on = false;
  if (exchange && do_attend && !P.offload) {
    const int my_tiles = ((k_sel * cs + kTile - 1) / kTile + csize - 1) / csize;
    early_on = my_tiles <= kPrefetchMaxTiles && (tid % csize) == static_cast<int>(crank);
  }
  auto early = [&](int ci) {
    if (!early_on) return;
    const int rows = min(cs, C - ci * cs);
    const size_t off = static_cast<size_t>(ci) * cs * kRowBytes;
    bulk_prefetch_l2(kplane + off, static_cast<uint32_t>(rows) * kRowBytes);
    bulk_prefetch_l2(vplane + off, static_cast<uint32_t>(rows) * kRowBytes);
  };

  // ---- copies that do not depend on this step's query start before the dependency wait ----
  bool attn_armed = false;
  if (scoring) {
    for (int j = warp; j < min(sc_n, kDecStages); j += W) issue_score(j);
  } else if (!dynamic) {
    setup_attn(n_tok);
    for (int j = warp; j < min(at_n, kDecStages); j += W) issue_attn(j);
    attn_armed = true;
  }
  const uint32_t* qg = reinterpret_cast<const uint32_t*>(P.q[li]) +
                       (static_cast<size_t>(ub) * Hq + static_cast<size_t>(uh) * G) * (kHeadDim / 2);
  // the query is written by whatever precedes this launch, so it may only be READ after the wait; asking L2
  // for its lines reads nothing and lets the loads below meet them there
  if (warp == W - 1 && lane * 32 < G * (kHeadDim / 2)) prefetch_l2_line(qg + lane * 32);

  HKV_STAMP(1)
  pdl_wait();
  HKV_STAMP(2)

  // the group's queries as B fragments of  S^T = X Q^T  (columns >= G are zero)
  uint32_t qb[8][2 * NT];
  {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int head = nt * 8 + g;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        qb[kk][2 * nt] = (head < G) ? __ldg(&qg[head * 64 + kk * 8 + t]) : 0u;
        qb[kk][2 * nt + 1] = (head < G) ? __ldg(&qg[head * 64 + kk * 8 + 4 + t]) : 0u;
      }
    }
  }

  HKV_STAMP(3)
  // =============================================================================================
  // chunk scoring + top-k selection (dynamic units)
  // =============================================================================================
  if (scoring) {
    if (clustered) { cluster_wait(); bar_pending = false; }   // every CTA of the cluster runs: remote stores are safe
    const uint32_t sc_addr = smem_u32(sc_smem), sbar_addr = smem_u32(&bars[kScoreBar]);
    float wlo = INFINITY, whi = -INFINITY;    // bounds of the scores this warp computed (same in every lane)

    const int mt_cnt = (sc_row1 - sc_row0 + 15) >> 4;                 // 16-row groups of this CTA
    const int n_items = sc_fine ? mt_cnt : sc_n;
    for (int it = warp; it < n_items; it += W) {
      const int piece = sc_fine ? (it >> 2) : it;                       // staged piece the item reads
      const int m_lo = sc_fine ? it : it * 4, m_hi = sc_fine ? it + 1 : min(mt_cnt, it * 4 + 4);
      const int stage = piece % kDecStages;
      if (!wait_tile(stage, static_cast<uint32_t>(piece))) {
        if (lane == 0) { atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT); err[1] = kErrScoreWait; }
        dead = true;
        break;
      }
      const uint32_t mbase = smem_u32(smem + stage * kStageBytes);
      for (int m = m_lo; m < m_hi; ++m) {
        const int mt = m & 3;                                           // group within the piece
        const int r0 = sc_row0 + piece * kScoreTile;                    // first chunk of the piece
        float acc[2][NT][4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) acc[e][nt][0] = acc[e][nt][1] = acc[e][nt][2] = acc[e][nt][3] = 0.f;
        }
        // piece p of a row sits at p ^ key, and rows start on 256-byte boundaries: the address of piece
        // 2 kk + a_piece is the row's address with the fixed low bits below, XOR (kk << 5)
        const uint32_t key = a_row & 7;     // tiles start at multiples of 16 chunks
        const uint32_t rowaddr = (mbase + (mt * 16 + a_row) * kRowBytes) | ((key >> 1) << 5) | (((a_piece ^ key) & 1u) << 4);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          uint32_t a0, a1, a2, a3;
          ldsm_x4(a0, a1, a2, a3, rowaddr ^ (kk << 5));
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma_bf16(acc[kk & 1][nt], a0, a1, a2, a3, qb[kk][2 * nt], qb[kk][2 * nt + 1]);
        }
        // chunk score = sum over the group's heads of <q_g, mean_c> (variant: their maximum; the
        // columns past the group hold zero queries and must not take part in it)
        float v0, v1;
        if (P.group_max) {
          v0 = v1 = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int h0 = nt * 8 + 2 * t;
            if (h0 < G) {
              v0 = fmaxf(v0, acc[0][nt][0] + acc[1][nt][0]);
              v1 = fmaxf(v1, acc[0][nt][2] + acc[1][nt][2]);
            }
            if (h0 + 1 < G) {
              v0 = fmaxf(v0, acc[0][nt][1] + acc[1][nt][1]);
              v1 = fmaxf(v1, acc[0][nt][3] + acc[1][nt][3]);
            }
          }
          v0 = fmaxf(v0, __shfl_xor_sync(0xffffffffu, v0, 1));
          v0 = fmaxf(v0, __shfl_xor_sync(0xffffffffu, v0, 2));
          v1 = fmaxf(v1, __shfl_xor_sync(0xffffffffu, v1, 1));
          v1 = fmaxf(v1, __shfl_xor_sync(0xffffffffu, v1, 2));
        } else {
          v0 = v1 = 0.f;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            v0 += (acc[0][nt][0] + acc[1][nt][0]) + (acc[0][nt][1] + acc[1][nt][1]);
            v1 += (acc[0][nt][2] + acc[1][nt][2]) + (acc[0][nt][3] + acc[1][nt][3]);
          }
          v0 += __shfl_xor_sync(0xffffffffu, v0, 1);
          v0 += __shfl_xor_sync(0xffffffffu, v0, 2);
          v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
          v1 += __shfl_xor_sync(0xffffffffu, v1, 2);
        }
        // Lanes of row group g now hold the scores of chunks g (v0) and g + 8 (v1) of this 16-chunk group.
        // Regroup: every lane gets the four consecutive scores 4t .. 4t+3, the unit of the exchange.
        const int cbase = r0 + mt * 16 + 4 * t;
        float4 quad;
        {
          float a[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int src = (((t & 1) << 2) + i) << 2;      // a lane of row group 4 (t & 1) + i
            const float x0 = __shfl_sync(0xffffffffu, v0, src), x1 = __shfl_sync(0xffffffffu, v1, src);
            a[i] = (t & 2) ? x1 : x0;
            if (cbase + i >= n_chunks) a[i] = -INFINITY;    // padding of the last group: never selected
          }
          quad = make_float4(a[0], a[1], a[2], a[3]);
          float mn = INFINITY, mx = -INFINITY;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (cbase + i < n_chunks) { mn = fminf(mn, a[i]); mx = fmaxf(mx, a[i]); }
          }
          mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1)); mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          wlo = fminf(wlo, mn);
          whi = fmaxf(whi, mx);
        }
        if (!exchange) {   // no selection in shared memory: the scores go to global memory
          if (g == 0) {
            if (cbase < n_chunks) gscores[cbase] = quad.x;
            if (cbase + 1 < n_chunks) gscores[cbase + 1] = quad.y;
            if (cbase + 2 < n_chunks) gscores[cbase + 2] = quad.z;
            if (cbase + 3 < n_chunks) gscores[cbase + 3] = quad.w;
          }
        } else if (!clustered) {
          if (g == 0) *reinterpret_cast<float4*>(sc_smem + cbase) = quad;
        } else {
          for (int s = g; s < csize; s += 8) st_async_f32x4(mapa(sc_addr + cbase * 4, s), quad, mapa(sbar_addr, s));
        }
      }
      __syncwarp();
      if (!sc_fine && it + kDecStages < sc_n) issue_score(it + kDecStages);
    }
    seq0 = static_cast<uint32_t>(sc_n);
    if (exchange) {
      // this warp's bounds, to every CTA (a warp that gave up sends them too: the byte count must add up)
      const int slot = static_cast<int>(crank) * W + warp;
      if (!clustered) { if (lane == 0) bounds[slot] = make_float2(wlo, whi); }
      else if (lane < csize) st_async_f32x2(mapa(smem_u32(&bounds[slot]), lane), wlo, whi, mapa(sbar_addr, lane));
    }
    HKV_STAMP(4)

    int emitted = 0;
    if (identity) {
      emitted = n_chunks;
      __syncthreads();   // the ring turns from chunk means to K/V tiles: every warp must be done with its means
    } else if (exchange) {
      // every score of the unit is on its way to this CTA: wait for the bytes, not for the cluster
      if (clustered) {
        if (!mbar_wait_bounded_cluster(&bars[kScoreBar], 0u)) {
          if (lane == 0) { atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT); err[1] = kErrExchangeWait; }
          dead = true;
        }
      } else {
        __syncthreads();
      }
      dead = __syncthreads_or(dead ? 1 : 0) != 0;
      HKV_STAMP(5)
      if (!dead) {
        float lo = INFINITY, hi = -INFINITY;
        for (int i = lane; i < csize * W; i += 32) { const float2 b2 = bounds[i]; lo = fminf(lo, b2.x); hi = fmaxf(hi, b2.y); }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
          hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
        }
        uint2* cand = reinterpret_cast<uint2*>(smem + kCandOff);
        const int ipt = (n_chunks + W * 32 - 1) / (W * 32);
        auto stamp = [&](int k2) { HKV_STAMP(20 + k2) };
        emitted = -1;
        if (ipt <= 1) emitted = block_topk_blocked<W, 1, 256>(sc_smem, n_chunks, n_mt * 16, k_sel, lo, hi, sel16, hist, cand, misc, early, stamp);
        else if (ipt <= 2) emitted = block_topk_blocked<W, 2, 256>(sc_smem, n_chunks, n_mt * 16, k_sel, lo, hi, sel16, hist, cand, misc, early, stamp);
        else if (ipt <= 4) emitted = block_topk_blocked<W, 4, 512>(sc_smem, n_chunks, n_mt * 16, k_sel, lo, hi, sel16, hist, cand, misc, early, stamp);
        else if (ipt <= 8) emitted = block_topk_blocked<W, 8, 512>(sc_smem, n_chunks, n_mt * 16, k_sel, lo, hi, sel16, hist, cand, misc, early, stamp);
        if (emitted < 0) {
          // crowded threshold bin (or more scores than the fast path takes): the general selection, its
          // scratch in the idle ring
          emitted = block_topk_smem<W>(
              sc_smem, n_chunks, k_sel, [&](int pos, int i) { sel16[pos] = static_cast<uint16_t>(i); },
              reinterpret_cast<int*>(smem));
          fence_proxy_async();   // the ring goes back to the bulk copies
          __syncthreads();
        }
        sel_in_smem = true;
      }
    } else {
      // more chunks than shared memory holds: selection on the scores in global memory; every CTA of the
      // cluster writes the same list to the same place
      __threadfence();
      if (clustered) { cluster_arrive(); cluster_wait(); } else { __syncthreads(); }
      HKV_STAMP(5)
      int* fb = reinterpret_cast<int*>(smem);
      emitted = block_select_emit(
          n_chunks, k_sel, [&](int i) { return float_key(__ldcg(&gscores[i])); }, [](int) { return false; },
          [&](int pos, int i) { gsel[pos] = i; }, fb, fb + 256, fb + 256 + 96);
      fence_proxy_async();
      __syncthreads();
    }
    int nv = emitted * cs;
    if (emitted > 0) {
      const int last = identity ? n_chunks - 1 : (sel_in_smem ? static_cast<int>(sel16[emitted - 1]) : gsel[emitted - 1]);
      if (last == n_chunks - 1) nv -= n_chunks * cs - C;   // the sequence's last chunk may be short
    }
    HKV_STAMP(6)
    setup_attn(nv);
    // the attention's first copies are what the step waits for: start them before anything else
    if (do_attend && !dead) {
      for (int j = warp; j < min(at_n, kDecStages); j += W) issue_attn(j);
      attn_armed = true;
    }
    // what later calls may ask for (scores, selected ids, attended tokens), off the critical path
    if (exchange && !dead) {
      for (int i = wb_lo + tid; i < wb_hi; i += W * 32) gscores[i] = sc_smem[i];
    }
    if (crank == 0 && !dead) {
      if (identity) { for (int i = tid; i < n_chunks; i += W * 32) gsel[i] = i; }
      else if (sel_in_smem) { for (int i = tid; i < emitted; i += W * 32) gsel[i] = sel16[i]; }
      if (tid == 0) *n_valid_g = nv;
    }
    if (!do_attend) return;
    // "my selection is done": from here on my score area is free to receive the peers' partial results
    if (clustered && kPushMerge && !bar_pending) { cluster_arrive_relaxed(); bar_pending = true; }
  } else if (dynamic) {
    setup_attn(__ldcg(n_valid_g));   // attention only: the list of an earlier selection
  }

  // =============================================================================================
  // flash-decoding over the unit's token list
  // =============================================================================================
  const float sc = P.scale_log2e;
  if (!attn_armed && !dead) {
    for (int j = warp; j < min(at_n, kDecStages); j += W) issue_attn(j);
  }

  HKV_STAMP(7)
  float o[8][NT][4];
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[dt][nt][0] = o[dt][nt][1] = o[dt][nt][2] = o[dt][nt][3] = 0.f;
  }
  float mrun[NT][2], lrun[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) { mrun[nt][0] = mrun[nt][1] = -INFINITY; lrun[nt][0] = lrun[nt][1] = 0.f; }

  // the loop over this warp's tiles, compiled twice: rows whose 16-byte pieces follow the staged row index (the
  // usual case: the permutation key is then a per-thread constant) and rows that carry their own keys
  auto run_tiles = [&](auto keys_c) {
  constexpr bool KEYS = decltype(keys_c)::value;
  for (int j = warp; j < at_n && !dead; j += W) {
    const int stage = (seq0 + j) % kDecStages;
    uint8_t* st = smem + stage * kStageBytes;
    const int v0 = (at_tile0 + j) * kTile;
    const int nrow = min(kTile, n_valid - v0);
    if (!wait_tile(stage, seq0 + static_cast<uint32_t>(j))) {
      if (lane == 0) { atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT); err[1] = kErrDecodeWait; }
      dead = true;
      break;
    }
#ifdef HKV_PROFILE
    if (j == 0) { HKV_STAMP(14) }
    if (warp == 0 && j == W) { HKV_STAMP(19) }
#endif
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(st + 2 * kTile * kRowBytes);
#ifdef HKV_CHECKED
    HKV_CHECK(!KEYS || keys[lane] < 8u, 110);
    HKV_CHECK(nrow >= 1, 111);
    dead = __any_sync(0xffffffffu, dead);
    if (dead) break;
#endif
    const bool partial = nrow < kTile;
    if (partial) {
      // rows past the end were not copied: clear them so that stale bits cannot poison P*V
      for (int r = nrow; r < kTile; ++r) {
        reinterpret_cast<uint2*>(st + r * kRowBytes)[lane] = make_uint2(0u, 0u);
        reinterpret_cast<uint2*>(st + kTile * kRowBytes + r * kRowBytes)[lane] = make_uint2(0u, 0u);
      }
      fence_proxy_async();
      __syncwarp();
    }
    const uint32_t kbase = smem_u32(st), vbase = kbase + kTile * kRowBytes;

    // S^T = K Q^T : rows = tokens (two 16-row tiles), columns = query heads; the reduction over the
    // head dimension runs as two interleaved accumulation chains.  Piece p of a row sits at
    // p ^ key:  (2 kk + a_piece) ^ key = ((kk ^ (key >> 1)) << 1) | ((a_piece ^ key) & 1); rows start on
    // 256-byte boundaries, so that address is the row's with fixed low bits, XOR (kk << 5).
    float s[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      float s2[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        s[mt][nt][0] = s[mt][nt][1] = s[mt][nt][2] = s[mt][nt][3] = 0.f;
        s2[nt][0] = s2[nt][1] = s2[nt][2] = s2[nt][3] = 0.f;
      }
      const int r = mt * 16 + a_row;
      const uint32_t key = KEYS ? keys[r] : static_cast<uint32_t>(a_row & 7);
      const uint32_t rowaddr = (kbase + r * kRowBytes) | ((key >> 1) << 5) | (((a_piece ^ key) & 1u) << 4);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        uint32_t a0, a1, a2, a3;
        ldsm_x4(a0, a1, a2, a3, rowaddr ^ (kk << 5));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (kk & 1) mma_bf16(s2[nt], a0, a1, a2, a3, qb[kk][2 * nt], qb[kk][2 * nt + 1]);
          else mma_bf16(s[mt][nt], a0, a1, a2, a3, qb[kk][2 * nt], qb[kk][2 * nt + 1]);
        }
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        s[mt][nt][0] += s2[nt][0]; s[mt][nt][1] += s2[nt][1];
        s[mt][nt][2] += s2[nt][2]; s[mt][nt][3] += s2[nt][3];
      }
    }

    // online softmax per query head (this thread: heads 2t, 2t+1 of each column tile; tokens g, g+8
    // of each row tile); logits stay unscaled, the scale enters the exponent's fused multiply-add
    uint32_t pb[2][NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      if (partial) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          if (mt * 16 + g >= nrow) s[mt][nt][0] = s[mt][nt][1] = -INFINITY;
          if (mt * 16 + g + 8 >= nrow) s[mt][nt][2] = s[mt][nt][3] = -INFINITY;
        }
      }
      float mx0 = fmaxf(fmaxf(s[0][nt][0], s[0][nt][2]), fmaxf(s[1][nt][0], s[1][nt][2]));
      float mx1 = fmaxf(fmaxf(s[0][nt][1], s[0][nt][3]), fmaxf(s[1][nt][1], s[1][nt][3]));
#pragma unroll
      for (int off = 4; off <= 16; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
      }
      const float mn0 = fmaxf(mrun[nt][0], mx0 * sc), mn1 = fmaxf(mrun[nt][1], mx1 * sc);
      if (__any_sync(0xffffffffu, mn0 != mrun[nt][0] || mn1 != mrun[nt][1])) {
        // a running maximum moved: bring the accumulators to the new reference
        const float c0 = fast_exp2(mrun[nt][0] - mn0), c1 = fast_exp2(mrun[nt][1] - mn1);
        mrun[nt][0] = mn0;
        mrun[nt][1] = mn1;
        lrun[nt][0] *= c0;
        lrun[nt][1] *= c1;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
          o[dt][nt][0] *= c0;
          o[dt][nt][1] *= c1;
          o[dt][nt][2] *= c0;
          o[dt][nt][3] *= c1;
        }
      }
      float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const float p0 = fast_exp2(fmaf(s[mt][nt][0], sc, -mn0)), p1 = fast_exp2(fmaf(s[mt][nt][1], sc, -mn1));
        const float p2 = fast_exp2(fmaf(s[mt][nt][2], sc, -mn0)), p3 = fast_exp2(fmaf(s[mt][nt][3], sc, -mn1));
        ps0 += p0 + p2;
        ps1 += p1 + p3;
        // P^T as the B operand of O^T += V^T P^T: tokens along k, heads along n
        pb[mt][nt][0] = movmatrix_trans(pack_bf16(p0, p1));
        pb[mt][nt][1] = movmatrix_trans(pack_bf16(p2, p3));
      }
      lrun[nt][0] += ps0;
      lrun[nt][1] += ps1;
    }

    // O^T += V^T P^T : rows = head-dim (eight 16-row tiles), k = tokens (two 16-token steps)
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      const int r = ks * 16 + v_row;
      const uint32_t key = KEYS ? keys[r] : static_cast<uint32_t>(v_row & 7);
      const uint32_t rowaddr = (vbase + r * kRowBytes) | ((key >> 1) << 5) | (((v_piece ^ key) & 1u) << 4);
#pragma unroll
      for (int dt = 0; dt < 8; ++dt) {
        uint32_t a0, a1, a2, a3;
        ldsm_x4_trans(a0, a1, a2, a3, rowaddr ^ (dt << 5));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(o[dt][nt], a0, a1, a2, a3, pb[ks][nt][0], pb[ks][nt][1]);
      }
    }
    __syncwarp();
#ifdef HKV_PROFILE
    if (j == 0) { HKV_STAMP(17) }
#endif
    if (j + kDecStages < at_n) issue_attn(j + kDecStages);
#ifdef HKV_PROFILE
    if (j == 0) { HKV_STAMP(18) }
#endif
  }

  };
  if (need_keys) run_tiles(std::true_type{}); else run_tiles(std::false_type{});

  HKV_STAMP(8)
  // a warp that gave up tells the others, so that nobody parks results over copies still in flight
  if (__syncthreads_or(dead ? 1 : 0)) {
    // leave only after every armed stage had another bounded chance to receive its copies
    for (int s2 = 0; s2 < kDecStages; ++s2) {
      const uint32_t a = armed[s2];
      if (a != 0u) mbar_wait_bounded(&bars[s2], ((a - 1u) / kDecStages) & 1u);
    }
    __syncthreads();
  }
  // the ring is idle from here on: it now holds the partial results

  HKV_STAMP(9)
  // ---- merge the warps of this CTA ----
  // each warp parks (m, l, O): O as [16 heads][kParkStride] floats, then m[16], l[16]
  {
    float* wo = reinterpret_cast<float*>(smem + warp * kParkBytes);
    float* wm = wo + 16 * kParkStride;
    float* wl = wm + 16;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float l0 = lrun[nt][0], l1 = lrun[nt][1];
#pragma unroll
      for (int off = 4; off <= 16; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
      }
      const int h0 = nt * 8 + 2 * t;
#pragma unroll
      for (int dt = 0; dt < 8; ++dt) {
        wo[h0 * kParkStride + dt * 16 + g] = o[dt][nt][0];
        wo[(h0 + 1) * kParkStride + dt * 16 + g] = o[dt][nt][1];
        wo[h0 * kParkStride + dt * 16 + g + 8] = o[dt][nt][2];
        wo[(h0 + 1) * kParkStride + dt * 16 + g + 8] = o[dt][nt][3];
      }
      if (g == 0) {
        wm[h0] = mrun[nt][0]; wm[h0 + 1] = mrun[nt][1];
        wl[h0] = l0; wl[h0 + 1] = l1;
      }
    }
  }
  __syncthreads();
  HKV_STAMP(16)

  const size_t out_row0 = static_cast<size_t>(ub) * Hq + static_cast<size_t>(uh) * G;
  float* part = reinterpret_cast<float*>(smem + (W * kParkBytes));
  float2* part_ml = reinterpret_cast<float2*>(smem + (W * kParkBytes) + kMaxGroup * kHeadDim * 4);
  // Push merge (groups up to 8): every CTA sends each owner its share of (m, l, O) into the owner's score
  // area, which is idle by now (peers have signalled the end of their selection), crediting the owner's
  // merge barrier; an owner reduces from its own shared memory once its bytes are in.
  const uint32_t recv_acc = smem_u32(smem + kScoresOff), recv_ml = recv_acc + kRecvMlOff;
  const uint32_t mbar_addr = smem_u32(&bars[kMergeBar]);
  if (clustered && kPushMerge && bar_pending) { cluster_wait(); bar_pending = false; }
  // items = (row, group of four columns): independent loads, one pass for groups up to 4, two up to 8
  for (int item = tid; item < G * 32; item += W * 32) {
    const int row = item >> 5, dq = item & 31;
    float mw[W], M = -INFINITY;
#pragma unroll
    for (int w2 = 0; w2 < W; ++w2) {
      mw[w2] = reinterpret_cast<const float*>(smem + w2 * kParkBytes)[16 * kParkStride + row];
      M = fmaxf(M, mw[w2]);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w2 = 0; w2 < W; ++w2) {
        const float* po = reinterpret_cast<const float*>(smem + w2 * kParkBytes);
        const float f = fast_exp2(mw[w2] - M);
        const float4 v = *reinterpret_cast<const float4*>(po + row * kParkStride + dq * 4);
        acc.x += v.x * f; acc.y += v.y * f; acc.z += v.z * f; acc.w += v.w * f;
        L += po[16 * kParkStride + 16 + row] * f;
      }
    }
    if (!clustered) {
      const float inv = L > 0.f ? 1.f / L : 0.f;
      const size_t off = (out_row0 + row) * kHeadDim + dq * 4;
      if (P.out_f32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(P.out[li]) + off) =
            make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
      } else {
        uint2 pk;
        pk.x = pack_bf16(acc.x * inv, acc.y * inv);
        pk.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(P.out[li]) + off) = pk;
      }
    } else if (kPushMerge) {
      const int e0 = row * kHeadDim + dq * 4;
      const int owner = fastdiv(e0, per_magic);
      st_async_f32x4(mapa(recv_acc + (static_cast<int>(crank) * per + (e0 - owner * per)) * 4, owner), acc, mapa(mbar_addr, owner));
      // the row's (m, l) goes to every owner: the 32 lanes of an item row hold the same pair, lane s sends to owner s
      if (dq < csize && own_cnt(dq) > 0)
        st_async_f32x2(mapa(recv_ml + (static_cast<int>(crank) * G + row) * 8, dq), M, L, mapa(mbar_addr, dq));
    } else {
      *reinterpret_cast<float4*>(part + row * kHeadDim + dq * 4) = acc;
      if (dq == 0) part_ml[row] = make_float2(M, L);
    }
  }
  HKV_STAMP(10)
  if (!clustered) return;

  if (kPushMerge) {
    const int e_lo = static_cast<int>(crank) * per, e_hi = min(total, e_lo + per);
    if (tid >= e_hi - e_lo) return;    // nothing of this thread's is left; peers only write to this CTA, which stays until its reducers leave
    if (!mbar_wait_bounded_cluster(&bars[kMergeBar], 0u)) {
      if (atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT) == 0) err[1] = kErrMergeWait;
      return;
    }
    HKV_STAMP(11)
    const float* racc = reinterpret_cast<const float*>(smem + kScoresOff);
    const float2* rml = reinterpret_cast<const float2*>(smem + kScoresOff + kRecvMlOff);
    for (int e = e_lo + tid; e < e_hi; e += W * 32) {
      const int row = e >> 7, le = e - e_lo;
      // senders in two halves of eight (the second only for clusters above eight CTAs); fixed order
      float ms[kMaxCluster], ls[kMaxCluster], av[kMaxCluster];
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) { ms[s2] = -INFINITY; ls[s2] = 0.f; av[s2] = 0.f; }
#pragma unroll
      for (int s2 = 0; s2 < 8; ++s2) {
        if (s2 < csize) {
          const float2 ml = rml[s2 * G + row];
          ms[s2] = ml.x; ls[s2] = ml.y; av[s2] = racc[s2 * per + le];
        }
      }
      if (csize > 8) {
#pragma unroll
        for (int s2 = 8; s2 < kMaxCluster; ++s2) {
          if (s2 < csize) {
            const float2 ml = rml[s2 * G + row];
            ms[s2] = ml.x; ls[s2] = ml.y; av[s2] = racc[s2 * per + le];
          }
        }
      }
      float M = -INFINITY;
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) M = fmaxf(M, ms[s2]);
      float acc = 0.f, L = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
          const float f = fast_exp2(ms[s2] - M);
          acc += av[s2] * f;
          L += ls[s2] * f;
        }
        if (csize > 8) {
#pragma unroll
          for (int s2 = 8; s2 < kMaxCluster; ++s2) {
            const float f = fast_exp2(ms[s2] - M);
            acc += av[s2] * f;
            L += ls[s2] * f;
          }
        }
      }
      const float r = L > 0.f ? __fdividef(acc, L) : 0.f;
      const size_t off = out_row0 * kHeadDim + e;
      if (P.out_f32) reinterpret_cast<float*>(P.out[li])[off] = r;
      else reinterpret_cast<__nv_bfloat16*>(P.out[li])[off] = __float2bfloat16_rn(r);
    }
    HKV_STAMP(13)
    return;
  }

  // ---- merge the CTAs of the cluster through distributed shared memory ----
  if (bar_pending) cluster_wait();
  cluster_arrive();
  cluster_wait();
  HKV_STAMP(11)
  {
    const uint32_t part_addr = smem_u32(part), ml_addr = smem_u32(part_ml);
    const int per2 = (total + csize - 1) / csize;
    const int e_end = min(total, static_cast<int>(crank + 1) * per2);
    for (int e = static_cast<int>(crank) * per2 + tid; e < e_end; e += W * 32) {
      const int row = e >> 7;
      float ms[kMaxCluster], ls[kMaxCluster], av[kMaxCluster];
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) {
        if (s2 < csize) {
          const float2 ml = ld_cluster_f32x2(mapa(ml_addr + row * 8, s2));
          ms[s2] = ml.x;
          ls[s2] = ml.y;
          av[s2] = ld_cluster_f32(mapa(part_addr + e * 4, s2));
        } else {
          ms[s2] = -INFINITY; ls[s2] = 0.f; av[s2] = 0.f;
        }
      }
      float M = -INFINITY;
#pragma unroll
      for (int s2 = 0; s2 < kMaxCluster; ++s2) M = fmaxf(M, ms[s2]);
      float acc = 0.f, L = 0.f;
      if (M > -INFINITY) {
#pragma unroll
        for (int s2 = 0; s2 < kMaxCluster; ++s2) {
          const float f = exp2f(ms[s2] - M);
          acc += av[s2] * f;
          L += ls[s2] * f;
        }
      }
      const float r = L > 0.f ? acc / L : 0.f;
      const size_t off = out_row0 * kHeadDim + e;
      if (P.out_f32) reinterpret_cast<float*>(P.out[li])[off] = r;
      else reinterpret_cast<__nv_bfloat16*>(P.out[li])[off] = __float2bfloat16_rn(r);
    }
  }
  HKV_STAMP(12)
  // nobody leaves while its partial may still be read
  cluster_arrive();
  cluster_wait();
  HKV_STAMP(13)
}

// warps per CTA of each instance: the wide-group kernel needs twice the registers per thread
constexpr int warps_of(int nt) { return nt == 1 ? kMaxWarps : 4; }

template <int NT>
void fill_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int n_clusters, int cluster, bool pdl,
                 cudaStream_t stream) {
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(static_cast<unsigned>(n_clusters) * cluster, 1, 1);
  cfg.blockDim = dim3(warps_of(NT) * 32, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.numAttrs = 1;
  if (pdl) {
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
}

// Once per device and kernel instance: shared-memory size, permission for clusters above eight CTAs, and
// for every cluster size how many clusters the device can hold at once (function attributes and
// occupancy belong to the device that is current when they are set / asked for).
struct ClusterCaps {
  bool ready = false;
  int max_active[kMaxCluster + 1] = {};
};
constexpr int kMaxDevices = 64;
std::mutex g_caps_mutex;

template <int NT>
cudaError_t configure(const ClusterCaps** out) {
  static ClusterCaps caps_of[kMaxDevices];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_caps_mutex);
  ClusterCaps& caps = caps_of[dev];
  if (!caps.ready) {
    e = cudaFuncSetAttribute(decode_kernel<NT, warps_of(NT)>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<NT, warps_of(NT)>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    for (int c = 1; c <= kMaxCluster; ++c) {
      cudaLaunchConfig_t cfg;
      cudaLaunchAttribute attr[2];
      fill_config<NT>(cfg, attr, 1, c, false, nullptr);
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, decode_kernel<NT, warps_of(NT)>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
      caps.max_active[c] = n;
    }
    caps.ready = true;
  }
  *out = &caps;
  return cudaSuccess;
}

template <int NT>
cudaError_t launch_nt(const DecodeParams& params, int total_units, cudaStream_t stream) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  fill_config<NT>(cfg, attr, total_units, params.cluster, params.pdl != 0, stream);
  return cudaLaunchKernelEx(&cfg, decode_kernel<NT, warps_of(NT)>, params);
}

}  // namespace

size_t decode_smem_bytes() { return kSmemBytes; }

constexpr int kLatencyCluster = 10;

int choose_cluster(int total_units, int max_tiles, const int* max_active) {
  // The largest even size (or 1) that (a) the device can hold in ONE wave of clusters, (b) leaves every
  // CTA at least two tiles of the longest unit.  max_active[c] = clusters of size c resident at once.
  // Even sizes only: two CTAs share an SM, and an odd cluster leaves half an SM idle (measured: 13 CTAs
  // per unit are slower than 12).  Sizes need not be powers of two.
  // Short lists (at most 16 tiles per CTA at ten CTAs per unit) are bound by the step's chain of latencies,
  // not by bandwidth; there ten CTAs per unit measured best at every batch size tried (1 .. 6 sequences of
  // four KV heads), larger clusters paying more for their barriers and exchanges than they gain.
  int c = 1;
  for (int t = 2; t <= kMaxCluster; t += 2)
    if (max_active[t] >= total_units && t * 2 <= max_tiles) c = t;
  if (c > kLatencyCluster && max_tiles <= kLatencyCluster * 16) c = kLatencyCluster;
  return c;
}

cudaError_t decode_cluster_caps(int group, const int** max_active) {
  const ClusterCaps* caps = nullptr;
  cudaError_t e = group > 8 ? configure<2>(&caps) : configure<1>(&caps);
  if (e != cudaSuccess) return e;
  *max_active = caps->max_active;
  return cudaSuccess;
}

#ifdef HKV_CHECKED
namespace {
// Checked build only: one CTA waits, bounded, on an mbarrier that nothing ever arrives on, and records the
// give-up in the error word like every other wait of the library does.
__global__ void selftest_wait_kernel(int32_t* err) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
  __syncthreads();
  if (!mbar_wait_bounded(&bar, 0u)) {
    if (threadIdx.x == 0 && atomicCAS(&err[0], 0, HKV_ERR_TIMEOUT) == 0) err[1] = kErrSelfTest;
  }
}
}  // namespace
cudaError_t launch_selftest_wait(int32_t* err_word, cudaStream_t stream) {
  selftest_wait_kernel<<<1, 64, 0, stream>>>(err_word);
  return cudaGetLastError();
}
#endif

cudaError_t launch_decode(const DecodeParams& params, int total_units, cudaStream_t stream) {
  if (total_units <= 0) return cudaSuccess;
  if (params.group > 8) return launch_nt<2>(params, total_units, stream);
  return launch_nt<1>(params, total_units, stream);
}

}  // namespace hkv
