// a6 on the 5th-generation tensor cores: sparse attention (Eq. 3) for the MLA latent shape
// (H = 64 heads, d_qk = 576, d_v = 512, the value is the first 512 dims of the key row).
//
// One thread block = one query (or one row split of one sequence in decode).  Its 64 heads are the M = 64
// rows of every MMA; the attended cache rows stream through a ring of three 64-key shared tiles:
//
//   warps 8-11  gather: rows [window | sink | sparse] (or the caller's row list) -> 128B-swizzled K-major tiles, up to
//               three tiles in flight.  Scattered rows are copied with coalesced 16-byte cp.async (a row whole, by one
//               warp, in back-to-back instructions), each tile handed over through an mbarrier when it has landed;
//               tiles of 64 consecutive window rows come as nine TMA boxes instead.  A TMA gather of the scattered
//               rows (cp.async.bulk.tensor ... tile::gather4: four cache rows x one 64-dim column block = 512 bytes
//               per instruction, 144 per tile) is built in as well (AttnArgs::gather4) and measured 1.3 x slower: the
//               TMA unit takes about 26 cycles per such instruction.
//               Q arrives the same way: its rope dims (512-575) stay in shared memory as an MMA operand, dims 0-511
//               are staged in the last tile buffer for the softmax warps
//               With two P V issuers (prefill) warps 6-7 have no MMAs to issue and copy rows as a fifth and sixth gather
//               warp (11 or 10 rows of a tile each instead of 16: measured 1 % faster).
//   warps 4-7   one thread each issues tcgen05.mma.  Back-to-back MMAs into one accumulator run far below the pipe's
//               rate at these small shapes, so each product is cut into independent accumulation chains:
//                 S = Q K^T   issuers 0 and 1: dims 256x .. 256x+255 with Q from tensor memory (16 steps of M64 N64
//                             K16) plus two rope steps with Q from shared memory; the partial sum of issuer x lands in
//                             lane half x of the S buffer
//                 O += P V    with P from tensor memory; V is the key tile read MN-major, so each cache row is fetched
//                             once.  Two layouts (AttnArgs::pv_issuers):
//                             2 (prefill)  issuer x: value dims 256x .. 256x+255 (M64 N256 K16 x 4 per tile), P from lane
//                                          half x, O in lane half x: an issuer owns everything in its lane half
//                             4 (decode)   issuer x: value dims 128x .. 128x+127 (M64 N128 K16 x 4 per tile)
//               A thread takes whichever of "next P V" / "next Q K^T" is ready, P V first (its completion frees a key
//               buffer, and the refill of that buffer is the longest latency of the ring).  The S buffer of tile i+1 still holds
//               P of tile i-1 in its first columns.  With four issuers Q K^T(i+1) waits for the completion barrier of
//               P V(i-1); the P V issuers that do no Q K^T release a key buffer as early as possible, which is what a
//               decode step, waiting on HBM gathers, needs.  With two issuers the P V that reads those columns and the
//               Q K^T that overwrites them are issued by the same thread, in that order, and touch only that thread's
//               lane half, so the tensor core's in-order execution of one thread's MMAs keeps them apart: Q K^T(i+1)
//               is queued right behind P V(i-1) and the pipe never idles for a barrier round trip between them (4 % of
//               a prefill step).  AttnArgs::qk_waits_pv (tuning knob LSA_TUNE_ATTN_PV_WAIT) brings the barrier back;
//               both ways give the same bits, which a test checks.
//   warps 0-3   softmax: move Q to tensor memory once; per tile tcgen05.ld of both partial sums, add, running max
//               with lazy rescaling of O, exp2, fp32 row sums, P as bf16 -> tensor memory (A operand of P V); at the
//               end O / l through shared memory to global in whole rows
//
// An M = 64 accumulator occupies 16 of the 32 lanes of each TMEM quarter, so two of them share a column range.  All
// 512 columns are in use:
//   columns   0-255   O[:, 0:256] in lanes 0-15, O[:, 256:512] in lanes 16-31
//   columns 256-383   Q[:, 0:512] as packed bf16: dims 0-255 in lanes 0-15, dims 256-511 in lanes 16-31 (an MMA reads
//                     its TMEM operand from the lanes its accumulator lives in)
//   columns 384-511   S buffers 0 and 1 (64 columns each): the first chain's partial sum in lanes 0-15, the second's in
//                     lanes 16-31.  Lanes l and l+16 of a softmax warp share head row l: they swap halves, so lane l
//                     finishes keys 0-31 and lane l+16 keys 32-63 of the tile.  P (32 columns = 64 bf16, one copy
//                     per lane half) overwrites the first half of the S buffer it came from.
#include "lsa_internal.h"
#include "lsa_tc.cuh"

#ifdef LSA_TIMELINE
// Instrumented build only (-DLSA_TIMELINE; the default library has none of this): SM-clock stamps of the attention
// kernel, one slot per event and block, each written by one thread; read back with lsa_debug_timeline.
enum TlEvent {
  kTlEntry = 0,     // block entry
  kTlSetup,         // barriers initialised, tensor memory allocated
  kTlDepWait,       // griddepcontrol.wait returned (thread 0)
  kTlQInTmem,       // MMA issuer 0: Q is in tensor memory
  kTlTile0Landed,   // MMA issuer 0: first key tile landed
  kTlS0,            // first S tile complete (softmax thread 0)
  kTlLastP,         // last P handed to the issuers
  kTlLastPV,        // last P V complete
  kTlStaged,        // thread 0: its part of O staged in shared memory
  kTlSynced,        // block barrier after the tile loop passed
  kTlSent,          // rows for the peer blocks written (split launches)
  kTlClusterSync,   // cluster barrier passed
  kTlMerged,        // merge done
  kTlExit,          // last instruction of thread 0
  kTlTile0Issued,   // gather thread 0: copies of the first tile issued
  kTlQIssued,       // gather thread 0: Q requested
  // steady state: tiles kTlProbe .. kTlProbe + 3 of the block, slot = event + tile - kTlProbe
  kTlKFreed = 16,   // gather thread 0: the tile's buffer is free (k_empty passed)
  kTlKIssued = 20,  // gather thread 0: the tile's copies are issued
  kTlKLanded = 24,  // (unused)
  kTlQkIssue0 = 28, // issuer 0: about to issue the tile's Q K^T
  kTlQkIssue1 = 32, // issuer 0: Q K^T issued
  kTlSFull = 36,    // softmax thread 0: the tile's S complete
  kTlSLoaded = 40,  // ... partial sums read and exchanged
  kTlPHanded = 44,  // ... P handed over
  kTlPvIssue0 = 48, // issuer 0: about to issue the tile's P V
  kTlPvIssue1 = 52, // issuer 0: P V issued
  kTlPvDone = 56,   // (unused)
  kTlQkMmas = 60,   // issuer 0: the tile's Q K^T MMAs issued, commit not yet
  kTlPvMmas = 64,   // issuer 0: the tile's P V MMAs issued, commits not yet
  kTlPHanded1 = 68, kTlPHanded2 = 72, kTlPHanded3 = 76,   // softmax warps 1-3: P handed over
  kTlSpinsQk = 80, kTlSpinsPv = 84,   // issuer 0: failed polls before the tile's Q K^T / P V (a count, not a time)
  kTlCount = 88
};
#ifndef LSA_TL_PROBE
#define LSA_TL_PROBE 10
#endif
constexpr int kTlProbe = LSA_TL_PROBE;
#define LSA_TL_VAL(cond, i, k, v)                                                       \
  do {                                                                                   \
    const unsigned blk_ = blockIdx.x + gridDim.x * blockIdx.y;                           \
    if ((cond) && (i) >= kTlProbe && (i) < kTlProbe + 4 && blk_ < 1024)                  \
      g_timeline[blk_ * kTlCount + (k) + (i) - kTlProbe] = g_timeline[blk_ * kTlCount] + (v); \
  } while (0)
#define LSA_TL_TILE(cond, i, k) do { if ((cond) && (i) >= kTlProbe && (i) < kTlProbe + 4) LSA_TL((k) + (i) - kTlProbe); } while (0)
__device__ long long g_timeline[1024 * kTlCount];
__device__ long long g_wall[1024 * 2];   // globaltimer (ns) at entry and exit
#define LSA_WALL(k)                                                                      \
  do {                                                                                   \
    const unsigned blk_ = blockIdx.x + gridDim.x * blockIdx.y;                           \
    long long t_;                                                                        \
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                              \
    if (blk_ < 1024) g_wall[blk_ * 2 + (k)] = t_;                                        \
  } while (0)
extern "C" __attribute__((visibility("default"))) int lsa_debug_wall(long long* host, int n_blocks) {
  return cudaMemcpyFromSymbol(host, g_wall, sizeof(long long) * 2 * (n_blocks < 1024 ? n_blocks : 1024)) == cudaSuccess ? 0 : -1;
}
#define LSA_TL(k)                                                                        \
  do {                                                                                   \
    const unsigned blk_ = blockIdx.x + gridDim.x * blockIdx.y;                           \
    if (blk_ < 1024) g_timeline[blk_ * kTlCount + (k)] = clock64();                       \
  } while (0)
#define LSA_TL_IF(cond, k) do { if (cond) LSA_TL(k); } while (0)
extern "C" __attribute__((visibility("default"))) int lsa_debug_timeline(long long* host, int n_blocks) {
  return cudaMemcpyFromSymbol(host, g_timeline, sizeof(long long) * kTlCount * (n_blocks < 1024 ? n_blocks : 1024)) == cudaSuccess ? 0 : -1;
}
#else
#define LSA_TL(k)
#define LSA_TL_IF(cond, k)
#define LSA_TL_TILE(cond, i, k)
#define LSA_TL_VAL(cond, i, k, v)
#define LSA_WALL(k)
#endif

namespace lsa {

namespace {

constexpr int kH = 64, kDQK = 576, kDV = 512;
constexpr int kTileKeys = 64;
constexpr int kAtoms = kDQK / 64;            // 9 column blocks of 64 dims (128 bytes) per row
constexpr int kAtomBytes = 64 * 128;         // 64 rows x 128 bytes
constexpr int kHalfKeys = 32;

constexpr int kSoftmaxWarps = 4, kMmaWarps = 4, kLoadWarps = 4;
constexpr int kThreadsAttnTc = 32 * (kSoftmaxWarps + kMmaWarps + kLoadWarps);
constexpr uint32_t kTmemColsAttn = 512;
constexpr int kKBufs = 3;                    // 64-key tile buffers in shared memory
constexpr uint32_t kColQ = 256;              // Q[:, 0:512] as packed bf16: 128 columns, dims 0-255 | 256-511 by lane half
constexpr uint32_t kColS = 384;              // two S / P buffers of 64 columns
constexpr uint32_t kSBuf = 64;
constexpr float kLog2eTc = 1.4426950408889634f;
constexpr int kMaxClusterSplit = 8;          // row splits of one sequence = blocks of one cluster (portable limit)
constexpr float kRescaleGap = 8.f;           // rescale O only when the row max grows by more than 2^8

struct AttnTcSmem {
  alignas(1024) uint8_t q_rope[kAtomBytes];                 // Q[:, 512:576], 64 rows x 128 B
  alignas(1024) uint8_t k[kKBufs][kAtoms][kAtomBytes];      // [tile buffer][column block][64 rows x 128 B]
  alignas(8) uint64_t q_full, q_tmem, k_full[kKBufs], k_empty[kKBufs], s_full[2], p_ready[2];
  alignas(8) uint64_t recv_full;          // two-split launches: the peer's rows and log-sum-exps have arrived
  uint32_t tmem_slot;
  alignas(16) float lse_own[kH];          // split launches: this block's log-sum-exp per head (log2 units)
  alignas(16) float lse_peer[kH / 2];     // two-split launches: the peer's, for the heads this block finishes
};
constexpr int kPitchPart = kDV * 4 + 16;                  // staged fp32 row of a partial result, padded against bank conflicts
// Two-split launches stage their rows in the order the softmax warps read them out of tensor memory: per warp (16
// rows) four column steps, each [value-dim half][row][64 floats] = 8 KB, the 16-byte chunks of a row's 256-byte piece
// XOR-swizzled by the row (no bank conflicts either way).  A step's 8 KB is contiguous, so the rows the peer finishes
// leave step by step, one bulk copy each, while the rest is still being read out; the peer's rows land behind the
// staged ones in the same layout.
constexpr int kPairRowBytes = kDV * 4;
constexpr int kRecvOffset = kH * kPairRowBytes;
constexpr uint32_t kRecvBytes = (kH / 2) * kDV * 4 + (kH / 2) * 4;
static_assert(kRecvOffset + (kH / 2) * kPairRowBytes <= kKBufs * kAtoms * kAtomBytes, "staged and received rows must fit the key buffers");
static_assert(kH * kPitchPart <= kKBufs * kAtoms * kAtomBytes, "staged rows must fit the key buffers");

// ---- thread-block cluster: barrier and loads from a peer block's shared memory
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of the cluster barrier on their own: a thread arrives when it is done with a phase and waits later,
// where it needs every thread of the cluster to have arrived.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
// Address of this block's shared-memory location `addr` in the block of rank `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_smem(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// Bulk copy from this block's shared memory into a peer block's (addresses from peer_smem); the bytes are counted on
// the peer's mbarrier.  16-byte aligned addresses, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_peer, uint32_t src, uint32_t bytes, uint32_t bar_peer) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_peer), "r"(src), "r"(bytes), "r"(bar_peer) : "memory");
}
// With n_split > 1 the kernel must be launched with clusters of (1, n_split, 1) blocks: the splits of one sequence
// are co-scheduled and merge their partial results themselves (no second kernel).  Block s finishes heads
// [s * 64 / n_split, (s + 1) * 64 / n_split): every block stages its rows (normalised, fp32) in shared memory and keeps
// its own share there.
//   Two splits (the decode configuration): the other 32 rows and their log-sum-exps are pushed straight into the
//   peer's shared memory, behind its staged rows, by bulk copies that count bytes on the peer's mbarrier.  The cluster
//   barrier is used in halves: a thread arrives when it has left the tile loop and waits before the first copy (the
//   peer's key buffers must be out of use before they receive), and once more around the end, so that no block leaves
//   while the other may still write into it.  Nothing goes through global memory.
//   Four or eight splits: the other rows (one bulk copy per row) and all log-sum-exps go to the global scratch, where
//   they stay in L2; after one cluster barrier the owner of a row combines its own part with the others'.  (Loads from
//   a peer's shared memory moved the same rows at about a quarter of the L2 path's rate.)
//
// q_tma != 0: q_map describes q as a bf16 matrix [n_query * 64, 576] and Q arrives as nine TMA boxes; otherwise the
// gather warps copy it with cp.async.  k_tma != 0 (contiguous caches only): k_map describes the cache rows, and key
// tiles that lie wholly inside the window, 64 consecutive rows, arrive as nine TMA boxes as well.  k_g4 != 0: g_map
// describes the cache rows with a box one row high, and every other key tile is gathered four rows per instruction.
//
// One instantiation per way the kernel is used, so that each holds only the code of its mode (the instruction caches
// hold far less than the whole kernel, and the three warp roles run their loops side by side):
//   kRows       the caller's row lists are walked (else [window | sink | sparse] of a contiguous cache)
//   kPv         threads that issue P V: 2 = an issuer owns a lane half, 4 = one issuer per 128 value dims
//   kClustered  the blocks of a cluster are row splits of one sequence and merge their results
template <bool kRows, int kPv, bool kClustered>
__global__ void __launch_bounds__(kThreadsAttnTc, 1) sparse_attn_tc_kernel(const __grid_constant__ CUtensorMap q_map, int q_tma,
                                                                            const __grid_constant__ CUtensorMap k_map, int k_tma,
                                                                            const __grid_constant__ CUtensorMap g_map, int k_g4,
                                                                            AttnArgs p) {
  extern __shared__ uint8_t smem_raw[];
  AttnTcSmem& sm = *reinterpret_cast<AttnTcSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qi = blockIdx.x, split = blockIdx.y;
  const void* const q_ptr = p.q;
  const void* const k_ptr = p.k;
  void* const out_ptr = p.out;
  float* const lse_ptr = p.lse;
  float* const part_out = p.part_out;
  float* const part_lse = p.part_lse;

  constexpr int n_pv = kPv;
  constexpr bool clustered = kClustered;
  const bool pair = kClustered && p.n_split == 2;   // two splits exchange their rows through shared memory
  const bool dead = tc::status_raised(p.status);   // an earlier block of this launch (or an earlier launch) gave up on a wait
  if (dead && !clustered) return;

  // ---- set-up
  if (tid == 0) {
    LSA_TL(kTlEntry);
    LSA_WALL(0);
    tc::mbar_init(smem_u32(&sm.q_full), q_tma ? 1 : 32 * kLoadWarps);
    tc::mbar_init(smem_u32(&sm.q_tmem), kSoftmaxWarps);
    for (int b = 0; b < kKBufs; ++b) {
      tc::mbar_init(smem_u32(&sm.k_full[b]), 32 * (kLoadWarps + (kPv == 2 ? 2 : 0)));
      tc::mbar_init(smem_u32(&sm.k_empty[b]), n_pv);
    }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(smem_u32(&sm.s_full[b]), 2);
      tc::mbar_init(smem_u32(&sm.p_ready[b]), kSoftmaxWarps);
    }
    if constexpr (kClustered) {
      tc::mbar_init(smem_u32(&sm.recv_full), 1);
      if (p.n_split == 2) tc::mbar_expect_tx(smem_u32(&sm.recv_full), kRecvBytes);   // armed once; used once per launch
    }
    tc::fence_mbar_init();
  }
  if (warp == kSoftmaxWarps) {
    tc::tmem_alloc(smem_u32(&sm.tmem_slot), kTmemColsAttn);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = sm.tmem_slot;
  if (tid == 0) LSA_TL(kTlSetup);
  // Programmatic dependent launch: this block may have been placed while the previous kernel of the stream was still
  // draining; what that kernel wrote is read, and what it may still read is overwritten, only after
  // griddepcontrol.wait.  The next kernel's blocks may be placed from then on.
  // rows_stable: the row lists (and the caches, as always) were complete before the previous kernel started, so the
  // gather warps read them and put the first two key tiles in flight while that kernel drains, and wait only before
  // they request Q; every other thread waits here.
  const bool early_rows = kRows && p.rows_stable != 0 && q_tma != 0;   // block-uniform
  const bool gather_warp = warp >= kSoftmaxWarps + kMmaWarps - (kPv == 2 ? 2 : 0);
  auto dependency_wait = [&]() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  };
  // Q is requested before anything else that depends on the previous kernel: a block cannot start without it, and in
  // prefill it comes from HBM.
  auto request_q = [&]() {
    // nine boxes, dealt to lane 0 of the four gather warps (an issued TMA copy costs its thread 200-300 cycles); the
    // first of them arrives on the barrier with the byte count of all nine (a box that completes before that only
    // makes the count negative for a moment: the phase cannot end before the arrival)
    const int qw = warp - (kSoftmaxWarps + kMmaWarps);
    if (q_tma && lane == 0 && qw >= 0) {
      const uint32_t stage = smem_u32(sm.k[kKBufs - 1]);
      if (qw == 0) tc::mbar_expect_tx(smem_u32(&sm.q_full), kH * kDQK * 2);
      for (int a = qw; a < kAtoms; a += kLoadWarps)
        tc::tma_load_2d(a < 8 ? stage + a * kAtomBytes : smem_u32(sm.q_rope), &q_map, a * 64, qi * kH, smem_u32(&sm.q_full));
      if (qw == 0) LSA_TL(kTlQIssued);
    }
  };
  if (!(early_rows && gather_warp)) {
    dependency_wait();
    if (tid == 0) LSA_TL(kTlDepWait);
    request_q();
  }

  // ---- this query's row list (same conventions as the mma.sync kernel)
  const int64_t t = p.paged ? static_cast<int64_t>(p.ctx_len[qi]) - 1 : p.q_pos0 + qi;
  int n_sink = 0, n_sp = 0, n_win = 0, n_tot;
  int64_t win0 = 0;
  const int32_t* rows = nullptr;
  if constexpr (kRows) {
    rows = p.rows + static_cast<int64_t>(qi) * p.rows_ld;
    n_tot = p.n_rows[qi];
  } else {
    n_sink = static_cast<int>(min64(p.S, t + 1));
    win0 = max64(p.S, t - p.W + 1);
    n_win = static_cast<int>(max64(0, t - win0 + 1));
    n_sp = p.n_sparse[qi];
    n_tot = n_sink + n_sp + n_win;
  }
  const int32_t* sp = p.sparse_idx ? p.sparse_idx + static_cast<int64_t>(qi) * p.Ksp : nullptr;
  // Without a row list the keys are visited as [window | sink | sparse] (the order within one softmax is free): the
  // window is a run of consecutive cache rows, so its whole tiles need no per-row addressing.
  auto row_of = [&](int i) -> int32_t {
    if (i >= n_tot) return -1;
    if constexpr (kRows) {
      return checked_row(rows[i], p.n_key, p.status);
    } else {
      if (i < n_win) return static_cast<int32_t>(win0 + i);
      if (i < n_win + n_sink) return i - n_win;
      return checked_row(sp[i - n_win - n_sink], p.n_key, p.status);
    }
  };
  const int tiles_all = (n_tot + kTileKeys - 1) / kTileKeys;
  const int tiles_per = (tiles_all + p.n_split - 1) / p.n_split;
  const int tile_begin = split * tiles_per;
  int n_tiles = max(0, min(tiles_all, tile_begin + tiles_per) - tile_begin);
  if (dead) n_tiles = 0;   // the peers of this cluster still expect this block at the cluster barrier

  // With two P V issuers the other two MMA warps have nothing to issue and gather as well.
  constexpr int kGw = kLoadWarps + (kPv == 2 ? 2 : 0);
  if (warp >= kSoftmaxWarps + kMmaWarps - (kGw - kLoadWarps)) {
    // ================= gather warps =================
    // gw 0..3: warps 8-11 (they also fetch Q and issue the TMA loads); gw 4..5: warps 6-7
    const int gw = warp >= kSoftmaxWarps + kMmaWarps ? warp - (kSoftmaxWarps + kMmaWarps) : kLoadWarps + warp - (kSoftmaxWarps + kMmaWarps - 2);
    const int lt = gw * 32 + lane;
    if (gw < kLoadWarps) {
      // Q of this query: the rope part (dims 512-575) stays in shared memory as an MMA operand; dims 0-511 are staged
      // in the last key buffer for the softmax warps, which move them to tensor memory.  As TMA boxes they complete
      // q_full by themselves; as cp.async copies they form the first group, handed over with the first key tile.
      // Both ways leave dims 64a .. 64a+63 of the 64 rows in column block a of that buffer, 128-byte swizzled.
      const uint32_t stage = smem_u32(sm.k[kKBufs - 1]);
      if (!q_tma) {
        const uint8_t* qg = reinterpret_cast<const uint8_t*>(q_ptr) + static_cast<int64_t>(qi) * kH * kDQK * 2;
        for (int e = lt; e < kH * 8; e += 32 * kLoadWarps) {
          const int r = e >> 3, c = e & 7;
          cp_async16(smem_u32(sm.q_rope) + r * 128 + ((c ^ (r & 7)) << 4), qg + r * kDQK * 2 + 512 * 2 + c * 16, 16);
        }
        for (int e = lt; e < kH * 64; e += 32 * kLoadWarps) {
          const int r = e >> 6, c = e & 63;
          cp_async16(stage + (c >> 3) * kAtomBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4), qg + r * kDQK * 2 + c * 16, 16);
        }
        cp_async_commit();
      }
    }
    // Every gather warp works on every tile: warp w copies rows 16w .. 16w+15, so a freed buffer is refilled by all
    // four warps at once.  Lanes 0-15 look up the cache row of their key once; the row number is then broadcast
    // and the 72 16-byte chunks of that row are copied by consecutive lanes (coalesced 512-byte requests: a row is
    // fetched whole, by one warp, in back-to-back instructions.  Spreading the chunks of a tile evenly over the warps,
    // every instruction full, was measured at 1.3 x the time, in prefill and in decode).
    // rows of a tile a warp copies: 16 each with four warps; 11, 11, 11, 11, 10, 10 with six
    const int row_first = kGw == 4 ? 16 * gw : (gw <= 4 ? 11 * gw : 54);
    const int n_my_rows = kGw == 4 ? 16 : (gw < 4 ? 11 : 10);
    const uint8_t* kg = reinterpret_cast<const uint8_t*>(k_ptr);
    auto tile_by_tma = [&](int i) -> bool {   // block-uniform
      return !kRows && k_tma && (tile_begin + i + 1) * kTileKeys <= n_win;
    };
    // TMA gather (k_g4): thread lt < 128 fetches row quad lt / 8 (tile rows 4 * quad .. + 3) of column block lt % 8, and
    // the threads with lt % 8 == 0 also the rope block: 144 instructions per tile.
    const bool g4 = k_g4 != 0;   // block-uniform
    const int quad = (lt >> 3) & 15, atom0 = lt & 7;
    auto my_key_row = [&](int i) -> int32_t {
      return (!g4 && i < n_tiles && lane < n_my_rows && !tile_by_tma(i)) ? row_of((tile_begin + i) * kTileKeys + row_first + lane) : -1;
    };
    auto my_quad_rows = [&](int i) -> int4 {
      int4 r = make_int4(0, 0, 0, 0);
      if (g4 && gw < kLoadWarps && i < n_tiles && !tile_by_tma(i)) {
        const int i0 = (tile_begin + i) * kTileKeys + 4 * quad;
        if (kRows && i0 + 3 < n_tot && ((reinterpret_cast<uintptr_t>(rows + i0) & 15u) == 0)) {
          r = *reinterpret_cast<const int4*>(rows + i0);
        } else {
          r.x = row_of(i0); r.y = row_of(i0 + 1); r.z = row_of(i0 + 2); r.w = row_of(i0 + 3);
        }
        // rows past the end of the list are masked in the softmax: any readable row will do
        r.x = max(r.x, 0); r.y = max(r.y, 0); r.z = max(r.z, 0); r.w = max(r.w, 0);
      }
      return r;
    };
    int32_t my_row = my_key_row(0);
    int4 my_rows4 = my_quad_rows(0);
    bool waited = !early_rows;   // this thread has executed the dependency wait
    // Copies of up to three tiles are in flight: a tile is handed to the MMA issuers (k_full) when its cp.async group
    // has landed, which is looked at after the next tile's copies are issued, or at once when no buffer is free.
    int first_pend = 0, n_pend = 0;   // tiles first_pend .. first_pend + n_pend - 1 are issued but not handed over
    bool q_handed = q_tma != 0 || gw >= kLoadWarps;   // TMA completes q_full by itself; the extra warps fetch no Q
    auto hand_over_q = [&]() {        // call after a wait that covers the first group
      tc::fence_proxy_async();
      tc::mbar_arrive(smem_u32(&sm.q_full));
      q_handed = true;
    };
    auto hand_over_oldest = [&]() {
      if (n_pend >= 3) cp_async_wait<2>();
      else if (n_pend == 2) cp_async_wait<1>();
      else cp_async_wait<0>();
      if (!q_handed) hand_over_q();
      tc::fence_proxy_async();
      tc::mbar_arrive(smem_u32(&sm.k_full[first_pend % kKBufs]));
      ++first_pend;
      --n_pend;
    };
    for (int i = 0; i < n_tiles; ++i) {
      const int b = i % kKBufs;
      const uint32_t par = ((i / kKBufs) & 1) ^ 1;
      const int32_t next_row = my_key_row(i + 1);   // fetched before the wait: off the critical path
      const int4 next_rows4 = my_quad_rows(i + 1);
      // Q and the first tile go out alone: requested together with the next tiles they would share the memory pipe
      // with them and the first Q K^T would start two tiles' worth of traffic later
      if (i == 1) while (n_pend > 0) hand_over_oldest();
      if (i == kKBufs - 1) {
        if (!waited) {   // two tiles are in flight: now the previous kernel must be done, then Q goes out
          dependency_wait();
          request_q();
          waited = true;
        }
        // first use of the buffer that staged Q: the softmax warps must have moved Q to tensor memory
        while (n_pend > 0 && !__all_sync(0xffffffffu, tc::mbar_test(smem_u32(&sm.q_tmem), 0))) hand_over_oldest();
        if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.q_tmem), 0, p.status))) break;
      }
      while (n_pend > 0 && !__all_sync(0xffffffffu, tc::mbar_test(smem_u32(&sm.k_empty[b]), par))) hand_over_oldest();
      if (!__all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.k_empty[b]), par, p.status))) break;
      LSA_TL_TILE(lt == 0, i, kTlKFreed);
      if (tile_by_tma(i)) {
        // 64 consecutive window rows: nine boxes that complete k_full by byte count; the (empty) cp.async group
        // below keeps the hand-over bookkeeping the same for every kind of tile.  An issued TMA copy costs its thread
        // 200-300 cycles, so the nine boxes are dealt to the gather warps (each announces the bytes of its own)
        if (lane == 0 && gw < kAtoms) {
          const int n_mine = (kAtoms - gw + kGw - 1) / kGw;
          tc::mbar_expect_tx_only(smem_u32(&sm.k_full[b]), n_mine * kAtomBytes);
          const int row0 = static_cast<int>(win0) + (tile_begin + i) * kTileKeys;
          for (int a = gw; a < kAtoms; a += kGw)
            tc::tma_load_2d(smem_u32(sm.k[b][a]), &k_map, a * 64, row0, smem_u32(&sm.k_full[b]));
        }
      } else if (g4) {
        // scattered rows: four rows x 64 dims per instruction, straight into their place in the swizzled tile
        if (lt == 0) tc::mbar_expect_tx_only(smem_u32(&sm.k_full[b]), kAtoms * kAtomBytes);
        if (gw < kLoadWarps)
          tc::tma_gather4_2d(smem_u32(sm.k[b][atom0]) + quad * 512, &g_map, atom0 * 64, my_rows4.x, my_rows4.y, my_rows4.z,
                             my_rows4.w, smem_u32(&sm.k_full[b]));
        if (gw < kLoadWarps && atom0 == 0)
          tc::tma_gather4_2d(smem_u32(sm.k[b][kAtoms - 1]) + quad * 512, &g_map, (kAtoms - 1) * 64, my_rows4.x, my_rows4.y,
                             my_rows4.z, my_rows4.w, smem_u32(&sm.k_full[b]));
      } else {
#pragma unroll 4
        for (int rr = 0; rr < n_my_rows; ++rr) {
          const int32_t row = __shfl_sync(0xffffffffu, my_row, rr);
          const int r = row_first + rr;
          const uint8_t* src = kg + static_cast<int64_t>(row >= 0 ? row : 0) * p.ld_k * 2;
          const int nb = row >= 0 ? 16 : 0;
#pragma unroll
          for (int c = lane; c < 72; c += 32)
            cp_async16(smem_u32(sm.k[b][c >> 3]) + r * 128 + (((c & 7) ^ (r & 7)) << 4), src + c * 16, nb);
        }
      }
      cp_async_commit();
      LSA_TL_IF(lt == 0 && i == 0, kTlTile0Issued);
      LSA_TL_TILE(lt == 0, i, kTlKIssued);
      ++n_pend;
      if (n_pend == kKBufs) hand_over_oldest();
      my_row = next_row;
      my_rows4 = next_rows4;
    }
    while (n_pend > 0) hand_over_oldest();
    if (!q_handed) {
      cp_async_wait<0>();
      hand_over_q();
    }
    if (!waited) {   // fewer than three tiles: Q has not been requested yet
      dependency_wait();
      request_q();
    }
  } else if (warp >= kSoftmaxWarps) {
    // ================= MMA issuers =================
    const int x = warp - kSoftmaxWarps;   // 0..3
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t idesc_qk = tc::idesc_bf16(kH, kTileKeys, 0, 0);
      constexpr uint32_t idesc_pv = n_pv == 4 ? tc::idesc_bf16(kH, 128, 0, 1) : tc::idesc_bf16(kH, 256, 0, 1);   // B = V read MN-major
      bool ok = tc::mbar_wait(smem_u32(&sm.q_full), 0, p.status) && tc::mbar_wait(smem_u32(&sm.q_tmem), 0, p.status);
      LSA_TL_IF(x == 0, kTlQInTmem);
      // Descriptors are built once; inside the loops only the start-address word moves (one add per operand).
      constexpr uint32_t kBufBytes = kAtoms * kAtomBytes;
      const uint64_t dqr = tc::smem_desc_sw128(smem_u32(sm.q_rope), 16, 1024);
      const uint64_t dk0 = tc::smem_desc_sw128(smem_u32(sm.k), 16, 1024);           // K-major view (Q K^T)
      const uint64_t dv0 = tc::desc_advance(tc::smem_desc_sw128(smem_u32(sm.k), kAtomBytes, 1024), (n_pv == 4 ? 2 : 4) * x * kAtomBytes);  // MN-major view (P V)
      constexpr uint32_t kLane16 = 16u << 16;
      // Q K^T (issuers 0 and 1): chain x = dims 256x .. 256x+255 with Q from tensor memory (lane half x), plus two of
      // the four rope steps with Q from shared memory; its partial sum goes to lane half x of the S buffer
      const uint32_t q_src = tmem_base + (x & 1) * kLane16 + kColQ;
      const uint32_t s_dst = tmem_base + (x & 1) * kLane16 + kColS;
      // P V (all four issuers): value dims 128x .. 128x+127 = columns 128*(x&1) .. of the accumulator in lane half
      // x>>1; P is read from the same lane half
      const uint32_t o_dst = n_pv == 4 ? tmem_base + (x >> 1) * kLane16 + (x & 1) * 128 : tmem_base + (x & 1) * kLane16;
      const uint32_t p_src = tmem_base + (n_pv == 4 ? (x >> 1) : (x & 1)) * kLane16 + kColS;
      auto issue_qk = [&](int i) {
        tc::fence_after_sync();
        const uint32_t d = s_dst + (i & 1) * kSBuf;
        const uint64_t dkb = tc::desc_advance(dk0, (i % kKBufs) * kBufBytes);
#pragma unroll
        for (int s = 0; s < 16; ++s)   // dims 256x + 16s .. +15: column block 4x + s/4, 32-byte slice s%4
          tc::umma_ts(d, q_src + 8 * s, tc::desc_advance(dkb, (4 * x + (s >> 2)) * kAtomBytes + (s & 3) * 32), idesc_qk, s != 0);
#pragma unroll
        for (int s = 0; s < 2; ++s)    // rope dims 512 + 32x + 16s .. +15
          tc::umma_ss(d, tc::desc_advance(dqr, (2 * x + s) * 32), tc::desc_advance(dkb, 8 * kAtomBytes + (2 * x + s) * 32), idesc_qk, 1);
        LSA_TL_TILE(x == 0, i, kTlQkMmas);
        tc::umma_commit(smem_u32(&sm.s_full[i & 1]));
      };
      auto issue_pv = [&](int j) {   // O[:, 128x : 128x+128] += P_j V_j
        tc::fence_after_sync();
        const uint64_t dvb = tc::desc_advance(dv0, (j % kKBufs) * kBufBytes);
#pragma unroll
        for (int kk = 0; kk < kTileKeys / 16; ++kk)   // keys 16*kk .. +15
          tc::umma_ts(o_dst, p_src + (j & 1) * kSBuf + kk * 8, tc::desc_advance(dvb, kk * 2048), idesc_pv, (j > 0) || (kk > 0));
        LSA_TL_TILE(x == 0, j, kTlPvMmas);
        // one completion signal per tile: "P V of tile j done" frees the key buffer for the gather warps and tells the
        // softmax warps (and, with four issuers, the Q K^T issuers) that O and the P columns may be touched again.
        // Several parties watch the same phase: it cannot flip twice before they have looked, because the P V of tile
        // j + 3 needs work of theirs that comes after the look.
        tc::umma_commit(smem_u32(&sm.k_empty[j % kKBufs]));
      };
      const bool does_qk = x < 2;
      const bool wait_pv = p.qk_waits_pv != 0 || n_pv != 2;
      // Two in-order queues, "next Q K^T" (at most one tile ahead of the softmax it feeds) and "next P V".
      // Whatever follows a batch of MMAs in this thread - a clock read, a barrier probe - waits until the batch has
      // left the issue stage, which costs a hundred cycles and more each time: the clock is read only while spinning
      // and a P V ends with one commit.  Whichever of the two is ready goes first; when both are, Q K^T (the softmax it
      // feeds is the longer chain).  Issuing the ready P V right behind a Q K^T without looking at the barriers in
      // between was measured: faster while whole window tiles stream in, slower on gathered tiles, where the later
      // completion of that P V holds up the refill of its key buffer; dropped.
      auto pv_done = [&](int j) -> bool {   // j >= 0
        return tc::mbar_test(smem_u32(&sm.k_empty[j % kKBufs]), (j / kKBufs) & 1);
      };
      int qk_next = does_qk ? 0 : n_tiles, pv_next = x < n_pv ? 0 : n_tiles;
      long long t_idle = 0;
      uint32_t spins = 0;
      while (ok && pv_next < n_tiles) {
        bool did = false;
        // P V first: its completion frees a key buffer, and the refill of that buffer is the longest latency of the ring
        if ((!does_qk || pv_next < qk_next) && tc::mbar_test(smem_u32(&sm.p_ready[pv_next & 1]), (pv_next >> 1) & 1)) {
          LSA_TL_TILE(x == 0, pv_next, kTlPvIssue0);
          issue_pv(pv_next++);
          LSA_TL_TILE(x == 0, pv_next - 1, kTlPvIssue1);
          did = true;
        }
        if (!did && qk_next < n_tiles && qk_next <= pv_next + 1) {
          // S buffer qk_next&1 also holds P of tile qk_next-2: it is free once that tile's P V has completed
          if (tc::mbar_test(smem_u32(&sm.k_full[qk_next % kKBufs]), (qk_next / kKBufs) & 1) &&
              (!wait_pv || qk_next < 2 || pv_done(qk_next - 2))) {
            LSA_TL_IF(x == 0 && qk_next == 0, kTlTile0Landed);
            LSA_TL_TILE(x == 0, qk_next, kTlQkIssue0);
            issue_qk(qk_next++);
            LSA_TL_TILE(x == 0, qk_next - 1, kTlQkIssue1);
            did = true;
          }
        }
        if (did) {
          spins = 0;
        } else if ((++spins & 255u) == 0) {
          // bounded: nothing became ready for about a second (the clock is read only while spinning)
          if (tc::status_raised(p.status)) {
            ok = false;
          } else {
            const long long now = clock64();
            if (spins == 256u) {
              t_idle = now;
            } else if (now - t_idle > tc::kWaitCycles) {
              report_status(p.status, kDevTimeout);
              ok = false;
            }
          }
        }
      }
    }
  } else {
    // ================= softmax warps =================
    const int quarter = warp;                 // TMEM lanes 32*warp .. +31
    const int r16 = lane & 15, hi = lane >> 4;
    const int row = 16 * quarter + r16;       // head; lanes l and l+16 share it: keys 0-31 / 32-63, O dims 0-255 / 256-511
    const uint32_t lane_addr = static_cast<uint32_t>(32 * quarter) << 16;
    bool ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.q_full), 0, p.status));
    {
      // Q[row, 256*hi : 256*hi+256] from the staging buffer -> 128 columns of this lane, in the order the tensor core
      // reads an A operand (two consecutive dims per 32-bit column)
      const uint8_t* qs = sm.k[kKBufs - 1][0] + row * 128;
#pragma unroll 1
      for (int part = 0; part < 2; ++part) {
        uint32_t w[64];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int c = 32 * hi + 16 * part + j;
          const uint4 u = *reinterpret_cast<const uint4*>(qs + (c >> 3) * kAtomBytes + (((c & 7) ^ (row & 7)) << 4));
          w[4 * j] = u.x; w[4 * j + 1] = u.y; w[4 * j + 2] = u.z; w[4 * j + 3] = u.w;
        }
        tc::tmem_st64(tmem_base + lane_addr + kColQ + part * 64, w);
        tc::tmem_st_wait();
      }
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(smem_u32(&sm.q_tmem));
    }
    const float zs = p.sm_scale * kLog2eTc;
    float m_used = -INFINITY, l_run = 0.f;    // m_used is kept identical in both lanes of a row; l_run is a partial sum
    for (int i = 0; i < n_tiles && ok; ++i) {
      const int b = i & 1;
      ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.s_full[b]), (i >> 1) & 1, p.status));
      if (!ok) break;
      LSA_TL_IF(tid == 0 && i == 0, kTlS0);
      LSA_TL_TILE(tid == 0, i, kTlSFull);
      tc::fence_after_sync();
      const uint32_t s_addr = tmem_base + lane_addr + kColS + b * kSBuf;
      uint32_t v[32];
      {
        // This lane holds one chain's partial sums for all 64 keys, its partner lane (l ^ 16) the other's.  Lane l
        // keeps keys 0-31, lane l+16 keys 32-63: send the half the partner finishes, add the one it sends.
        uint32_t s64[64];
        tc::tmem_ld64(s_addr, s64);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float give = __uint_as_float(hi ? s64[j] : s64[32 + j]);
          const float keep = __uint_as_float(hi ? s64[32 + j] : s64[j]);
          v[j] = __float_as_uint(keep + __shfl_xor_sync(0xffffffffu, give, 16));
        }
      }
      LSA_TL_TILE(tid == 0, i, kTlSLoaded);
      // logits in log2 units, ragged tail masked
      const int n_valid = n_tot - (tile_begin + i) * kTileKeys - kHalfKeys * hi;   // keys of this lane's half that exist
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float z = j < n_valid ? __uint_as_float(v[j]) * zs : -INFINITY;
        v[j] = __float_as_uint(z);
        mx = fmaxf(mx, z);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      // running max, moved only when it grows by more than kRescaleGap (O and l are then rescaled)
      float alpha = 1.f;
      if (i == 0) {
        m_used = mx;
      } else if (mx > m_used + kRescaleGap) {
        alpha = exp2f(m_used - mx);
        m_used = mx;
      }
      if (__any_sync(0xffffffffu, alpha != 1.f)) {
        // O may be touched only between P V of tile i-1 (done) and P V of tile i (not yet released)
        ok = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.k_empty[(i - 1) % kKBufs]), ((i - 1) / kKBufs) & 1, p.status));
        if (!ok) break;
        tc::fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < 256; c += 64) {
          uint32_t o[64];
          tc::tmem_ld64(tmem_base + lane_addr + c, o);
          tc::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 64; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
          tc::tmem_st64(tmem_base + lane_addr + c, o);
        }
        tc::tmem_st_wait();
        l_run *= alpha;
        tc::fence_before_sync();
      }
      // P = exp2(z - m), fp32 row sum, bf16 pack
      uint32_t pk[16];
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float p0 = exp2f(__uint_as_float(v[2 * j]) - m_used);
        const float p1 = exp2f(__uint_as_float(v[2 * j + 1]) - m_used);
        sum += p0 + p1;
        pk[j] = pack_bf16(p0, p1);
      }
      l_run += sum;
      {
        // The A operand of P V sits in tensor memory, in the lanes of the accumulator it feeds: both lanes of a
        // row need all 64 keys, so the two halves are swapped in, then written as 32 columns of packed bf16.
        uint32_t full[32];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t other = __shfl_xor_sync(0xffffffffu, pk[j], 16);
          full[j] = hi ? other : pk[j];
          full[16 + j] = hi ? pk[j] : other;
        }
        tc::tmem_st32(s_addr, full);   // over the first 32 columns of the S buffer this lane has just read
        tc::tmem_st_wait();
        tc::fence_before_sync();
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(smem_u32(&sm.p_ready[b]));
      LSA_TL_TILE(tid == 0, i, kTlPHanded);
      LSA_TL_TILE(tid == 32, i, kTlPHanded1);
      LSA_TL_TILE(tid == 64, i, kTlPHanded2);
      LSA_TL_TILE(tid == 96, i, kTlPHanded3);
    }
    if (tid == 0) LSA_TL(kTlLastP);
    // ---- epilogue: O / l
    const float l_row = l_run + __shfl_xor_sync(0xffffffffu, l_run, 16);
    const float m_row = m_used;
    bool have_o = ok && n_tiles > 0;
    if (have_o) have_o = __all_sync(0xffffffffu, tc::mbar_wait(smem_u32(&sm.k_empty[(n_tiles - 1) % kKBufs]), ((n_tiles - 1) / kKBufs) & 1, p.status));
    tc::fence_after_sync();
    if (pair) cluster_arrive();   // this thread has left the tile loop, and every P V of the block has completed
    if (tid == 0) LSA_TL(kTlLastPV);
    const float inv = (have_o && l_row > 0.f) ? 1.f / l_row : 0.f;
    const float lse2 = (have_o && l_row > 0.f) ? m_row + log2f(l_row) : -INFINITY;   // log2 domain
    uint8_t* stage = &sm.k[0][0][0];
    if (!clustered) {
      // The block's output is one contiguous piece of memory (64 rows of 512 bf16).  A thread owns half a row, so
      // direct stores would scatter 16-byte pieces over 32 rows per instruction; instead each warp lays its 16 rows
      // out in the (now idle) key buffers, with a 16-byte pad per row against bank conflicts, and every row leaves
      // as one bulk copy.
      constexpr int kRowBytes = kDV * 2, kPitch = kRowBytes + 16;
      uint8_t* my_stage = stage + row * kPitch + hi * (kRowBytes / 2);
#pragma unroll 1
      for (int c = 0; c < 256; c += 64) {
        uint32_t o[64];
        if (have_o) {
          tc::tmem_ld64(tmem_base + lane_addr + c, o);
          tc::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 64; ++j) o[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint4 w4;
          w4.x = pack_bf16(__uint_as_float(o[8 * j + 0]) * inv, __uint_as_float(o[8 * j + 1]) * inv);
          w4.y = pack_bf16(__uint_as_float(o[8 * j + 2]) * inv, __uint_as_float(o[8 * j + 3]) * inv);
          w4.z = pack_bf16(__uint_as_float(o[8 * j + 4]) * inv, __uint_as_float(o[8 * j + 5]) * inv);
          w4.w = pack_bf16(__uint_as_float(o[8 * j + 6]) * inv, __uint_as_float(o[8 * j + 7]) * inv);
          *reinterpret_cast<uint4*>(my_stage + (c + 8 * j) * 2) = w4;
        }
      }
      tc::fence_proxy_async();
      __syncwarp();
      uint8_t* dst = reinterpret_cast<uint8_t*>(reinterpret_cast<__nv_bfloat16*>(out_ptr) + static_cast<int64_t>(qi) * kH * kDV);
      if (hi == 0) {   // one bulk copy per row, issued by the lane that staged the row's first half
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     :: "l"(dst + static_cast<int64_t>(row) * kRowBytes), "r"(smem_u32(stage + row * kPitch)), "n"(kRowBytes) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the staging buffer must outlive the copy
      }
      if (hi == 0 && lse_ptr != nullptr) lse_ptr[static_cast<int64_t>(qi) * kH + row] = lse2 / kLog2eTc;
    } else {
      // partial result of a split: normalised fp32 rows in the key buffers
      const bool foreign = pair && row / (kH / 2) != split;   // warp-uniform: a warp stages 16 consecutive rows
      const uint32_t peer = static_cast<uint32_t>(split ^ 1);
      const int peer_row0 = (kH / 2) * (split ^ 1);
      uint32_t bar_peer = 0, dst_peer = 0;
      if (foreign) {
        // into the peer's shared memory, once every thread of the peer has left its tile loop (first half of the
        // cluster barrier: its key buffers, which receive the rows, are then out of use)
        cluster_wait();
        bar_peer = peer_smem(smem_u32(&sm.recv_full), peer);
        dst_peer = peer_smem(smem_u32(stage + kRecvOffset + (16 * quarter - peer_row0) * kPairRowBytes), peer);
      }
      uint8_t* my_row = stage + row * kPitchPart;                        // (four or eight splits: padded rows)
      uint8_t* my_warp = stage + 16 * quarter * kPairRowBytes;           // (two splits: this warp's 32 KB)
#pragma unroll 1
      for (int c = 0; c < 256; c += 64) {
        uint32_t o[64];
        if (have_o) {
          tc::tmem_ld64(tmem_base + lane_addr + c, o);
          tc::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 64; ++j) o[j] = 0u;
        }
        if (pair) {
          uint8_t* piece = my_warp + (c / 64) * 8192 + hi * 4096 + r16 * 256;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            *reinterpret_cast<float4*>(piece + ((j ^ r16) << 4)) =
                make_float4(__uint_as_float(o[4 * j]) * inv, __uint_as_float(o[4 * j + 1]) * inv,
                            __uint_as_float(o[4 * j + 2]) * inv, __uint_as_float(o[4 * j + 3]) * inv);
          if (foreign) {
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0)
              bulk_copy_to_peer(dst_peer + (c / 64) * 8192, smem_u32(my_warp + (c / 64) * 8192), 8192, bar_peer);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)   // 16-byte chunk hi * 64 + c / 4 + j of the row
            *reinterpret_cast<float4*>(my_row + ((hi * 64 + c / 4 + j) << 4)) =
                make_float4(__uint_as_float(o[4 * j]) * inv, __uint_as_float(o[4 * j + 1]) * inv,
                            __uint_as_float(o[4 * j + 2]) * inv, __uint_as_float(o[4 * j + 3]) * inv);
        }
      }
      if (hi == 0) {
        sm.lse_own[row] = lse2;
        if (!pair) part_lse[(static_cast<int64_t>(qi) * p.n_split + split) * kH + row] = lse2;
      }
      // Rows that another block of the cluster finishes leave as soon as this warp has staged them, while the other
      // softmax warps are still staging.
      tc::fence_proxy_async();
      __syncwarp();
      if (pair) {
        if (foreign) {
          if (lane == 0)   // the log-sum-exps of the warp's 16 rows
            bulk_copy_to_peer(peer_smem(smem_u32(&sm.lse_peer[16 * quarter - peer_row0]), peer), smem_u32(&sm.lse_own[16 * quarter]),
                              16 * 4, bar_peer);
        } else {
          cluster_wait();   // (every thread passes the first half of the barrier once)
        }
      } else {
        const int rows_per = kH / p.n_split;
        if (hi == 0 && row / rows_per != split) {   // one bulk copy per row (2 KB), issued by the lane that holds its first half
          float* dst = part_out + ((static_cast<int64_t>(qi) * p.n_split + split) * kH + row) * kDV;
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                       :: "l"(dst), "r"(smem_u32(stage + row * kPitchPart)), "n"(kDV * 4) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
    }
  }
  // the threads of the other roles have left the tile loop too
  if (pair && warp >= kSoftmaxWarps) cluster_arrive();
  if (tid == 0) LSA_TL(kTlStaged);
  tc::fence_before_sync();
  __syncthreads();
  if (tid == 0) LSA_TL(kTlSynced);
  if (warp == kSoftmaxWarps) tc::tmem_dealloc(tmem_base, kTmemColsAttn);
  if (clustered) {
    // ---- merge of the splits (Sec. 4.1.1: online-softmax rescaling) for this block's heads: weights
    // 2^(lse_j - max) / sum, O = sum_j w_j O_j, bf16 to global.
    const int n = p.n_split;
    const int rows_per = kH / n;
    const int row0 = split * rows_per;
    const uint8_t* stage = &sm.k[0][0][0];
    constexpr int kWarps = kThreadsAttnTc / 32;
    if (pair) {
      if (warp >= kSoftmaxWarps) cluster_wait();   // (the softmax warps completed this phase before they sent)
      // the peer's rows for this block's heads, and their log-sum-exps, are in shared memory when the byte count is met
      (void)tc::mbar_wait(smem_u32(&sm.recv_full), 0, p.status);
      if (tid == 0) LSA_TL(kTlClusterSync);
      // Second use of the cluster barrier: a block may leave once the peer has everything it was sent (until then the
      // copies still read this block's shared memory).  A thread arrives as soon as it has seen this block's own
      // bytes complete and waits at the very end, by when the peer has normally long arrived.
      cluster_arrive();
      __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(out_ptr) + (static_cast<int64_t>(qi) * kH + row0) * kDV;
#pragma unroll
      for (int rl = warp; rl < kH / 2; rl += kWarps) {   // a warp finishes a row: lane l the chunks l, l + 32, ...
        const int R = row0 + rl;
        const float l_own = sm.lse_own[R], l_peer = sm.lse_peer[rl];
        const float m = fmaxf(l_own, l_peer);
        float w_own = m > -INFINITY ? exp2f(l_own - m) : 0.f, w_peer = m > -INFINITY ? exp2f(l_peer - m) : 0.f;
        const float den = w_own + w_peer;
        const float r_den = den > 0.f ? 1.f / den : 0.f;
        w_own *= r_den;
        w_peer *= r_den;
        if (lane == 0 && lse_ptr != nullptr)
          lse_ptr[static_cast<int64_t>(qi) * kH + R] = den > 0.f ? (m + log2f(den)) / kLog2eTc : -INFINITY;
        // row R = row R % 16 of staging warp R / 16 (here and in the peer, whose warp 2 * split + rl / 16 sent it)
        const uint8_t* a_warp = stage + (R >> 4) * (16 * kPairRowBytes);
        const uint8_t* b_warp = stage + kRecvOffset + (rl >> 4) * (16 * kPairRowBytes);
        const int r16m = R & 15;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int chunk = lane + 32 * u;   // 16-byte chunk of the row: value-dim half chunk / 64, step (chunk % 64) / 16
          const int ch = (chunk >> 6) * 4096 + ((chunk & 63) >> 4) * 8192 + r16m * 256 + (((chunk & 15) ^ r16m) << 4);
          const float4 a = *reinterpret_cast<const float4*>(a_warp + ch), b = *reinterpret_cast<const float4*>(b_warp + ch);
          uint2 o;
          o.x = pack_bf16(w_own * a.x + w_peer * b.x, w_own * a.y + w_peer * b.y);
          o.y = pack_bf16(w_own * a.z + w_peer * b.z, w_own * a.w + w_peer * b.w);
          *reinterpret_cast<uint2*>(out + static_cast<int64_t>(rl) * kDV + (lane + 32 * u) * 4) = o;
        }
      }
      if (tid == 0) LSA_TL(kTlMerged);
      cluster_wait();   // (see the arrival above)
    } else {
      if (warp < kSoftmaxWarps) {   // the threads that sent rows wait until they are written (not only read out of shared memory)
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __threadfence();
      }
      if (tid == 0) LSA_TL(kTlSent);
      cluster_sync_all();   // every block of the cluster has written its rows
      if (tid == 0) LSA_TL(kTlClusterSync);
    // Warp w finishes rows w, w + 12, ... of this block's share (at most three).  Lane 8k + j first fetches the
    // log-sum-exp of split j for the warp's k-th row, so that all of them are in flight together.
    const int k_of = lane >> 3, j_of = lane & 7;
    const int rl_mine = warp + kWarps * k_of;
    float my_l = -INFINITY;
    if (k_of < 3 && rl_mine < rows_per && j_of < n)
      my_l = j_of == split ? sm.lse_own[row0 + rl_mine]
                           : __ldcg(part_lse + (static_cast<int64_t>(qi) * n + j_of) * kH + row0 + rl_mine);
    float m = my_l;
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    float wgt = m > -INFINITY ? exp2f(my_l - m) : 0.f;
    float den = wgt;
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) den += __shfl_xor_sync(0xffffffffu, den, d);
    wgt = den > 0.f ? wgt / den : 0.f;
    if (lse_ptr != nullptr && j_of == 0 && k_of < 3 && rl_mine < rows_per)
      lse_ptr[static_cast<int64_t>(qi) * kH + row0 + rl_mine] = den > 0.f ? (m + log2f(den)) / kLog2eTc : -INFINITY;
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(out_ptr) + (static_cast<int64_t>(qi) * kH + row0) * kDV;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      const int rl = warp + kWarps * k;   // warp-uniform
      if (rl < rows_per) {
        float4 acc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < n; ++j) {
          const float w = __shfl_sync(0xffffffffu, wgt, 8 * k + j);
          float4 v[4];
          if (j == split) {
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const float4*>(stage + (row0 + rl) * kPitchPart + (lane + 32 * u) * 16);
          } else {
            const float4* src = reinterpret_cast<const float4*>(part_out + ((static_cast<int64_t>(qi) * n + j) * kH + row0 + rl) * kDV);
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldcg(src + lane + 32 * u);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            acc[u].x += w * v[u].x; acc[u].y += w * v[u].y; acc[u].z += w * v[u].z; acc[u].w += w * v[u].w;
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          uint2 o;
          o.x = pack_bf16(acc[u].x, acc[u].y);
          o.y = pack_bf16(acc[u].z, acc[u].w);
          *reinterpret_cast<uint2*>(out + static_cast<int64_t>(rl) * kDV + (lane + 32 * u) * 4) = o;
        }
      }
    }
    if (tid == 0) LSA_TL(kTlMerged);
    }   // four or eight splits
  }
  if (tid == 0) {
    LSA_TL(kTlExit);
    LSA_WALL(1);
  }
}

}  // namespace

// Largest cluster of full-SM blocks of this kernel the device can place (queried once per process).
static_assert(sizeof(AttnTcSmem) + 1024 <= 227 * 1024, "shared memory of the attention kernel exceeds one SM");

using AttnTcKernel = void (*)(CUtensorMap, int, CUtensorMap, int, CUtensorMap, int, AttnArgs);

// The instantiation that serves a call (see the kernel's template parameters).
static AttnTcKernel pick_kernel(const AttnArgs& a) {
  const bool rows = a.rows != nullptr;
  if (!rows) return a.pv_issuers == 4 ? sparse_attn_tc_kernel<false, 4, false> : sparse_attn_tc_kernel<false, 2, false>;
  if (a.n_split > 1) return a.pv_issuers == 4 ? sparse_attn_tc_kernel<true, 4, true> : sparse_attn_tc_kernel<true, 2, true>;
  return a.pv_issuers == 4 ? sparse_attn_tc_kernel<true, 4, false> : sparse_attn_tc_kernel<true, 2, false>;
}

static int max_cluster_blocks() {
  static const int n = [] {
    const size_t smem = sizeof(AttnTcSmem) + 1024;
    AttnTcKernel kernel = sparse_attn_tc_kernel<true, 4, true>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) return 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1, kMaxClusterSplit);
    cfg.blockDim = dim3(kThreadsAttnTc);
    cfg.dynamicSmemBytes = smem;
    int size = 0;
    const cudaError_t eq = cudaOccupancyMaxPotentialClusterSize(&size, kernel, &cfg);
    if (eq != cudaSuccess) {
      (void)cudaGetLastError();
      return 1;
    }
    return size < 1 ? 1 : size;
  }();
  return n;
}

// Row splits the tcgen05 kernel can merge inside a cluster: a power of two that divides the 64 heads, at most 8 blocks
// and at most what the device can co-schedule.
bool attn_tc_split_ok(int n_split) {
  if (n_split == 1) return true;
  return (n_split == 2 || n_split == 4 || n_split == 8) && n_split <= max_cluster_blocks();
}

bool attn_tc_supported(const AttnArgs& a) {
  return a.H == kH && a.DQK == kDQK && a.DV == kDV && a.v == a.k && a.ld_v == a.ld_k;
}

cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t st, int64_t* n_launch) {
  if (a.n_query == 0) return cudaSuccess;
  const size_t smem = sizeof(AttnTcSmem) + 1024;
  if (a.n_split > 1 && a.rows == nullptr) return cudaErrorInvalidValue;   // row splits walk row lists
  AttnTcKernel kernel = pick_kernel(a);
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  CUtensorMap q_map{}, k_map{}, g_map{};
  const int q_tma = (reinterpret_cast<uintptr_t>(a.q) & 15u) == 0 &&
                    make_map_bf16_rows(&q_map, a.q, kDQK, static_cast<uint64_t>(a.n_query) * kH, kH);
  // contiguous cache: the last query sees rows 0 .. q_pos0 + n_query - 1, so the cache holds at least that many
  const int k_tma = !a.paged && a.rows == nullptr && a.ld_k % 8 == 0 && (reinterpret_cast<uintptr_t>(a.k) & 15u) == 0 &&
                    make_map_bf16_rows(&k_map, a.k, static_cast<uint64_t>(a.ld_k), static_cast<uint64_t>(a.q_pos0 + a.n_query), kTileKeys);
  // gather of scattered rows by TMA: any cache whose base and row pitch TMA can address; a paged pool's row count is
  // not known here (every row number comes from the caller's list), so its map spans the whole coordinate range
  const uint64_t g_rows = a.paged || a.rows != nullptr ? 0x7fffffffull : static_cast<uint64_t>(a.q_pos0 + a.n_query);
  const int k_g4 = a.gather4 && a.ld_k % 8 == 0 && (reinterpret_cast<uintptr_t>(a.k) & 15u) == 0 &&
                   make_map_bf16_rows(&g_map, a.k, static_cast<uint64_t>(a.ld_k), g_rows, 1);
  if (a.n_split <= 1) {
    kernel<<<dim3(a.n_query, 1, 1), kThreadsAttnTc, smem, st>>>(q_map, q_tma, k_map, k_tma, g_map, k_g4, a);
  } else {
    if (!attn_tc_split_ok(a.n_split)) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(a.n_query, a.n_split, 1);
    cfg.blockDim = dim3(kThreadsAttnTc);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2]{};
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = static_cast<unsigned>(a.n_split);
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol.wait in the kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    e = cudaLaunchKernelEx(&cfg, kernel, q_map, q_tma, k_map, k_tma, g_map, k_g4, a);
    if (e != cudaSuccess) return e;
  }
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace lsa
