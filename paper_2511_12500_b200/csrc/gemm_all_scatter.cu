// GEMM + all-scatter over the emulated symmetric heap, three schedules (Section 4, Listings 2-5).
//
// Two persistent, warp-specialised tcgen05 kernels share this file:
//   gemm_all_scatter_pair_kernel  a cluster of two CTAs per 256 x 256 tile (cta_group::2), tile ids claimed in
//                                 raster order; the default whenever M > 128 and N/world > 128 (ragged edges are
//                                 zero-filled by the loads and clipped by the stores)
//   gemm_all_scatter_kernel       one CTA per 128 x 256 or 128 x 128 tile, static tile stride or stream-K; the
//                                 skinny and the tiny shapes (TMA zero fill on loads, masks on stores)
// Warp roles in a producer CTA:
//   warp 0      TMA producer  (cp.async.bulk.tensor -> 128B-swizzled shared-memory stages, mbarrier ring)
//   warp 1      MMA issuer    (one thread; tcgen05.mma into a double-buffered TMEM accumulator)
//   warps 2..5  epilogue      (tcgen05.ld -> fp32 -> fp16/bf16 -> pair kernel: swizzled shared-memory boxes, TMA
//                              stores by one thread; single-CTA kernel: 16-byte global stores -> flags or lock)
//   warps 6..9  consumer      (pair kernel, optional: acquire flags, OUT = C + bias)
// What happens to a finished tile depends on the schedule:
//   bulk_synchronous       store to the owner rank's slot; a second kernel scatters and publishes
//   fused_sequential       store to all W slots from registers, then publish W ready flags
//   workgroup_specialized  store to the owner slot, cas(lock, 0->1, release); reserved communication
//                          CTAs poll the locks (acquire), copy the tile to the other W-1 slots with
//                          TMA and publish the flags.  Tiles of the last wave (raster id >= seq_from) are
//                          scattered and published by their producers instead: nothing is left to overlap with
// Because the TMEM accumulator is double buffered, the epilogue of tile i (including the W-way
// scatter) overlaps the main loop of tile i+1 inside one CTA.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <climits>
#include <cmath>
#include <cstring>
#include <mutex>

#include "iris_device.cuh"
#include "sm100_ptx.cuh"

namespace iris {

constexpr int BM = 128;           // rows of a compute tile = rows of a publication tile
constexpr int BK = 64;            // 64 x 16-bit = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;        // K of one tcgen05.mma for 16-bit inputs
constexpr int kGemmThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kConsWarps = 4;     // optional consumer warps appended to every producer CTA of the pair kernel
constexpr int kGemmThreadsFused = kGemmThreads + 32 * kConsWarps;
constexpr int kConsUnroll = 16;   // 16-byte loads in flight per consumer lane
constexpr int kPairBNc = 256;     // pair tile width (also used by the fused consumer's item decode)
constexpr int kSchedDepth = 4;    // pair kernel: tile ids in flight between the claiming thread and the other roles
constexpr int kCommWarps = 6;     // communication CTA: every warp is a communicator with a 32 KB tile buffer
constexpr int kTileBytes = IRIS_TILE * IRIS_TILE * 2;
constexpr int kMnBlockBytes = 64 * BK * 2;   // B_r [K, N_local]: one [64 k][64 n] block of a stage, as its TMA box lands
constexpr int kSmemPayload = 192 * 1024;
constexpr int kSmemCtrl = 1024;
constexpr int kStoreBoxBytes = BM * 64 * 2;                 // 16 KB: 128 rows x 64 columns, one TMA store box (128B-swizzled rows)
constexpr int kEpiStageBytes = 2 * kStoreBoxBytes;          // single-CTA kernel: 128 converted columns of a tile on their way out
constexpr int kSmemTotal = kSmemPayload + kEpiStageBytes + kSmemCtrl + 1024;  // + slack to align the base to 1024
constexpr int kCommSmemTotal = kSmemPayload + kSmemCtrl + 1024;               // the communication kernel of the two-stream form
static_assert(kSmemTotal <= 232448, "shared memory per CTA");

template <int BN>
struct TileCfg {
  static constexpr int kStageBytes = BM * BK * 2 + BN * BK * 2;
  static constexpr int kStages = kSmemPayload / kStageBytes;  // 4 for BN=256, 6 for BN=128
  static constexpr int kTmemCols = 2 * BN;                    // two accumulators
};

struct alignas(64) GemmParams {
  CUtensorMap tmA;                    // A [M, K], box 64 x 128, 128B swizzle
  CUtensorMap tmB[IRIS_MAX_WORLD];    // B_r [N_local, K], box 64 x BN, 128B swizzle; or B_r [K, N_local], box 64 (n) x 64 (k), 128B swizzle
  CUtensorMap tmBn[IRIS_MAX_WORLD];   // pair kernel, fuse_last: B_r [N_local, K] with a box of 64 x (remainder columns / 2) rows
  CUtensorMap tmC[IRIS_MAX_WORLD];    // C of slot s viewed as [W][M][N_local], box 128 x 128 x 1, no swizzle
  CUtensorMap tmC4;                   // C of all slots as one tensor [slot][rank][M][N_local] (slots equally spaced: every heap
                                      // handle), box 128 x 128 x 1 x 1, no swizzle: the communication warps' copies
  CUtensorMap tmC4s;                  // the same tensor, box 64 x 128 x 1 x 1, 128B swizzle: the epilogues' stores
  CUtensorMap tmCs[IRIS_MAX_WORLD];   // slots at arbitrary addresses: C of slot s as [W][M][N_local], box 64 x 128 x 1, 128B swizzle
  int one_map;                        // 1 = tmC4 / tmC4s are valid; 0 = slots at arbitrary addresses, per-slot maps tmC[]
  HeapTable tab;
  uint64_t c_off, flag_off, lock_off;
  uint64_t timeout_ns;
  int32_t* status;
  int M, N, K, n_local;
  int tiles_m;          // compute tile rows: ceil(M / 128), or ceil(M / 256) for CTA pairs
  int ctiles_per_rank;  // compute tiles per rank along N: ceil(N_local / BN)
  int ptiles_per_rank;  // publication tiles per rank along N: ceil(N_local / 128)
  int total_ctiles;     // tiles_m * W * ctiles_per_rank
  int total_ptiles;     // ptiles_m * W * ptiles_per_rank
  int kblocks;          // ceil(K / 64)
  int ptiles_m;         // publication tile rows: ceil(M / 128)
  int dynamic;          // pair kernel: 1 = tiles are claimed from *tile_counter in raster order, 0 = static stride
  int32_t* tile_counter;
  const uint8_t* bias;  // fused consumer: bias[N] of the element type (NULL = no consumer warps)
  uint64_t out_off;     // fused consumer: OUT region in every slot
  int gemm_ctas, comm_ctas;
  int rank_first, rank_count;   // the ranks whose shards this call computes and scatters (all: 0, W)
  int streamk;          // single-CTA kernel: 1 = equal k-step ranges per CTA (tiles may be computed in parts)
  float* ws;            // stream-K: two fp32 tile slots per CTA for partial sums
  int32_t* arrive;      // stream-K: per compute tile, how many parts have been parked
  int seq_from;         // compute tiles with raster id >= seq_from are scattered by their producer (Listing 4's loop); 0 in
                        // fused_sequential mode, the first tile of the last wave in workgroup_specialized mode
  int takeover;         // pair kernel, workgroup_specialized: 1 = a producer also keeps (scatters itself) a tile below seq_from
                        // when the communication CTAs could not drain their backlog plus this tile before the kernel ends
  int32_t* backlog;     // publication tiles handed over and not yet published ([0]), tiles kept by that rule ([1])
  uint32_t t_pt_ns;     // estimate: time a communication warp needs for one publication tile, its CTA's port shared by all warps
  uint32_t t_tile_ns;   // estimate: main-loop time of one compute tile
  int fuse_last;        // pair kernel: 1 = a shard's last full 256-column tile and the narrow remainder after it are ONE work unit
                        // (two MMA groups on the same A stages, one accumulator each): the remainder no longer costs its own
                        // loads of A.  ctiles_per_rank / total_ctiles then count work units, one fewer per shard than tiles
  int kb_per_stage;     // pair kernel: 64-wide k-blocks per operand stage (2: the boxes of two adjacent k-blocks are requested together)
  int stage_bytes;      // pair kernel: bytes of one operand stage (32 KB per k-block, plus the remainder's B rows with fuse_last) ...
  int n_stages;         // ... and how many of them the 192 KB ring holds (3 to 6)
  int b1_bytes;         // fuse_last: bytes of the remainder's B box per CTA
  int sub_bytes;        // pair kernel: bytes of one k-block's operands inside a stage (32 KB, plus the remainder's B rows with fuse_last)
  int half_stage;       // pair kernel, two k-blocks per stage: 1 = the last stage of the ring has room for one k-block only
  int b_mn;             // 1 = B_r is [K, N_local] row-major (N contiguous): 64 x 64 boxes, MN-major descriptor; 0 = [N_local, K]
  int pace_stores;      // pair kernel: 1 = the epilogue spreads a tile's box stores over most of the next tile's main loop
  int raster_group;
  int mode;
  int32_t epoch;
};

struct CtrlBlock {  // lives in shared memory after the payload area
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint64_t comm_full[kCommWarps];
  uint64_t sched_full[kSchedDepth];
  uint64_t sched_empty[kSchedDepth];
  volatile int32_t sched_tile[kSchedDepth];
  uint32_t tmem_base;
  volatile int abort;
  volatile int last_part;   // stream-K: this CTA parked the last part of the tile and reduces it
  volatile int keep_tile;   // pair kernel: this CTA scatters the current tile itself
};

struct TileCoord { int tm, rank, jn; };

// Tile id -> coordinates, grouped like Triton's GROUP_SIZE_M swizzle (Section 3.4): ids run down
// `raster_group` tile rows before moving to the next tile column, so CTAs that run at the same
// time share A row panels and B column panels in L2.
__device__ __forceinline__ TileCoord decode_ctile(int id, const GemmParams& p) {
  const int tiles_n = p.rank_count * p.ctiles_per_rank;
  const int per_group = p.raster_group * tiles_n;
  const int g = id / per_group;
  const int first_m = g * p.raster_group;
  const int gsz = min(p.raster_group, p.tiles_m - first_m);
  const int in = id - g * per_group;
  const int tn = in / gsz;
  TileCoord c;
  c.tm = first_m + in % gsz;
  c.rank = p.rank_first + tn / p.ctiles_per_rank;
  c.jn = tn % p.ctiles_per_rank;
  return c;
}

// Bounded mbarrier wait.  Returns false when the deadline passed (recorded in the status block) or
// when another thread of the CTA already gave up.
template <bool CLUSTER_ACQUIRE = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const GemmParams& p, CtrlBlock* ctrl, int tile) {
  auto poll = [&]() { return CLUSTER_ACQUIRE ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity); };
  if (poll()) return true;
  const uint64_t start = globaltimer_ns();
  uint32_t spins = 0;
  while (!poll()) {
    if ((++spins & 63u) == 0) {
      if (ctrl->abort) return false;
      if (globaltimer_ns() - start > p.timeout_ns) {
        report_timeout(p.status, KID_GEMM, tile, -1, (int)parity, (int)(bar & 0xFFFF));
        ctrl->abort = 1;
        return false;
      }
    }
  }
  return true;
}

template <bool BF16>
__device__ __forceinline__ uint32_t pack2(uint32_t lo_bits, uint32_t hi_bits) {
  const float lo = __uint_as_float(lo_bits), hi = __uint_as_float(hi_bits);
  if (BF16) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);  // .x = lo (lower address), .y = hi
    return *reinterpret_cast<uint32_t*>(&v);
  } else {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
  }
}

}  // namespace iris

// Scratch of iris_gemm_all_scatter_noalloc(): a status block (first 64 words) followed by one lock per
// publication tile.  It lives in the library image, so every GPU that loads the library holds these
// 65 792 bytes until the process exits.  Device code names the array directly; host code must not use
// the name as an address (it is only a host-side stand-in) and asks cudaGetSymbolAddress() instead.
constexpr int kNoAllocStatusWords = 64;
constexpr int kNoAllocMaxTiles = 16384;
static __device__ __align__(256) int32_t g_noalloc_scratch[kNoAllocStatusWords + kNoAllocMaxTiles];

namespace iris {

// Address of lock[t]: in the owner rank's heap slot, or (STATIC_LOCKS) in the library's static scratch.
template <bool STATIC_LOCKS>
__device__ __forceinline__ int32_t* lock_addr(const GemmParams& p, int rank, int t) {
  if (STATIC_LOCKS) return &g_noalloc_scratch[kNoAllocStatusWords + t];
  return reinterpret_cast<int32_t*>(p.tab.base[rank] + p.lock_off) + t;
}

// ------------------------------------------------------------------------------------------------
// Communication CTA (workgroup-specialised mode), Listing 5's `else` branch.
// Each of the CTA's six warps is an independent communicator with its own 32 KB tile buffer and its own
// mbarrier.  Work items are publication tiles numbered in the producers' raster order (item k = sub-tile
// k % SUBS of compute tile k / SUBS; a CTA pair's 256-row tile has SUBS_M = 2 rows of them; a work unit of the pair kernel may hold two compute tiles),
// dealt round-robin to the communicator warps, so a warp sees its
// tiles become ready roughly first-in first-out.
//   poll     all 32 lanes watch 32 of the warp's pending items at once: one acquire-ordered load of
//            lock[t] per lane; a ballot collects the ready set
//   claim    the ready lanes take their locks together: cas(lock, 1 -> 0, acquire, gpu)
//   copy     per ready tile (ids handed over by shuffles): lane 0 issues one TMA load of the owner's tile
//            and, once it has landed, W-1 TMA stores from the same buffer (iris.put to every other rank),
//            then waits until the stores have been performed
//   publish  lanes 0..W-1 write the tile's ready flag in slot `lane` with release semantics
// ------------------------------------------------------------------------------------------------
template <bool STATIC_LOCKS, int SUBS, int SUBS_M = 1>
__device__ void comm_cta(const GemmParams& p, CtrlBlock* ctrl, uint8_t* payload, int warp, int lane, int comm_block) {
  constexpr uint32_t kFull = 0xFFFFFFFFu;
  const int W = p.tab.world;
  const int ncw = p.comm_ctas * kCommWarps;
  const int cw = comm_block * kCommWarps + warp;   // comm_block: this CTA's index among the communication CTAs
  const int L = p.fuse_last ? 2 : 1;               // compute tiles per work unit (pair kernel with fused shard tails: up to two)
  const int per_unit = SUBS * SUBS_M * L;
  const int items = min(p.total_ctiles, p.seq_from) * per_unit;   // the tail wave's tiles are scattered by their producers
  const int n_my = cw < items ? (items - cw + ncw - 1) / ncw : 0;  // items cw, cw + ncw, ...
  const int pt_n = W * p.ptiles_per_rank;
  const uint32_t buf = ptx::smem_u32(payload + warp * kTileBytes);
  const uint32_t bar = ptx::smem_u32(&ctrl->comm_full[warp]);
  uint32_t bar_phase = 0;
  int widx = lane < n_my ? lane : -1;  // index into this warp's item list that this lane watches
  int next = n_my < 32 ? n_my : 32;
  uint64_t last_progress = globaltimer_ns();
  uint32_t spins = 0;
  bool ok = true;
  // item -> publication tile, recomputed only when the lane moves to a new item
  // (t < 0 with widx >= 0: the compute tile has no such sub-tile; nothing to do)
  int t = -1, rank = 0;
  auto assign = [&]() {
    t = -1;
    if (widx < 0) return;
    const int k = cw + widx * ncw;
    const TileCoord tc = decode_ctile(k / per_unit, p);
    const int l = (k % per_unit) / (SUBS * SUBS_M), sub = k % (SUBS * SUBS_M);
    if (l == 1 && tc.jn != p.ctiles_per_rank - 1) return;   // only a shard's last unit has a second tile
    const int pj = (tc.jn + l) * SUBS + sub % SUBS;
    const int tm = tc.tm * SUBS_M + sub / SUBS;  // publication tile row
    rank = tc.rank;
    if (pj < p.ptiles_per_rank && tm < p.ptiles_m) t = tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
  };
  assign();
  while (ok && __any_sync(kFull, widx >= 0)) {
    bool ready = false;
    int state = 0;   // 1: the producer handed the tile over; 2: the producer scattered and published it itself
    if (widx >= 0) {
      if (t >= 0) state = ld_acquire_gpu(lock_addr<STATIC_LOCKS>(p, rank, t));
      ready = t < 0 || state == 1 || state == 2;
    }
    const uint32_t mask = __ballot_sync(kFull, ready);
    if (mask == 0) {
      if ((++spins & 15u) == 0) {
        bool expired = false;
        if (lane == 0) {
          expired = ctrl->abort != 0;
          if (!expired && globaltimer_ns() - last_progress > p.timeout_ns) {
            report_timeout(p.status, KID_GEMM, t, -2, 0, 1);
            ctrl->abort = 1;
            expired = true;
          }
        }
        if (__any_sync(kFull, expired)) ok = false;
      }
      continue;
    }
    // claim (Listing 5, communication branch): every ready lane takes its lock, state -> 0, acquire at gpu scope
    if (ready && t >= 0) (void)cas_acquire_gpu(lock_addr<STATIC_LOCKS>(p, rank, t), state, 0);
    __syncwarp();
    uint32_t todo = mask;
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const int rt = __shfl_sync(kFull, t, src);
      const int rrank = __shfl_sync(kFull, rank, src);
      const int rstate = __shfl_sync(kFull, state, src);
      if (rt < 0 || rstate == 2) continue;   // no such sub-tile, or nothing left to do but the lock reset above
      const int tm = rt / pt_n, pj = (rt % pt_n) % p.ptiles_per_rank;
      bool fail = false;
      if (lane == 0) {
        fence_proxy_async();  // producers' generic-proxy stores (acquired above) -> our async-proxy read
        ptx::mbar_arrive_expect_tx(bar, kTileBytes);
        if (p.one_map) ptx::tma_load_4d(buf, &p.tmC4, pj * IRIS_TILE, tm * IRIS_TILE, rrank, rrank, bar);
        else ptx::tma_load_3d(buf, &p.tmC[rrank], pj * IRIS_TILE, tm * IRIS_TILE, rrank, bar);
        if (!mbar_wait(bar, bar_phase, p, ctrl, rt)) {
          fail = true;
        } else {
          for (int s = 0; s < W; ++s) {
            if (s == rrank) continue;
            if (p.one_map) ptx::tma_store_4d(&p.tmC4, pj * IRIS_TILE, tm * IRIS_TILE, rrank, s, buf);
            else ptx::tma_store_3d(&p.tmC[s], pj * IRIS_TILE, tm * IRIS_TILE, rrank, buf);
          }
          ptx::bulk_commit_group();
          ptx::bulk_wait_group<0>();  // stores performed: the buffer is free and the tile may be published
          fence_proxy_async();        // async-proxy writes above -> the generic-proxy release of the flags below
        }
      }
      bar_phase ^= 1;
      if (__any_sync(kFull, fail)) { ok = false; break; }
      // bar.warp.sync orders lane 0's wait for the bulk stores (and its proxy fence) before the other lanes' flag
      // releases: a vote converges the warp but is not a memory barrier
      __syncwarp();
      if (lane < W) st_release_flag(reinterpret_cast<int32_t*>(p.tab.base[lane] + p.flag_off) + rt, p.epoch, p.tab.flags_sys);
      if (p.takeover && lane == 0) atomicAdd(p.backlog, -1);
      __syncwarp();
    }
    // lanes whose item was handled move on to the next unwatched items, in lane order
    if (mask & (1u << lane)) {
      const int cand = next + __popc(mask & ((1u << lane) - 1u));
      widx = cand < n_my ? cand : -1;
      assign();
    }
    next = min(n_my, next + __popc(mask));
    last_progress = globaltimer_ns();
  }
}

// ------------------------------------------------------------------------------------------------
// The single-CTA GEMM + scatter kernel.
//
// Work is handed out as segments (tile, kb0, kb1) of the k-loop:
//   static stride   CTA c takes whole tiles c, c + NUM, ... (the listings' loop): every segment is a full tile
//   stream-K        the T x KB k-steps of all tiles are cut into NUM equal, contiguous ranges, one per CTA, so
//                   every SM streams the same number of operand bytes whatever T mod NUM is (the skinny,
//                   memory-bound shapes: one tile row, a tile count that is not a multiple of the SM count).
//                   A tile that straddles two or more ranges is computed in parts: each part's fp32 accumulator
//                   goes to a workspace slot, the part that arrives last (one atomic per part) adds the parts in
//                   k order -- a fixed order, so the result does not depend on who was last -- converts,
//                   scatters and publishes.
// ------------------------------------------------------------------------------------------------
struct Segment { int tile, kb0, kb1; bool first; };

struct SegmentIter {
  long long u, u_end;   // stream-K: next k-step unit and end of this CTA's range
  int tile, stride;     // static: next tile and stride
  bool streamk, started;
  __device__ __forceinline__ SegmentIter(const GemmParams& p, int cta) : started(false) {
    streamk = p.streamk != 0;
    const long long units = (long long)p.total_ctiles * p.kblocks;
    u = streamk ? units * cta / p.gemm_ctas : 0;
    u_end = streamk ? units * (cta + 1) / p.gemm_ctas : 0;
    tile = cta;
    stride = p.gemm_ctas;
  }
  __device__ __forceinline__ bool next(const GemmParams& p, Segment& s) {
    if (streamk) {
      if (u >= u_end) return false;
      s.tile = (int)(u / p.kblocks);
      s.kb0 = (int)(u % p.kblocks);
      s.kb1 = (int)min((long long)p.kblocks, s.kb0 + (u_end - u));
      s.first = !started;
      u += s.kb1 - s.kb0;
    } else {
      if (tile >= p.total_ctiles) return false;
      s.tile = tile; s.kb0 = 0; s.kb1 = p.kblocks; s.first = !started;
      tile += stride;
    }
    started = true;
    return true;
  }
};

// stream-K bookkeeping: which CTA's range holds k-step unit x, and where that CTA's range starts
__device__ __forceinline__ int streamk_cta_of(long long x, long long units, int ctas) { return (int)(((x + 1) * ctas + units - 1) / units - 1); }
__device__ __forceinline__ long long streamk_begin(int cta, long long units, int ctas) { return units * cta / ctas; }

template <int BN, bool BF16, bool STATIC_LOCKS = false>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_all_scatter_kernel(const __grid_constant__ GemmParams p) {
  using Cfg = TileCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* payload = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  CtrlBlock* ctrl = reinterpret_cast<CtrlBlock*>(payload + kSmemPayload + kEpiStageBytes);
  const int warp = (int)threadIdx.x / 32, lane = (int)threadIdx.x % 32;
  const bool is_comm = (int)blockIdx.x >= p.gemm_ctas;
  const int W = p.tab.world;

  if (threadIdx.x == 0) {
    for (int i = 0; i < Cfg::kStages; ++i) { ptx::mbar_init(ptx::smem_u32(&ctrl->full[i]), 1); ptx::mbar_init(ptx::smem_u32(&ctrl->empty[i]), 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_full[i]), 1); ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_empty[i]), 4); }
    for (int i = 0; i < kCommWarps; ++i) ptx::mbar_init(ptx::smem_u32(&ctrl->comm_full[i]), 1);
    ctrl->abort = 0;
    ptx::fence_mbar_init();
    fence_proxy_async();
    if (p.kblocks > 0 && !is_comm) {
      ptx::prefetch_tensormap(&p.tmA);
      for (int r = p.rank_first; r < p.rank_first + p.rank_count; ++r) ptx::prefetch_tensormap(&p.tmB[r]);
    }
    if (is_comm) {
      if (p.one_map) ptx::prefetch_tensormap(&p.tmC4);
      else for (int r = 0; r < W; ++r) ptx::prefetch_tensormap(&p.tmC[r]);
    } else {
      if (p.one_map) ptx::prefetch_tensormap(&p.tmC4s);
      else for (int r = 0; r < W; ++r) ptx::prefetch_tensormap(&p.tmCs[r]);
    }
  }
  if (warp == 1 && !is_comm) {
    ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), Cfg::kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();

  if (is_comm) {
    comm_cta<STATIC_LOCKS, BN / IRIS_TILE>(p, ctrl, payload, warp, lane, (int)blockIdx.x - p.gemm_ctas);
  } else if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      SegmentIter it(p, (int)blockIdx.x);
      Segment sg;
      while (ok && it.next(p, sg)) {
        const TileCoord tc = decode_ctile(sg.tile, p);
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (!mbar_wait(ptx::smem_u32(&ctrl->empty[stage]), phase ^ 1, p, ctrl, sg.tile)) { ok = false; break; }
          const uint32_t bar = ptx::smem_u32(&ctrl->full[stage]);
          uint8_t* sa = payload + stage * Cfg::kStageBytes;
          ptx::mbar_arrive_expect_tx(bar, Cfg::kStageBytes);
          ptx::tma_load_2d(ptx::smem_u32(sa), &p.tmA, kb * BK, tc.tm * BM, bar);
          if (p.b_mn) {   // B_r [K, N_local]: one [64 k][64 n] block per 64 columns of the tile
#pragma unroll
            for (int nb = 0; nb < BN / 64; ++nb)
              ptx::tma_load_2d(ptx::smem_u32(sa + BM * BK * 2 + nb * kMnBlockBytes), &p.tmB[tc.rank], tc.jn * BN + nb * 64, kb * BK, bar);
          } else {
            ptx::tma_load_2d(ptx::smem_u32(sa + BM * BK * 2), &p.tmB[tc.rank], kb * BK, tc.jn * BN, bar);
          }
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      const uint32_t idesc = ptx::idesc_f16(BM, BN, BF16 ? 1 : 0) | (p.b_mn ? ptx::kIdescBMnMajor : 0u);
      const uint64_t b_kstep = p.b_mn ? (uint64_t)(2 * 1024 >> 4) : 2u;   // 16 k: two 8-row swizzle atoms (MN-major), or +32 bytes in the row (K-major)
      const uint32_t tmem_base = ctrl->tmem_base;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      SegmentIter it(p, (int)blockIdx.x);
      Segment sg;
      while (ok && it.next(p, sg)) {
        if (!mbar_wait(ptx::smem_u32(&ctrl->tmem_empty[acc]), acc_phase ^ 1, p, ctrl, sg.tile)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
          if (!mbar_wait(ptx::smem_u32(&ctrl->full[stage]), phase, p, ctrl, sg.tile)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(payload + stage * Cfg::kStageBytes);
          const uint64_t adesc = ptx::smem_desc_k_sw128(sa);
          const uint64_t bdesc = p.b_mn ? ptx::smem_desc_mn_sw128(sa + BM * BK * 2, kMnBlockBytes) : ptx::smem_desc_k_sw128(sa + BM * BK * 2);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)  // +32 bytes per K step: +2 in the (>>4) address field
            ptx::mma_f16_ss(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)k * b_kstep, idesc, (kb > sg.kb0) || k != 0);
          ptx::mma_commit(ptx::smem_u32(&ctrl->empty[stage]));  // stage reusable once these MMAs have read it
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        ptx::mma_commit(ptx::smem_u32(&ctrl->tmem_full[acc]));  // accumulator (of this segment) complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5, lane quadrant = warp % 4 ----------------
    const int quad = warp & 3;
    const int et = (int)threadIdx.x - 64;  // 0..127
    int acc = 0;
    uint32_t acc_phase = 0;
    const uint32_t tmem_base = ctrl->tmem_base;
    const long long units = (long long)p.total_ctiles * p.kblocks;
    SegmentIter it(p, (int)blockIdx.x);
    Segment sg;
    while (it.next(p, sg)) {
      const int tile = sg.tile;
      const TileCoord tc = decode_ctile(tile, p);
      const bool ok = mbar_wait(ptx::smem_u32(&ctrl->tmem_full[acc]), acc_phase, p, ctrl, tile);
      if (ptx::bar_red_or(1, kEpiThreads, !ok)) break;  // uniform decision for all four warps
      ptx::tc_fence_after();
      const bool whole = sg.kb0 == 0 && sg.kb1 == p.kblocks;   // this CTA computed the tile's entire k range
      const bool seq = tile >= p.seq_from;                      // scatter from registers (Listing 4) or hand over (Listing 5)
      const int row_in_tile = quad * 32 + lane;
      const int col_in_shard = tc.jn * BN;
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN);

      // The converted tile leaves through shared memory: a lane owns a row, so a store straight from its registers would
      // put 16 bytes into each of 32 different lines per instruction (measured: twice the payload crosses the SM's port).
      // Instead 128 columns at a time are staged as two 64-column boxes in the 128B-swizzle layout of the store maps
      // (16-byte piece j of row r at position j ^ (r % 8): a warp's 512 bytes per instruction spread over all banks)
      // and one thread sends them out with TMA -- whole 128-byte lines, clipped by the maps at row M and column N_local.
      const uint32_t stg = ptx::smem_u32(payload + kSmemPayload);
      auto stage_chunk = [&](const uint32_t (&v)[32], int ch) {
        const uint32_t row_base = stg + (uint32_t)(((ch >> 1) & 1) * kStoreBoxBytes + row_in_tile * 128);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 q;
          if (p.kblocks == 0) {
            q = make_uint4(0, 0, 0, 0);  // K == 0: the sum is empty
          } else {
            q.x = pack2<BF16>(v[8 * i + 0], v[8 * i + 1]);
            q.y = pack2<BF16>(v[8 * i + 2], v[8 * i + 3]);
            q.z = pack2<BF16>(v[8 * i + 4], v[8 * i + 5]);
            q.w = pack2<BF16>(v[8 * i + 6], v[8 * i + 7]);
          }
          const int piece = (ch & 1) * 4 + i;
          ptx::st_shared_v4(row_base + (uint32_t)((piece ^ (row_in_tile & 7)) << 4), q);
        }
      };
      // Sends the staged columns [128 * half, 128 * half + 128) of the tile to every slot (Listing 4) or to the owner's
      // (Listings 3 and 5).  After the last half the stores have been performed (the tile may be published); after an
      // earlier one the boxes have been read and may be refilled.
      auto flush_half = [&](int half, bool last) {
        fence_proxy_async();   // this thread's shared-memory writes -> the TMA unit's reads
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        if (et == 0) {
          for (int s = 0; s < W; ++s) {
            if (!seq && s != tc.rank) continue;
#pragma unroll
            for (int b = 0; b < 2; ++b) {
              const int col = col_in_shard + half * IRIS_TILE + 64 * b;
              if (col >= p.n_local) continue;
              if (p.one_map) ptx::tma_store_4d(&p.tmC4s, col, tc.tm * BM, tc.rank, s, stg + (uint32_t)(b * kStoreBoxBytes));
              else ptx::tma_store_3d(&p.tmCs[s], col, tc.tm * BM, tc.rank, stg + (uint32_t)(b * kStoreBoxBytes));
            }
          }
          ptx::bulk_commit_group();
          if (last) {
            ptx::bulk_wait_group<0>();
            fence_proxy_async();   // async-proxy writes above -> the generic-proxy release (flags or lock) after the barrier
          } else {
            ptx::bulk_wait_group_read<0>();
          }
        }
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
      };
      auto release_accumulator = [&]() {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->tmem_empty[acc]));
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      };
      constexpr int kChunks = BN / 32;

      bool publish = true;
      if (whole) {
#pragma unroll 1
        for (int ch = 0; ch < kChunks; ++ch) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(t_addr + (uint32_t)(ch * 32), v);
          ptx::tmem_wait_ld();
          stage_chunk(v, ch);
          if ((ch & 3) == 3) {
            if (ch == kChunks - 1) release_accumulator();   // accumulator drained: hand it back to the MMA warp
            flush_half(ch >> 2, ch == kChunks - 1);
          }
        }
      } else {
        // ---- stream-K: a part of the tile.  Park the fp32 partial sums, then see whether we are the last part. ----
        // Workspace layout of a part: [chunk of 32 columns][row][32 floats], so a lane writes 128 contiguous bytes and a
        // warp 4 KB.
        float* mine = p.ws + (size_t)(2 * (int)blockIdx.x + (sg.first ? 0 : 1)) * (BM * BN) + (size_t)row_in_tile * 32;
#pragma unroll 1
        for (int ch = 0; ch < kChunks; ++ch) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(t_addr + (uint32_t)(ch * 32), v);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 8; ++i)
            st_global_v4(mine + (size_t)ch * (BM * 32) + 4 * i, make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
        }
        release_accumulator();
        const int c_lo = streamk_cta_of((long long)tile * p.kblocks, units, p.gemm_ctas);
        const int c_hi = streamk_cta_of((long long)tile * p.kblocks + p.kblocks - 1, units, p.gemm_ctas);
        __threadfence();   // the partial sums are visible device-wide before our arrival is counted
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        if (et == 0) ctrl->last_part = atomic_rmw<false>(p.arrive + tile, 0, 1, IRIS_SEM_ACQ_REL, IRIS_SCOPE_GPU) == c_hi - c_lo;
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        publish = ctrl->last_part != 0;
        if (publish) {
          __threadfence();
#pragma unroll 1
          for (int ch = 0; ch < kChunks; ++ch) {
            float sum[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) sum[i] = 0.0f;
            for (int c = c_lo; c <= c_hi; ++c) {   // parts in k order: CTA c_lo holds the lowest k range
              const bool its_first = streamk_begin(c, units, p.gemm_ctas) >= (long long)tile * p.kblocks;
              const float* part = p.ws + (size_t)(2 * c + (its_first ? 0 : 1)) * (BM * BN) + (size_t)ch * (BM * 32) + (size_t)row_in_tile * 32;
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const uint4 w = ld_global_v4(part + 4 * i);
                sum[4 * i + 0] += __uint_as_float(w.x);
                sum[4 * i + 1] += __uint_as_float(w.y);
                sum[4 * i + 2] += __uint_as_float(w.z);
                sum[4 * i + 3] += __uint_as_float(w.w);
              }
            }
            uint32_t v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(sum[i]);
            stage_chunk(v, ch);
            if ((ch & 3) == 3) flush_half(ch >> 2, ch == kChunks - 1);
          }
        }
      }
      if (publish && p.mode != IRIS_MODE_BULK_SYNCHRONOUS) {
        // the tile's stores have been performed and fenced by the issuing thread before the barrier that ended
        // flush_half; the releases below are cumulative over them
        const int subs = BN / IRIS_TILE;
        const int pt_n = W * p.ptiles_per_rank;
        if (seq) {
          if (et < subs * W) {
            const int sub = et / W, s = et % W;
            const int pj = tc.jn * subs + sub;
            if (pj < p.ptiles_per_rank) {
              const int t = tc.tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
              st_release_flag(reinterpret_cast<int32_t*>(p.tab.base[s] + p.flag_off) + t, p.epoch, p.tab.flags_sys);
            }
          }
        } else if (et < subs) {
          const int pj = tc.jn * subs + et;
          if (pj < p.ptiles_per_rank) {
            const int t = tc.tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
            // hand-over (Listing 5, producer branch): lock 0 -> 1, release at gpu scope
            (void)cas_release_gpu(lock_addr<STATIC_LOCKS>(p, tc.rank, t), 0, 1);
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1 && !is_comm) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(ctrl->tmem_base, Cfg::kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Fused consumer warps (optional).  The flag-gated consumer of Section 4.1 running inside the same launch:
// four extra warps in every producer CTA take (publication tile, slot) items in the producers' raster
// order, wait -- acquire load of flag[s][t], bounded, with back-off so the spinning does not steal issue
// slots from the MMA and TMA warps -- and then stream the tile: OUT[s] = C[s] + bias.  The consumer is
// HBM-bound and the GEMM tensor-bound, so sharing the SMs costs the GEMM little and hides the consumer's
// 2 x W x M x N x 2 bytes behind it; per SM this is under 10 GB/s.
// ------------------------------------------------------------------------------------------------
template <bool BF16>
__device__ void consumer_warp(const GemmParams& p, CtrlBlock* ctrl, int cwarp, int lane) {
  constexpr uint32_t kFull = 0xFFFFFFFFu;
  constexpr int SUBS = kPairBNc / IRIS_TILE, SUBS_M = 2;
  const int W = p.tab.world;
  const int ncons = p.gemm_ctas * kConsWarps;
  const int pt_n = W * p.ptiles_per_rank;
  const int L = p.fuse_last ? 2 : 1, per_unit = SUBS * SUBS_M * L;
  const long long items = (long long)p.total_ctiles * per_unit * W;
  for (long long q = (long long)blockIdx.x * kConsWarps + cwarp; q < items; q += ncons) {
    const int k = (int)(q / W), s = (int)(q % W);
    const TileCoord tc = decode_ctile(k / per_unit, p);
    const int l = (k % per_unit) / (SUBS * SUBS_M), sub = k % (SUBS * SUBS_M);
    if (l == 1 && tc.jn != p.ctiles_per_rank - 1) continue;   // only a shard's last unit has a second tile
    const int pj = (tc.jn + l) * SUBS + sub % SUBS;
    const int tm = tc.tm * SUBS_M + sub / SUBS;
    if (pj >= p.ptiles_per_rank || tm >= p.ptiles_m) continue;
    const int t = tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
    int ok = 1;
    if (lane == 0) {
      const int32_t* flag = reinterpret_cast<const int32_t*>(p.tab.base[s] + p.flag_off) + t;
      int32_t seen = ld_acquire_gpu(flag);
      if (seen < p.epoch) {
        const uint64_t start = globaltimer_ns();
        uint32_t spins = 0;
        while ((seen = ld_acquire_gpu(flag)) < p.epoch) {
          __nanosleep(400);
          if ((++spins & 15u) == 0) {
            if (ctrl->abort) { ok = 0; break; }
            if (globaltimer_ns() - start > p.timeout_ns) {
              report_timeout(p.status, KID_CONSUMER, t, s, seen, p.epoch);
              ctrl->abort = 1;
              ok = 0;
              break;
            }
          }
        }
      }
    }
    ok = __shfl_sync(kFull, ok, 0);
    __syncwarp();   // bar.warp.sync orders lane 0's acquire of the flag before every lane's reads of the tile
    if (!ok) return;
    const int rows = min(IRIS_TILE, p.M - tm * IRIS_TILE);
    const uint64_t col0 = (uint64_t)tc.rank * p.n_local + (uint64_t)pj * IRIS_TILE;
    const uint64_t tile_off = ((uint64_t)(tm * IRIS_TILE) * p.N + col0) * 2;
    const uint64_t src = p.tab.base[s] + p.c_off + tile_off;
    const uint64_t dst = p.tab.base[s] + p.out_off + tile_off;
    const int ch = lane & 15;  // 16-byte chunk within the 256-byte tile row
    const int cols = min(IRIS_TILE, p.n_local - pj * IRIS_TILE);
    if (ch * 8 >= cols) continue;  // ragged shard: the last publication tile is narrower (whole chunks: N_local % 8 == 0)
    const uint4 b = *reinterpret_cast<const uint4*>(p.bias + (col0 + (uint64_t)ch * 8) * 2);
    // 2 rows per pass, kConsUnroll passes (= 8 KB per warp) in flight: at ~2 us of loaded-memory latency that is
    // ~4 GB/s per warp, several times the 1.3 GB/s each warp must sustain to keep up with the GEMM.
    for (int r0 = lane >> 4; r0 < rows; r0 += 2 * kConsUnroll) {
      uint4 v[kConsUnroll];
#pragma unroll
      for (int u = 0; u < kConsUnroll; ++u)
        if (r0 + 2 * u < rows) v[u] = ld_global_v4(reinterpret_cast<const void*>(src + ((uint64_t)(r0 + 2 * u) * p.N + (uint64_t)ch * 8) * 2));
#pragma unroll
      for (int u = 0; u < kConsUnroll; ++u)
        if (r0 + 2 * u < rows) {
          uint4 o;
          o.x = add2<BF16>(v[u].x, b.x);
          o.y = add2<BF16>(v[u].y, b.y);
          o.z = add2<BF16>(v[u].z, b.z);
          o.w = add2<BF16>(v[u].w, b.w);
          st_global_v4(reinterpret_cast<void*>(dst + ((uint64_t)(r0 + 2 * u) * p.N + (uint64_t)ch * 8) * 2), o);
        }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant: a cluster of two CTAs (one TPC) computes a 256 x 256 tile with tcgen05 cta_group::2.
// CTA r of the pair owns rows [128 r, 128 r + 128) of the tile: it TMA-loads its own 128 x 64 slice of A
// and its own half (128 of the 256 columns) of the B tile -- no multicast, every CTA fetches only what
// it keeps -- and the leader's MMA thread issues one 256 x 256 x 16 instruction for both: each SM's
// tensor core reads its A slice locally and both B halves.  Per CTA and k-step 32 KB are pulled in instead
// of 48 KB for the same flops per SM: 64 B/clk, which the SM's port to the L2 sustains, instead of 96, which
// it does not (the single-CTA kernel's tensor pipe is 67 % busy, this one's 92 %).
// Accumulators: 2 x 256 columns of TMEM in each CTA (rows of its own half).  Shared memory: a 192 KB ring of operand
// stages -- 3 stages of 64 KB holding two 64-wide k-blocks each (sub-stages [A 16 KB | B 16 KB]), whose boxes are
// requested back to back; with a fused remainder's B rows in every sub-stage, two such stages and a last one of a
// single k-block (or one k-block per stage when asked for or when five k-blocks would not fit) -- and two 16 KB
// store boxes (128 converted columns of the CTA's half tile, 128B-swizzled for the TMA stores).
//   full[s]        leader only; the leader's producer expects 64 KB, all four loads (two per CTA) complete on it
//   empty[s]       both CTAs; the leader's tcgen05.commit multicasts the arrival to the pair
//   tmem_full[a]   both CTAs; multicast commit after a tile's last MMA
//   tmem_empty[a]  leader only; 8 arrivals = 4 epilogue warps x 2 CTAs (the peer's arrive remotely)
// ------------------------------------------------------------------------------------------------
constexpr int kPairBN = 256;
// Columns the pair's MMA computes for tile column jn of a shard: the full 256, or -- last tile of a ragged shard --
// what is left, rounded up to 32 (one epilogue chunk; the instruction's N has to be a multiple of 16).  A narrower
// instruction takes proportionally fewer tensor cycles; the rows of B beyond the shard that it reads are zero-filled
// by the load and the columns they produce are clipped by the stores.
__device__ __forceinline__ int pair_tile_cols(const GemmParams& p, int jn) {
  const int left = p.n_local - jn * kPairBN;
  return left >= kPairBN ? kPairBN : ((left + 31) & ~31);
}
constexpr int kPairStageBytes = 2 * BM * BK * 2;            // 32 KB: A slice + B half of one 64-wide k-block
constexpr int kPairRingBytes = 192 * 1024;                  // operand stages: 3 x 64 KB (two k-blocks per stage), 6 x 32 KB, or fewer, larger ones
constexpr int kPairMaxStages = 6;
constexpr int kPairStoreBytes = 2 * kStoreBoxBytes;         // 32 KB: 128 converted columns of this CTA's half tile on their way out
constexpr int kPairSmemPayload = kPairRingBytes + kPairStoreBytes;   // 224 KB
constexpr int kPairSmemTotal = kPairSmemPayload + kSmemCtrl + 1024;
static_assert(kPairSmemPayload >= kCommWarps * kTileBytes, "communication warps' tile buffers share the payload area");
static_assert(kPairSmemTotal <= 232448, "shared memory per CTA");

template <bool BF16, bool STATIC_LOCKS = false, bool CONSUMER = false, int KBS = 2>
__global__ void __launch_bounds__(CONSUMER ? kGemmThreadsFused : kGemmThreads, 1) gemm_all_scatter_pair_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* payload = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  CtrlBlock* ctrl = reinterpret_cast<CtrlBlock*>(payload + kPairSmemPayload);
  const int warp = (int)threadIdx.x / 32, lane = (int)threadIdx.x % 32;
  const int cta_rank = (int)ptx::cluster_ctarank();
  const bool leader = cta_rank == 0;
  const bool is_comm = (int)blockIdx.x >= p.gemm_ctas;   // gemm_ctas is even: a pair is never split
  const int pair_id = (int)blockIdx.x >> 1, gemm_pairs = p.gemm_ctas >> 1;
  const int W = p.tab.world;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPairMaxStages; ++i) { ptx::mbar_init(ptx::smem_u32(&ctrl->full[i]), 1); ptx::mbar_init(ptx::smem_u32(&ctrl->empty[i]), 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_full[i]), 1); ptx::mbar_init(ptx::smem_u32(&ctrl->tmem_empty[i]), 8); }
    for (int i = 0; i < kCommWarps; ++i) ptx::mbar_init(ptx::smem_u32(&ctrl->comm_full[i]), 1);
    // tile feed: one publisher; readers = the leader's MMA thread + 4 epilogue warps, the peer's producer + 4 epilogue warps
    for (int i = 0; i < kSchedDepth; ++i) { ptx::mbar_init(ptx::smem_u32(&ctrl->sched_full[i]), 1); ptx::mbar_init(ptx::smem_u32(&ctrl->sched_empty[i]), 10); }
    ctrl->abort = 0;
    ptx::fence_mbar_init();
    fence_proxy_async();
    if (p.kblocks > 0 && !is_comm) {
      ptx::prefetch_tensormap(&p.tmA);
      for (int r = p.rank_first; r < p.rank_first + p.rank_count; ++r) ptx::prefetch_tensormap(&p.tmB[r]);
    }
    if (p.one_map) ptx::prefetch_tensormap(is_comm ? &p.tmC4 : &p.tmC4s);
    else for (int r = 0; r < p.tab.world; ++r) ptx::prefetch_tensormap(is_comm ? &p.tmC[r] : &p.tmCs[r]);
  }
  if (warp == 1 && !is_comm) {
    ptx::tmem_alloc_pair(ptx::smem_u32(&ctrl->tmem_base), 2 * kPairBN);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();   // the peer's barriers exist before anything of ours can signal them
  ptx::tc_fence_after();

  // Tile feed.  Lane 0 of the leader's producer warp decides which tile the pair computes next -- the next id
  // of the raster order from a global counter (dynamic), or pair_id + n * gemm_pairs (static, the listings'
  // loop) -- and publishes it through a small ring in both CTAs' shared memory; every other role takes its
  // tile ids from the ring.  -1 ends the stream.
  auto feed_take = [&](int& j, uint32_t& ph, int& slot) -> int {   // -2: the wait expired
    if (!mbar_wait<true>(ptx::smem_u32(&ctrl->sched_full[j]), ph, p, ctrl, -4)) return -2;
    const int tile = ctrl->sched_tile[j];
    slot = j;
    if (++j == kSchedDepth) { j = 0; ph ^= 1; }
    return tile;
  };
  auto feed_release = [&](int slot) { ptx::mbar_arrive_cluster(ptx::mapa(ptx::smem_u32(&ctrl->sched_empty[slot]), 0)); };

  if (warp >= kGemmThreads / 32) {
    if (CONSUMER && !is_comm) consumer_warp<BF16>(p, ctrl, warp - kGemmThreads / 32, lane);
  } else if (is_comm) {
    comm_cta<STATIC_LOCKS, kPairBN / IRIS_TILE, 2>(p, ctrl, payload, warp, lane, (int)blockIdx.x - p.gemm_ctas);
  } else if (warp == 0) {
    // ---------------- TMA producer (both CTAs); the leader's also claims and publishes the tiles ----------------
    if (lane == 0) {
      int stage = 0, fj = 0, fslot = 0;
      uint32_t phase = 0, fph = 0;
      int static_next = pair_id;
      auto claim = [&]() -> int {
        int t;
        if (p.dynamic) t = atomicAdd(p.tile_counter, 1);
        else { t = static_next; static_next += gemm_pairs; }
        return t;
      };
      int claimed = leader ? claim() : 0;
      for (;;) {
        int tile;
        if (leader) {
          tile = claimed < p.total_ctiles ? claimed : -1;
          if (!mbar_wait(ptx::smem_u32(&ctrl->sched_empty[fj]), fph ^ 1, p, ctrl, -5)) break;
          ctrl->sched_tile[fj] = tile;
          ptx::st_shared_cluster_u32(ptx::mapa(ptx::smem_u32((const void*)&ctrl->sched_tile[fj]), 1), (uint32_t)tile);
          ptx::mbar_arrive(ptx::smem_u32(&ctrl->sched_full[fj]));
          ptx::mbar_arrive_cluster(ptx::mapa(ptx::smem_u32(&ctrl->sched_full[fj]), 1));   // release.cluster: after the remote store
          if (++fj == kSchedDepth) { fj = 0; fph ^= 1; }
          if (tile >= 0) claimed = claim();   // the next claim's latency hides behind this tile's loads
        } else {
          tile = feed_take(fj, fph, fslot);
          if (tile != -2) feed_release(fslot);
        }
        if (tile < 0) break;
        const TileCoord tc = decode_ctile(tile, p);
        const int ncols = pair_tile_cols(p, tc.jn);   // this CTA keeps rows [cta_rank * ncols / 2, ...) of the B tile
        // a shard's last unit with fuse_last: the remainder tile's B rows ride in the same stage, after A and B
        const bool fused = p.fuse_last && tc.jn == p.ctiles_per_rank - 1;
        const int ncols1 = fused ? pair_tile_cols(p, tc.jn + 1) : 0;
        bool ok = true;
        constexpr int kbs = KBS;   // 64-wide k-blocks per stage (= p.kb_per_stage)
        for (int kb = 0, nk; kb < p.kblocks; kb += nk) {
          // k-blocks in this stage: kbs, one in the ring's short last stage, one at the end of an odd count
          nk = min((kbs == 2 && p.half_stage && stage == p.n_stages - 1) ? 1 : kbs, p.kblocks - kb);
          if (!mbar_wait(ptx::smem_u32(&ctrl->empty[stage]), phase ^ 1, p, ctrl, tile)) { ok = false; break; }
          const uint32_t full_local = ptx::smem_u32(&ctrl->full[stage]);
          if (leader) ptx::mbar_arrive_expect_tx(full_local, 2 * nk * (kPairStageBytes + (fused ? p.b1_bytes : 0)));
          const uint32_t full_leader = ptx::mapa(full_local, 0);
          const uint32_t sa = ptx::smem_u32(payload + stage * p.stage_bytes);
          const uint32_t sub = (uint32_t)p.sub_bytes;
          // A stage is nk sub-stages [A 16 KB | B 16 KB | (fused unit) the remainder's B rows].  The boxes of adjacent k-blocks
          // (the next 128 bytes of the same rows) are requested back to back: measured with a load-only probe on L2-resident
          // data, one SM sustains 46-55 B/clk with one k-block per stage and 76-88 B/clk with two, and this main loop needs 64.
#pragma unroll
          for (int j = 0; j < kbs; ++j)
            if (j < nk) ptx::tma_load_2d_pair(sa + j * sub, &p.tmA, (kb + j) * BK, tc.tm * 2 * BM + cta_rank * BM, full_leader);
          if (p.b_mn) {   // this CTA's half of the tile's columns as two [64 k][64 n] blocks per k-block
            const int n0 = tc.jn * kPairBN + cta_rank * (ncols / 2);
#pragma unroll
            for (int j = 0; j < kbs; ++j)
              if (j < nk) {
                ptx::tma_load_2d_pair(sa + j * sub + BM * BK * 2, &p.tmB[tc.rank], n0, (kb + j) * BK, full_leader);
                ptx::tma_load_2d_pair(sa + j * sub + BM * BK * 2 + kMnBlockBytes, &p.tmB[tc.rank], n0 + 64, (kb + j) * BK, full_leader);
              }
          } else {
#pragma unroll
            for (int j = 0; j < kbs; ++j)
              if (j < nk) ptx::tma_load_2d_pair(sa + j * sub + BM * BK * 2, &p.tmB[tc.rank], (kb + j) * BK, tc.jn * kPairBN + cta_rank * (ncols / 2), full_leader);
          }
          if (fused) {
#pragma unroll
            for (int j = 0; j < kbs; ++j)
              if (j < nk) ptx::tma_load_2d_pair(sa + j * sub + kPairStageBytes, &p.tmBn[tc.rank], (kb + j) * BK, (tc.jn + 1) * kPairBN + cta_rank * (ncols1 / 2), full_leader);
          }
          if (++stage == p.n_stages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && leader) {
      const uint32_t tmem_base = ctrl->tmem_base;
      int stage = 0, acc = 0, fj = 0, fslot = 0;
      uint32_t phase = 0, acc_phase = 0, fph = 0;
      for (;;) {
        const int tile = feed_take(fj, fph, fslot);
        if (tile != -2) feed_release(fslot);
        if (tile < 0) break;
        const TileCoord tc = decode_ctile(tile, p);
        const bool fused = p.fuse_last && tc.jn == p.ctiles_per_rank - 1;
        // accumulator(s): one per compute tile of the unit, taken in order from the two buffers
        const int a0 = acc;
        if (!mbar_wait(ptx::smem_u32(&ctrl->tmem_empty[acc]), acc_phase ^ 1, p, ctrl, tile)) break;
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        const int a1 = acc;
        if (fused) {
          if (!mbar_wait(ptx::smem_u32(&ctrl->tmem_empty[acc]), acc_phase ^ 1, p, ctrl, tile)) break;
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(a0 * kPairBN), d_tmem1 = tmem_base + (uint32_t)(a1 * kPairBN);
        const uint32_t b_major = p.b_mn ? ptx::kIdescBMnMajor : 0u;
        const uint32_t idesc = ptx::idesc_f16(2 * BM, pair_tile_cols(p, tc.jn), BF16 ? 1 : 0) | b_major;
        const uint32_t idesc1 = fused ? ptx::idesc_f16(2 * BM, pair_tile_cols(p, tc.jn + 1), BF16 ? 1 : 0) : 0u;
        const uint64_t b_kstep = p.b_mn ? (uint64_t)(2 * 1024 >> 4) : 2u;
        bool ok = true;
        constexpr int kbs = KBS;
        for (int kb = 0, nk; kb < p.kblocks; kb += nk) {
          nk = min((kbs == 2 && p.half_stage && stage == p.n_stages - 1) ? 1 : kbs, p.kblocks - kb);
          if (!mbar_wait(ptx::smem_u32(&ctrl->full[stage]), phase, p, ctrl, tile)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = ptx::smem_u32(payload + stage * p.stage_bytes);
#pragma unroll
          for (int j = 0; j < kbs; ++j) {
            if (j >= nk) break;
            const uint32_t sj = sa + j * (uint32_t)p.sub_bytes;
            const uint64_t adesc = ptx::smem_desc_k_sw128(sj);
            const uint64_t bdesc = p.b_mn ? ptx::smem_desc_mn_sw128(sj + BM * BK * 2, kMnBlockBytes) : ptx::smem_desc_k_sw128(sj + BM * BK * 2);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
              ptx::mma_f16_ss_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)k * b_kstep, idesc, (kb | j | k) != 0);
            if (fused) {   // the remainder tile: same A sub-stage, its own B rows, the other accumulator
              const uint64_t b1desc = ptx::smem_desc_k_sw128(sj + kPairStageBytes);
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k)
                ptx::mma_f16_ss_pair(d_tmem1, adesc + (uint64_t)(k * 2), b1desc + (uint64_t)(k * 2), idesc1, (kb | j | k) != 0);
            }
          }
          ptx::mma_commit_pair(ptx::smem_u32(&ctrl->empty[stage]), 3);  // both CTAs may refill this stage
          if (++stage == p.n_stages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        ptx::mma_commit_pair(ptx::smem_u32(&ctrl->tmem_full[a0]), 3);  // accumulator complete in both CTAs
        if (fused) ptx::mma_commit_pair(ptx::smem_u32(&ctrl->tmem_full[a1]), 3);
      }
    }
  } else {
    // ---------------- epilogue: warps 2..5 of both CTAs, each CTA drains its own 128 rows ----------------
    const int quad = warp & 3;
    const int et = (int)threadIdx.x - 64;
    int acc = 0, fj = 0, fslot = 0;
    uint32_t acc_phase = 0, fph = 0;
    const uint32_t tmem_base = ctrl->tmem_base;
    uint64_t prev_issue = 0;               // thread 0: when the previous tile's stores started
    uint32_t period_ns = p.t_tile_ns;      // thread 0: time between two tiles of this CTA (estimate, then measured)
    bool stop = false;
    while (!stop) {
      const int tile = feed_take(fj, fph, fslot);   // a work unit: one compute tile, or a shard's last full tile plus its remainder
      __syncwarp();
      if (tile != -2 && lane == 0) feed_release(fslot);
      const TileCoord tc0 = decode_ctile(tile >= 0 ? tile : 0, p);
      const int nsub = (tile >= 0 && p.fuse_last && tc0.jn == p.ctiles_per_rank - 1) ? 2 : 1;
      for (int l = 0; l < nsub; ++l) {   // the unit's compute tiles, one accumulator each, in the order the MMA thread took them
      // uniform decision for all four warps: stop on the end marker or on any failed wait
      bool ok = tile >= 0;
      if (ok) ok = mbar_wait(ptx::smem_u32(&ctrl->tmem_full[acc]), acc_phase, p, ctrl, tile);
      if (ptx::bar_red_or(1, kEpiThreads, !ok)) { stop = true; break; }
      TileCoord tc = tc0;
      tc.jn += l;
      ptx::tc_fence_after();
      const int tm = tc.tm * 2 + cta_rank;  // publication tile row of this CTA's half
      const int row_in_half = quad * 32 + lane;
      const int col_in_shard = tc.jn * kPairBN;
      // Scatter to every slot (Listing 4) or store locally and hand over (Listings 3, 5).  Below seq_from the
      // workgroup-specialised schedule hands over unless the takeover rule (decided by thread 0 further down) keeps the tile.
      bool seq = tile >= p.seq_from;
      // Convert and stage this CTA's 128 x 256 half in shared memory, 128 columns at a time, as two 64-column boxes in the
      // 128B-swizzle layout of the store maps: a lane owns a row, so its 16-byte pieces go to (piece ^ row % 8) and a
      // warp's 512 bytes per instruction spread over all banks.  One thread sends the boxes out with TMA: whole 128-byte
      // lines, clipped by the maps at row M and column N_local, to the owner's slot or (Listing 4's loop over all ranks)
      // to all.  (The previous tile's stores have been waited for before the barrier at the top of this loop.)
      // Stores and operand loads leave the SM through one queue: a burst of W x 4 boxes (512 KB, 9 us of the port) holds
      // up the loads of the tile that is being multiplied meanwhile for longer than the stage ring covers.  So the boxes
      // go out one at a time, spread over three quarters of the time this CTA takes per tile (measured from the previous
      // tile; nothing is left to protect in the last wave, which goes at once).  The accumulator goes back to the MMA
      // warp when its last column has been read, before the second half's stores.
      constexpr int cpr = 4;                              // 32-column chunks per round: 128 columns, two store boxes
      const uint32_t stg = ptx::smem_u32(payload + kPairRingBytes);
      const int chunks = pair_tile_cols(p, tc.jn) / 32;   // 8, fewer for the narrow last tile of a ragged shard
      const int halves = (chunks + cpr - 1) / cpr;
      const int a_cur = acc;
      uint32_t gap_ns = 0;     // thread 0: pause between two boxes
      uint64_t due = 0;        // thread 0: when the next box may go
      for (int hf = 0; hf < halves; ++hf) {
        const int ch_end = min(chunks, cpr * hf + cpr);
#pragma unroll 1
        for (int ch = cpr * hf; ch < ch_end; ++ch) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a_cur * kPairBN + ch * 32), v);
          ptx::tmem_wait_ld();
          const uint32_t row_base = stg + (uint32_t)((((ch - cpr * hf) >> 1)) * kStoreBoxBytes + row_in_half * 128);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 q;
            if (p.kblocks == 0) {
              q = make_uint4(0, 0, 0, 0);   // K == 0: the sum is empty
            } else {
              q.x = pack2<BF16>(v[8 * i + 0], v[8 * i + 1]);
              q.y = pack2<BF16>(v[8 * i + 2], v[8 * i + 3]);
              q.z = pack2<BF16>(v[8 * i + 4], v[8 * i + 5]);
              q.w = pack2<BF16>(v[8 * i + 6], v[8 * i + 7]);
            }
            const int piece = (ch & 1) * 4 + i;
            ptx::st_shared_v4(row_base + (uint32_t)(((piece ^ (row_in_half & 7)) << 4)), q);
          }
        }
        if (hf == halves - 1) {   // accumulator drained: hand it back to the MMA warp before the last stores go out
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa(ptx::smem_u32(&ctrl->tmem_empty[acc]), 0));
          if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        fence_proxy_async();   // this thread's shared-memory writes -> the TMA unit's reads
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        if (et == 0) {
          if (hf == 0) {
            if (p.takeover && !seq && tm < p.ptiles_m) {
              // Hand over only what the communication warps can still finish: their backlog plus this CTA's publication
              // tiles, at t_pt_ns each spread over all of them, against the main-loop time of the waves still to come.
              // Near the end of the kernel (and whenever they fall behind) the producers' own store ports take the rest.
              const int mine = min(kPairBN / IRIS_TILE, p.ptiles_per_rank - tc.jn * (kPairBN / IRIS_TILE));
              const int waves_left = (p.total_ctiles - 1 - tile) / (p.gemm_ctas >> 1);
              const int queued = ld_relaxed_gpu(p.backlog);
              seq = (uint64_t)(queued + mine) * p.t_pt_ns > (uint64_t)waves_left * p.t_tile_ns * (uint64_t)(p.comm_ctas * kCommWarps);
              if (seq) atomicAdd(p.backlog + 1, 1);
              else atomicAdd(p.backlog, mine);
            }
            ctrl->keep_tile = seq ? 1 : 0;
            const uint64_t t0 = globaltimer_ns();
            if (l == 0) {   // per work unit
              if (prev_issue != 0) period_ns = (uint32_t)min((uint64_t)(4u * p.t_tile_ns + 1000u), t0 - prev_issue);
              prev_issue = t0;
            }
            int boxes = 0;
#pragma unroll
            for (int b = 0; b < kPairBN / 64; ++b) boxes += col_in_shard + 64 * b < p.n_local ? 1 : 0;
            const bool last_wave = tile >= p.total_ctiles - (p.gemm_ctas >> 1);
            // (a tile that is handed over goes at once: the communication CTAs are waiting for it)
            const bool hand_over = !seq && p.mode == IRIS_MODE_WORKGROUP_SPECIALIZED;
            // (nor is the first tile of a two-tile unit paced: the second accumulator waits behind it and the MMA thread behind both)
            gap_ns = (p.pace_stores && !last_wave && !hand_over && l == nsub - 1) ? (period_ns / 4u * 3u) / (uint32_t)(boxes * (seq ? W : 1)) : 0u;
            due = t0;
          }
          if (tm < p.ptiles_m) {
            for (int s = 0; s < W; ++s) {
              if (!seq && s != tc.rank) continue;
#pragma unroll
              for (int b = 0; b < cpr / 2; ++b) {
                const int col = col_in_shard + hf * cpr * 32 + 64 * b;
                if (col < p.n_local) {
                  // (with two-tile units among the work only the round after the accumulator's release is paced: a unit
                  // that needs both accumulators would wait behind a paced first round for 3/8 of a tile time)
                  if (gap_ns && (!p.fuse_last || hf == halves - 1)) {
                    while (globaltimer_ns() < due) __nanosleep(64);
                    due += gap_ns;
                  }
                  if (p.one_map) ptx::tma_store_4d(&p.tmC4s, col, tm * BM, tc.rank, s, stg + (uint32_t)(b * kStoreBoxBytes));
                  else ptx::tma_store_3d(&p.tmCs[s], col, tm * BM, tc.rank, stg + (uint32_t)(b * kStoreBoxBytes));
                }
              }
            }
            ptx::bulk_commit_group();
          }
          if (hf == halves - 1) {
            ptx::bulk_wait_group<0>();   // stores performed: the boxes are free and the tile may be published
            fence_proxy_async();         // async-proxy writes above -> the generic-proxy release (flags or lock) after the barrier
          } else {
            ptx::bulk_wait_group_read<0>();   // the boxes have been read and may be refilled
          }
        }
        if (hf != halves - 1) asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
      }
      if (p.mode != IRIS_MODE_BULK_SYNCHRONOUS) {
        asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        seq = ctrl->keep_tile != 0;   // (the next write to keep_tile comes after the barrier at the top of the loop)
        constexpr int subs = kPairBN / IRIS_TILE;
        const int pt_n = W * p.ptiles_per_rank;
        if (tm < p.ptiles_m) {
          if (seq) {
            if (et < subs * W) {
              const int sub = et / W, s = et % W;
              const int pj = tc.jn * subs + sub;
              if (pj < p.ptiles_per_rank) {   // a ragged shard's last tile may have only one publication tile
                const int t = tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
                st_release_flag(reinterpret_cast<int32_t*>(p.tab.base[s] + p.flag_off) + t, p.epoch, p.tab.flags_sys);
              }
            } else if (p.takeover && tile < p.seq_from && et >= 64 && et < 64 + subs) {
              // a tile the communication warps are watching: tell its warp that only the lock is left to reset
              const int pj = tc.jn * subs + (et - 64);
              if (pj < p.ptiles_per_rank) {
                const int t = tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
                (void)cas_release_gpu(lock_addr<STATIC_LOCKS>(p, tc.rank, t), 0, 2);
              }
            }
          } else if (et < subs) {
            const int pj = tc.jn * subs + et;
            if (pj < p.ptiles_per_rank) {
              const int t = tm * pt_n + tc.rank * p.ptiles_per_rank + pj;
              (void)cas_release_gpu(lock_addr<STATIC_LOCKS>(p, tc.rank, t), 0, 1);
            }
          }
        }
      }
      }   // compute tiles of the unit
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();   // the leader's MMAs read the peer's shared memory and both write both TMEMs: leave together
  if (warp == 1 && !is_comm) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(ctrl->tmem_base, 2 * kPairBN);
  }
}

// ------------------------------------------------------------------------------------------------
// Unfused producer-consumer (Section 4.1): the communication role as a kernel of its own.  The GEMM kernel runs with
// producer CTAs only on one stream; this kernel, launched right after it on a second stream with as many CTAs as the
// producers leave SMs free, is the consumer of the lock handshake: the same 32-lane acquire poll, claim, TMA copy to
// the other W-1 slots and flag publication as the communication CTAs of the single launch (comm_cta above).
// The dependency runs one way only: nothing in the GEMM kernel waits for this one, and every wait here has its
// deadline, so the pair completes (or reports a timeout) whichever kernel the hardware happens to start first.
// SUBS x SUBS_M: publication tiles per compute tile of the producing kernel (its work-item order).
// ------------------------------------------------------------------------------------------------
template <int SUBS, int SUBS_M>
__global__ void __launch_bounds__(kCommWarps * 32, 1) scatter_comm_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* payload = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  CtrlBlock* ctrl = reinterpret_cast<CtrlBlock*>(payload + kSmemPayload);   // (kCommSmemTotal: no epilogue staging here)
  const int warp = (int)threadIdx.x / 32, lane = (int)threadIdx.x % 32;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kCommWarps; ++i) ptx::mbar_init(ptx::smem_u32(&ctrl->comm_full[i]), 1);
    ctrl->abort = 0;
    ptx::fence_mbar_init();
    fence_proxy_async();
    if (p.one_map) ptx::prefetch_tensormap(&p.tmC4);
    else for (int r = 0; r < p.tab.world; ++r) ptx::prefetch_tensormap(&p.tmC[r]);
  }
  __syncthreads();
  comm_cta<false, SUBS, SUBS_M>(p, ctrl, payload, warp, lane, (int)blockIdx.x);
}

// ------------------------------------------------------------------------------------------------
// Bulk-synchronous second kernel (Listing 3, all_scatter): per publication tile, iris.put the owner's
// tile to every other rank, then publish the W ready flags.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) all_scatter_kernel(const __grid_constant__ HeapTable tab, uint64_t c_off, uint64_t flag_off, int M, int N, int n_local,
                                                          int tiles_m, int ptiles_per_rank, int rank_first, int rank_count, int32_t epoch) {
  const int W = tab.world;
  const int pt_n = W * ptiles_per_rank, pt_sel = rank_count * ptiles_per_rank;
  const int total = tiles_m * pt_sel;
  for (int it = blockIdx.x; it < total; it += gridDim.x) {
    const int tm = it / pt_sel, rank = rank_first + (it % pt_sel) / ptiles_per_rank, pj = (it % pt_sel) % ptiles_per_rank;
    const int t = tm * pt_n + rank * ptiles_per_rank + pj;
    const int rows = min(IRIS_TILE, M - tm * IRIS_TILE);
    const int cols = min(IRIS_TILE, n_local - pj * IRIS_TILE);
    const int cpr = cols / 8;  // 16-byte chunks per row
    const uint64_t local = tab.base[rank] + c_off + ((uint64_t)(tm * IRIS_TILE) * N + (uint64_t)rank * n_local + (uint64_t)pj * IRIS_TILE) * 2;
    for (int i0 = threadIdx.x; i0 < rows * cpr; i0 += 256 * 4) {
      uint4 v[4];
      uint64_t off[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * 256;
        if (i < rows * cpr) {
          off[u] = ((uint64_t)(i / cpr) * N + (uint64_t)(i % cpr) * 8) * 2;
          v[u] = ld_global_v4(reinterpret_cast<const void*>(local + off[u]));
        }
      }
      for (int s = 0; s < W; ++s) {
        if (s == rank) continue;
        const uint64_t remote = translate(local, rank, s, tab);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (i0 + u * 256 < rows * cpr) st_global_v4(reinterpret_cast<void*>(remote + off[u]), v[u]);
      }
    }
    __syncthreads();
    if ((int)threadIdx.x < W) st_release_flag(reinterpret_cast<int32_t*>(tab.base[threadIdx.x] + flag_off) + t, epoch, tab.flags_sys);
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

static int make_map(CUtensorMap* m, int dtype, int rank, void* base, const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
                    CUtensorMapSwizzle swz, const char* what) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return fail(IRIS_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(m, dtype == IRIS_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, (cuuint32_t)rank, base, dims, strides, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(IRIS_ERR_CUDA, "cuTensorMapEncodeTiled(%s) failed with CUresult %d", what, (int)r);
  return IRIS_OK;
}

// The dynamic shared-memory limit is an attribute of (function, device): set it once per device a kernel is
// launched on.  `done` is that kernel's per-device record; the device is the current one.
constexpr int kMaxDevices = 64;
static int ensure_smem_limit(const void* kern, int bytes, bool (&done)[kMaxDevices]) {
  int dev = 0;
  IRIS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < kMaxDevices && done[dev]) return IRIS_OK;
  IRIS_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (dev >= 0 && dev < kMaxDevices) done[dev] = true;
  return IRIS_OK;
}

template <int BN, bool BF16, bool STATIC_LOCKS = false>
static int launch_gemm(const GemmParams& p, int grid, bool cooperative, cudaStream_t st) {
  auto kern = gemm_all_scatter_kernel<BN, BF16, STATIC_LOCKS>;
  static bool configured[kMaxDevices] = {};
  if (int rc = ensure_smem_limit(reinterpret_cast<const void*>(kern), kSmemTotal, configured)) return rc;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = kSmemTotal;
  cfg.stream = st;
  if (cooperative) {   // CTAs that wait on one another: refuse, with a clear message, a grid that cannot be resident all at once
    int per_sm = 0, dev = 0, sms = 0;
    IRIS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kGemmThreads, kSmemTotal));
    IRIS_CUDA_TRY(cudaGetDevice(&dev));
    IRIS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (grid > per_sm * sms)
      return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter: %d CTAs cannot be co-resident (%d per SM x %d SMs)", grid, per_sm, sms);
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // CTAs that wait on one another must be co-resident
  attr[0].val.cooperative = cooperative ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  IRIS_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p));
  return IRIS_OK;
}

template <bool BF16, bool STATIC_LOCKS, bool CONSUMER, int KBS>
static int launch_gemm_pair_kbs(const GemmParams& p, int grid, cudaStream_t st, int* max_pairs_out);

// (the kernel is instantiated for one and for two k-blocks per operand stage: p.kb_per_stage selects)
template <bool BF16, bool STATIC_LOCKS = false, bool CONSUMER = false>
static int launch_gemm_pair(const GemmParams& p, int grid, cudaStream_t st, int* max_pairs_out) {
  return p.kb_per_stage == 1 ? launch_gemm_pair_kbs<BF16, STATIC_LOCKS, CONSUMER, 1>(p, grid, st, max_pairs_out)
                             : launch_gemm_pair_kbs<BF16, STATIC_LOCKS, CONSUMER, 2>(p, grid, st, max_pairs_out);
}

template <bool BF16, bool STATIC_LOCKS, bool CONSUMER, int KBS>
static int launch_gemm_pair_kbs(const GemmParams& p, int grid, cudaStream_t st, int* max_pairs_out) {
  auto kern = gemm_all_scatter_pair_kernel<BF16, STATIC_LOCKS, CONSUMER, KBS>;
  static bool configured[kMaxDevices] = {};
  if (int rc = ensure_smem_limit(reinterpret_cast<const void*>(kern), kPairSmemTotal, configured)) return rc;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(max_pairs_out ? 2 : grid));
  cfg.blockDim = dim3(CONSUMER ? kGemmThreadsFused : kGemmThreads);
  cfg.dynamicSmemBytes = kPairSmemTotal;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_pairs_out) {  // query only: how many pairs can be resident at once
    IRIS_CUDA_TRY(cudaOccupancyMaxActiveClusters(max_pairs_out, kern, &cfg));
    return IRIS_OK;
  }
  IRIS_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p));
  return IRIS_OK;
}

template <int SUBS, int SUBS_M>
static int launch_scatter_comm(const GemmParams& p, cudaStream_t st) {
  auto kern = scatter_comm_kernel<SUBS, SUBS_M>;
  static bool configured[kMaxDevices] = {};
  if (int rc = ensure_smem_limit(reinterpret_cast<const void*>(kern), kCommSmemTotal, configured)) return rc;
  kern<<<p.comm_ctas, kCommWarps * 32, kCommSmemTotal, st>>>(p);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

// How many CTAs to reserve for communication when the caller does not say.  A communication CTA moves
// one tile read plus W-1 tile writes per publication tile; one SM sustains about 55 GB/s of such TMA
// traffic while the other SMs run the GEMM (measured with per-phase %globaltimer stamps in the
// communicator warps).  The split c : (S - c) that lets both sides finish together solves
// c / (S - c) = x with x = (communication SM-seconds) / (GEMM SM-seconds); a 35 % margin covers the
// tail, where the last tiles become ready only when the GEMM ends.
static int auto_comm_ctas(int M, int N, int K, int W, int sms) {
  const double bytes = (double)W * M * N * 2.0;
  const double t_gemm = std::max(2.0 * M * N * (double)K / 1.45e15, ((double)M * K + (double)N * K) * 2.0 / 6.0e12);
  const double x = 1.35 * (bytes / 55e9) / (t_gemm * sms + 1e-12);
  int c = (int)std::ceil(sms * x / (1.0 + x));
  return std::max(4, std::min(c, sms / 3));
}

// CTA-pair kernel with the takeover rule: producers keep what the communication CTAs cannot finish, so the count only
// has to balance two things -- every communication pair is a producer pair less (and can add a wave), every byte the
// communicators do not take is stored through the producers' own ports instead.  Model per candidate count c:
// waves = ceil(tiles / pairs), t = waves * t_tile + (remote bytes - what c SMs move in that time) / (producer SMs' ports);
// the smallest t among the counts that leave at least half of the scatter to the communication CTAs (the schedule
// stays what its name says; measured differences between the candidates are a few per cent).  Kept bytes are paced
// by the producers' epilogues and cost about two thirds of their raw port time.  Constants: 45 GB/s sustained per communication SM (57 at best), 57 GB/s per
// producer port, 270 ns per k-step of a pair tile.
static int auto_comm_ctas_pair(int total_ctiles, int kblocks, double remote_bytes, int grid) {
  int best_c = 2;
  double best_t = 1e30;
  for (int c = 2; c <= grid - 2 && c <= 64; c += 2) {
    const int pairs = std::min((grid - c) / 2, std::max(1, total_ctiles));
    const double waves = std::ceil((double)total_ctiles / pairs);
    const double t_gemm = waves * (kblocks * 0.27e-6 + 2e-6);
    const double cap = c * 45e9 * t_gemm;
    if (cap < remote_bytes * 0.5 && c < std::min(grid - 2, 64) - 1) continue;
    const double kept = std::max(0.0, remote_bytes - cap);
    const double t = t_gemm + 0.67 * kept / (2.0 * pairs * 57e9);
    if (t < best_t * 0.999) { best_t = t; best_c = c; }
  }
  return best_c;
}

// ---- launch plans ---------------------------------------------------------------------------------------
// What a plan needs to know about where the slots are: a heap handle's (equally spaced from `base`, status block in
// the handle) or raw addresses (base == NULL: one tensor map per slot, single-CTA kernel only).
struct PlanEnv {
  HeapTable tab;
  char* base;          // slots bytes_per_rank apart from here, or nullptr: slots wherever tab.base says
  uint64_t bpr;
  int sm_count;
  int32_t* status;
  bool pair_any_base;  // with base == nullptr: the CTA-pair kernel may still be chosen (it then stores through per-slot maps)
};
struct Plan { GemmParams p; int bn, grid; bool pair, streamk; };

// Compute-tile width of the single-CTA kernel when the caller does not choose one.
static int default_block_n(int M, int nl, int W, int sm_count) {
  int bn = (nl % 256 == 0 || nl > 1024) ? 256 : 128;
  // Few tiles (the skinny shapes): when the 128-wide tiles all fit in one wave they put more SMs to work on the
  // B panels; when they need a second, partly filled wave (config 4: 224 tiles on 148 SMs) one wave of 256-wide
  // tiles is faster (measured 0.127 vs 0.142 ms) although a quarter of the SMs then idle.
  if ((int64_t)((M + BM - 1) / BM) * W * ((nl + 127) / 128) <= sm_count) bn = 128;
  if (nl <= 128) bn = 128;
  return bn;
}

struct PlanKey {
  const void* heap; const void* slot[IRIS_MAX_WORLD]; const void* status; uint64_t bytes_per_rank; int flags_sys;
  const void* A; const void* B[IRIS_MAX_WORLD];
  int M, N, K, world, mode, dtype;
  uint64_t c_off, flag_off, lock_off;
  int comm_ctas, max_ctas, raster_group, block_n, cta_pair, static_schedule, stream_k, wg_tail, fused_consumer, rank_first, rank_count, pace_stores, b_layout, fuse_tail, stage_k;
  uint64_t spin_timeout_ns;
};
// A few plans are kept (round-robin replacement): a step that alternates between calls -- one per rank shard in the
// host-buffer pipeline, several schedules in a comparison -- finds each of them again on its next pass.
constexpr int kPlanSlots = 16;
static std::mutex g_plan_mutex;
static Plan g_plan[kPlanSlots];
static PlanKey g_plan_key[kPlanSlots];
static bool g_plan_valid[kPlanSlots] = {};
static int g_plan_next = 0;

static void make_key(PlanKey* k, const iris_gemm_args* a, const iris_heap* h) {
  std::memset(k, 0, sizeof(*k));   // padding too: keys are compared with memcmp
  k->heap = h; k->status = h->status; k->bytes_per_rank = h->bytes_per_rank; k->flags_sys = h->flags_sys;
  for (int r = 0; r < h->world && r < IRIS_MAX_WORLD; ++r) k->slot[r] = h->slot_base[r];
  k->A = a->A;
  const int r_end = a->rank_count ? a->rank_first + a->rank_count : a->world;
  for (int r = a->rank_first; r < r_end && r < IRIS_MAX_WORLD; ++r) k->B[r] = a->B_shards ? a->B_shards[r] : nullptr;
  k->M = a->M; k->N = a->N; k->K = a->K; k->world = a->world; k->mode = a->mode; k->dtype = a->dtype;
  k->c_off = a->c_off; k->flag_off = a->flag_off; k->lock_off = a->lock_off;
  k->comm_ctas = a->comm_ctas; k->max_ctas = a->max_ctas; k->raster_group = a->raster_group; k->block_n = a->block_n;
  k->cta_pair = a->cta_pair; k->static_schedule = a->static_schedule; k->stream_k = a->stream_k; k->wg_tail = a->wg_tail;
  k->rank_first = a->rank_first; k->rank_count = a->rank_count; k->pace_stores = a->pace_stores; k->b_layout = a->b_layout; k->fuse_tail = a->fuse_tail; k->stage_k = a->stage_k;
  k->fused_consumer = a->consumer_bias != nullptr;   // the split between producers and communicators depends on it
  k->spin_timeout_ns = a->spin_timeout_ns;
}

int64_t num_tiles(int M, int N, int world) {
  if (M < 0 || N < 0 || world < 1 || world > IRIS_MAX_WORLD || N % world != 0) return -1;
  const int64_t nl = N / world;
  return (int64_t)((M + IRIS_TILE - 1) / IRIS_TILE) * world * ((nl + IRIS_TILE - 1) / IRIS_TILE);
}

// Tile geometry, grid split and tensor maps of one call: everything but the epoch.  The arguments have been checked.
static int build_plan(const iris_gemm_args* a, const PlanEnv& env, Plan& out) {
  GemmParams& p = out.p;
  int& bn = out.bn;
  int& grid = out.grid;
  bool& pair = out.pair;
  bool& streamk = out.streamk;
  const int W = a->world, nl = a->N / W;
  const int rank_first = a->rank_first, rank_count = a->rank_count ? a->rank_count : W;   // 0, 0 = every rank
  const bool wg = a->mode == IRIS_MODE_WORKGROUP_SPECIALIZED;
  const bool fused_consumer = a->consumer_bias != nullptr;
  std::memset(&p, 0, sizeof(p));
  bn = a->block_n ? a->block_n : default_block_n(a->M, nl, W, env.sm_count);
  if (nl <= 128) bn = 128;
  // CTA pairs (256 x 256 tiles) need at least two tile rows.  A shard that is not a whole number of 256-column
  // tiles is fine: TMA zero-fills the missing B rows, stores and flags are masked, and the last tile's MMA is only
  // as wide as what is left of the shard (rounded up to 32 columns), so the padding costs next to nothing.
  const bool pair_ok = a->M > BM && nl > BM && a->block_n != 128 && env.sm_count >= 4 && (env.base != nullptr || env.pair_any_base);
  if (a->cta_pair > 0 && !pair_ok) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter: cta_pair needs M > 128, N/world > 128 and block_n != 128");
  pair = pair_ok && a->cta_pair >= 0;
  int max_pairs = 0;
  if (pair) {
    const int rc = a->dtype == IRIS_BF16 ? launch_gemm_pair<true>(p, 0, nullptr, &max_pairs) : launch_gemm_pair<false>(p, 0, nullptr, &max_pairs);
    if (rc != IRIS_OK) return rc;
    if (max_pairs < 2) {
      if (a->cta_pair > 0) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter: no room for CTA pairs on this device");
      pair = false;
    }
  }
  if (pair) {   // a cap on the grid that leaves no room for whole pairs: fall back to single-CTA tiles unless pairs were demanded
    const int cap = a->max_ctas ? std::min(a->max_ctas, env.sm_count) : env.sm_count;
    if ((cap & ~1) < (wg ? 4 : 2)) {
      if (a->cta_pair > 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: max_ctas too small for CTA pairs");
      pair = false;
    }
  }
  if (pair) bn = kPairBN;
  // Ragged shard on the pair kernel: the remainder after the last full 256-column tile is computed by the pair that
  // computes that tile, on the same A stages (a 64-column tile of its own would pull in as much of A as a full one).
  p.fuse_last = (pair && a->fuse_tail >= 0 && a->b_layout == IRIS_B_N_BY_K && nl > kPairBN && nl % kPairBN != 0) ? 1 : 0;
  if (p.fuse_last && wg && a->fuse_tail == 0) {
    // workgroup_specialized hands the last wave to the producers: with fewer than three waves of the (longer, fewer) fused
    // units that wave is too large a share of the work (measured: 4096 x 2560 x 8192, two waves, 0.247 vs 0.223 ms)
    const int64_t units = (int64_t)((a->M + 2 * BM - 1) / (2 * BM)) * rank_count * (nl / kPairBN);
    const int pairs_guess = std::max(1, (a->max_ctas ? std::min(a->max_ctas, env.sm_count) : env.sm_count) / 2);
    if (units < 3 * (int64_t)pairs_guess) p.fuse_last = 0;
  }
  // Operand stages of the pair kernel: two 64-wide k-blocks per stage (3 stages of 64 KB; with a fused remainder of up to
  // 96 columns two stages and a one-k-block stage, e.g. 72 + 72 + 36 KB) unless the caller asks for one (6 of 32 KB) or
  // the fused remainder's B rows leave no room for five k-blocks (then one k-block per stage, 4 stages).
  p.kb_per_stage = a->stage_k == 64 ? 1 : 2;
  p.sub_bytes = kPairStageBytes;
  if (p.fuse_last) {
    const int rem32 = ((nl % kPairBN) + 31) & ~31;
    p.b1_bytes = (rem32 / 2) * BK * 2;
    p.sub_bytes = kPairStageBytes + (int)align_up((uint64_t)p.b1_bytes, 1024);
  }
  // Two k-blocks per stage need five k-blocks' worth of ring to pay (measured: with room for two such stages only, the
  // 448-column shard runs 9-13 % slower than with four or five one-k-block stages); unless the caller insists, fall back.
  if (p.kb_per_stage == 2 && a->stage_k == 0 && kPairRingBytes < 5 * p.sub_bytes) p.kb_per_stage = 1;
  p.stage_bytes = p.kb_per_stage * p.sub_bytes;
  p.n_stages = std::min(kPairMaxStages, kPairRingBytes / p.stage_bytes);
  // what is left of the ring after the two-k-block stages holds one more k-block (remainders up to 96 columns: 72 + 72 + 36 KB)
  p.half_stage = (p.kb_per_stage == 2 && p.n_stages < kPairMaxStages && kPairRingBytes - p.n_stages * p.stage_bytes >= p.sub_bytes) ? 1 : 0;
  p.n_stages += p.half_stage;
  p.tab = env.tab;
  p.c_off = a->c_off;
  p.flag_off = a->flag_off;
  p.lock_off = a->lock_off;
  p.timeout_ns = a->spin_timeout_ns ? a->spin_timeout_ns : kDefaultTimeoutNs;
  p.status = env.status;
  p.M = a->M; p.N = a->N; p.K = a->K; p.n_local = nl;
  p.ptiles_m = (a->M + BM - 1) / BM;
  p.tiles_m = pair ? (a->M + 2 * BM - 1) / (2 * BM) : p.ptiles_m;
  p.ctiles_per_rank = (nl + bn - 1) / bn - p.fuse_last;   // work units per rank along N
  p.ptiles_per_rank = (nl + IRIS_TILE - 1) / IRIS_TILE;
  p.rank_first = rank_first; p.rank_count = rank_count;
  p.total_ctiles = p.tiles_m * rank_count * p.ctiles_per_rank;
  p.total_ptiles = p.ptiles_m * rank_count * p.ptiles_per_rank;
  p.kblocks = (a->K + BK - 1) / BK;
  // 2048 rows per raster group: with tiles claimed in raster order the running tiles then cover about
  // 8 x 9 pair tiles, the near-square footprint that minimises operand re-reads from HBM (measured).
  p.raster_group = a->raster_group ? a->raster_group : (pair ? 8 : 16);
  p.mode = a->mode;
  p.epoch = a->epoch;
  p.b_mn = a->b_layout == IRIS_B_K_BY_N ? 1 : 0;
  grid = a->max_ctas ? std::min(a->max_ctas, env.sm_count) : env.sm_count;
  if (pair) {
    grid = std::min(grid & ~1, 2 * max_pairs);
    if (grid < (wg ? 4 : 2)) return fail(IRIS_ERR_ARG, "gemm_all_scatter: max_ctas too small for CTA pairs");
    if (wg) {
      int comm = a->comm_ctas;
      // (with consumer warps in the producer CTAs their ports are busy with OUT = C + bias: the communication CTAs
      // then get the whole scatter, as they do without the takeover rule)
      if (!comm) comm = a->wg_tail == 0 && !fused_consumer ? auto_comm_ctas_pair(p.total_ctiles, p.kblocks, (double)(W - 1) * a->M * nl * rank_count * 2.0, grid)
                                                            : auto_comm_ctas(a->M, nl * rank_count, a->K, W, grid);
      comm = std::max(2, std::min((comm + 1) & ~1, grid - 2));   // whole pairs on both sides
      p.comm_ctas = comm;
      p.gemm_ctas = 2 * std::min((grid - comm) / 2, p.total_ctiles);
    } else {
      p.comm_ctas = 0;
      p.gemm_ctas = 2 * std::min(grid / 2, p.total_ctiles);
    }
    // The fewest producer pairs that still finish in the same number of waves: on this power-capped part an SM
    // that would only idle through the last, partly filled wave is better left out, the others then clock higher
    // (W = 8, 1024 x 16384 x 16384: 256 tiles on 64 pairs instead of 74, fused_sequential 0.425 -> 0.398 ms).
    if (p.total_ctiles > 0) {
      const int units = p.gemm_ctas / 2;
      const int waves = (p.total_ctiles + units - 1) / units;
      p.gemm_ctas = 2 * ((p.total_ctiles + waves - 1) / waves);
    }
  } else if (wg) {
    if (grid < 2) return fail(IRIS_ERR_ARG, "gemm_all_scatter: workgroup_specialized needs at least 2 CTAs");
    int comm = a->comm_ctas ? a->comm_ctas : auto_comm_ctas(a->M, nl * rank_count, a->K, W, grid);
    comm = std::min(comm, std::min(grid - 1, p.total_ptiles));
    p.comm_ctas = comm;
    p.gemm_ctas = std::min(grid - comm, p.total_ctiles);
  } else {
    p.comm_ctas = 0;
    p.gemm_ctas = std::min(grid, p.total_ctiles);
  }
  // stream-K (single-CTA kernel): when the tile count leaves the last wave badly filled, cut the k-steps of all
  // tiles into equal ranges instead, one per producer CTA.
  streamk = false;
  if (!pair && a->stream_k >= 0 && p.kblocks > 0) {
    const int producers = wg ? std::max(1, std::min(grid, env.sm_count) - p.comm_ctas) : grid;
    const int64_t waves = (p.total_ctiles + producers - 1) / producers;
    const bool badly_filled = (int64_t)p.total_ctiles * 10 < waves * producers * 9;      // < 90 % of the slots used
    const bool enough_k = (int64_t)p.total_ctiles * p.kblocks >= (int64_t)producers * 4 && p.kblocks >= 8;
    (void)badly_filled;   // measured: on the skinny shapes this was meant for, operand streaming -- not the wave fill -- is the
                          // limit and the parts' round trip through the workspace costs more than it saves: on request only
    if (enough_k && a->stream_k > 0) {
      streamk = true;
      p.gemm_ctas = producers;
    }
  }
  p.streamk = streamk ? 1 : 0;
  grid = p.gemm_ctas + p.comm_ctas;
  // Which tiles the producers scatter themselves.  In workgroup_specialized mode the tiles of the last wave
  // (raster ids >= total - producer units; every unit's final tile is one of them) have no GEMM work left to
  // overlap with, so handing them to a few communication CTAs would leave their store ports as the only ones
  // busy at the end of the kernel: the producers write those tiles to all W slots and publish them, as in
  // fused_sequential mode.  wg_tail: -1 = never (Listing 5 for every tile), n > 0 = the last n compute tiles.
  p.takeover = 0;
  p.t_tile_ns = (uint32_t)std::min<int64_t>((int64_t)p.kblocks * 260, 1 << 28);   // 512 tensor cycles per k-step at full clocks
  p.pace_stores = pair && a->pace_stores >= 0 ? 1 : 0;
  if (a->mode == IRIS_MODE_FUSED_SEQUENTIAL) p.seq_from = 0;
  else if (!wg || a->wg_tail < 0) p.seq_from = INT_MAX;
  else {
    const int units = pair ? p.gemm_ctas / 2 : p.gemm_ctas;
    p.seq_from = std::max(0, p.total_ctiles - (a->wg_tail > 0 ? a->wg_tail : units));
    // wg_tail = 0 on the pair kernel: producers also keep tiles the communication CTAs could not finish in time.
    // Estimates: one SM's port stores at most 57 GB/s, shared by the CTA's communicator warps; a k-step of a pair
    // tile takes 512 tensor cycles.
    if (pair && a->wg_tail == 0) {
      p.takeover = 1;
      p.t_pt_ns = (uint32_t)((uint64_t)kCommWarps * kTileBytes * (W - 1) / 45);   // 45 GB/s: what a communication SM sustains
    }
  }

  // Tensor maps.  K == 0 has no operand to describe; the kernel then never issues a load.
  if (a->K > 0) {
    const cuuint64_t dimsA[2] = {(cuuint64_t)a->K, (cuuint64_t)a->M};
    const cuuint64_t strA[1] = {(cuuint64_t)a->K * 2};
    const cuuint32_t boxA[2] = {BK, BM};
    int rc = make_map(&p.tmA, a->dtype, 2, const_cast<void*>(a->A), dimsA, strA, boxA, CU_TENSOR_MAP_SWIZZLE_128B, "A");
    if (rc != IRIS_OK) return rc;
    for (int r = rank_first; r < rank_first + rank_count; ++r) {
      if (a->b_layout == IRIS_B_K_BY_N) {   // Listing 2's operand as printed: [K, N_local], N contiguous
        const cuuint64_t dimsB[2] = {(cuuint64_t)nl, (cuuint64_t)a->K};
        const cuuint64_t strB[1] = {(cuuint64_t)nl * 2};
        const cuuint32_t boxB[2] = {64, BK};
        rc = make_map(&p.tmB[r], a->dtype, 2, const_cast<void*>(a->B_shards[r]), dimsB, strB, boxB, CU_TENSOR_MAP_SWIZZLE_128B, "B [K, N_local]");
      } else {
        const cuuint64_t dimsB[2] = {(cuuint64_t)a->K, (cuuint64_t)nl};
        const cuuint32_t boxB[2] = {BK, (cuuint32_t)(pair ? kPairBN / 2 : bn)};   // a pair's CTA loads its half of the tile
        rc = make_map(&p.tmB[r], a->dtype, 2, const_cast<void*>(a->B_shards[r]), dimsB, strA, boxB, CU_TENSOR_MAP_SWIZZLE_128B, "B");
        if (rc == IRIS_OK && p.fuse_last) {
          const cuuint32_t boxBn[2] = {BK, (cuuint32_t)(p.b1_bytes / (BK * 2))};
          rc = make_map(&p.tmBn[r], a->dtype, 2, const_cast<void*>(a->B_shards[r]), dimsB, strA, boxBn, CU_TENSOR_MAP_SWIZZLE_128B, "B (remainder columns)");
        }
      }
      if (rc != IRIS_OK) return rc;
    }
  }
  if (env.base) {
    // C of every slot as one 4-D tensor [slot][rank][row][column]: the slots of a heap handle are bytes_per_rank apart.
    const cuuint64_t dims4[4] = {(cuuint64_t)nl, (cuuint64_t)a->M, (cuuint64_t)W, (cuuint64_t)W};
    const cuuint64_t str4[3] = {(cuuint64_t)a->N * 2, (cuuint64_t)nl * 2, (cuuint64_t)env.bpr};
    const cuuint32_t box4[4] = {IRIS_TILE, IRIS_TILE, 1, 1}, box4s[4] = {64, BM, 1, 1};
    p.one_map = 1;
    if (wg) {
      int rc = make_map(&p.tmC4, a->dtype, 4, env.base + a->c_off, dims4, str4, box4, CU_TENSOR_MAP_SWIZZLE_NONE, "C (all slots)");
      if (rc != IRIS_OK) return rc;
    }
    int rc = make_map(&p.tmC4s, a->dtype, 4, env.base + a->c_off, dims4, str4, box4s, CU_TENSOR_MAP_SWIZZLE_128B, "C (all slots, epilogue stores)");
    if (rc != IRIS_OK) return rc;
  } else {
    // slots at arbitrary addresses: C of slot s as [rank][row][column], per slot one map for the communication CTAs'
    // copies and one for the epilogue's stores
    p.one_map = 0;
    for (int s = 0; s < W; ++s) {
      const cuuint64_t dimsC[3] = {(cuuint64_t)nl, (cuuint64_t)a->M, (cuuint64_t)W};
      const cuuint64_t strC[2] = {(cuuint64_t)a->N * 2, (cuuint64_t)nl * 2};
      const cuuint32_t boxC[3] = {IRIS_TILE, IRIS_TILE, 1}, boxCs[3] = {64, BM, 1};
      int rc = wg ? make_map(&p.tmC[s], a->dtype, 3, reinterpret_cast<void*>(env.tab.base[s] + a->c_off), dimsC, strC, boxC, CU_TENSOR_MAP_SWIZZLE_NONE, "C") : IRIS_OK;
      if (rc != IRIS_OK) return rc;
      rc = make_map(&p.tmCs[s], a->dtype, 3, reinterpret_cast<void*>(env.tab.base[s] + a->c_off), dimsC, strC, boxCs, CU_TENSOR_MAP_SWIZZLE_128B, "C (epilogue stores)");
      if (rc != IRIS_OK) return rc;
    }
  }
  return IRIS_OK;
}

// Streams and events of iris_gemm_all_scatter_host's copy / compute / copy-back pipeline.
constexpr int kHostPipeChunks = 8;
struct HostPipe {
  cudaStream_t s[3];
  cudaEvent_t b_ready, a_ready[kHostPipeChunks + 1], c_ready[kHostPipeChunks + 1];
};

void free_host_pipe(iris_heap* h) {
  HostPipe* hp = static_cast<HostPipe*>(h->host_pipe);
  if (!hp) return;
  for (cudaStream_t st : hp->s) if (st) cudaStreamDestroy(st);
  if (hp->b_ready) cudaEventDestroy(hp->b_ready);
  for (int i = 0; i <= kHostPipeChunks; ++i) {
    if (hp->a_ready[i]) cudaEventDestroy(hp->a_ready[i]);
    if (hp->c_ready[i]) cudaEventDestroy(hp->c_ready[i]);
  }
  delete hp;
  h->host_pipe = nullptr;
}

}  // namespace iris

using namespace iris;

extern "C" {

int64_t iris_num_tiles(int M, int N, int world) {
  const int64_t n = num_tiles(M, N, world);
  return n < 0 ? fail(IRIS_ERR_ARG, "iris_num_tiles: bad arguments") : n;
}

size_t iris_gemm_heap_bytes(int M, int N, int world) {
  const int64_t nt = num_tiles(M, N, world);
  if (nt < 0) return 0;
  return (size_t)(align_up((uint64_t)M * N * 2, 256) + 2 * align_up((uint64_t)nt * 4, 256) + 256);
}

// Checks, plan and launches of one call.  unfused: the workgroup-specialised schedule as two kernels, producers on
// `stream` and the communication kernel on `comm_stream` (Section 4.1's unfused producer-consumer pattern).
static int enqueue_gemm_all_scatter(const iris_gemm_args* a, void* stream, bool unfused, void* comm_stream) {
  if (!a) return fail(IRIS_ERR_ARG, "gemm_all_scatter: NULL args");
  iris_heap* h = a->heap;
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "gemm_all_scatter: bad heap handle");
  const int W = a->world;
  if (W != h->world) return fail(IRIS_ERR_ARG, "gemm_all_scatter: world=%d differs from the heap's world=%d", W, h->world);
  if (a->mode < IRIS_MODE_BULK_SYNCHRONOUS || a->mode > IRIS_MODE_WORKGROUP_SPECIALIZED) return fail(IRIS_ERR_ARG, "gemm_all_scatter: unknown mode %d", a->mode);
  if (a->dtype != IRIS_F16 && a->dtype != IRIS_BF16) return fail(IRIS_ERR_ARG, "gemm_all_scatter: unknown dtype %d", a->dtype);
  if (a->M < 0 || a->N < 0 || a->K < 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: negative dimension");
  if (a->N % W != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: N=%d is not a multiple of world=%d", a->N, W);
  const int nl = a->N / W;
  if (nl % 8 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: N/world=%d must be a multiple of 8 (16-byte stores)", nl);
  if (a->K % 8 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: K=%d must be a multiple of 8 (16-byte row pitch)", a->K);
  if (a->block_n != 0 && a->block_n != 128 && a->block_n != 256) return fail(IRIS_ERR_ARG, "gemm_all_scatter: block_n must be 0, 128 or 256");
  if (a->epoch < 1) return fail(IRIS_ERR_ARG, "gemm_all_scatter: epoch must be >= 1");
  if (a->c_off % 256 != 0 || a->flag_off % 4 != 0 || a->lock_off % 4 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: misaligned heap offsets");
  if (a->comm_ctas < 0 || a->max_ctas < 0 || a->raster_group < 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: negative tuning parameter");
  if (a->cta_pair < -1 || a->cta_pair > 1) return fail(IRIS_ERR_ARG, "gemm_all_scatter: cta_pair must be -1, 0 or 1");
  if (a->pace_stores < -1 || a->pace_stores > 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: pace_stores must be 0 or -1");
  if (a->wg_tail < -1) return fail(IRIS_ERR_ARG, "gemm_all_scatter: wg_tail must be -1, 0 or a tile count");
  if (a->stream_k < -1 || a->stream_k > 1) return fail(IRIS_ERR_ARG, "gemm_all_scatter: stream_k must be -1, 0 or 1");
  if (a->stage_k != 0 && a->stage_k != 64 && a->stage_k != 128) return fail(IRIS_ERR_ARG, "gemm_all_scatter: stage_k must be 0, 64 or 128");
  if (a->fuse_tail < -1 || a->fuse_tail > 1) return fail(IRIS_ERR_ARG, "gemm_all_scatter: fuse_tail must be -1, 0 or 1");
  if (a->b_layout != IRIS_B_N_BY_K && a->b_layout != IRIS_B_K_BY_N) return fail(IRIS_ERR_ARG, "gemm_all_scatter: unknown b_layout %d", a->b_layout);
  if (a->rank_first < 0 || a->rank_count < 0 || a->rank_first + a->rank_count > W || (a->rank_count == 0 && a->rank_first != 0))
    return fail(IRIS_ERR_ARG, "gemm_all_scatter: rank range [%d, %d) outside [0, %d)", a->rank_first, a->rank_first + a->rank_count, W);
  const int rank_first = a->rank_first, rank_count = a->rank_count ? a->rank_count : W;   // 0, 0 = every rank
  // A heap over several processes: the locks of a shard live in its owner's slot and are handled with gpu-scope atomics,
  // and only the owner holds that shard of B, so a process computes its own rank's shard and nothing else.
  if (h->local_rank >= 0 && (rank_first != h->local_rank || rank_count != 1))
    return fail(IRIS_ERR_ARG, "gemm_all_scatter: on a heap over several processes rank_first must be the local rank (%d) and rank_count 1", h->local_rank);
  const int64_t nt = num_tiles(a->M, a->N, W);
  const uint64_t bpr = h->bytes_per_rank;
  const uint64_t c_bytes = (uint64_t)a->M * a->N * 2;
  if (a->c_off > bpr || c_bytes > bpr - a->c_off) return fail(IRIS_ERR_RANGE, "gemm_all_scatter: C leaves the slot");
  if (a->flag_off > bpr || (uint64_t)nt * 4 > bpr - a->flag_off) return fail(IRIS_ERR_RANGE, "gemm_all_scatter: flags leave the slot");
  const bool wg = a->mode == IRIS_MODE_WORKGROUP_SPECIALIZED;
  if (wg && (a->lock_off > bpr || (uint64_t)nt * 4 > bpr - a->lock_off)) return fail(IRIS_ERR_RANGE, "gemm_all_scatter: locks leave the slot");
  auto overlaps = [](uint64_t o1, uint64_t n1, uint64_t o2, uint64_t n2) { return n1 && n2 && o1 < o2 + n2 && o2 < o1 + n1; };
  if (overlaps(a->c_off, c_bytes, a->flag_off, (uint64_t)nt * 4) || (wg && (overlaps(a->c_off, c_bytes, a->lock_off, (uint64_t)nt * 4) || overlaps(a->flag_off, (uint64_t)nt * 4, a->lock_off, (uint64_t)nt * 4))))
    return fail(IRIS_ERR_ARG, "gemm_all_scatter: C, flag and lock regions overlap");
  const bool fused_consumer = a->consumer_bias != nullptr;
  if (fused_consumer && h->local_rank >= 0)
    return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter: consumer_bias consumes every slot; on a heap over several processes call iris_consume_bias, which reads the local slot");
  if (unfused) {
    if (!wg) return fail(IRIS_ERR_ARG, "gemm_all_scatter_unfused: the two-kernel form is the workgroup_specialized schedule (mode %d given)", a->mode);
    // consumer warps inside the producer kernel would wait for flags that the second kernel publishes, while that one
    // waits for the producers: two launches waiting on one another.  The consumer goes on a stream of its own instead.
    if (fused_consumer) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter_unfused: consumer_bias is not supported here; launch iris_consume_bias on its own stream");
  }
  if (fused_consumer) {
    if ((uint64_t)a->consumer_bias % 16 != 0 || a->consumer_out_off % 16 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: consumer bias / OUT offset must be 16-byte aligned");
    if (a->consumer_out_off > bpr || c_bytes > bpr - a->consumer_out_off) return fail(IRIS_ERR_RANGE, "gemm_all_scatter: OUT leaves the slot");
    if (overlaps(a->consumer_out_off, c_bytes, a->c_off, c_bytes) || overlaps(a->consumer_out_off, c_bytes, a->flag_off, (uint64_t)nt * 4) ||
        (wg && overlaps(a->consumer_out_off, c_bytes, a->lock_off, (uint64_t)nt * 4)))
      return fail(IRIS_ERR_ARG, "gemm_all_scatter: OUT overlaps C, the flags or the locks");
  }
  if (a->M == 0 || a->N == 0) return IRIS_OK;  // empty output: nothing to compute, nothing to publish
  if (!a->A && a->K > 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: A is NULL");
  if (!a->B_shards) return fail(IRIS_ERR_ARG, "gemm_all_scatter: B_shards is NULL");
  if ((uint64_t)a->A % 16 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: A must be 16-byte aligned");
  for (int r = rank_first; r < rank_first + rank_count; ++r)
    if (a->K > 0 && (!a->B_shards[r] || (uint64_t)a->B_shards[r] % 16 != 0)) return fail(IRIS_ERR_ARG, "gemm_all_scatter: B_shards[%d] is NULL or not 16-byte aligned", r);

  // The launch plan (tile geometry, grid split, tensor maps) depends on everything but the epoch; timing loops
  // call with the same arguments over and over, so recent plans are kept and re-used when nothing else changed.
  GemmParams p;
  int bn = 0, grid = 0;
  bool pair = false, streamk = false;
  PlanKey key;
  make_key(&key, a, h);
  bool hit = false;
  {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    for (int i = 0; i < kPlanSlots && !hit; ++i) {
      if (g_plan_valid[i] && std::memcmp(&key, &g_plan_key[i], sizeof(key)) == 0) {
        p = g_plan[i].p; bn = g_plan[i].bn; grid = g_plan[i].grid; pair = g_plan[i].pair; streamk = g_plan[i].streamk;
        hit = true;
      }
    }
  }
  auto build = [&]() -> int {
    PlanEnv env{h->table(), h->base, h->bytes_per_rank, h->sm_count, h->status, true};
    Plan pl;
    const int rc = build_plan(a, env, pl);
    p = pl.p; bn = pl.bn; grid = pl.grid; pair = pl.pair; streamk = pl.streamk;
    return rc;
  };
  if (!hit) {
    const int brc = build();
    if (brc != IRIS_OK) return brc;
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    const int i = g_plan_next;
    g_plan_next = (g_plan_next + 1) % kPlanSlots;
    g_plan[i].p = p; g_plan[i].bn = bn; g_plan[i].grid = grid; g_plan[i].pair = pair; g_plan[i].streamk = streamk;
    g_plan_key[i] = key;
    g_plan_valid[i] = true;
  }
  p.epoch = a->epoch;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc;
  const bool bf = a->dtype == IRIS_BF16;
  if (streamk) {
    // two fp32 tile slots per producer CTA, then one arrival counter per compute tile (zeroed for every launch)
    const size_t slots_bytes = (size_t)2 * p.gemm_ctas * BM * bn * sizeof(float);
    const size_t need = slots_bytes + align_up((uint64_t)p.total_ctiles * 4, 256);
    if (need > h->ws_bytes) {
      if (h->ws) { IRIS_CUDA_TRY(cudaStreamSynchronize(st)); cudaFree(h->ws); }
      h->ws = nullptr; h->ws_bytes = 0;
      if (cudaMalloc(&h->ws, need) != cudaSuccess) { cudaGetLastError(); return fail(IRIS_ERR_NOMEM, "gemm_all_scatter: stream-K workspace (%zu bytes)", need); }
      h->ws_bytes = need;
    }
    p.ws = static_cast<float*>(h->ws);
    p.arrive = reinterpret_cast<int32_t*>(static_cast<char*>(h->ws) + slots_bytes);
    IRIS_CUDA_TRY(cudaMemsetAsync(p.arrive, 0, (size_t)p.total_ctiles * 4, st));
  }
  if (pair) {
    p.dynamic = a->static_schedule ? 0 : 1;
    p.tile_counter = h->status + 16;   // spare words of the status block; every launch starts them at zero
    p.backlog = h->status + 17;        // [17] publication tiles waiting for the communication CTAs, [18] tiles kept by producers
    if (p.dynamic || p.takeover) IRIS_CUDA_TRY(cudaMemsetAsync(p.tile_counter, 0, 3 * sizeof(int32_t), st));
  }
  const bool cons_in_kernel = pair && fused_consumer && a->mode != IRIS_MODE_BULK_SYNCHRONOUS;  // BSP publishes in its 2nd kernel
  if (cons_in_kernel) { p.bias = static_cast<const uint8_t*>(a->consumer_bias); p.out_off = a->consumer_out_off; }
  // unfused: the producers alone; they wait on nothing outside their own CTA (pair), so no cooperative launch is needed
  const int ggrid = unfused ? p.gemm_ctas : grid;
  const bool coop = wg && !unfused;
  if (unfused) {   // fork: the second stream starts after whatever precedes the producers on the first (the counter resets above)
    if (!h->ev_fork) {
      IRIS_CUDA_TRY(cudaEventCreateWithFlags(reinterpret_cast<cudaEvent_t*>(&h->ev_fork), cudaEventDisableTiming));
      IRIS_CUDA_TRY(cudaEventCreateWithFlags(reinterpret_cast<cudaEvent_t*>(&h->ev_join), cudaEventDisableTiming));
    }
    IRIS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(h->ev_fork), st));
  }
  if (cons_in_kernel) rc = bf ? launch_gemm_pair<true, false, true>(p, ggrid, st, nullptr) : launch_gemm_pair<false, false, true>(p, ggrid, st, nullptr);
  else if (pair)      rc = bf ? launch_gemm_pair<true>(p, ggrid, st, nullptr) : launch_gemm_pair<false>(p, ggrid, st, nullptr);
  else if (bn == 256) rc = bf ? launch_gemm<256, true>(p, ggrid, coop, st) : launch_gemm<256, false>(p, ggrid, coop, st);
  else                rc = bf ? launch_gemm<128, true>(p, ggrid, coop, st) : launch_gemm<128, false>(p, ggrid, coop, st);
  if (rc != IRIS_OK) return rc;
  if (unfused) {
    // The producers are launched first; the communication kernel follows on its own stream and takes the SMs they left.
    // join: work enqueued on `stream` after this call sees the finished scatter.
    cudaStream_t cst = static_cast<cudaStream_t>(comm_stream);
    IRIS_CUDA_TRY(cudaStreamWaitEvent(cst, static_cast<cudaEvent_t>(h->ev_fork), 0));
    if (pair)           rc = launch_scatter_comm<2, 2>(p, cst);
    else if (bn == 256) rc = launch_scatter_comm<2, 1>(p, cst);
    else                rc = launch_scatter_comm<1, 1>(p, cst);
    if (rc != IRIS_OK) return rc;
    IRIS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(h->ev_join), cst));
    IRIS_CUDA_TRY(cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(h->ev_join), 0));
  }
  if (a->mode == IRIS_MODE_BULK_SYNCHRONOUS) {
    // Listing 3: the second kernel on the same stream; the kernel boundary is the synchronisation.
    const int g2 = std::min(p.total_ptiles, h->sm_count * 8);
    all_scatter_kernel<<<g2, 256, 0, st>>>(p.tab, a->c_off, a->flag_off, a->M, a->N, nl, p.ptiles_m, p.ptiles_per_rank, rank_first, rank_count, a->epoch);
    IRIS_CUDA_TRY(cudaGetLastError());
  }
  // Where the consumer does not ride inside the GEMM launch (single-CTA tiles, bulk-synchronous) it follows on
  // the same stream: same flags, same result.
  if (fused_consumer && !cons_in_kernel)
    return iris_consume_bias_ranks(h, a->c_off, a->consumer_out_off, a->flag_off, a->consumer_bias, a->M, a->N, W, rank_first, rank_count, a->dtype, a->epoch, 0,
                                   a->spin_timeout_ns, stream);
  return IRIS_OK;
}

int iris_gemm_all_scatter_ex(const iris_gemm_args* a, void* stream) { return enqueue_gemm_all_scatter(a, stream, false, nullptr); }

int iris_gemm_all_scatter_unfused(const iris_gemm_args* a, void* producer_stream, void* comm_stream) {
  if (producer_stream == comm_stream) return fail(IRIS_ERR_ARG, "gemm_all_scatter_unfused: the two kernels need two different streams");
  return enqueue_gemm_all_scatter(a, producer_stream, true, comm_stream);
}

static void short_form_layout(int M, int N, int world, uint64_t* flag_off, uint64_t* lock_off) {
  const int64_t nt = num_tiles(M, N, world);
  *flag_off = align_up((uint64_t)M * N * 2, 256);
  *lock_off = *flag_off + align_up((uint64_t)(nt > 0 ? nt : 0) * 4, 256);
}

// The short form and the host-buffer entry point choose where flags and locks live, so they also initialise them:
// on the heap's first such call, and whenever (M, N) -- hence the layout -- changes, both arrays are zeroed in every
// slot on `st` before the launch (stale locks would break Listing 5's handshake, stale flags >= epoch would let a
// consumer read early).  The epoch keeps growing, so zeroed flags are always "not yet published".
static int short_form_init(iris_heap* heap, int M, int N, int world, cudaStream_t st) {
  if (heap->sf_M == M && heap->sf_N == N) return IRIS_OK;
  const int64_t nt = num_tiles(M, N, world);
  uint64_t flag_off, lock_off;
  short_form_layout(M, N, world, &flag_off, &lock_off);
  const uint64_t bytes = (lock_off - flag_off) * 2;   // both arrays, each rounded up to 256 bytes
  if (nt > 0) {
    if (flag_off > heap->bytes_per_rank || bytes > heap->bytes_per_rank - flag_off) return fail(IRIS_ERR_RANGE, "gemm_all_scatter: flags and locks leave the slot");
    for (int s = 0; s < world; ++s)
      IRIS_CUDA_TRY(cudaMemsetAsync(heap->slot_base[s] + flag_off, 0, bytes, st));
  }
  heap->sf_M = M; heap->sf_N = N;
  return IRIS_OK;
}

static int short_form(const void* A, const void* const* B_shards, iris_heap* heap, int M, int N, int K, int world, int mode, int dtype, void* stream,
                      const void* bias = nullptr, uint64_t out_off = 0) {
  if (!heap_ok(heap)) return fail(IRIS_ERR_STATE, "gemm_all_scatter: bad heap handle");
  if (heap->local_rank >= 0) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter: the short form computes every rank's shard; on a heap over several processes call iris_gemm_all_scatter_ex with rank_first = the local rank");
  if (num_tiles(M, N, world) < 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter: bad M/N/world");
  iris_gemm_args a;
  std::memset(&a, 0, sizeof(a));
  a.A = A; a.B_shards = B_shards; a.heap = heap;
  a.M = M; a.N = N; a.K = K; a.world = world; a.mode = mode; a.dtype = dtype;
  a.c_off = 0;
  short_form_layout(M, N, world, &a.flag_off, &a.lock_off);
  a.epoch = heap->epoch + 1;
  a.consumer_bias = bias;
  a.consumer_out_off = out_off;
  int rc = short_form_init(heap, M, N, world, static_cast<cudaStream_t>(stream));
  if (rc != IRIS_OK) return rc;
  rc = iris_gemm_all_scatter_ex(&a, stream);
  if (rc == IRIS_OK) heap->epoch = a.epoch;
  return rc;
}

int gemm_all_scatter(const void* A, const void* const* B_shards, iris_heap* heap, int M, int N, int K, int world, int mode) {
  return short_form(A, B_shards, heap, M, N, K, world, mode, IRIS_BF16, nullptr);
}

int iris_gemm_takeover_stats(const iris_heap* heap, int32_t out[2]) {
  if (!heap_ok(heap) || !out) return fail(IRIS_ERR_ARG, "iris_gemm_takeover_stats: bad argument");
  int32_t w[2];
  IRIS_CUDA_TRY(cudaSetDevice(heap->device));
  IRIS_CUDA_TRY(cudaMemcpy(w, heap->status + 17, sizeof(w), cudaMemcpyDeviceToHost));
  out[0] = w[1];
  out[1] = w[0];
  return IRIS_OK;
}

uint64_t iris_gemm_out_offset(int M, int N, int world) {
  if (num_tiles(M, N, world) < 0) return 0;
  uint64_t flag_off, lock_off;
  short_form_layout(M, N, world, &flag_off, &lock_off);
  return lock_off + (lock_off - flag_off);
}

int iris_gemm_all_scatter_host(const void* A_host, const void* const* B_shards_host, void* C_host, int32_t* flags_host, const void* bias_host,
                               void* OUT_host, iris_heap* heap, int M, int N, int K, int world, int mode, int dtype, int out_slot) {
  if (!heap_ok(heap)) return fail(IRIS_ERR_STATE, "gemm_all_scatter_host: bad heap handle");
  if (heap->local_rank >= 0) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter_host: not available on a heap over several processes");
  if (world != heap->world || out_slot < 0 || out_slot >= world) return fail(IRIS_ERR_ARG, "gemm_all_scatter_host: bad world or out_slot");
  const int64_t nt = num_tiles(M, N, world);
  if (nt < 0 || K < 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_host: bad M/N/K/world");
  if ((M > 0 && N > 0) && (!A_host || !B_shards_host || !C_host)) return fail(IRIS_ERR_ARG, "gemm_all_scatter_host: NULL buffer");
  if ((bias_host == nullptr) != (OUT_host == nullptr)) return fail(IRIS_ERR_ARG, "gemm_all_scatter_host: bias_host and OUT_host go together");
  const size_t c_bytes = (size_t)M * N * 2;
  const uint64_t out_off = iris_gemm_out_offset(M, N, world);
  if (bias_host && out_off + c_bytes > heap->bytes_per_rank) return fail(IRIS_ERR_RANGE, "gemm_all_scatter_host: heap slot too small for OUT");
  const size_t a_bytes = (size_t)M * K * 2, b_bytes = (size_t)N * K * 2, shard_bytes = world ? b_bytes / world : 0;
  const size_t stage_b_need = b_bytes + (bias_host ? align_up((uint64_t)N * 2, 256) : 0);
  IRIS_CUDA_TRY(cudaSetDevice(heap->device));
  IRIS_CUDA_TRY(cudaDeviceSynchronize());   // the call owns the heap from here on; it returns only when everything is done
  if (a_bytes > heap->stage_a_bytes) {
    if (heap->stage_a) cudaFree(heap->stage_a);
    heap->stage_a = nullptr; heap->stage_a_bytes = 0;
    if (cudaMalloc(&heap->stage_a, a_bytes) != cudaSuccess) { cudaGetLastError(); return fail(IRIS_ERR_NOMEM, "gemm_all_scatter_host: staging for A"); }
    heap->stage_a_bytes = a_bytes;
  }
  if (stage_b_need > heap->stage_b_bytes) {
    if (heap->stage_b) cudaFree(heap->stage_b);
    heap->stage_b = nullptr; heap->stage_b_bytes = 0;
    if (cudaMalloc(&heap->stage_b, stage_b_need) != cudaSuccess) { cudaGetLastError(); return fail(IRIS_ERR_NOMEM, "gemm_all_scatter_host: staging for B"); }
    heap->stage_b_bytes = stage_b_need;
  }
  HostPipe* hp = static_cast<HostPipe*>(heap->host_pipe);
  if (!hp) {
    hp = new HostPipe();
    std::memset(hp, 0, sizeof(*hp));
    heap->host_pipe = hp;
    for (int i = 0; i < 3; ++i) IRIS_CUDA_TRY(cudaStreamCreateWithFlags(&hp->s[i], cudaStreamNonBlocking));
    IRIS_CUDA_TRY(cudaEventCreateWithFlags(&hp->b_ready, cudaEventDisableTiming));
    for (int i = 0; i <= kHostPipeChunks; ++i) {
      IRIS_CUDA_TRY(cudaEventCreateWithFlags(&hp->a_ready[i], cudaEventDisableTiming));
      IRIS_CUDA_TRY(cudaEventCreateWithFlags(&hp->c_ready[i], cudaEventDisableTiming));
    }
  }
  cudaStream_t s_in = hp->s[0], s_run = hp->s[1], s_out = hp->s[2];

  // Three streams: host-to-device copies, kernels, device-to-host copies.  The smaller operand goes first and whole,
  // the other one in blocks; every block is its own gemm_all_scatter, and its part of C (and OUT) starts back to the
  // host as soon as its kernels are done, so the host link carries both directions at once and the GEMM hides behind
  // the copies.
  //   by ranks (A is the smaller operand)  block = one rank's shard B_r: the call covers ranks [r, r+1), all rows --
  //                                        what that rank of a real job would run -- and returns a column block
  //   by rows  (B is the smaller operand)  block = rows [r0, r1) of A: C, OUT, flags and locks of a row block are
  //                                        contiguous in the short form's layout, so a block is the same call with
  //                                        shifted offsets, and returns whole rows
  uint64_t flag_off, lock_off;
  short_form_layout(M, N, world, &flag_off, &lock_off);
  const int nl = world ? N / world : 0;
  const int64_t tiles_per_row = (int64_t)world * ((nl + IRIS_TILE - 1) / IRIS_TILE);
  const bool by_ranks = world >= 2 && world <= kHostPipeChunks && a_bytes <= b_bytes && c_bytes > 0;
  int rows_per_block = M;   // by rows: whole problem unless it is tall enough to be worth cutting (blocks of whole pair tiles)
  if (!by_ranks && M >= 1024) rows_per_block = std::max(512, (int)align_up((uint64_t)(M + kHostPipeChunks - 1) / kHostPipeChunks, 256));
  const int blocks = by_ranks ? world : std::max(1, rows_per_block ? (M + rows_per_block - 1) / rows_per_block : 1);

  const void* dB[IRIS_MAX_WORLD] = {nullptr};
  for (int r = 0; r < world; ++r) dB[r] = static_cast<char*>(heap->stage_b) + (size_t)r * shard_bytes;
  void* dbias = static_cast<char*>(heap->stage_b) + b_bytes;
  if (bias_host && N > 0) IRIS_CUDA_TRY(cudaMemcpyAsync(dbias, bias_host, (size_t)N * 2, cudaMemcpyHostToDevice, s_in));
  if (by_ranks) {
    if (a_bytes) IRIS_CUDA_TRY(cudaMemcpyAsync(heap->stage_a, A_host, a_bytes, cudaMemcpyHostToDevice, s_in));
  } else {
    for (int r = 0; r < world; ++r)
      if (shard_bytes) IRIS_CUDA_TRY(cudaMemcpyAsync(const_cast<void*>(dB[r]), B_shards_host[r], shard_bytes, cudaMemcpyHostToDevice, s_in));
  }
  IRIS_CUDA_TRY(cudaEventRecord(hp->b_ready, s_in));
  IRIS_CUDA_TRY(cudaStreamWaitEvent(s_run, hp->b_ready, 0));

  char* slot = heap->slot_base[out_slot];
  if (int irc = short_form_init(heap, M, N, world, s_run)) return irc;
  const int32_t epoch = heap->epoch + 1;
  for (int blk = 0; blk < blocks; ++blk) {
    const int r0 = by_ranks ? 0 : blk * rows_per_block;
    const int rows = by_ranks ? M : std::min(rows_per_block, M - r0);
    const size_t a_off = (size_t)r0 * K * 2, row_off = (size_t)r0 * N * 2;
    if (by_ranks) {
      if (shard_bytes) IRIS_CUDA_TRY(cudaMemcpyAsync(const_cast<void*>(dB[blk]), B_shards_host[blk], shard_bytes, cudaMemcpyHostToDevice, s_in));
    } else if (rows > 0 && K > 0) {
      IRIS_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(heap->stage_a) + a_off, static_cast<const char*>(A_host) + a_off, (size_t)rows * K * 2, cudaMemcpyHostToDevice, s_in));
    }
    IRIS_CUDA_TRY(cudaEventRecord(hp->a_ready[blk], s_in));
    IRIS_CUDA_TRY(cudaStreamWaitEvent(s_run, hp->a_ready[blk], 0));
    iris_gemm_args a;
    std::memset(&a, 0, sizeof(a));
    a.A = static_cast<char*>(heap->stage_a) + a_off;
    a.B_shards = dB; a.heap = heap;
    a.M = rows; a.N = N; a.K = K; a.world = world; a.mode = mode; a.dtype = dtype;
    a.c_off = row_off;
    a.flag_off = flag_off + (uint64_t)(r0 / IRIS_TILE) * tiles_per_row * 4;
    a.lock_off = lock_off + (uint64_t)(r0 / IRIS_TILE) * tiles_per_row * 4;
    a.epoch = epoch;
    if (by_ranks) { a.rank_first = blk; a.rank_count = 1; }
    // with a bias the consumer is part of the same call (inside the GEMM launch where the kernel supports it)
    a.consumer_bias = (bias_host && c_bytes) ? dbias : nullptr;
    a.consumer_out_off = out_off + row_off;
    const int rc = iris_gemm_all_scatter_ex(&a, s_run);
    if (rc != IRIS_OK) { cudaDeviceSynchronize(); return rc; }
    IRIS_CUDA_TRY(cudaEventRecord(hp->c_ready[blk], s_run));
    IRIS_CUDA_TRY(cudaStreamWaitEvent(s_out, hp->c_ready[blk], 0));
    if (rows > 0 && N > 0) {
      if (by_ranks) {   // rank blk's columns of every row
        const size_t col_off = (size_t)blk * nl * 2, pitch = (size_t)N * 2;
        IRIS_CUDA_TRY(cudaMemcpy2DAsync(static_cast<char*>(C_host) + col_off, pitch, slot + col_off, pitch, (size_t)nl * 2, (size_t)M, cudaMemcpyDeviceToHost, s_out));
        if (bias_host) IRIS_CUDA_TRY(cudaMemcpy2DAsync(static_cast<char*>(OUT_host) + col_off, pitch, slot + out_off + col_off, pitch, (size_t)nl * 2, (size_t)M, cudaMemcpyDeviceToHost, s_out));
      } else {
        IRIS_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(C_host) + row_off, slot + row_off, (size_t)rows * N * 2, cudaMemcpyDeviceToHost, s_out));
        if (bias_host) IRIS_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(OUT_host) + row_off, slot + out_off + row_off, (size_t)rows * N * 2, cudaMemcpyDeviceToHost, s_out));
      }
    }
  }
  heap->epoch = epoch;
  if (flags_host && nt > 0)
    for (int s = 0; s < world; ++s)
      IRIS_CUDA_TRY(cudaMemcpyAsync(flags_host + (size_t)s * nt, heap->slot_base[s] + flag_off, (size_t)nt * 4, cudaMemcpyDeviceToHost, s_out));
  IRIS_CUDA_TRY(cudaStreamSynchronize(s_out));
  IRIS_CUDA_TRY(cudaStreamSynchronize(s_in));
  return iris_status_check(heap, s_run, nullptr);
}

// The one entry point that allocates nothing (see the header).  Workgroup-specialised schedule with the
// locks and the status block in g_noalloc_scratch.
int iris_gemm_all_scatter_noalloc(const void* A, const void* const* B_shards, const uint64_t* slot_bases, size_t bytes_per_rank, int M, int N,
                                  int K, int world, int dtype, uint64_t c_off, uint64_t flag_off, int32_t epoch, void* stream) {
  if (world < 1 || world > IRIS_MAX_WORLD) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: world=%d not in [1,%d]", world, IRIS_MAX_WORLD);
  if (!slot_bases) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: slot_bases is NULL");
  if (dtype != IRIS_F16 && dtype != IRIS_BF16) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: unknown dtype %d", dtype);
  if (M < 0 || N < 0 || K < 0 || N % world != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: bad M/N/K (N must be a multiple of world)");
  const int nl = N / world;
  if (nl % 8 != 0 || K % 8 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: N/world and K must be multiples of 8");
  if (epoch < 1 || c_off % 256 != 0 || flag_off % 4 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: epoch must be >= 1, c_off %% 256 == 0, flag_off %% 4 == 0");
  const int64_t nt = num_tiles(M, N, world);
  if (nt > kNoAllocMaxTiles)
    return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter_noalloc: %lld publication tiles exceed the static scratch limit of %d (use iris_gemm_all_scatter_ex with locks in the heap)",
                (long long)nt, kNoAllocMaxTiles);
  const uint64_t c_bytes = (uint64_t)M * N * 2;
  if (c_off > bytes_per_rank || c_bytes > bytes_per_rank - c_off || flag_off > bytes_per_rank || (uint64_t)nt * 4 > bytes_per_rank - flag_off)
    return fail(IRIS_ERR_RANGE, "gemm_all_scatter_noalloc: C or the flags leave the slot");
  if (c_bytes && nt && c_off < flag_off + (uint64_t)nt * 4 && flag_off < c_off + c_bytes) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: C and flag regions overlap");
  for (int r = 0; r < world; ++r)
    if (slot_bases[r] == 0 || slot_bases[r] % 256 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: slot_bases[%d] is NULL or not 256-byte aligned", r);
  if (M == 0 || N == 0) return IRIS_OK;
  if (K > 0) {
    if (!A || (uint64_t)A % 16 != 0 || !B_shards) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: A/B_shards NULL or A not 16-byte aligned");
    for (int r = 0; r < world; ++r)
      if (!B_shards[r] || (uint64_t)B_shards[r] % 16 != 0) return fail(IRIS_ERR_ARG, "gemm_all_scatter_noalloc: B_shards[%d] is NULL or not 16-byte aligned", r);
  }

  // Set-up, once per device, with that device current: the device address of the static scratch.  (The record is
  // filled without a lock: two threads making a device's first call at the same time both look the address up and
  // store the same value.)
  static int32_t* scratch_of_device[kMaxDevices] = {nullptr};
  int dev = -1, sms = 0;
  IRIS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter_noalloc: device ordinal %d not supported", dev);
  if (!scratch_of_device[dev]) {
    void* sym = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&sym, g_noalloc_scratch);
    if (e != cudaSuccess || !sym) return fail(IRIS_ERR_CUDA, "gemm_all_scatter_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
    scratch_of_device[dev] = static_cast<int32_t*>(sym);
  }
  int32_t* scratch = scratch_of_device[dev];
  IRIS_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (sms < 2) return fail(IRIS_ERR_UNSUPPORTED, "gemm_all_scatter_noalloc: needs at least 2 SMs");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps the previous call's contents: the status block and the locks in use must start at zero.
  IRIS_CUDA_TRY(cudaMemsetAsync(scratch, 0, (size_t)(kNoAllocStatusWords + nt) * 4, st));

  // The plan is the one iris_gemm_all_scatter_ex builds for workgroup_specialized with default tuning (same function:
  // CTA-pair tiles where the shape allows them, single-CTA tiles otherwise), with the slots at the caller's addresses
  // (one store map per slot) and the locks, the work-unit counter and the status block in the scratch.
  iris_gemm_args a;
  std::memset(&a, 0, sizeof(a));
  a.A = A; a.B_shards = B_shards;
  a.M = M; a.N = N; a.K = K; a.world = world; a.mode = IRIS_MODE_WORKGROUP_SPECIALIZED; a.dtype = dtype;
  a.c_off = c_off; a.flag_off = flag_off; a.epoch = epoch;
  PlanEnv env{};
  for (int r = 0; r < world; ++r) env.tab.base[r] = slot_bases[r];
  env.tab.bytes_per_rank = bytes_per_rank;
  env.tab.world = world;
  env.base = nullptr;
  env.bpr = bytes_per_rank;
  env.sm_count = sms;
  env.status = scratch;
  env.pair_any_base = true;
  Plan pl;
  int rc = build_plan(&a, env, pl);
  if (rc != IRIS_OK) return rc;
  if (pl.streamk) return fail(IRIS_ERR_STATE, "gemm_all_scatter_noalloc: unexpected plan");
  pl.p.epoch = epoch;
  const bool bf = dtype == IRIS_BF16;
  if (pl.pair) {
    pl.p.dynamic = 1;
    pl.p.tile_counter = scratch + 16;   // spare words of the scratch's status block, zeroed above with the rest
    pl.p.backlog = scratch + 17;
    rc = bf ? launch_gemm_pair<true, true>(pl.p, pl.grid, st, nullptr) : launch_gemm_pair<false, true>(pl.p, pl.grid, st, nullptr);
  } else if (pl.bn == 256) rc = bf ? launch_gemm<256, true, true>(pl.p, pl.grid, true, st) : launch_gemm<256, false, true>(pl.p, pl.grid, true, st);
  else              rc = bf ? launch_gemm<128, true, true>(pl.p, pl.grid, true, st) : launch_gemm<128, false, true>(pl.p, pl.grid, true, st);
  if (rc != IRIS_OK) return rc;
  // the status words come back on the caller's stream (no other stream is touched), then one wait for that stream
  int32_t host_status[kStatusWords] = {0};
  IRIS_CUDA_TRY(cudaMemcpyAsync(host_status, scratch, sizeof(host_status), cudaMemcpyDeviceToHost, st));
  IRIS_CUDA_TRY(cudaStreamSynchronize(st));
  if (host_status[0] != 0)
    return fail(host_status[0], "gemm_all_scatter_noalloc: device-side wait expired: block=%d tile=%d", host_status[2], host_status[3]);
  return IRIS_OK;
}



}  // extern "C"
