// Flag-gated consumer: waits (acquire; gpu scope, system scope on a heap over several processes) for a publication tile's ready flag in a slot, then
// reads that tile of C and writes OUT = C + bias.  This is the consumer side of the paper's
// producer-consumer handshake (Section 4.1): poll the tile's flag with acquire-ordered loads and touch
// the data only once it has been seen set.  HBM-bound: 16-byte coalesced accesses, one warp
// instruction covers 512 contiguous bytes of a row, several CTAs per SM for latency hiding.
#include "iris_device.cuh"

namespace iris {

constexpr int kConsThreads = 256;

template <bool BF16>
__global__ void __launch_bounds__(kConsThreads) consume_bias_kernel(const __grid_constant__ HeapTable tab, uint64_t c_off, uint64_t out_off, uint64_t flag_off,
                                                                    const uint8_t* bias, int M, int N, int n_local, int tiles_m,
                                                                    int ptiles_per_rank, int rank_first, int rank_count, int slot_first, int slot_count,
                                                                    int32_t epoch, uint64_t timeout_ns, int32_t* status) {
  const int W = tab.world;
  const int pt_n = W * ptiles_per_rank;            // publication tiles per tile row, all ranks (the flag index uses this)
  const int pt_sel = rank_count * ptiles_per_rank; // ... of the ranks this call covers
  const int items = tiles_m * pt_sel * slot_count;  // (tile, slot) pairs, tile-major so early tiles are consumed first everywhere
  for (int it = blockIdx.x; it < items; it += gridDim.x) {
    const int ti = it / slot_count, s = slot_first + it % slot_count;
    const int tm = ti / pt_sel, rank = rank_first + (ti % pt_sel) / ptiles_per_rank, pj = (ti % pt_sel) % ptiles_per_rank;
    const int t = tm * pt_n + rank * ptiles_per_rank + pj;
    // ---- acquire the tile in slot s ----
    int failed = 0;
    if (threadIdx.x == 0) {
      const int32_t* flag = reinterpret_cast<const int32_t*>(tab.base[s] + flag_off) + t;
      int32_t seen = ld_acquire_flag(flag, tab.flags_sys);
      if (seen < epoch) {
        const uint64_t start = globaltimer_ns();
        uint32_t spins = 0;
        while ((seen = ld_acquire_flag(flag, tab.flags_sys)) < epoch) {
          __nanosleep(256);   // the tile is still being produced: leave the issue slots to whoever shares this SM
          if ((++spins & 31u) == 0 && globaltimer_ns() - start > timeout_ns) {
            report_timeout(status, KID_CONSUMER, t, s, seen, epoch);
            failed = 1;
            break;
          }
        }
      }
    }
    // the barrier orders thread 0's acquire before every thread's reads of the tile
    if (__syncthreads_or(failed)) return;
    const int rows = min(IRIS_TILE, M - tm * IRIS_TILE);
    const int cols = min(IRIS_TILE, n_local - pj * IRIS_TILE);
    const int cpr = cols / 8;
    const uint64_t col0 = (uint64_t)rank * n_local + (uint64_t)pj * IRIS_TILE;
    const uint64_t tile_off = ((uint64_t)(tm * IRIS_TILE) * N + col0) * 2;
    const uint64_t src = tab.base[s] + c_off + tile_off;
    const uint64_t dst = tab.base[s] + out_off + tile_off;
    for (int i0 = threadIdx.x; i0 < rows * cpr; i0 += kConsThreads * 4) {
      uint4 v[4], b[4];
      uint64_t off[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kConsThreads;
        if (i < rows * cpr) {
          const int r = i / cpr, ch = i % cpr;
          off[u] = ((uint64_t)r * N + (uint64_t)ch * 8) * 2;
          v[u] = ld_global_v4(reinterpret_cast<const void*>(src + off[u]));
          b[u] = *reinterpret_cast<const uint4*>(bias + (col0 + (uint64_t)ch * 8) * 2);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (i0 + u * kConsThreads < rows * cpr) {
          uint4 o;
          o.x = add2<BF16>(v[u].x, b[u].x);
          o.y = add2<BF16>(v[u].y, b[u].y);
          o.z = add2<BF16>(v[u].z, b[u].z);
          o.w = add2<BF16>(v[u].w, b[u].w);
          st_global_v4(reinterpret_cast<void*>(dst + off[u]), o);
        }
      }
    }
  }
}

}  // namespace iris

using namespace iris;

extern "C" int iris_consume_bias(iris_heap* h, uint64_t c_off, uint64_t out_off, uint64_t flag_off, const void* bias, int M, int N, int world,
                                 int dtype, int32_t epoch, int ctas, uint64_t timeout_ns, void* stream) {
  return iris_consume_bias_ranks(h, c_off, out_off, flag_off, bias, M, N, world, 0, world, dtype, epoch, ctas, timeout_ns, stream);
}

extern "C" int iris_consume_bias_ranks(iris_heap* h, uint64_t c_off, uint64_t out_off, uint64_t flag_off, const void* bias, int M, int N, int world,
                                       int rank_first, int rank_count, int dtype, int32_t epoch, int ctas, uint64_t timeout_ns, void* stream) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_consume_bias: bad heap handle");
  if (world != h->world) return fail(IRIS_ERR_ARG, "iris_consume_bias: world differs from the heap's");
  if (rank_first < 0 || rank_count < 0 || rank_first + rank_count > world) return fail(IRIS_ERR_ARG, "iris_consume_bias: rank range outside [0, world)");
  if (dtype != IRIS_F16 && dtype != IRIS_BF16) return fail(IRIS_ERR_ARG, "iris_consume_bias: unknown dtype");
  if (M < 0 || N < 0 || N % world != 0 || (N / world) % 8 != 0) return fail(IRIS_ERR_ARG, "iris_consume_bias: bad M/N (N/world must be a multiple of 8)");
  if (c_off % 16 != 0 || out_off % 16 != 0 || flag_off % 4 != 0) return fail(IRIS_ERR_ARG, "iris_consume_bias: misaligned offsets");
  if (M == 0 || N == 0 || rank_count == 0) return IRIS_OK;
  if (!bias || (uint64_t)bias % 16 != 0) return fail(IRIS_ERR_ARG, "iris_consume_bias: bias is NULL or not 16-byte aligned");
  const uint64_t bpr = h->bytes_per_rank, bytes = (uint64_t)M * N * 2;
  const int nl = N / world;
  const int tiles_m = (M + IRIS_TILE - 1) / IRIS_TILE, ptr_ = (nl + IRIS_TILE - 1) / IRIS_TILE;
  const uint64_t nt = (uint64_t)tiles_m * world * ptr_;
  if (c_off > bpr || bytes > bpr - c_off || out_off > bpr || bytes > bpr - out_off || flag_off > bpr || nt * 4 > bpr - flag_off)
    return fail(IRIS_ERR_RANGE, "iris_consume_bias: a region leaves the slot");
  if (c_off < out_off + bytes && out_off < c_off + bytes) return fail(IRIS_ERR_ARG, "iris_consume_bias: C and OUT overlap");
  // every slot of a one-process heap (each emulated rank consumes its copy); this process's own slot otherwise
  const int slot_first = h->local_rank >= 0 ? h->local_rank : 0, slot_count = h->local_rank >= 0 ? 1 : world;
  const uint64_t items = (uint64_t)tiles_m * rank_count * ptr_ * slot_count;
  uint64_t grid = ctas > 0 ? (uint64_t)ctas : (uint64_t)h->sm_count * 8;
  if (grid > items) grid = items;
  const uint64_t to = timeout_ns ? timeout_ns : kDefaultTimeoutNs;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == IRIS_BF16)
    consume_bias_kernel<true><<<(int)grid, kConsThreads, 0, st>>>(h->table(), c_off, out_off, flag_off, static_cast<const uint8_t*>(bias), M, N, nl, tiles_m, ptr_, rank_first, rank_count, slot_first, slot_count, epoch, to, h->status);
  else
    consume_bias_kernel<false><<<(int)grid, kConsThreads, 0, st>>>(h->table(), c_off, out_off, flag_off, static_cast<const uint8_t*>(bias), M, N, nl, tiles_m, ptr_, rank_first, rank_count, slot_first, slot_count, epoch, to, h->status);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}
