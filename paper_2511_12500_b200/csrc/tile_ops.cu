// Tile put / get, int32 atomics on heap addresses, and the all-store / all-load microbenchmark
// kernels (Table 3; Section 5.1).  All of this is HBM-bound byte movement: 16-byte coalesced
// accesses, enough loads in flight per thread, grids sized in multiples of the SM count.
#include "iris_device.cuh"

namespace iris {

// ---- 2-D copy between two (already range-checked) regions; translation happens here ----------
// Each side is either used as given (rank pair {-1, -1}: a local heap address or a buffer outside the heap)
// or translated from the caller's address space to the rank whose memory is touched (Section 3.3).
//   put   src as given,            dst translate(from -> to)
//   get   src translate(from -> to), dst as given
//   copy  src translate(cur -> from), dst translate(cur -> to)
//   load / store: like get / put with the local side outside the heap (the value-based API of Table 3,
//   with a device buffer standing in for the registers)
struct Xlate { int from, to; };
template <bool VEC16>
__global__ void __launch_bounds__(256) copy2d_kernel(const __grid_constant__ HeapTable tab, uint64_t src, uint64_t dst, size_t rows, size_t row_bytes,
                                                     size_t src_pitch, size_t dst_pitch, Xlate xs, Xlate xd) {
  const uint64_t s = xs.from >= 0 ? translate(src, xs.from, xs.to, tab) : src;
  const uint64_t d = xd.from >= 0 ? translate(dst, xd.from, xd.to, tab) : dst;
  const size_t unit = VEC16 ? 16 : 1;
  const size_t per_row = row_bytes / unit;
  const size_t total = rows * per_row;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t r = i / per_row, c = (i % per_row) * unit;
    if (VEC16) {
      st_global_v4(reinterpret_cast<void*>(d + r * dst_pitch + c), ld_global_v4(reinterpret_cast<const void*>(s + r * src_pitch + c)));
    } else {
      *reinterpret_cast<uint8_t*>(d + r * dst_pitch + c) = *reinterpret_cast<const uint8_t*>(s + r * src_pitch + c);
    }
  }
}

// ---- atomics -------------------------------------------------------------------------------------
template <bool IS_CAS>
__global__ void __launch_bounds__(256) atomic_vec_kernel(const __grid_constant__ HeapTable tab, uint64_t ptr, size_t count, size_t stride, int from_rank, int to_rank,
                                                         int32_t cmp, int32_t val, int sem, int scope, int32_t* old_out) {
  const uint64_t p = translate(ptr, from_rank, to_rank, tab);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
    const int32_t old = atomic_rmw<IS_CAS>(reinterpret_cast<int32_t*>(p + i * stride), cmp, val, sem, scope);
    if (old_out) old_out[i] = old;
  }
}

// The other read-modify-write atomics of Table 3 (xchg, and, or, xor, min, max), same sem x scope choice.
#define IRIS_RMW_CASE(SEMV, SCOPEV, SEMS, SCOPES)                                                                      \
  if (sem == SEMV && scope == SCOPEV) {                                                                                \
    switch (op) {                                                                                                      \
      case IRIS_OP_XCHG: asm volatile("atom." SEMS "." SCOPES ".global.exch.b32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break; \
      case IRIS_OP_AND:  asm volatile("atom." SEMS "." SCOPES ".global.and.b32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;  \
      case IRIS_OP_OR:   asm volatile("atom." SEMS "." SCOPES ".global.or.b32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;   \
      case IRIS_OP_XOR:  asm volatile("atom." SEMS "." SCOPES ".global.xor.b32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;  \
      case IRIS_OP_MIN:  asm volatile("atom." SEMS "." SCOPES ".global.min.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;  \
      case IRIS_OP_MAX:  asm volatile("atom." SEMS "." SCOPES ".global.max.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;  \
      default:           asm volatile("atom." SEMS "." SCOPES ".global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(val) : "memory"); break;  \
    }                                                                                                                  \
    return old;                                                                                                        \
  }

__device__ __forceinline__ int32_t atomic_op(int32_t* p, int op, int32_t val, int sem, int scope) {
  int32_t old = 0;
  IRIS_RMW_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_BLOCK, "relaxed", "cta")
  IRIS_RMW_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_GPU, "relaxed", "gpu")
  IRIS_RMW_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_SYS, "relaxed", "sys")
  IRIS_RMW_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_BLOCK, "acquire", "cta")
  IRIS_RMW_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_GPU, "acquire", "gpu")
  IRIS_RMW_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_SYS, "acquire", "sys")
  IRIS_RMW_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_BLOCK, "release", "cta")
  IRIS_RMW_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_GPU, "release", "gpu")
  IRIS_RMW_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_SYS, "release", "sys")
  IRIS_RMW_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_BLOCK, "acq_rel", "cta")
  IRIS_RMW_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_GPU, "acq_rel", "gpu")
  IRIS_RMW_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_SYS, "acq_rel", "sys")
  return old;
}
#undef IRIS_RMW_CASE

__global__ void __launch_bounds__(256) atomic_op_kernel(const __grid_constant__ HeapTable tab, uint64_t ptr, size_t count, size_t stride, int from_rank,
                                                        int to_rank, int op, int32_t val, int sem, int scope, int32_t* old_out) {
  const uint64_t p = translate(ptr, from_rank, to_rank, tab);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
    const int32_t old = atomic_op(reinterpret_cast<int32_t*>(p + i * stride), op, val, sem, scope);
    if (old_out) old_out[i] = old;
  }
}

// ---- 64-bit atomic_add / atomic_cas (Table 3's atomics on uint64 words), same sem x scope choice -----------
#define IRIS_ATOM64_CASE(SEMV, SCOPEV, SEMS, SCOPES)                                                         \
  if (sem == SEMV && scope == SCOPEV) {                                                                      \
    if (IS_CAS)                                                                                              \
      asm volatile("atom." SEMS "." SCOPES ".global.cas.b64 %0, [%1], %2, %3;"                               \
                   : "=l"(old) : "l"(p), "l"(cmp), "l"(val) : "memory");                                     \
    else                                                                                                     \
      asm volatile("atom." SEMS "." SCOPES ".global.add.u64 %0, [%1], %2;" : "=l"(old) : "l"(p), "l"(val) : "memory"); \
    return old;                                                                                              \
  }

template <bool IS_CAS>
__device__ __forceinline__ uint64_t atomic_rmw64(uint64_t* p, uint64_t cmp, uint64_t val, int sem, int scope) {
  uint64_t old = 0;
  IRIS_ATOM64_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_BLOCK, "relaxed", "cta")
  IRIS_ATOM64_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_GPU, "relaxed", "gpu")
  IRIS_ATOM64_CASE(IRIS_SEM_RELAXED, IRIS_SCOPE_SYS, "relaxed", "sys")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_BLOCK, "acquire", "cta")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_GPU, "acquire", "gpu")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQUIRE, IRIS_SCOPE_SYS, "acquire", "sys")
  IRIS_ATOM64_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_BLOCK, "release", "cta")
  IRIS_ATOM64_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_GPU, "release", "gpu")
  IRIS_ATOM64_CASE(IRIS_SEM_RELEASE, IRIS_SCOPE_SYS, "release", "sys")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_BLOCK, "acq_rel", "cta")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_GPU, "acq_rel", "gpu")
  IRIS_ATOM64_CASE(IRIS_SEM_ACQ_REL, IRIS_SCOPE_SYS, "acq_rel", "sys")
  return old;
}
#undef IRIS_ATOM64_CASE

template <bool IS_CAS>
__global__ void __launch_bounds__(256) atomic_vec64_kernel(const __grid_constant__ HeapTable tab, uint64_t ptr, size_t count, size_t stride, int from_rank,
                                                           int to_rank, uint64_t cmp, uint64_t val, int sem, int scope, uint64_t* old_out) {
  const uint64_t p = translate(ptr, from_rank, to_rank, tab);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
    const uint64_t old = atomic_rmw64<IS_CAS>(reinterpret_cast<uint64_t*>(p + i * stride), cmp, val, sem, scope);
    if (old_out) old_out[i] = old;
  }
}

template <bool IS_CAS>
__global__ void __launch_bounds__(256) atomic_contended_kernel(const __grid_constant__ HeapTable tab, uint64_t ptr, size_t threads, int from_rank, int to_rank,
                                                               int32_t cmp, int32_t val, int sem, int scope, int32_t* old_out) {
  int32_t* p = reinterpret_cast<int32_t*>(translate(ptr, from_rank, to_rank, tab));
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < threads; i += (size_t)gridDim.x * blockDim.x) {
    const int32_t old = atomic_rmw<IS_CAS>(p, cmp, IS_CAS ? val + (int32_t)i : val, sem, scope);
    if (old_out) old_out[i] = old;
  }
}

// ---- all-store / all-load ---------------------------------------------------------------------
// push: work item (r, i): rank r reads tile i of its block once and stores it into all W slots
//       (iris.put to every rank, self included), then publishes W flags.
// pull: work item (s, r, i): rank s loads tile i of rank r's block (iris.get) into its own
//       receive area, then publishes its own flag.
constexpr int kAllStoreThreads = 256;
constexpr int kUnroll = 4;

__global__ void __launch_bounds__(kAllStoreThreads) all_store_kernel(const __grid_constant__ HeapTable tab, uint64_t payload_off, uint64_t recv_off, uint64_t flag_off,
                                                                     size_t S, size_t tile_bytes, int32_t epoch, int pull) {
  const int W = tab.world;
  const size_t T = (S + tile_bytes - 1) / tile_bytes;
  const size_t items = pull ? (size_t)W * W * T : (size_t)W * T;
  for (size_t it = blockIdx.x; it < items; it += gridDim.x) {
    size_t rem = it;
    int s_only = -1;
    if (pull) { s_only = (int)(rem / ((size_t)W * T)); rem %= (size_t)W * T; }
    const int r = (int)(rem / T);
    const size_t i = rem % T;
    const size_t begin = i * tile_bytes;
    const size_t bytes = (begin + tile_bytes <= S) ? tile_bytes : S - begin;
    const size_t chunks = bytes / 16;
    // Addresses in the acting rank's space, then translated (Section 3.3: translate, then operate).
    //   push: acting rank r; source is local, destination recv_off + r*S in rank s.
    //   pull: acting rank s; source payload in rank r, destination local.
    const int actor = pull ? s_only : r;
    const uint64_t src_local = tab.base[actor] + payload_off + begin;
    const uint64_t dst_local = tab.base[actor] + recv_off + (uint64_t)r * S + begin;
    const uint64_t src = pull ? translate(src_local, actor, r, tab) : src_local;
    for (size_t c0 = threadIdx.x; c0 < chunks; c0 += (size_t)kAllStoreThreads * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const size_t c = c0 + (size_t)u * kAllStoreThreads;
        if (c < chunks) v[u] = ld_global_v4(reinterpret_cast<const void*>(src + c * 16));
      }
      if (pull) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const size_t c = c0 + (size_t)u * kAllStoreThreads;
          if (c < chunks) st_global_v4(reinterpret_cast<void*>(dst_local + c * 16), v[u]);
        }
      } else {
        for (int s = 0; s < W; ++s) {
          const uint64_t dst = translate(dst_local, r, s, tab);
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const size_t c = c0 + (size_t)u * kAllStoreThreads;
            if (c < chunks) st_global_v4(reinterpret_cast<void*>(dst + c * 16), v[u]);
          }
        }
      }
    }
    // All of this CTA's stores for the tile precede the barrier; the release by the publishing
    // thread is cumulative over them.
    __syncthreads();
    const uint64_t flag_local = tab.base[actor] + flag_off + ((uint64_t)r * T + i) * 4;
    if (pull) {
      if (threadIdx.x == 0) cas_release_gpu(reinterpret_cast<int32_t*>(flag_local), epoch - 1, epoch);
    } else if ((int)threadIdx.x < W) {
      cas_release_gpu(reinterpret_cast<int32_t*>(translate(flag_local, r, (int)threadIdx.x, tab)), epoch - 1, epoch);
    }
  }
}

static int check_region(const iris_heap* h, const void* p, int rank, size_t rows, size_t row_bytes, size_t pitch, const char* what) {
  const uint64_t base = (uint64_t)h->slot_base[rank];
  const uint64_t a = (uint64_t)p;
  if (a < base || a - base >= h->bytes_per_rank) return fail(IRIS_ERR_RANGE, "%s: address is outside rank %d's heap", what, rank);
  // span = (rows - 1) * pitch + row_bytes must fit in what is left of the slot; compared by division so that huge
  // rows / pitch values cannot wrap the product
  const uint64_t avail = h->bytes_per_rank - (a - base);
  if (row_bytes > avail || (rows > 1 && pitch > 0 && (uint64_t)(rows - 1) > (avail - row_bytes) / pitch))
    return fail(IRIS_ERR_RANGE, "%s: region leaves rank %d's heap", what, rank);
  return IRIS_OK;
}

static int grid_for(const iris_heap* h, size_t work_threads, int per_sm) {
  size_t blocks = (work_threads + 255) / 256;
  const size_t cap = (size_t)h->sm_count * per_sm;
  if (blocks > cap) blocks = cap;
  return blocks < 1 ? 1 : (int)blocks;
}

// kind: 0 put, 1 get, 2 copy, 3 load (dst outside the heap), 4 store (src outside the heap)
static int move2d(iris_heap* h, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch, size_t dst_pitch,
                  int cur_rank, int from_rank, int to_rank, void* stream, int kind, const char* name) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "%s: bad heap handle", name);
  if (from_rank < 0 || from_rank >= h->world || to_rank < 0 || to_rank >= h->world || cur_rank < 0 || cur_rank >= h->world)
    return fail(IRIS_ERR_ARG, "%s: rank out of range", name);
  if (rows == 0 || row_bytes == 0) return IRIS_OK;
  if (!src || !dst) return fail(IRIS_ERR_ARG, "%s: NULL pointer", name);
  if (src_pitch < row_bytes || dst_pitch < row_bytes) return fail(IRIS_ERR_ARG, "%s: pitch smaller than row_bytes", name);
  // Heap-side addresses are given in the caller's (cur_rank's) space; translation preserves offsets, so checking
  // them against the caller's slot also bounds the translated region.  Buffers outside the heap are the caller's.
  int rc = IRIS_OK;
  if (kind != 4) rc = check_region(h, src, cur_rank, rows, row_bytes, src_pitch, name);
  if (rc != IRIS_OK) return rc;
  if (kind != 3) rc = check_region(h, dst, cur_rank, rows, row_bytes, dst_pitch, name);
  if (rc != IRIS_OK) return rc;
  Xlate xs{-1, -1}, xd{-1, -1};
  switch (kind) {
    case 0: xd = {from_rank, to_rank}; break;                              // put
    case 1: xs = {from_rank, to_rank}; break;                              // get
    case 2: xs = {cur_rank, from_rank}; xd = {cur_rank, to_rank}; break;   // copy
    case 3: xs = {from_rank, to_rank}; break;                              // load
    default: xd = {from_rank, to_rank}; break;                             // store
  }
  const bool vec = ((uint64_t)src % 16 == 0) && ((uint64_t)dst % 16 == 0) && row_bytes % 16 == 0 && src_pitch % 16 == 0 && dst_pitch % 16 == 0;
  const size_t work = rows * (vec ? row_bytes / 16 : row_bytes);
  const int grid = grid_for(h, work, 8);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (vec)
    copy2d_kernel<true><<<grid, 256, 0, st>>>(h->table(), (uint64_t)src, (uint64_t)dst, rows, row_bytes, src_pitch, dst_pitch, xs, xd);
  else
    copy2d_kernel<false><<<grid, 256, 0, st>>>(h->table(), (uint64_t)src, (uint64_t)dst, rows, row_bytes, src_pitch, dst_pitch, xs, xd);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

static int atomic_common(iris_heap* h, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, int sem, int scope, const char* name,
                         size_t word = 4) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "%s: bad heap handle", name);
  if (from_rank < 0 || from_rank >= h->world || to_rank < 0 || to_rank >= h->world) return fail(IRIS_ERR_ARG, "%s: rank out of range", name);
  if (sem < IRIS_SEM_RELAXED || sem > IRIS_SEM_ACQ_REL || scope < IRIS_SCOPE_BLOCK || scope > IRIS_SCOPE_SYS) return fail(IRIS_ERR_ARG, "%s: bad sem/scope", name);
  if (count == 0) return 1;  // nothing to do
  if (!ptr || (uint64_t)ptr % word != 0 || stride % word != 0 || (count > 1 && stride == 0))
    return fail(IRIS_ERR_ARG, "%s: pointer/stride must be %zu-byte aligned", name, word);
  return check_region(h, ptr, from_rank, count, word, stride ? stride : word, name);
}

}  // namespace iris

using namespace iris;

extern "C" {

int iris_put_tile(iris_heap* h, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch, size_t dst_pitch,
                  int from_rank, int to_rank, void* stream) {
  return move2d(h, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, from_rank, to_rank, stream, 0, "iris_put_tile");
}

int iris_get_tile(iris_heap* h, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch, size_t dst_pitch,
                  int from_rank, int to_rank, void* stream) {
  return move2d(h, src, dst, rows, row_bytes, src_pitch, dst_pitch, from_rank, from_rank, to_rank, stream, 1, "iris_get_tile");
}

int iris_copy_tile(iris_heap* h, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch, size_t dst_pitch, int cur_rank,
                   int from_rank, int to_rank, void* stream) {
  return move2d(h, src, dst, rows, row_bytes, src_pitch, dst_pitch, cur_rank, from_rank, to_rank, stream, 2, "iris_copy_tile");
}

int iris_load_tile(iris_heap* h, const void* src, void* out, size_t rows, size_t row_bytes, size_t src_pitch, size_t out_pitch, int from_rank,
                   int to_rank, void* stream) {
  return move2d(h, src, out, rows, row_bytes, src_pitch, out_pitch, from_rank, from_rank, to_rank, stream, 3, "iris_load_tile");
}

int iris_store_tile(iris_heap* h, const void* values, void* dst, size_t rows, size_t row_bytes, size_t values_pitch, size_t dst_pitch, int from_rank,
                    int to_rank, void* stream) {
  return move2d(h, values, dst, rows, row_bytes, values_pitch, dst_pitch, from_rank, from_rank, to_rank, stream, 4, "iris_store_tile");
}

int iris_atomic_rmw(iris_heap* h, int op, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, int32_t value, int sem, int scope,
                    int32_t* old_out, void* stream) {
  if (op < IRIS_OP_ADD || op > IRIS_OP_MAX) return fail(IRIS_ERR_ARG, "iris_atomic_rmw: unknown op %d", op);
  int rc = atomic_common(h, ptr, count, stride, from_rank, to_rank, sem, scope, "iris_atomic_rmw");
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_op_kernel<<<grid_for(h, count, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, count, stride, from_rank, to_rank, op, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_add(iris_heap* h, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, int32_t value, int sem, int scope,
                    int32_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, count, stride, from_rank, to_rank, sem, scope, "iris_atomic_add");
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_vec_kernel<false><<<grid_for(h, count, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, count, stride, from_rank, to_rank, 0, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_cas(iris_heap* h, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, int32_t compare, int32_t value, int sem,
                    int scope, int32_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, count, stride, from_rank, to_rank, sem, scope, "iris_atomic_cas");
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_vec_kernel<true><<<grid_for(h, count, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, count, stride, from_rank, to_rank, compare, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_add_u64(iris_heap* h, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, uint64_t value, int sem, int scope,
                        uint64_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, count, stride, from_rank, to_rank, sem, scope, "iris_atomic_add_u64", 8);
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_vec64_kernel<false><<<grid_for(h, count, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, count, stride, from_rank, to_rank, 0, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_cas_u64(iris_heap* h, void* ptr, size_t count, size_t stride, int from_rank, int to_rank, uint64_t compare, uint64_t value, int sem,
                        int scope, uint64_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, count, stride, from_rank, to_rank, sem, scope, "iris_atomic_cas_u64", 8);
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_vec64_kernel<true><<<grid_for(h, count, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, count, stride, from_rank, to_rank, compare, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_add_contended(iris_heap* h, void* ptr, size_t threads, int from_rank, int to_rank, int32_t value, int sem, int scope,
                              int32_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, threads ? 1 : 0, 4, from_rank, to_rank, sem, scope, "iris_atomic_add_contended");
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_contended_kernel<false><<<grid_for(h, threads, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, threads, from_rank, to_rank, 0, value, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_atomic_cas_contended(iris_heap* h, void* ptr, size_t threads, int from_rank, int to_rank, int32_t compare, int32_t value_base, int sem,
                              int scope, int32_t* old_out, void* stream) {
  int rc = atomic_common(h, ptr, threads ? 1 : 0, 4, from_rank, to_rank, sem, scope, "iris_atomic_cas_contended");
  if (rc != IRIS_OK) return rc > 0 ? IRIS_OK : rc;
  atomic_contended_kernel<true><<<grid_for(h, threads, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), (uint64_t)ptr, threads, from_rank, to_rank, compare, value_base, sem, scope, old_out);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

int iris_all_store_bench(iris_heap* h, uint64_t payload_off, uint64_t recv_off, uint64_t flag_off, size_t S, size_t tile_bytes, int32_t epoch,
                         int ctas, int pull, void* stream) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_all_store_bench: bad heap handle");
  if (h->local_rank >= 0) return fail(IRIS_ERR_UNSUPPORTED, "iris_all_store_bench: emulates every rank in one process; not available on a heap over several processes");
  if (S == 0) return IRIS_OK;
  if (S % 16 != 0 || tile_bytes == 0 || tile_bytes % 16 != 0 || tile_bytes > 32768) return fail(IRIS_ERR_ARG, "iris_all_store_bench: S and tile_bytes must be multiples of 16, tile_bytes <= 32768");
  if (payload_off % 16 != 0 || recv_off % 16 != 0 || flag_off % 4 != 0) return fail(IRIS_ERR_ARG, "iris_all_store_bench: misaligned offsets");
  const uint64_t bpr = h->bytes_per_rank, W = (uint64_t)h->world;
  const uint64_t T = (S + tile_bytes - 1) / tile_bytes;
  if (payload_off > bpr || S > bpr - payload_off || recv_off > bpr || W * S > bpr - recv_off || flag_off > bpr || W * T * 4 > bpr - flag_off)
    return fail(IRIS_ERR_RANGE, "iris_all_store_bench: a region leaves the slot");
  const bool overlap = (payload_off < recv_off + W * S) && (recv_off < payload_off + S);
  if (overlap) return fail(IRIS_ERR_ARG, "iris_all_store_bench: payload and receive areas overlap");
  const uint64_t items = pull ? W * W * T : W * T;
  uint64_t grid = ctas > 0 ? (uint64_t)ctas : (uint64_t)h->sm_count * 8;
  if (grid > items) grid = items;
  all_store_kernel<<<(int)grid, kAllStoreThreads, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), payload_off, recv_off, flag_off, S, tile_bytes, epoch, pull);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

}  // extern "C"
