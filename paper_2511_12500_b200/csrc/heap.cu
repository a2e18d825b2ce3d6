// Symmetric heap over W equal slots of one device allocation, bump allocator, pointer
// translation, status block.  (Section 3.1 symmetric heap; Section 3.2 initialisation steps 3, 6.)
#include <cstring>

#include "iris_device.cuh"

namespace iris {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

__global__ void flags_fill_kernel(const __grid_constant__ HeapTable tab, uint64_t off, size_t count, int32_t value) {
  const size_t total = count * (size_t)tab.world;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int s = (int)(i / count);
    reinterpret_cast<int32_t*>(tab.base[s] + off)[i % count] = value;
  }
}

}  // namespace iris

using namespace iris;

extern "C" {

const char* iris_last_error(void) { return g_err; }
const char* iris_version(void) { return "iris-b200 0.1 (sm_100a)"; }

int iris_heap_create_ex(int world, size_t bytes_per_rank, void* external_base, iris_heap** out) {
  if (!out) return fail(IRIS_ERR_ARG, "iris_heap_create: out is NULL");
  *out = nullptr;
  if (world < 1 || world > IRIS_MAX_WORLD) return fail(IRIS_ERR_ARG, "iris_heap_create: world=%d not in [1,%d]", world, IRIS_MAX_WORLD);
  if (bytes_per_rank == 0 || bytes_per_rank % 256 != 0)
    return fail(IRIS_ERR_ARG, "iris_heap_create: bytes_per_rank=%zu must be a positive multiple of 256", bytes_per_rank);
  if (external_base && (reinterpret_cast<uintptr_t>(external_base) % 256 != 0))
    return fail(IRIS_ERR_ARG, "iris_heap_create: external base must be 256-byte aligned");
  int dev = 0;
  IRIS_CUDA_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  IRIS_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(IRIS_ERR_UNSUPPORTED, "iris_heap_create: device is sm_%d%d, this library is sm_100a only", prop.major, prop.minor);
  iris_heap* h = new iris_heap();
  std::memset(h, 0, sizeof(*h));
  h->world = world;
  h->device = dev;
  h->bytes_per_rank = bytes_per_rank;
  h->sm_count = prop.multiProcessorCount;
  if (external_base) {
    h->base = static_cast<char*>(external_base);
    h->owns = false;
  } else {
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, (size_t)world * bytes_per_rank);
    if (e != cudaSuccess) {
      delete h;
      cudaGetLastError();
      return fail(IRIS_ERR_NOMEM, "iris_heap_create: cudaMalloc(%zu) failed: %s", (size_t)world * bytes_per_rank, cudaGetErrorString(e));
    }
    h->base = static_cast<char*>(p);
    h->owns = true;
    // flags, locks and everything else start at zero (a caller-owned backing store is left as the caller prepared it)
    e = cudaMemset(p, 0, (size_t)world * bytes_per_rank);
    if (e != cudaSuccess) {
      cudaFree(p);
      delete h;
      cudaGetLastError();
      return fail(IRIS_ERR_CUDA, "iris_heap_create: cudaMemset: %s", cudaGetErrorString(e));
    }
  }
  for (int r = 0; r < world; ++r) h->slot_base[r] = h->base + (size_t)r * bytes_per_rank;
  h->local_rank = -1;
  h->sf_M = h->sf_N = -1;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->status), 256);
  if (e == cudaSuccess) e = cudaMemset(h->status, 0, 256);
  if (e != cudaSuccess) {
    if (h->owns) cudaFree(h->base);
    delete h;
    cudaGetLastError();
    return fail(IRIS_ERR_NOMEM, "iris_heap_create: status block: %s", cudaGetErrorString(e));
  }
  h->magic = kHeapMagic;
  *out = h;
  return IRIS_OK;
}

int iris_heap_create_from_bases(int world, size_t bytes_per_rank, const uint64_t* bases, int local_rank, iris_heap** out) {
  if (!out) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: out is NULL");
  *out = nullptr;
  if (!bases) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: bases is NULL");
  if (world < 1 || world > IRIS_MAX_WORLD) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: world=%d not in [1,%d]", world, IRIS_MAX_WORLD);
  if (local_rank < 0 || local_rank >= world) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: local_rank=%d not in [0,%d)", local_rank, world);
  if (bytes_per_rank == 0 || bytes_per_rank % 256 != 0)
    return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: bytes_per_rank=%zu must be a positive multiple of 256", bytes_per_rank);
  for (int r = 0; r < world; ++r) {
    if (bases[r] == 0 || bases[r] % 256 != 0) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: base of slot %d must be a 256-byte aligned device address", r);
    for (int q = 0; q < r; ++q) {
      const uint64_t lo = bases[q] < bases[r] ? bases[q] : bases[r], hi = bases[q] < bases[r] ? bases[r] : bases[q];
      if (hi - lo < bytes_per_rank) return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: slots %d and %d overlap", q, r);
    }
  }
  int dev = 0;
  IRIS_CUDA_TRY(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  IRIS_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(IRIS_ERR_UNSUPPORTED, "iris_heap_create_from_bases: device is sm_%d%d, this library is sm_100a only", prop.major, prop.minor);
  for (int r = 0; r < world; ++r) {   // every slot must be device memory this process can address (its own or a mapped peer's)
    cudaPointerAttributes pa;
    const cudaError_t e = cudaPointerGetAttributes(&pa, reinterpret_cast<const void*>(bases[r]));
    if (e != cudaSuccess || (pa.type != cudaMemoryTypeDevice && pa.type != cudaMemoryTypeManaged)) {
      cudaGetLastError();
      return fail(IRIS_ERR_ARG, "iris_heap_create_from_bases: base of slot %d is not device memory known to this process", r);
    }
  }
  iris_heap* h = new iris_heap();
  std::memset(h, 0, sizeof(*h));
  h->world = world;
  h->device = dev;
  h->bytes_per_rank = bytes_per_rank;
  h->sm_count = prop.multiProcessorCount;
  h->base = nullptr;
  h->owns = false;
  for (int r = 0; r < world; ++r) h->slot_base[r] = reinterpret_cast<char*>(bases[r]);
  h->local_rank = local_rank;
  h->flags_sys = 1;
  h->sf_M = h->sf_N = -1;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->status), 256);
  if (e == cudaSuccess) e = cudaMemset(h->status, 0, 256);
  if (e != cudaSuccess) {
    delete h;
    cudaGetLastError();
    return fail(IRIS_ERR_NOMEM, "iris_heap_create_from_bases: status block: %s", cudaGetErrorString(e));
  }
  h->magic = kHeapMagic;
  *out = h;
  return IRIS_OK;
}

int iris_heap_local_rank(const iris_heap* h) { return heap_ok(h) ? h->local_rank : fail(IRIS_ERR_STATE, "bad heap handle"); }

// ---- one rank's slot as memory other processes can map (Section 3.2, steps 3-5: allocate, exchange handles, open) ----
int iris_ipc_alloc(size_t bytes, void** ptr_out) {
  if (!ptr_out) return fail(IRIS_ERR_ARG, "iris_ipc_alloc: ptr_out is NULL");
  *ptr_out = nullptr;
  if (bytes == 0) return fail(IRIS_ERR_ARG, "iris_ipc_alloc: bytes must be positive");
  void* p = nullptr;
  cudaError_t e = cudaMalloc(&p, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(IRIS_ERR_NOMEM, "iris_ipc_alloc: cudaMalloc(%zu) failed: %s", bytes, cudaGetErrorString(e));
  }
  e = cudaMemset(p, 0, bytes);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    cudaFree(p);
    cudaGetLastError();
    return fail(IRIS_ERR_CUDA, "iris_ipc_alloc: cudaMemset: %s", cudaGetErrorString(e));
  }
  *ptr_out = p;
  return IRIS_OK;
}

int iris_ipc_free(void* ptr) {
  if (!ptr) return IRIS_OK;
  IRIS_CUDA_TRY(cudaDeviceSynchronize());
  IRIS_CUDA_TRY(cudaFree(ptr));
  return IRIS_OK;
}

int iris_ipc_export(void* ptr, unsigned char* handle_out) {
  static_assert(sizeof(cudaIpcMemHandle_t) == IRIS_IPC_HANDLE_BYTES, "handle size");
  if (!ptr || !handle_out) return fail(IRIS_ERR_ARG, "iris_ipc_export: NULL argument");
  cudaIpcMemHandle_t hd;
  IRIS_CUDA_TRY(cudaIpcGetMemHandle(&hd, ptr));
  std::memcpy(handle_out, &hd, sizeof(hd));
  return IRIS_OK;
}

int iris_ipc_open(const unsigned char* handle, void** ptr_out) {
  if (!handle || !ptr_out) return fail(IRIS_ERR_ARG, "iris_ipc_open: NULL argument");
  *ptr_out = nullptr;
  cudaIpcMemHandle_t hd;
  std::memcpy(&hd, handle, sizeof(hd));
  void* p = nullptr;
  const cudaError_t e = cudaIpcOpenMemHandle(&p, hd, cudaIpcMemLazyEnablePeerAccess);
  if (e != cudaSuccess) {
    cudaGetLastError();   // a refused handle must not show up as the next launch's error
    return fail(IRIS_ERR_CUDA, "iris_ipc_open: %s", cudaGetErrorString(e));
  }
  *ptr_out = p;
  return IRIS_OK;
}

int iris_ipc_close(void* ptr) {
  if (!ptr) return IRIS_OK;
  IRIS_CUDA_TRY(cudaDeviceSynchronize());
  IRIS_CUDA_TRY(cudaIpcCloseMemHandle(ptr));
  return IRIS_OK;
}

iris_heap* iris_heap_create(int world, size_t bytes_per_rank) {
  iris_heap* h = nullptr;
  return iris_heap_create_ex(world, bytes_per_rank, nullptr, &h) == IRIS_OK ? h : nullptr;
}

int iris_heap_destroy(iris_heap* h) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_heap_destroy: bad handle");
  cudaDeviceSynchronize();
  if (h->owns) cudaFree(h->base);
  cudaFree(h->status);
  if (h->stage_a) cudaFree(h->stage_a);
  if (h->stage_b) cudaFree(h->stage_b);
  if (h->ws) cudaFree(h->ws);
  iris::free_host_pipe(h);
  if (h->ev_fork) cudaEventDestroy(static_cast<cudaEvent_t>(h->ev_fork));
  if (h->ev_join) cudaEventDestroy(static_cast<cudaEvent_t>(h->ev_join));
  h->magic = 0;
  delete h;
  cudaGetLastError();
  return IRIS_OK;
}

int iris_heap_world(const iris_heap* h) { return heap_ok(h) ? h->world : fail(IRIS_ERR_STATE, "bad heap handle"); }
size_t iris_heap_bytes_per_rank(const iris_heap* h) { return heap_ok(h) ? h->bytes_per_rank : 0; }
int32_t iris_heap_epoch(const iris_heap* h) { return heap_ok(h) ? h->epoch : 0; }

void* iris_heap_base(const iris_heap* h, int rank) {
  if (!heap_ok(h) || rank < 0 || rank >= h->world) {
    set_error("iris_heap_base: bad handle or rank");
    return nullptr;
  }
  return h->slot_base[rank];
}

int iris_heap_bases(const iris_heap* h, uint64_t* out) {
  if (!heap_ok(h) || !out) return fail(IRIS_ERR_ARG, "iris_heap_bases: bad handle or NULL out");
  for (int r = 0; r < h->world; ++r) out[r] = (uint64_t)h->slot_base[r];
  return IRIS_OK;
}

int iris_malloc(iris_heap* h, size_t bytes, size_t align, uint64_t* offset_out) {
  if (!heap_ok(h) || !offset_out) return fail(IRIS_ERR_ARG, "iris_malloc: bad handle or NULL offset_out");
  if (align == 0) align = 256;
  if (align < 16 || (align & (align - 1)) != 0) return fail(IRIS_ERR_ARG, "iris_malloc: align=%zu must be a power of two >= 16", align);
  const uint64_t start = align_up(h->bump, align);
  if (start > h->bytes_per_rank || bytes > h->bytes_per_rank - start)
    return fail(IRIS_ERR_NOMEM, "iris_malloc: %zu bytes at offset %llu exceed bytes_per_rank=%zu", bytes, (unsigned long long)start, h->bytes_per_rank);
  h->bump = start + bytes;
  *offset_out = start;
  return IRIS_OK;
}

int iris_heap_reset(iris_heap* h) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_heap_reset: bad handle");
  h->bump = 0;
  return IRIS_OK;
}

int iris_translate(const iris_heap* h, const void* ptr, int from_rank, int to_rank, void** out) {
  if (!heap_ok(h) || !out) return fail(IRIS_ERR_ARG, "iris_translate: bad handle or NULL out");
  if (from_rank < 0 || from_rank >= h->world || to_rank < 0 || to_rank >= h->world)
    return fail(IRIS_ERR_ARG, "iris_translate: rank out of range (from=%d to=%d world=%d)", from_rank, to_rank, h->world);
  const uint64_t from_base = (uint64_t)h->slot_base[from_rank];
  const uint64_t to_base = (uint64_t)h->slot_base[to_rank];
  const uint64_t p = (uint64_t)ptr;
  if (p < from_base || p - from_base >= h->bytes_per_rank)
    return fail(IRIS_ERR_RANGE, "iris_translate: pointer is outside rank %d's heap", from_rank);
  *out = reinterpret_cast<void*>(to_base + (p - from_base));
  return IRIS_OK;
}

int iris_status_check(iris_heap* h, void* stream, int32_t* detail) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_status_check: bad handle");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  IRIS_CUDA_TRY(cudaStreamSynchronize(st));
  int32_t host[kStatusWords];
  IRIS_CUDA_TRY(cudaMemcpy(host, h->status, sizeof(host), cudaMemcpyDeviceToHost));
  if (detail) std::memcpy(detail, host, sizeof(host));
  if (host[0] != 0) {
    IRIS_CUDA_TRY(cudaMemset(h->status, 0, sizeof(host)));
    return fail(host[0], "device-side wait expired: kernel=%d block=%d tile=%d slot=%d seen=%d expected=%d", host[1], host[2], host[3], host[4], host[5], host[6]);
  }
  return IRIS_OK;
}

int iris_flags_fill(iris_heap* h, uint64_t off, size_t count, int32_t value, void* stream) {
  if (!heap_ok(h)) return fail(IRIS_ERR_STATE, "iris_flags_fill: bad handle");
  if (off % 4 != 0) return fail(IRIS_ERR_ARG, "iris_flags_fill: offset must be a multiple of 4");
  if (off > h->bytes_per_rank || count > (h->bytes_per_rank - off) / 4) return fail(IRIS_ERR_RANGE, "iris_flags_fill: region leaves the slot");
  if (count == 0) return IRIS_OK;
  const size_t total = count * (size_t)h->world;
  const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  flags_fill_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(h->table(), off, count, value);
  IRIS_CUDA_TRY(cudaGetLastError());
  return IRIS_OK;
}

}  // extern "C"
