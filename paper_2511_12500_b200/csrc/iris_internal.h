// Host-side internals shared by the translation units of libiris_b200.so.
#pragma once

#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "iris_b200.h"

namespace iris {

constexpr uint32_t kHeapMagic = 0x49524953u;  // "IRIS"
constexpr int kStatusWords = 8;               // {code, kernel, block, tile, slot, seen, expected, 0}
constexpr uint64_t kDefaultTimeoutNs = 2000000000ull;

// Kernel ids recorded in the status block.
enum { KID_GEMM = 1, KID_SCATTER = 2, KID_CONSUMER = 3, KID_ALLSTORE = 4 };

// The table every kernel receives by value: the B200 form of the paper's `heap_bases` tensor
// (Section 3.3: 64 bytes at W = 8; here it sits in constant-bank kernel parameters).
struct HeapTable {
  uint64_t base[IRIS_MAX_WORLD];
  uint64_t bytes_per_rank;
  int world;
  int flags_sys;   // 1 = slots may live on other devices or in other processes: ready flags are released and acquired at system scope
};

void set_error(const char* fmt, ...);
int fail(int code, const char* fmt, ...);

#define IRIS_CUDA_TRY(expr)                                                                    \
  do {                                                                                         \
    cudaError_t e_ = (expr);                                                                   \
    if (e_ != cudaSuccess) return ::iris::fail(IRIS_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

}  // namespace iris

struct iris_heap {
  uint32_t magic;
  int world;
  int device;
  size_t bytes_per_rank;
  char* base;          // device; nullptr when the slots are not one contiguous range (iris_heap_create_from_bases)
  char* slot_base[IRIS_MAX_WORLD];   // slot r starts here (base + r * bytes_per_rank for a contiguous heap)
  int local_rank;      // heap over several processes / devices: the slot that lives in this process's own memory; -1 otherwise
  int flags_sys;       // see HeapTable
  bool owns;
  uint64_t bump;       // next free offset
  int32_t* status;     // device, kStatusWords int32
  int32_t epoch;       // last epoch used by the short-form call
  int sf_M, sf_N;      // short form / host entry point: the (M, N) whose flag and lock arrays have been zeroed (-1: none yet)
  int sm_count;
  // staging for the host-buffer entry point
  void* stage_a;
  void* stage_b;
  size_t stage_a_bytes, stage_b_bytes;
  // stream-K workspace (partial sums + arrival counters), allocated on first use
  void* ws;
  size_t ws_bytes;
  // streams and events of the host-buffer entry point's copy/compute pipeline, created on first use
  void* host_pipe;
  // fork / join events of the two-stream (unfused) form of the workgroup-specialised schedule, created on first use
  void* ev_fork;
  void* ev_join;
  iris::HeapTable table() const {
    iris::HeapTable t{};
    for (int r = 0; r < world; ++r) t.base[r] = (uint64_t)slot_base[r];
    t.bytes_per_rank = bytes_per_rank;
    t.world = world;
    t.flags_sys = flags_sys;
    return t;
  }
};

namespace iris {
inline bool heap_ok(const iris_heap* h) { return h && h->magic == kHeapMagic; }
void free_host_pipe(iris_heap* h);   // gemm_all_scatter.cu
}  // namespace iris
