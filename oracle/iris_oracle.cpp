// CPU oracle for the GEMM + all-scatter path over an emulated symmetric heap.
//
// TEST INFRASTRUCTURE ONLY.  Nothing in the product library may include, link or call this file;
// only tests/, the smoke check and the benchmark's cpu_baseline leg use it.  It shares no code
// with the CUDA path: its own fp16/bf16 codec, its own loops, its own heap model.
//
// What it computes is the plain definition the method reaches faster (the paper states that GEMM +
// all-scatter is functionally the same as a matmul followed by an all-gather, Section 5.2):
//   * pointer translation                      (Listing 1, Section 3.3 "Pointer Translation")
//   * put / get / atomics on a heap image      (Table 3, Section 3.3)
//   * C = A . [B_0 | ... | B_{W-1}] with fp64 accumulation in ascending k and ONE rounding to the
//     16-bit output type                       (Listing 2; fp32 accumulation there, fp64 here)
//   * every rank's column shard copied into every rank's slot at the rank's column offset
//                                              (Listings 3-5: offset = rm*ldc + rn + rank*N_local)
//   * per-tile ready flags / locks end state   (Listing 5 handshake; Section 4.1 producer-consumer)
//   * flag-gated consumer  OUT = C + bias      (Section 4.1 producer-consumer, consumer side)
//   * the all-store microbenchmark end state   (Section 5.1, all-store)
//
// The heap is modelled as a host byte array image[W][bytes_per_rank]; "rank r's address p" is the
// pair (r, offset).  Parity status: every function here is pinned by tests/test_oracle_*.py
// (brute force in exact integer arithmetic, identities, numpy float64 matmul, codec tables,
// translation algebra).  Timing numbers are not pinned by the paper (it prints none).

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

constexpr int kF16 = 0;
constexpr int kBF16 = 1;
constexpr int64_t kTile = 128;  // publication tile edge (BLOCK_SIZE_M = BLOCK_SIZE_N = 128)

struct Fmt { int ebits, mbits, bias; };
inline Fmt fmt_of(int dtype) { return dtype == kF16 ? Fmt{5, 10, 15} : Fmt{8, 7, 127}; }

// 16-bit float -> double, by the IEEE definition (sign, biased exponent, fraction).
double decode1(int dtype, uint16_t bits) {
  const Fmt f = fmt_of(dtype);
  const int sign = bits >> 15;
  const int e = (bits >> f.mbits) & ((1 << f.ebits) - 1);
  const int m = bits & ((1 << f.mbits) - 1);
  double v;
  if (e == (1 << f.ebits) - 1) {
    v = m ? std::nan("") : INFINITY;
  } else if (e == 0) {
    v = std::ldexp((double)m, 1 - f.bias - f.mbits);  // subnormal or zero
  } else {
    v = std::ldexp((double)((1 << f.mbits) + m), e - f.bias - f.mbits);
  }
  return sign ? -v : v;
}

// double -> 16-bit float, round to nearest, ties to even, directly from the fp64 value
// (no intermediate fp32: that would round twice).
uint16_t encode1(int dtype, double x) {
  const Fmt f = fmt_of(dtype);
  const uint16_t sign = std::signbit(x) ? 0x8000u : 0u;
  const uint16_t exp_all = (uint16_t)(((1 << f.ebits) - 1) << f.mbits);
  if (std::isnan(x)) return (uint16_t)(sign | exp_all | (1u << (f.mbits - 1)));
  double a = std::fabs(x);
  if (std::isinf(a)) return (uint16_t)(sign | exp_all);
  if (a == 0.0) return sign;
  int e2;
  std::frexp(a, &e2);            // a = frac * 2^e2, frac in [0.5,1)  =>  floor(log2 a) = e2-1
  int e = e2 - 1;
  const int emin = 1 - f.bias;   // exponent of the smallest normal
  const int emax = (1 << f.ebits) - 2 - f.bias;
  if (e < emin) e = emin;        // subnormal range: fixed quantum 2^(emin - mbits)
  // a / 2^(e - mbits) is exact in fp64 (a power-of-two scaling); nearbyint rounds ties to even
  // in the default rounding mode.
  double q = std::nearbyint(std::ldexp(a, f.mbits - e));
  if (q >= std::ldexp(1.0, f.mbits + 1)) { q = std::ldexp(1.0, f.mbits); e += 1; }
  if (e > emax) return (uint16_t)(sign | exp_all);  // overflow -> inf
  const uint32_t qi = (uint32_t)q;
  if (qi < (1u << f.mbits)) return (uint16_t)(sign | qi);  // subnormal (exponent field 0)
  return (uint16_t)(sign | ((uint32_t)(e + f.bias) << f.mbits) | (qi - (1u << f.mbits)));
}

template <class F>
void parallel_rows(int64_t begin, int64_t end, int threads, F body) {
  if (threads < 1) threads = 1;
  const int64_t n = end - begin;
  if (n <= 0) return;
  if (threads > n) threads = (int)n;
  if (threads == 1) { for (int64_t i = begin; i < end; ++i) body(i); return; }
  std::atomic<int64_t> next(begin);
  std::vector<std::thread> pool;
  for (int t = 0; t < threads; ++t)
    pool.emplace_back([&] { for (;;) { int64_t i = next.fetch_add(1); if (i >= end) break; body(i); } });
  for (auto& th : pool) th.join();
}

inline bool bad_rank(int r, int world) { return r < 0 || r >= world; }
inline uint8_t* slot(uint8_t* image, uint64_t bpr, int r) { return image + (uint64_t)r * bpr; }

}  // namespace

extern "C" {

int orc_hw_threads() { unsigned n = std::thread::hardware_concurrency(); return n ? (int)n : 1; }

double orc_decode1(int dtype, uint16_t bits) { return decode1(dtype, bits); }
uint16_t orc_encode1(int dtype, double x) { return encode1(dtype, x); }
void orc_decode(int dtype, const uint16_t* in, int64_t n, double* out) { for (int64_t i = 0; i < n; ++i) out[i] = decode1(dtype, in[i]); }
void orc_encode(int dtype, const double* in, int64_t n, uint16_t* out) { for (int64_t i = 0; i < n; ++i) out[i] = encode1(dtype, in[i]); }

// Listing 1: offset of ptr inside from_rank's heap, added to to_rank's base.  Returns 0, or -1 for
// a bad rank, -2 when ptr is outside [bases[from], bases[from] + bytes_per_rank).
int orc_translate(const uint64_t* bases, int world, uint64_t bytes_per_rank, uint64_t ptr, int from_rank,
                  int to_rank, uint64_t* out) {
  if (bad_rank(from_rank, world) || bad_rank(to_rank, world)) return -1;
  const uint64_t from_base = bases[from_rank];
  if (ptr < from_base || ptr - from_base >= bytes_per_rank) return -2;
  const uint64_t offset = ptr - from_base;
  *out = bases[to_rank] + offset;
  return 0;
}

// Block [m0,m1) x [n0,n1) of C = A . Bcat^T where Bcat row n is row (n mod N_local) of shard
// n / N_local; A is [M,K], each shard [N_local,K], both K-contiguous.  Sum in fp64, ascending k,
// then one rounding.  c16: (m1-m0) x (n1-n0) row-major; c64 (optional): the unrounded sums.
int orc_gemm_block(int dtype, const uint16_t* A, const uint16_t* const* B_shards, int64_t M, int64_t N, int64_t K,
                   int world, int64_t m0, int64_t m1, int64_t n0, int64_t n1, uint16_t* c16, double* c64,
                   int threads) {
  if (world < 1 || N % world != 0 || m0 < 0 || m1 > M || n0 < 0 || n1 > N || m0 > m1 || n0 > n1) return -1;
  const int64_t n_local = N / world, bw = n1 - n0;
  // decode the needed B rows once: bdec[(n-n0)][k]
  std::vector<double> bdec((size_t)bw * (size_t)K);
  parallel_rows(n0, n1, threads, [&](int64_t n) {
    const uint16_t* brow = B_shards[n / n_local] + (n % n_local) * K;
    double* d = &bdec[(size_t)(n - n0) * (size_t)K];
    for (int64_t k = 0; k < K; ++k) d[k] = decode1(dtype, brow[k]);
  });
  parallel_rows(m0, m1, threads, [&](int64_t m) {
    std::vector<double> arow((size_t)K);
    for (int64_t k = 0; k < K; ++k) arow[k] = decode1(dtype, A[m * K + k]);
    for (int64_t n = n0; n < n1; ++n) {
      const double* b = &bdec[(size_t)(n - n0) * (size_t)K];
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += arow[k] * b[k];
      const size_t o = (size_t)(m - m0) * (size_t)bw + (size_t)(n - n0);
      if (c64) c64[o] = acc;
      c16[o] = encode1(dtype, acc);
    }
  });
  return 0;
}

// All-scatter end state: for every rank r and every slot s, rank r's columns
// [r*N_local, (r+1)*N_local) of the rounded C land in slot s at c_off + (m*N + n)*2.
int orc_all_scatter(uint8_t* image, int world, uint64_t bpr, uint64_t c_off, int64_t M, int64_t N,
                    const uint16_t* c_full) {
  if (world < 1 || N % world != 0 || c_off + (uint64_t)M * N * 2 > bpr) return -2;
  const int64_t n_local = N / world;
  for (int r = 0; r < world; ++r)        // the rank that produced the shard
    for (int s = 0; s < world; ++s) {    // the rank whose heap receives it (s == r: its own copy)
      uint16_t* dst = (uint16_t*)(slot(image, bpr, s) + c_off);
      for (int64_t m = 0; m < M; ++m)
        for (int64_t n = r * n_local; n < (r + 1) * n_local; ++n) dst[m * N + n] = c_full[m * N + n];
    }
  return 0;
}

// Publication tiles: 128 x 128, counted per rank shard so that no tile straddles two ranks:
// TM = ceil(M/128), TNl = ceil(N_local/128), t = tm*(W*TNl) + r*TNl + j.
int64_t orc_num_tiles(int64_t M, int64_t N, int world) {
  const int64_t n_local = N / world;
  return ((M + kTile - 1) / kTile) * world * ((n_local + kTile - 1) / kTile);
}

// End state of the ready flags: flag[s][t] == epoch in every slot, for every tile.
int orc_publish_flags(uint8_t* image, int world, uint64_t bpr, uint64_t flag_off, int64_t ntiles, int32_t epoch) {
  if (flag_off + (uint64_t)ntiles * 4 > bpr) return -2;
  for (int s = 0; s < world; ++s) {
    int32_t* f = (int32_t*)(slot(image, bpr, s) + flag_off);
    for (int64_t t = 0; t < ntiles; ++t) f[t] = epoch;
  }
  return 0;
}

// End state of the producer->communicator locks in workgroup-specialised mode: each lock went
// 0 -> 1 (producer, release) -> 0 (communicator, acquire), so it reads 0.  lock[t] lives in the
// slot of the rank that owns tile t.
int orc_consume_locks(uint8_t* image, int world, uint64_t bpr, uint64_t lock_off, int64_t M, int64_t N) {
  const int64_t n_local = N / world, tm_n = (M + kTile - 1) / kTile, tnl = (n_local + kTile - 1) / kTile;
  if (lock_off + (uint64_t)(tm_n * world * tnl) * 4 > bpr) return -2;
  for (int64_t tm = 0; tm < tm_n; ++tm)
    for (int r = 0; r < world; ++r)
      for (int64_t j = 0; j < tnl; ++j) {
        const int64_t t = tm * (world * tnl) + r * tnl + j;
        int32_t* lock = (int32_t*)(slot(image, bpr, r) + lock_off) + t;
        *lock = 0;
      }
  return 0;
}

// put: read rank `from`'s memory at src_off, write rank `to`'s memory at dst_off (Table 3: local -> remote).
int orc_put(uint8_t* image, int world, uint64_t bpr, uint64_t src_off, uint64_t dst_off, int64_t rows,
            int64_t row_bytes, int64_t src_pitch, int64_t dst_pitch, int from_rank, int to_rank) {
  if (bad_rank(from_rank, world) || bad_rank(to_rank, world)) return -1;
  if (rows == 0 || row_bytes == 0) return 0;
  if (src_off + (uint64_t)(rows - 1) * src_pitch + row_bytes > bpr || dst_off + (uint64_t)(rows - 1) * dst_pitch + row_bytes > bpr) return -2;
  std::vector<uint8_t> tmp((size_t)row_bytes);
  for (int64_t i = 0; i < rows; ++i) {
    std::memcpy(tmp.data(), slot(image, bpr, from_rank) + src_off + i * src_pitch, (size_t)row_bytes);
    std::memcpy(slot(image, bpr, to_rank) + dst_off + i * dst_pitch, tmp.data(), (size_t)row_bytes);
  }
  return 0;
}

// get: read rank `to`'s memory at src_off, write rank `from`'s memory at dst_off (Table 3: remote -> local).
int orc_get(uint8_t* image, int world, uint64_t bpr, uint64_t src_off, uint64_t dst_off, int64_t rows,
            int64_t row_bytes, int64_t src_pitch, int64_t dst_pitch, int from_rank, int to_rank) {
  if (bad_rank(from_rank, world) || bad_rank(to_rank, world)) return -1;
  if (rows == 0 || row_bytes == 0) return 0;
  if (src_off + (uint64_t)(rows - 1) * src_pitch + row_bytes > bpr || dst_off + (uint64_t)(rows - 1) * dst_pitch + row_bytes > bpr) return -2;
  std::vector<uint8_t> tmp((size_t)row_bytes);
  for (int64_t i = 0; i < rows; ++i) {
    std::memcpy(tmp.data(), slot(image, bpr, to_rank) + src_off + i * src_pitch, (size_t)row_bytes);
    std::memcpy(slot(image, bpr, from_rank) + dst_off + i * dst_pitch, tmp.data(), (size_t)row_bytes);
  }
  return 0;
}

// Sequential read-modify-write of `count` int32 words at off + i*stride in rank `to_rank`'s memory.
// old_out[i] receives the value before the operation.
int orc_atomic_add(uint8_t* image, int world, uint64_t bpr, uint64_t off, int64_t count, int64_t stride,
                   int to_rank, int32_t val, int32_t* old_out) {
  if (bad_rank(to_rank, world)) return -1;
  if (count > 0 && off + (uint64_t)(count - 1) * stride + 4 > bpr) return -2;
  for (int64_t i = 0; i < count; ++i) {
    int32_t* p = (int32_t*)(slot(image, bpr, to_rank) + off + i * stride);
    const int32_t old = *p;
    *p = (int32_t)((uint32_t)old + (uint32_t)val);
    if (old_out) old_out[i] = old;
  }
  return 0;
}

int orc_atomic_cas(uint8_t* image, int world, uint64_t bpr, uint64_t off, int64_t count, int64_t stride,
                   int to_rank, int32_t cmp, int32_t val, int32_t* old_out) {
  if (bad_rank(to_rank, world)) return -1;
  if (count > 0 && off + (uint64_t)(count - 1) * stride + 4 > bpr) return -2;
  for (int64_t i = 0; i < count; ++i) {
    int32_t* p = (int32_t*)(slot(image, bpr, to_rank) + off + i * stride);
    const int32_t old = *p;
    if (old == cmp) *p = val;
    if (old_out) old_out[i] = old;
  }
  return 0;
}

// The same two operations on uint64 words (Table 3's atomics, 64-bit operands): the addition wraps modulo 2^64,
// the compare-and-swap writes iff the word equals cmp; old_out[i] receives the value before the operation.
int orc_atomic_add_u64(uint8_t* image, int world, uint64_t bpr, uint64_t off, int64_t count, int64_t stride,
                       int to_rank, uint64_t val, uint64_t* old_out) {
  if (bad_rank(to_rank, world)) return -1;
  if (count > 0 && off + (uint64_t)(count - 1) * stride + 8 > bpr) return -2;
  for (int64_t i = 0; i < count; ++i) {
    uint64_t* p = (uint64_t*)(slot(image, bpr, to_rank) + off + i * stride);
    const uint64_t old = *p;
    *p = old + val;
    if (old_out) old_out[i] = old;
  }
  return 0;
}

int orc_atomic_cas_u64(uint8_t* image, int world, uint64_t bpr, uint64_t off, int64_t count, int64_t stride,
                       int to_rank, uint64_t cmp, uint64_t val, uint64_t* old_out) {
  if (bad_rank(to_rank, world)) return -1;
  if (count > 0 && off + (uint64_t)(count - 1) * stride + 8 > bpr) return -2;
  for (int64_t i = 0; i < count; ++i) {
    uint64_t* p = (uint64_t*)(slot(image, bpr, to_rank) + off + i * stride);
    const uint64_t old = *p;
    if (old == cmp) *p = val;
    if (old_out) old_out[i] = old;
  }
  return 0;
}

// Consumer: in every slot, OUT = C + bias (bias broadcast over rows), added in fp32 and rounded
// once to the 16-bit type.  The sum of two 16-bit floats rounded to fp32 and then to 16 bits is
// computed here as written: float add, then the codec.
int orc_consume_bias(uint8_t* image, int world, uint64_t bpr, int dtype, uint64_t c_off, uint64_t out_off,
                     int64_t M, int64_t N, const uint16_t* bias) {
  if (c_off + (uint64_t)M * N * 2 > bpr || out_off + (uint64_t)M * N * 2 > bpr) return -2;
  for (int s = 0; s < world; ++s) {
    const uint16_t* c = (const uint16_t*)(slot(image, bpr, s) + c_off);
    uint16_t* o = (uint16_t*)(slot(image, bpr, s) + out_off);
    for (int64_t m = 0; m < M; ++m)
      for (int64_t n = 0; n < N; ++n) {
        const float sum = (float)decode1(dtype, c[m * N + n]) + (float)decode1(dtype, bias[n]);
        o[m * N + n] = encode1(dtype, (double)sum);
      }
  }
  return 0;
}

// All-store: every rank r's block of S bytes (at payload_off in its own slot) lands in every slot
// s at recv_off + r*S; one int32 flag per (slot, source rank, tile) goes epoch-1 -> epoch.
int orc_all_store(uint8_t* image, int world, uint64_t bpr, uint64_t payload_off, uint64_t recv_off,
                  uint64_t flag_off, uint64_t S, uint64_t tile_bytes, int32_t epoch) {
  if (tile_bytes == 0) return -1;
  const uint64_t T = (S + tile_bytes - 1) / tile_bytes;
  if (payload_off + S > bpr || recv_off + (uint64_t)world * S > bpr || flag_off + (uint64_t)world * T * 4 > bpr) return -2;
  for (int r = 0; r < world; ++r)
    for (int s = 0; s < world; ++s) {
      std::memmove(slot(image, bpr, s) + recv_off + (uint64_t)r * S, slot(image, bpr, r) + payload_off, (size_t)S);
      int32_t* f = (int32_t*)(slot(image, bpr, s) + flag_off) + (uint64_t)r * T;
      for (uint64_t i = 0; i < T; ++i)
        if (f[i] == epoch - 1) f[i] = epoch;
    }
  return 0;
}

// Remaining read-modify-write atomics of Table 3 on int32 words of rank `to_rank`'s memory, applied
// sequentially: op 0 add, 1 xchg, 2 and, 3 or, 4 xor, 5 min (signed), 6 max (signed).
int orc_atomic_rmw(uint8_t* image, int world, uint64_t bpr, int op, uint64_t off, int64_t count, int64_t stride,
                   int to_rank, int32_t val, int32_t* old_out) {
  if (bad_rank(to_rank, world) || op < 0 || op > 6) return -1;
  if (count > 0 && off + (uint64_t)(count - 1) * stride + 4 > bpr) return -2;
  for (int64_t i = 0; i < count; ++i) {
    int32_t* p = (int32_t*)(slot(image, bpr, to_rank) + off + i * stride);
    const int32_t old = *p;
    int32_t neu = old;
    switch (op) {
      case 0: neu = (int32_t)((uint32_t)old + (uint32_t)val); break;
      case 1: neu = val; break;
      case 2: neu = old & val; break;
      case 3: neu = old | val; break;
      case 4: neu = old ^ val; break;
      case 5: neu = old < val ? old : val; break;
      case 6: neu = old > val ? old : val; break;
    }
    *p = neu;
    if (old_out) old_out[i] = old;
  }
  return 0;
}

// copy (Table 3: between any two ranks): the caller `cur_rank` names both regions in its own address
// space; bytes move from rank `from_rank`'s memory at src_off to rank `to_rank`'s memory at dst_off.
int orc_copy(uint8_t* image, int world, uint64_t bpr, uint64_t src_off, uint64_t dst_off, int64_t rows, int64_t row_bytes,
             int64_t src_pitch, int64_t dst_pitch, int from_rank, int to_rank) {
  if (bad_rank(from_rank, world) || bad_rank(to_rank, world)) return -1;
  if (rows == 0 || row_bytes == 0) return 0;
  if (src_off + (uint64_t)(rows - 1) * src_pitch + row_bytes > bpr || dst_off + (uint64_t)(rows - 1) * dst_pitch + row_bytes > bpr) return -2;
  std::vector<uint8_t> tmp((size_t)row_bytes);
  for (int64_t i = 0; i < rows; ++i) {
    std::memcpy(tmp.data(), slot(image, bpr, from_rank) + src_off + i * src_pitch, (size_t)row_bytes);
    std::memcpy(slot(image, bpr, to_rank) + dst_off + i * dst_pitch, tmp.data(), (size_t)row_bytes);
  }
  return 0;
}

}  // extern "C"
