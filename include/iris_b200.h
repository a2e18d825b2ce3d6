/*
 * iris_b200.h -- C ABI of the B200 (sm_100a) implementation of the GEMM + all-scatter path of
 * "Iris: First-Class Multi-GPU Programming Experience in Triton" (arXiv 2511.12500).
 *
 * The paper's W ranks are emulated as W equal partitions ("slots") of one allocation in a single
 * GPU's HBM.  Slot r plays the role of rank r's symmetric heap: an object allocated at offset o
 * exists at bases[r] + o in every slot (Section 3.1 "Adoption of Symmetric Heap Abstraction").
 *
 * Conventions
 *   - Every function returns an int status (IRIS_OK == 0, errors negative) unless stated otherwise;
 *     no exception crosses this boundary.  iris_last_error() gives a thread-local detail string.
 *   - "device pointer" = address in the GPU's global memory; "host pointer" = ordinary CPU memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls that
 *     take a stream only enqueue work; the caller synchronises.  Pointers are borrowed: they must
 *     stay valid until the enqueued work has run.
 *   - Argument errors are detected before anything is launched.  Problems that only the device
 *     can see (a bounded wait that ran out) are recorded in the heap's status block and reported
 *     by iris_status_check(); a kernel never traps and never spins without a deadline.
 *   - The library is sm_100a only and has no CPU fallback: on a machine without such a GPU every
 *     call that needs the device returns IRIS_ERR_CUDA.
 */
#ifndef IRIS_B200_H
#define IRIS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------------------------------ */
/* Status codes, enumerations                                                                  */
/* ------------------------------------------------------------------------------------------ */
enum {
  IRIS_OK = 0,
  IRIS_ERR_ARG = -1,         /* bad argument value / alignment / divisibility                  */
  IRIS_ERR_RANGE = -2,       /* an address or region leaves its rank's heap slot               */
  IRIS_ERR_NOMEM = -3,       /* heap exhausted or device allocation failed                     */
  IRIS_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (also: no usable GPU)        */
  IRIS_ERR_UNSUPPORTED = -5, /* valid request that this build cannot serve                     */
  IRIS_ERR_TIMEOUT = -6,     /* a device-side bounded wait expired (see iris_status_check)     */
  IRIS_ERR_STATE = -7        /* heap used after destroy / inconsistent handle                  */
};

enum { IRIS_F16 = 0, IRIS_BF16 = 1 }; /* element type of A, B, C, bias (accumulation is fp32) */

/* The three schedules of Section 4 ("Building Complex Multi-GPU Patterns"). */
enum {
  IRIS_MODE_BULK_SYNCHRONOUS = 0,     /* Listing 3: GEMM kernel, then an all-scatter kernel     */
  IRIS_MODE_FUSED_SEQUENTIAL = 1,     /* Listing 4: each tile stored to all ranks from registers */
  IRIS_MODE_WORKGROUP_SPECIALIZED = 2 /* Listing 5: producer CTAs + communication CTAs, locks   */
};

/* Memory order and scope of atomics (Table 3 note; Section 3.3 "Atomic Operations and Memory Model"). */
enum { IRIS_SEM_RELAXED = 0, IRIS_SEM_ACQUIRE = 1, IRIS_SEM_RELEASE = 2, IRIS_SEM_ACQ_REL = 3 };
enum { IRIS_SCOPE_BLOCK = 0, IRIS_SCOPE_GPU = 1, IRIS_SCOPE_SYS = 2 };
/* Read-modify-write atomics of Table 3 (atomic_cas has its own call). min / max compare as signed int32. */
enum { IRIS_OP_ADD = 0, IRIS_OP_XCHG = 1, IRIS_OP_AND = 2, IRIS_OP_OR = 3, IRIS_OP_XOR = 4, IRIS_OP_MIN = 5, IRIS_OP_MAX = 6 };

/* Storage of a B shard (iris_gemm_args.b_layout). */
enum {
  IRIS_B_N_BY_K = 0, /* [N/W, K], K contiguous: the K x N_local operand stored column-major            */
  IRIS_B_K_BY_N = 1  /* [K, N/W] row-major, N contiguous: Listing 2's K x N_local operand as printed   */
};

#define IRIS_MAX_WORLD 8
#define IRIS_TILE 128 /* publication tile edge: one ready flag per 128 x 128 block of C */

typedef struct iris_heap iris_heap;

const char* iris_last_error(void); /* never NULL; valid until the calling thread's next library call */
const char* iris_version(void);

/* ------------------------------------------------------------------------------------------ */
/* Symmetric heap (Section 3.2 "Constructor and Initialization", steps 3 and 6)                */
/* ------------------------------------------------------------------------------------------ */

/* Create a heap of `world` slots of `bytes_per_rank` bytes each on the current CUDA device.
 * 1 <= world <= IRIS_MAX_WORLD; bytes_per_rank > 0 and a multiple of 256.  The library allocates
 * world * bytes_per_rank bytes of device memory (plus a 256-byte status block), clears them to zero
 * (so flag and lock arrays placed anywhere in it start in their initial state) and owns them.
 * Returns NULL on failure (see iris_last_error). */
iris_heap* iris_heap_create(int world, size_t bytes_per_rank);

/* Same, with the status code returned and an optional caller-owned backing store:
 * external_base != NULL must be a 256-byte aligned device pointer to world * bytes_per_rank bytes
 * that outlives the heap (e.g. a torch tensor's storage); NULL = the library allocates.  A caller-owned
 * backing store is used as it is: before the first iris_gemm_all_scatter_ex on it the caller sets the lock array
 * to 0 and the flag array below the first epoch (iris_flags_fill); gemm_all_scatter() and
 * iris_gemm_all_scatter_host() choose their own layout and clear their flag and lock arrays themselves. */
int iris_heap_create_ex(int world, size_t bytes_per_rank, void* external_base, iris_heap** out);

/* A heap over several processes or devices (Section 3.1: one slot per rank, each in its owner's memory; Section 3.2
 * steps 3-6: allocate, exchange handles, open the peers' slots, build the table of bases).  bases[0..world) are HOST
 * values: the device address, in THIS process, of every rank's slot of bytes_per_rank bytes, each 256-byte aligned,
 * none overlapping another, each device memory this process can address (IRIS_ERR_ARG otherwise);
 * bases[local_rank] is this process's own allocation, the others are mappings of the peers' (iris_ipc_open, or any
 * mapping the caller made).  The heap owns none of them and the caller keeps them
 * alive until iris_heap_destroy.  Nothing is cleared.  What changes on such a heap:
 *   - ready flags are released and acquired at SYSTEM scope (every other scope in this header stays as written);
 *   - iris_gemm_all_scatter_ex / _unfused compute this rank's shard only: rank_first must be local_rank and
 *     rank_count 1 (IRIS_ERR_ARG otherwise).  The locks of the workgroup-specialised schedule are the local
 *     slot's; tiles go to every slot with TMA stores through one tensor map per slot;
 *   - iris_consume_bias[_ranks] reads and writes the local slot only;
 *   - gemm_all_scatter(), iris_gemm_all_scatter_host(), consumer_bias inside the launch and iris_all_store_bench
 *     emulate all ranks in one process and return IRIS_ERR_UNSUPPORTED.
 * Between ranks the caller orders things on the host (a barrier before the first launch, so that every rank's flags
 * are in their initial state, and before the memory is released).  Kernels of different ranks never wait for one
 * another except the consumer for flags, with the usual deadline. */
int iris_heap_create_from_bases(int world, size_t bytes_per_rank, const uint64_t* bases, int local_rank, iris_heap** out);
int iris_heap_local_rank(const iris_heap* heap); /* the local rank of a heap made from bases; -1 for a one-process heap */

/* One rank's slot as memory that other processes can map.  iris_ipc_alloc: `bytes` of device memory on the current
 * device, cleared to zero (a plain allocation of its own, so that the handle names exactly this range).
 * iris_ipc_export: writes IRIS_IPC_HANDLE_BYTES bytes that another process passes to iris_ipc_open (in that process:
 * a device address of the same memory, valid until iris_ipc_close).  A handle cannot be opened by the process that
 * exported it.  iris_ipc_free / iris_ipc_close synchronise the device first; NULL is a no-op.
 * Errors: IRIS_ERR_ARG (NULL), IRIS_ERR_NOMEM, IRIS_ERR_CUDA with the runtime's message in iris_last_error(). */
#define IRIS_IPC_HANDLE_BYTES 64
int iris_ipc_alloc(size_t bytes, void** ptr_out);
int iris_ipc_free(void* ptr);
int iris_ipc_export(void* ptr, unsigned char* handle_out);
int iris_ipc_open(const unsigned char* handle, void** ptr_out);
int iris_ipc_close(void* ptr);

/* Free the heap (and its memory if the library owns it).  Synchronises the device first. */
int iris_heap_destroy(iris_heap* heap);

int iris_heap_world(const iris_heap* heap);                /* get_num_ranks(); <0 on bad handle */
size_t iris_heap_bytes_per_rank(const iris_heap* heap);    /* 0 on bad handle                   */
void* iris_heap_base(const iris_heap* heap, int rank);     /* device pointer; NULL on bad rank  */
/* get_heap_bases(): writes `world` device addresses into the host array out[]. */
int iris_heap_bases(const iris_heap* heap, uint64_t* out);

/* Symmetric bump allocation: reserves `bytes` at one offset that is valid in every slot.
 * align: power of two >= 16 (0 = 256).  There is no per-object free; iris_heap_reset() releases
 * everything.  IRIS_ERR_NOMEM when the slot is exhausted.  offset_out: host pointer. */
int iris_malloc(iris_heap* heap, size_t bytes, size_t align, uint64_t* offset_out);
int iris_heap_reset(iris_heap* heap);

/* Pointer translation (Listing 1, Section 3.3): *out = base[to_rank] + (ptr - base[from_rank]).
 * `ptr` is a device address that is valid in from_rank's slot.  IRIS_ERR_RANGE if it is not inside
 * [base[from_rank], base[from_rank] + bytes_per_rank); IRIS_ERR_ARG for a bad rank.  Pure host
 * arithmetic; the kernels use the same formula on a by-value copy of the base table. */
int iris_translate(const iris_heap* heap, const void* ptr, int from_rank, int to_rank, void** out);

/* ------------------------------------------------------------------------------------------ */
/* Device-detected errors                                                                      */
/* ------------------------------------------------------------------------------------------ */

/* Synchronise `stream`, read the heap's status block and clear it.  Returns IRIS_OK, or
 * IRIS_ERR_TIMEOUT when a kernel gave up a bounded wait (detail[0..7], if not NULL, receives
 * {code, kernel id, block, tile, slot, value seen, value expected, 0} on the host). */
int iris_status_check(iris_heap* heap, void* stream, int32_t* detail);

/* ------------------------------------------------------------------------------------------ */
/* Tile memory operations and atomics on heap addresses (Table 3)                              */
/* ------------------------------------------------------------------------------------------ */

/* put: copy a 2-D region from from_rank's memory to to_rank's memory (local -> remote).
 * src and dst are device addresses valid in from_rank's slot, as in Listings 3 and 5 (where put
 * receives the same local address for both, with the caller's and the remote rank): the region is
 * read at src and written at translate(dst, from_rank, to_rank).  rows x row_bytes bytes; consecutive rows are
 * src_pitch / dst_pitch bytes apart (pitch >= row_bytes).  A 16-byte vector path is used when
 * both addresses, both pitches and row_bytes are multiples of 16, a byte path otherwise.
 * IRIS_ERR_RANGE if either region leaves its slot.  rows == 0 or row_bytes == 0: no-op. */
int iris_put_tile(iris_heap* heap, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch,
                  size_t dst_pitch, int from_rank, int to_rank, void* stream);

/* get: the mirror image (remote -> local): read translate(src, from_rank, to_rank), write dst
 * in from_rank's slot. */
int iris_get_tile(iris_heap* heap, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch,
                  size_t dst_pitch, int from_rank, int to_rank, void* stream);

/* copy (Table 3: between any two ranks): src and dst are addresses valid in cur_rank's slot; the region is read
 * at translate(src, cur_rank, from_rank) and written at translate(dst, cur_rank, to_rank).  Otherwise as put. */
int iris_copy_tile(iris_heap* heap, const void* src, void* dst, size_t rows, size_t row_bytes, size_t src_pitch,
                   size_t dst_pitch, int cur_rank, int from_rank, int to_rank, void* stream);

/* load / store (Table 3, value-based): like get / put, but the local side is a device buffer of the caller's
 * that need not lie in the heap (it stands in for the registers the paper's value-based calls use).
 * load: read translate(src, from_rank, to_rank) -> out.   store: values -> translate(dst, from_rank, to_rank).
 * Only the heap-side region is range-checked. */
int iris_load_tile(iris_heap* heap, const void* src, void* out, size_t rows, size_t row_bytes, size_t src_pitch,
                   size_t out_pitch, int from_rank, int to_rank, void* stream);
int iris_store_tile(iris_heap* heap, const void* values, void* dst, size_t rows, size_t row_bytes, size_t values_pitch,
                    size_t dst_pitch, int from_rank, int to_rank, void* stream);

/* atomic_add / atomic_cas on int32 words of to_rank's memory.  `ptr` is valid in from_rank's slot
 * and is translated first.  Vector form: `count` words, `stride_bytes` apart (multiple of 4), one
 * GPU thread per word; old_out (device pointer to count int32, or NULL) receives the previous
 * values.  sem / scope select the PTX qualifiers (.relaxed/.acquire/.release/.acq_rel,
 * .cta/.gpu/.sys). */
int iris_atomic_add(iris_heap* heap, void* ptr, size_t count, size_t stride_bytes, int from_rank, int to_rank,
                    int32_t value, int sem, int scope, int32_t* old_out, void* stream);
int iris_atomic_cas(iris_heap* heap, void* ptr, size_t count, size_t stride_bytes, int from_rank, int to_rank,
                    int32_t compare, int32_t value, int sem, int scope, int32_t* old_out, void* stream);

/* The same two atomics on uint64 words (Table 3's atomic_add / atomic_cas with 64-bit operands; Section 3.3's
 * sem x scope choice).  ptr and stride_bytes must be multiples of 8; the addition wraps modulo 2^64; old_out is
 * a device pointer to count uint64 (or NULL). */
int iris_atomic_add_u64(iris_heap* heap, void* ptr, size_t count, size_t stride_bytes, int from_rank, int to_rank,
                        uint64_t value, int sem, int scope, uint64_t* old_out, void* stream);
int iris_atomic_cas_u64(iris_heap* heap, void* ptr, size_t count, size_t stride_bytes, int from_rank, int to_rank,
                        uint64_t compare, uint64_t value, int sem, int scope, uint64_t* old_out, void* stream);

/* The remaining atomics (atomic_xchg / and / or / xor / min / max; IRIS_OP_ADD is accepted too), vector form
 * as iris_atomic_add: old_out receives the previous values. */
int iris_atomic_rmw(iris_heap* heap, int op, void* ptr, size_t count, size_t stride_bytes, int from_rank, int to_rank,
                    int32_t value, int sem, int scope, int32_t* old_out, void* stream);

/* Contended forms used by the protocol tests and the atomics microbenchmark: `threads` GPU
 * threads all operate on the SAME word.  add: each adds `value`; cas: thread i tries
 * compare -> value_base + i.  old_out: device pointer to `threads` int32 (or NULL). */
int iris_atomic_add_contended(iris_heap* heap, void* ptr, size_t threads, int from_rank, int to_rank, int32_t value,
                              int sem, int scope, int32_t* old_out, void* stream);
int iris_atomic_cas_contended(iris_heap* heap, void* ptr, size_t threads, int from_rank, int to_rank,
                              int32_t compare, int32_t value_base, int sem, int scope, int32_t* old_out,
                              void* stream);

/* Set `count` int32 words at heap offset `off` to `value` in every slot (flag / lock set-up). */
int iris_flags_fill(iris_heap* heap, uint64_t off, size_t count, int32_t value, void* stream);

/* All-store microbenchmark (Section 5.1, "all-store"): every rank r copies its block of S bytes
 * (at payload_off in its own slot) into every slot s at recv_off + r*S, in tiles of tile_bytes
 * (multiple of 16, <= 32768; the last tile of a block may be short), and after each tile's bytes
 * sets flag[s][r*T + i] with atomic_cas(epoch-1 -> epoch, release, gpu), T = ceil(S/tile_bytes).
 * S must be a multiple of 16.  ctas: grid size (0 = 8 per SM).  Reads W*S, writes W*W*S bytes.
 * pull != 0 runs the all-load form instead: every rank s fetches (get) block r from rank r's
 * slot into its own recv area; same end state. */
int iris_all_store_bench(iris_heap* heap, uint64_t payload_off, uint64_t recv_off, uint64_t flag_off, size_t S,
                         size_t tile_bytes, int32_t epoch, int ctas, int pull, void* stream);

/* ------------------------------------------------------------------------------------------ */
/* GEMM + all-scatter (Section 4, Listings 2-5)                                                */
/* ------------------------------------------------------------------------------------------ */

/* C = A . [B_0 | B_1 | ... | B_{W-1}] with fp32 accumulation, rounded once to the element type;
 * rank r owns columns [r*N/W, (r+1)*N/W).  Each finished tile is stored into EVERY rank's slot at
 * the tile's global offset (Listing 4: offset = rm*ldc + rn + cur_rank*N_local), and for each
 * 128 x 128 publication tile t and each slot s the int32 ready flag flag[s][t] is then written
 * with release semantics at gpu scope.
 *
 * Publication tiles are counted per rank shard so that none straddles two ranks:
 *   TM = ceil(M/128), TNl = ceil((N/W)/128), t = tm*(W*TNl) + r*TNl + j.
 *
 * Layout in every slot: C row-major [M, N] (ldc = N) at c_off; int32 flag[TM*W*TNl] at flag_off;
 * int32 lock[TM*W*TNl] at lock_off (workgroup-specialised mode only; lock t is used in the slot of
 * the rank owning tile t, must be 0 before the call and is 0 again afterwards: Listing 5's
 * cas(0->1, release) by the producer and cas(1->0, acquire) by the communication CTA).
 */
typedef struct iris_gemm_args {
  const void* A;               /* device: [M, K] row-major, K contiguous, 16-byte aligned        */
  const void* const* B_shards; /* HOST array of `world` DEVICE pointers, each 16-byte aligned; shard r
                                  is [N/W, K] with K contiguous (= the K x N_local operand of
                                  Listing 2 stored column-major) unless b_layout says otherwise  */
  iris_heap* heap;
  int M, N, K;                 /* N = global width; N % world == 0, (N/world) % 8 == 0, K % 8 == 0;
                                  M, N, K >= 0 (an empty problem publishes nothing and succeeds) */
  int world;                   /* must equal the heap's world                                    */
  int mode;                    /* IRIS_MODE_*                                                    */
  int dtype;                   /* IRIS_F16 or IRIS_BF16                                          */
  uint64_t c_off, flag_off, lock_off; /* offsets inside a slot; c_off % 256 == 0, others % 4     */
  int32_t epoch;               /* value written to the flags; callers use 1, 2, 3, ...           */
  int comm_ctas;               /* workgroup-specialised: communication CTAs (0 = chosen by the
                                  library: from a small model of waves and store-path time when
                                  the producers may take tiles over (wg_tail = 0, CTA-pair kernel:
                                  10 at the largest config), from the ratio of scatter bytes to
                                  GEMM time otherwise (16 there))                                */
  int max_ctas;                /* cap on the persistent grid (0 = one CTA per SM)                */
  int raster_group;            /* tile rows per raster group for L2 reuse (0 = 2048 rows)        */
  int block_n;                 /* compute-tile width: 0 = auto, 128 or 256                       */
  uint64_t spin_timeout_ns;    /* deadline of every device-side wait (0 = 2 s)                   */
  int cta_pair;                /* 0 = use 256 x 256 CTA-pair tiles (tcgen05 cta_group::2) when M > 128
                                  and N/world > 128 (a ragged last tile is padded);
                                  1 = use them whenever M > 128 and N/world > 128
                                  (IRIS_ERR_UNSUPPORTED otherwise); -1 = single-CTA tiles only   */
  int static_schedule;         /* CTA-pair kernel: 0 = pairs claim tile ids in raster order from
                                  an atomic counter as they become free; 1 = the listings' static
                                  loop tile = pid, pid + NUM, ... (the single-CTA kernel always
                                  uses the static loop)                                          */
  int stream_k;                /* single-CTA kernel: 1 = split the k-steps of all tiles into equal
                                  ranges, one per CTA; tiles that straddle ranges are computed in
                                  parts and reduced in k order through a workspace the heap
                                  allocates on first use; 0 and -1 = whole tiles only (measured
                                  faster on every benchmark shape, hence the default)            */
  int wg_tail;                 /* workgroup-specialised: which compute tiles the producers scatter
                                  themselves (to all W slots, as fused_sequential does) instead of
                                  handing them to the communication CTAs.
                                  0 = the last wave (the last P tiles of the raster order, P =
                                  producer CTAs or pairs: no GEMM work is left to overlap their
                                  scatter with) and, in the CTA-pair kernel, every tile that the
                                  communication CTAs could not finish before the kernel ends,
                                  judged when the tile completes from their backlog and the waves
                                  still to come (so too few communication CTAs cost little);
                                  n > 0 = exactly the last n tiles; -1 = none (Listing 5 for every
                                  tile).  The final heap image is the same in every case        */
  int rank_first, rank_count;  /* compute, scatter and publish only the shards of ranks
                                  [rank_first, rank_first + rank_count): what one rank of a real
                                  W-GPU job runs (its own N/world columns into every slot), and
                                  what a pipeline over shards runs per stage.  0, 0 = every rank.
                                  B_shards entries outside the range are not read; tiles, flags and
                                  locks of other ranks are not touched; a consumer that is part of
                                  the call covers the same ranks                                  */
  int pace_stores;             /* CTA-pair kernel: 0 = the epilogue thread sends a tile's store boxes
                                  out one by one, spread over three quarters of the time the CTA takes
                                  per tile, because a burst of W copies holds up the operand loads of
                                  the tile being multiplied meanwhile (same queue out of the SM);
                                  -1 = all at once                                                */
  const void* consumer_bias;   /* not NULL: also run the flag-gated consumer OUT = C + bias (see
                                  iris_consume_bias) as part of this call: inside the same launch,
                                  as extra warps that acquire each tile's flag while the GEMM is
                                  still running (CTA-pair kernel, fused_sequential and
                                  workgroup_specialized), or as a following kernel otherwise.
                                  Device pointer to N elements, 16-byte aligned                  */
  uint64_t consumer_out_off;   /* offset of OUT [M, N] in every slot (with consumer_bias)        */
  int b_layout;                /* IRIS_B_N_BY_K (0): shards are [N/W, K], K contiguous;
                                  IRIS_B_K_BY_N (1): shards are [K, N/W] row-major as Listing 2 prints
                                  its B operand.  The tensor cores then read B as an MN-major
                                  operand (transpose bit of the instruction descriptor, 64 x 64
                                  shared-memory blocks); results are bit-identical to the other
                                  layout's on the transposed data                                */
  int fuse_tail;               /* CTA-pair kernel, shards that are not a whole number of 256-column tiles
                                  (N/world > 256, K-contiguous B): 1 = the remainder columns are computed
                                  by the pair that computes the shard's last full tile, as a second MMA
                                  group on the same A stages with its own accumulator (a narrow tile of
                                  its own would load as much of A as a full one); -1 = the remainder is
                                  a tile of its own; 0 = the library chooses (fused, except in
                                  workgroup_specialized mode with fewer than three waves of work).
                                  Same results either way                                          */
  int stage_k;                 /* CTA-pair kernel: K extent of one operand stage in shared memory.  128 = two 64-wide
                                  k-blocks per stage, their TMA boxes requested back to back (3 stages of 64 KB):
                                  adjacent 128-byte pieces of the same operand rows in flight together is what lets
                                  one SM's loads keep up with its tensor core; 64 = one k-block per stage (6 stages
                                  of 32 KB).  0 = the library chooses: 128, except that stages which also carry a
                                  fused remainder (fuse_tail) of more than 96 columns hold one k-block (two such
                                  stages would be all that fits).  With a remainder of up to 96 columns the ring is
                                  two two-k-block stages and one one-k-block stage.  Same results              */
} iris_gemm_args;

/* Enqueue the whole operation on `stream` (bulk-synchronous: two kernels; otherwise one).
 * IRIS_ERR_ARG / IRIS_ERR_RANGE / IRIS_ERR_UNSUPPORTED are returned before any launch. */
int iris_gemm_all_scatter_ex(const iris_gemm_args* args, void* stream);

/* Unfused producer-consumer (Section 4.1 "Unfused producer-consumer"; Section 5.2 reports it as the best pattern on
 * the paper's hardware): the workgroup-specialised schedule as TWO kernels on TWO streams with a partition of the
 * SMs.  The GEMM kernel (producer CTAs only: tile -> owner slot -> lock 0 -> 1, release) is launched on
 * producer_stream; the communication kernel (lock 1 -> 0, acquire; copy to the other W-1 slots; publish the flags),
 * with comm_ctas CTAs -- at most what the producers leave free -- is launched right after it on comm_stream.
 * args->mode must be IRIS_MODE_WORKGROUP_SPECIALIZED; comm_ctas, wg_tail and every other field mean what they mean
 * for iris_gemm_all_scatter_ex, and the final heap image is the same.  consumer_bias is refused
 * (IRIS_ERR_UNSUPPORTED): a consumer goes on a stream of its own (iris_consume_bias), where it overlaps both.
 * Ordering: comm_stream first waits for what was enqueued on producer_stream before this call; after the call
 * producer_stream waits for the communication kernel, so work enqueued on producer_stream afterwards (and
 * iris_status_check on it) sees the finished scatter.  The two streams must differ.
 * The dependency between the kernels runs one way (the second waits for locks the first sets, never the reverse)
 * and every wait has the usual deadline: if the hardware starts the second kernel late the scatter merely
 * overlaps less, and if it cannot run at all within spin_timeout_ns the call ends with IRIS_ERR_TIMEOUT in the
 * status block, never with a hang. */
int iris_gemm_all_scatter_unfused(const iris_gemm_args* args, void* producer_stream, void* comm_stream);

/* The short form named by the problem statement.  bf16; C at offset 0 of every slot, flags at
 * align256(M*N*2), locks right after the flags (align256); epoch = a per-heap counter that starts
 * at 1 and grows by one per call (iris_heap_epoch() returns the last value used); default stream.
 * The heap must have been created with bytes_per_rank >= iris_gemm_heap_bytes(M, N, world).  On a heap's
 * first such call, and whenever (M, N) differ from the previous short-form or host-buffer call on it, the
 * flag and lock arrays of every slot are cleared on the stream before the launch. */
int gemm_all_scatter(const void* A, const void* const* B_shards, iris_heap* heap, int M, int N, int K, int world,
                     int mode);
size_t iris_gemm_heap_bytes(int M, int N, int world);
int32_t iris_heap_epoch(const iris_heap* heap);
/* Number of publication tiles TM*W*TNl (0 for an empty problem, <0 on bad arguments). */
int64_t iris_num_tiles(int M, int N, int world);

/* Flag-gated consumer (Section 4.1, producer-consumer: the consumer side).  For every slot s and
 * publication tile t: wait (acquire, gpu scope, bounded by timeout_ns, 0 = 2 s) until
 * flag[s][t] >= epoch, then OUT[s] = C[s] + bias on that tile; bias: device pointer to N elements
 * of `dtype`, broadcast over rows; the sum is formed in fp32 and rounded once.  OUT is a second
 * row-major [M, N] region at out_off in every slot.  ctas: grid size (0 = 8 per SM).
 * On a stream of its own the consumer may be launched while its producer is still running (that is the point of
 * the flags).  Launch it AFTER every kernel that publishes the flags it waits for has been launched: those kernels are
 * persistent, all their CTAs are resident from the start, and the consumer's CTAs then fill whatever the SMs have left
 * (beside a GEMM CTA, which takes all but 1 KB of an SM's shared memory, that is one consumer CTA per SM; the rest of
 * the grid follows as the GEMM's CTAs leave).  The other order is not supported.  A consumer CTA leaves only once its
 * tiles are published, every resident CTA reserves 1 KB of shared memory, and a GEMM CTA that arrives later fits only
 * on an SM holding at most one of them (the single-CTA workgroup-specialised kernel, a cooperative launch, did not
 * start at all behind a waiting consumer of 64 CTAs).  A publisher that finds no room never runs, and the wait ends by
 * its deadline (IRIS_ERR_TIMEOUT), not by making progress.  The same holds when a publishing kernel can only start
 * later (the second kernel of bulk_synchronous mode starts when the GEMM ends) or when two streams are released by
 * the same event and start in no fixed order: keep the consumer off the device until the publishers are running. */
int iris_consume_bias(iris_heap* heap, uint64_t c_off, uint64_t out_off, uint64_t flag_off, const void* bias, int M,
                      int N, int world, int dtype, int32_t epoch, int ctas, uint64_t timeout_ns, void* stream);
/* The same for the publication tiles of ranks [rank_first, rank_first + rank_count) only (the column
 * shards those ranks own, in every slot); rank_count = 0 does nothing. */
int iris_consume_bias_ranks(iris_heap* heap, uint64_t c_off, uint64_t out_off, uint64_t flag_off, const void* bias,
                            int M, int N, int world, int rank_first, int rank_count, int dtype, int32_t epoch,
                            int ctas, uint64_t timeout_ns, void* stream);

/* End-to-end form with HOST buffers: copies A and the W shards (and bias, if given) to device staging
 * owned by the heap (allocated on first use, reused afterwards), runs gemm_all_scatter in `mode` with
 * the short form's layout, then -- when bias_host != NULL -- the flag-gated consumer with OUT at
 * iris_gemm_out_offset(M, N, world); copies slot `out_slot`'s C ([M, N], to C_host), its OUT (to
 * OUT_host; bias_host and OUT_host are both NULL or both non-NULL) and the flags of all slots
 * (world * iris_num_tiles int32, slot-major, to flags_host; may be NULL) back, and returns after
 * everything has completed.  The work is pipelined over blocks of rows (M >= 1024: up to 8 blocks of
 * whole 256-row tiles) on three streams the heap handle owns: while block i computes, block i+1's rows
 * of A arrive and block i-1's rows of C and OUT leave, so both directions of the host link are busy
 * at once; every block is the same operation on its rows, and the result is the one an unblocked call
 * gives.  Synchronises the device on entry (the call owns the heap until it returns).  Host buffers
 * should be pinned for full copy speed.  With a bias the heap needs bytes_per_rank >=
 * iris_gemm_out_offset + M*N*2. */
int iris_gemm_all_scatter_host(const void* A_host, const void* const* B_shards_host, void* C_host,
                               int32_t* flags_host, const void* bias_host, void* OUT_host, iris_heap* heap,
                               int M, int N, int K, int world, int mode, int dtype, int out_slot);
/* Offset of OUT in the short form's layout: right after the lock array (256-byte aligned). */
uint64_t iris_gemm_out_offset(int M, int N, int world);

/* How the last workgroup-specialised launch of the CTA-pair kernel on this heap split the scatter:
 * out[0] = 128-row half tiles that their producers kept under the takeover rule (wg_tail = 0; the last
 * wave, which is never handed over, is not counted), out[1] = publication tiles still queued for the
 * communication CTAs (0 after a completed launch).  Synchronises the device; `out` is host memory. */
int iris_gemm_takeover_stats(const iris_heap* heap, int32_t out[2]);

/* ------------------------------------------------------------------------------------------ */
/* An entry point that allocates nothing                                                       */
/* ------------------------------------------------------------------------------------------ */

/* (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * Some callers of this library are not in a position to allocate device memory: a serving process
 * whose framework reserved all of HBM for its own pool at start-up, so that a cudaMalloc from a
 * plug-in would fail or eat into somebody else's budget; a latency-critical loop that cannot afford
 * the device-wide synchronisation an allocation or a free implies; code that runs under a memory
 * budget fixed in advance and audited.  Every other GEMM entry point needs an iris_heap handle, and
 * creating one allocates (the status block, and the heap itself unless a base is supplied), and the
 * workgroup-specialised schedule needs a zeroed lock array on top.  This call needs none of that:
 *
 *   - it takes the W slot base addresses directly (slot_bases: HOST array of `world` DEVICE
 *     addresses, each 256-byte aligned, each the start of bytes_per_rank bytes the caller owns);
 *     inputs A, B_shards and the outputs (C at c_off and int32 flags at flag_off in every slot)
 *     are the caller's, exactly as for iris_gemm_all_scatter_ex;
 *   - it runs the workgroup-specialised schedule; the per-tile locks and the status block live in
 *     a fixed array inside the library image (static __device__, 65 792 bytes, held by every GPU
 *     that loads the library until the process exits);
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Limit: at most 16 384 publication tiles, i.e. ceil(M/128) * world * ceil((N/world)/128) <= 16384
 * (the W=8, 8192 x 16384 output of the largest benchmark configuration has 8192).  Larger problems
 * are refused with IRIS_ERR_UNSUPPORTED and a message naming the limit; nothing is launched.
 *
 * The first call on a device looks up the device address of that array (with that device current)
 * and remembers it (the per-device record is filled without a lock: concurrent first calls store
 * the same value).  Every call clears the words it is going to use (the array keeps the previous
 * call's contents) on `stream`, launches on `stream`, reads the status words back on `stream` and
 * then WAITS for that stream -- no other stream is touched -- and returns IRIS_OK or
 * IRIS_ERR_TIMEOUT (a bounded device-side wait ran out).  Because every call waits for its stream,
 * no call may be made while that stream is being captured.  All calls share the one array: two
 * calls whose GPU work overlaps (different streams, different host threads) race on it and must be
 * serialised by the caller.
 * Other arguments, checks, layout and results are those of iris_gemm_all_scatter_ex in
 * IRIS_MODE_WORKGROUP_SPECIALIZED with default tuning: the launch plan (CTA-pair or single-CTA
 * tiles, tile width, grid split, which tiles the producers scatter themselves) is built by the
 * same code and the same kernels run -- with the locks and the work-unit counter in the static
 * array and, the slots being wherever the caller says, one store map per slot -- so the results
 * are bit-identical to that call's. */
int iris_gemm_all_scatter_noalloc(const void* A, const void* const* B_shards, const uint64_t* slot_bases,
                                  size_t bytes_per_rank, int M, int N, int K, int world, int dtype, uint64_t c_off,
                                  uint64_t flag_off, int32_t epoch, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IRIS_B200_H */
