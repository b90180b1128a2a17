/*
 * grand.h -- C ABI of the B200 (sm_100a) library for batched dynamic maintenance and search of a
 * Vamana-style proximity graph (GrAND).
 *
 * One handle = one index on one GPU = one mutator at a time.  The library owns the device-resident
 * vector store (row stride padded to 16 B), the fixed-stride adjacency array uint32[capacity x R]
 * with a degree counter per node, the live bitmap and a workspace pool that is allocated when the
 * index is created (the pre-allocated resource pool of Sec. 3.1): grand_insert_batch, grand_delete_batch,
 * grand_search and the host variants of the two update calls allocate nothing.  (grand_reverse_graph and
 * grand_search_host keep buffers of their own that grow with the largest request.)  The caller owns
 * every buffer it passes in, and the library keeps no caller pointer past a call.  Unless a
 * function says "host", pointer arguments are DEVICE pointers, row-major and densely packed.
 *
 * Batch semantics are deterministic (one legal outcome of the lock-free scheme of Sec. 4): every
 * search of a batch runs on the batch-start snapshot, reverse-edge candidates of one target merge
 * in (distance, id) order, ties break by id.  Distances: L2 = squared Euclidean, IP = negated dot
 * product; uint8/int8 vectors use exact int32 arithmetic, fp32 vectors accumulate in fp32.
 *
 * Errors: every function returns 0 (GRAND_OK) or a negative grand_status.  Update calls validate the
 * whole batch on the device before mutating anything, so a failing call leaves the index unchanged.
 * No exception crosses this boundary and there is no CPU fallback.
 */
#ifndef GRAND_H_
#define GRAND_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct grand_index grand_index; /* opaque */
typedef void* grand_stream;             /* a cudaStream_t; NULL = the default stream */

typedef enum { GRAND_U8 = 0, GRAND_I8 = 1, GRAND_F32 = 2 } grand_dtype;
typedef enum { GRAND_L2 = 0, GRAND_IP = 1 } grand_metric;
typedef enum { GRAND_MODE_VAMANA = 0, GRAND_MODE_FIXED_DEGREE = 1 } grand_mode;

typedef enum {
  GRAND_OK = 0,
  GRAND_ERR_INVALID_ARG = -1,  /* null pointer, k > L, parameter beyond a compile-time bound */
  GRAND_ERR_CAPACITY = -2,     /* id >= capacity, batch larger than max_batch, or a delete batch that touches more
                                  in-neighbour entries than max_delete_edges */
  GRAND_ERR_DUPLICATE_ID = -3, /* the same id twice in one batch */
  GRAND_ERR_ALREADY_LIVE = -4, /* insert of a live id */
  GRAND_ERR_NOT_LIVE = -5,     /* delete of an id that is not live */
  GRAND_ERR_UNSUPPORTED = -6,  /* Vamana mode with the IP metric and no mips_max_norm (alpha-pruning needs a metric) */
  GRAND_ERR_CUDA = -7,         /* a CUDA call failed; text in grand_last_error */
  GRAND_ERR_NOMEM = -9         /* device allocation failed (index creation, or growth of an introspection buffer) */
} grand_status;

#define GRAND_INVALID_ID 0xFFFFFFFFu
#define GRAND_MAX_R 128u      /* degree bound limit */
#define GRAND_MAX_L 512u      /* worklist size limit */
#define GRAND_MAX_ROW_BYTES 4096u /* dim * sizeof(element), after padding to 16 B */

/* Optional parameters; a zero field selects the default.  P, c and k follow the parameter list of
 * Alg. 5 / Alg. 6 (scratch capacity, replacement edges per repair, repair candidates). */
typedef struct {
  uint64_t capacity;  /* peak number of ids N; ids live in [0, N-1]; default 1<<20; < 2^31 */
  uint64_t max_batch; /* largest update batch; default 1<<17 */
  uint32_t P;         /* reverse-edge candidates kept per target and batch; default 64; <= 256 */
  uint32_t c;         /* replacement edges per repaired neighbour; default 2; <= 8 */
  uint32_t k_repair;  /* repair candidates per deleted node; default min(50, L); <= 128 */
  uint32_t vmax;      /* expansion cap of update searches; default 2*L; <= 1024 */
  uint32_t mode;      /* grand_mode; default GRAND_MODE_VAMANA.  GRAND_MODE_FIXED_DEGREE needs R <= L (Alg. 7 keeps
                         the R closest entries of a search result of L entries); else GRAND_ERR_INVALID_ARG */
  uint32_t hash_bits; /* log2 of the per-query visited cache in 4-byte words; 8..13, and 4 << hash_bits >= padded row bytes;
                         0 = default: 10, and on rows above 512 bytes up to three times that where shared memory is left over */
  uint32_t full_transpose; /* 1: every delete batch builds the whole reverse graph; default 0: only the rows of the
                              batch's nodes (the only rows the repair reads; identical result) */
  float mips_max_norm;     /* > 0: Vamana mode accepts the IP metric on fp32 vectors through the MIPS -> L2
                              reduction of Sec. 5.3, x -> [x, sqrt(M^2 - |x|^2)] with M = this bound on every base
                              vector's norm (an insert with a larger norm fails with GRAND_ERR_INVALID_ARG);
                              searches still return negated inner products */
  uint32_t visited_set_delete; /* 1: Alg. 6 exactly as printed - the in-neighbours of a deleted node are looked for
                              only in the visited set of its search (no reverse graph).  Edges from nodes that
                              the search did not visit stay behind; searches and rebuilds skip neighbours that
                              are not live.  Default 0: exact in-neighbours, no edge to a deleted node survives.
                              Vamana mode only. */
  uint64_t max_delete_edges;   /* most in-neighbour entries (sum of the in-degrees of its nodes) one delete batch may
                              touch; default min(3 * max_batch * R, capacity * R).  The workspace of the update
                              calls is sized from max_batch and this bound when the index is created; a delete
                              batch beyond it fails with GRAND_ERR_CAPACITY and leaves the index unchanged. */
  uint32_t snapshot_search;    /* 1: searches may run on other streams (and from other host threads) WHILE an update
                              batch runs.  The adjacency is kept twice; a batch works on the unpublished copy and
                              publishes it when it returns, so a search sees exactly the graph of the last batch
                              that had returned when the search was issued.  Costs capacity*R*4 bytes and one
                              copy of the changed rows per batch.  Default 0: one copy, and a search must not
                              overlap an update.  Only grand_search (device pointers) may overlap; the *_host
                              variants share one staging area with the update calls, and profiling
                              (grand_set_profiling) assumes one caller.  Not combinable with visited_set_delete. */
  /* device allocator hooks (default cudaMalloc / cudaFree); lets a host runtime pool the memory */
  void* (*dev_alloc)(size_t bytes, void* user);
  void (*dev_free)(void* ptr, void* user);
  void* user;
} grand_options;

/* Counters since creation (or the last grand_reset_stats).  Times are accumulated only while
 * profiling is on (grand_set_profiling), from CUDA events recorded on the caller's stream. */
typedef struct {
  uint64_t expansions;     /* worklist entries expanded by all beam searches */
  uint64_t dist_evals;     /* query-to-node distances evaluated by beam searches */
  uint64_t pair_dists;     /* node-to-node distances (prune, repair picks, rebuild) */
  uint64_t dirty_nodes;    /* adjacency rows rebuilt */
  uint64_t prunes;         /* RobustPrune invocations (forward + rebuild) */
  uint64_t requests;       /* reverse-edge / repair requests grouped */
  uint64_t kernel_launches; /* kernels launched through this handle */
  uint64_t rebuild_bytes;  /* bytes the dirty-node rebuild has to move: per rebuilt row its read and write (2 * R * 4),
                              its request tuples (12 each) and, when a prune runs, one vector per candidate */
  uint64_t picks_bytes;    /* bytes the delete repair has to move: one vector per (deleted node, surviving in- or
                              out-neighbour) pair plus the repair candidates' vectors once per deleted node */
  uint64_t prune_bytes;    /* forward RobustPrune: one vector per candidate looked at */
  uint64_t rebuild_prunes; /* rebuilt rows that went through a prune (the rest were appends / compactions) */
  double ms_search;        /* beam-search kernels (search, insert and delete searches) */
  double ms_prune;         /* forward RobustPrune */
  double ms_group;         /* request grouping, and the set-up kernels of the repair picks */
  double ms_rebuild;       /* dirty-node rebuild */
  double ms_transpose;     /* reverse-graph construction */
  double ms_picks;         /* delete repair picks (the pick kernel alone) */
  double ms_other;         /* validation, store write, publish / retire */
  uint64_t n_search_launches;  /* launches behind ms_search, ms_prune, ms_rebuild, ms_picks, ms_transpose: */
  uint64_t n_prune_launches;
  uint64_t n_rebuild_launches;
  uint64_t n_picks_launches;
  uint64_t n_transpose_launches;
  uint64_t picks_pair_dists; /* node-to-node distances evaluated by the repair picks alone ... */
  uint64_t prune_pair_dists; /* ... and by the forward RobustPrune alone (both are part of pair_dists) */
} grand_stats;

/* Index life cycle (problem statement of Sec. 3-4: capacity fixed at initialisation, ids in
 * [0, N-1], deleted ids reusable).  dim * sizeof(element) <= GRAND_MAX_ROW_BYTES, R <= GRAND_MAX_R,
 * L <= GRAND_MAX_L.  The device current at creation owns the index. */
int grand_create(uint32_t dim, uint32_t dtype, uint32_t metric, uint32_t R, uint32_t L, float alpha,
                 grand_index** out);
int grand_create_ex(uint32_t dim, uint32_t dtype, uint32_t metric, uint32_t R, uint32_t L, float alpha,
                    const grand_options* opts, grand_index** out);
int grand_destroy(grand_index* idx);

/* BatchInsert (Alg. 5 in Vamana mode, Alg. 7 in fixed-degree mode).  ids_dev: n distinct non-live ids;
 * vecs_dev: n x dim elements.  Work is enqueued on `stream`; the call returns after the batch is
 * applied (it reads back one status block). */
int grand_insert_batch(grand_index* idx, const uint32_t* ids_dev, const void* vecs_dev, uint64_t n,
                       grand_stream stream);

/* BatchDelete (Alg. 6 with in-neighbours from the on-demand CSR reverse graph of Alg. 8; Alg. 8 itself
 * in fixed-degree mode).  ids_dev: n distinct live ids.  After the call no row holds a deleted id. */
int grand_delete_batch(grand_index* idx, const uint32_t* ids_dev, uint64_t n, grand_stream stream);

/* BeamSearch (Alg. 1) from the medoid with worklist size L (k <= L <= GRAND_MAX_L; expansion cap 2L).
 * out_ids_dev: nq x k ids sorted by (distance, id), padded with GRAND_INVALID_ID; out_dists_dev: nq x k
 * int32 (uint8/int8 vectors; padding INT32_MAX) or float (fp32 vectors; padding +inf).  Asynchronous
 * on `stream`; concurrent searches on a quiescent index are allowed. */
int grand_search(const grand_index* idx, const void* queries_dev, uint64_t nq, uint32_t k, uint32_t L,
                 uint32_t* out_ids_dev, void* out_dists_dev, grand_stream stream);

/* The same three calls with HOST buffers (pinned memory gives asynchronous copies): the host-to-device
 * copy of the inputs and the device-to-host copy of the results happen inside the call, which returns
 * after they complete. */
int grand_insert_batch_host(grand_index* idx, const uint32_t* ids_host, const void* vecs_host, uint64_t n,
                            grand_stream stream);
int grand_delete_batch_host(grand_index* idx, const uint32_t* ids_host, uint64_t n, grand_stream stream);
int grand_search_host(grand_index* idx, const void* queries_host, uint64_t nq, uint32_t k, uint32_t L,
                      uint32_t* out_ids_host, void* out_dists_host, grand_stream stream);

/* Introspection for parity checks and measurement.  Any output pointer may be NULL.
 * adj_dev: capacity x R (unused slots hold GRAND_INVALID_ID); deg_dev: capacity; live_bitmap_dev:
 * ceil(capacity/32) words, bit v%32 of word v/32; entry_out_host: HOST pointer to the medoid id. */
int grand_export_graph(const grand_index* idx, uint32_t* adj_dev, uint32_t* deg_dev, uint32_t* live_bitmap_dev,
                       uint32_t* entry_out_host, grand_stream stream);
/* Replaces the whole state (tests, and loading a saved index).  vecs_dev: capacity x dim packed elements.  Every
 * degree must be <= R and every listed neighbour id < capacity, else GRAND_ERR_INVALID_ARG and nothing is replaced. */
int grand_import_graph(grand_index* idx, const uint32_t* adj_dev, const uint32_t* deg_dev,
                       const uint32_t* live_bitmap_dev, uint32_t entry, const void* vecs_dev, grand_stream stream);
/* Exact reverse graph in CSR (Alg. 8): off_dev has capacity+1 entries, row z of src_dev lists every live
 * v with z in N_out(v), ascending.  src_dev needs room for capacity*R entries in the worst case;
 * pass src_dev = NULL to obtain only offsets and *E_out_host (HOST pointer, total edges). */
int grand_reverse_graph(grand_index* idx, uint32_t* off_dev, uint32_t* src_dev, uint64_t* E_out_host,
                        grand_stream stream);

/* The same CSR reverse graph for callers that cannot allocate device memory: hosts whose memory plan is
 * frozen at start-up (a serving process that has handed all of HBM to its own pool, a sandboxed plug-in
 * barred from the driver's allocator, a real-time loop that cannot take cudaMalloc's implicit
 * synchronisation or its failure mid-request).  The paper has no counterpart for this call.  It needs no
 * index handle: adj_dev (n_nodes x R, unused slots ignored through deg_dev; every listed neighbour id must be
 * < n_nodes, otherwise the call returns GRAND_ERR_INVALID_ARG - such an edge is never followed, so nothing is
 * written outside the caller's buffers) and deg_dev (n_nodes) are the caller's inputs, off_dev (n_nodes + 1) and src_dev (src_capacity entries; NULL = offsets only) the caller's
 * outputs, E_out_host a HOST pointer to the edge count.  The result equals grand_reverse_graph on the same
 * graph.  Its working memory is one fixed device array inside the library, GRAND_NOALLOC_SCRATCH_BYTES per GPU
 * for the life of the process: n_nodes > GRAND_NOALLOC_MAX_NODES returns GRAND_ERR_CAPACITY, and so does a
 * src_dev too small for the edges found.  All calls on a device share that array (everything that must be
 * zero is cleared per call), so calls that overlap on the GPU race: serialise them.  The first call on each
 * device resolves the array's address and should be made during set-up, before any stream capture.  No
 * cudaMalloc, cudaFree or allocating library routine is called. */
#define GRAND_NOALLOC_MAX_NODES (1u << 20)
#define GRAND_NOALLOC_SCRATCH_BYTES ((GRAND_NOALLOC_MAX_NODES + GRAND_NOALLOC_MAX_NODES / 2048u + 64u) * 4u)
int grand_reverse_graph_noalloc(const uint32_t* adj_dev, const uint32_t* deg_dev, uint64_t n_nodes, uint32_t R,
                                uint32_t* off_dev, uint32_t* src_dev, uint64_t src_capacity, uint64_t* E_out_host,
                                grand_stream stream);

int grand_get_entry(const grand_index* idx, uint32_t* entry_out_host);
int grand_set_entry(grand_index* idx, uint32_t entry);
int grand_live_count(const grand_index* idx, uint64_t* n_out_host);
int grand_row_bytes(const grand_index* idx, uint32_t* row_bytes_out_host);

int grand_get_stats(const grand_index* idx, grand_stats* out_host);
int grand_reset_stats(grand_index* idx);
int grand_set_profiling(grand_index* idx, int on);

const char* grand_strerror(int status);
const char* grand_last_error(const grand_index* idx);

#ifdef __cplusplus
}
#endif
#endif /* GRAND_H_ */
