// Host-side launch interface between the C-ABI orchestration (grand_api.cu) and the kernel
// translation units.  Plain structs of device pointers and sizes; every launcher enqueues on the
// given stream and returns the cudaError_t of the launch.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace grand {

// Kernel launches are counted per index: the API entry point names the counter of its handle for the
// calling thread (LaunchScope), every launcher adds to it.
void count_launches(unsigned n);
struct LaunchScope {
  unsigned long long* prev;
  explicit LaunchScope(unsigned long long* counter);
  ~LaunchScope();
};

// Facts about the current device, looked up once per device (a process may drive several GPUs).
int sm_count();
// Lets `kernel` use the device's full opt-in dynamic shared memory; done once per (kernel, device).  `done` is a
// zero-initialised per-kernel table owned by the launcher (one slot per device index).
constexpr int kMaxDevices = 64;
struct SmemOptIn { int done[kMaxDevices]; };
cudaError_t allow_full_dynamic_smem(const void* kernel, SmemOptIn* done);

// Row layout shared by every distance kernel: a padded row has nchunk 16-byte chunks; a team of G
// lanes covers it with CPL chunks per lane.  layout_code selects the (G, CPL) instantiation.
struct Layout {
  uint32_t dim, dtype, metric;  // as stored (dim includes the extra coordinate of the MIPS -> L2 reduction)
  uint32_t udim;                // dimension of the caller's vectors and queries
  uint32_t esize, row_bytes, nchunk;
  int code;  // index into the (G, CPL) table, -1 = unsupported
  int G, CPL;
};
Layout make_layout(uint32_t dim, uint32_t dtype, uint32_t metric);

// Device-resident scalar state, read back by the host at the end of each update call.
struct DevState {
  int status;            // first error seen by a kernel (0 = ok); atomicMin of negative codes
  uint32_t entry;        // medoid
  uint32_t ndirty;       // length of the dirty list
  uint32_t cursor;       // segment allocator for grouped requests
  uint32_t work;         // dynamic work counter of the rebuild kernel
  uint32_t nheavy;       // dirty nodes listed for the warp-per-node rebuild (front of the work list) ...
  uint32_t nlight;       // ... and for the team-per-node append / compaction (back of the work list)
  uint32_t pad_;
  unsigned long long nlive;
  unsigned long long total_in;   // sum of in-degrees of the delete batch
  unsigned long long medoid_key; // argmin scratch
  unsigned long long counters[16];
};
// expansions, query-to-node distances, node-to-node distances, rebuilt rows, prunes, grouped requests; then the
// bytes the method itself has to move in the rebuild, repair-pick and forward-prune kernels (what each kernel
// counts is stated where it counts), and the rebuilt rows that went through a prune
enum { CTR_EXP = 0, CTR_DIST = 1, CTR_PAIR = 2, CTR_DIRTY = 3, CTR_PRUNE = 4, CTR_REQ = 5, CTR_RB_BYTES = 6, CTR_PK_BYTES = 7,
       CTR_FP_BYTES = 8, CTR_RB_PRUNED = 9, CTR_PK_PAIRS = 10, CTR_FP_PAIRS = 11 };  // + pair distances of the picks / forward prune alone

struct GraphView {
  const uint8_t* store;
  uint32_t* adj;
  uint32_t* deg;
  uint32_t* live;  // bitmap
  uint32_t* rowd;  // optional, cap x R: order-preserving bits of dist(u, adj[u][s]); 0xFFFFFFFF = not known
  uint8_t* rowpfx;  // per row: length of the leading run that is a RobustPrune output in ascending key
                    // order (no member of the run prunes a later member); appended entries follow it
  // visited-set delete mode only (else nullptr): rows may hold edges to ids that were deleted and later came
  // back with another vector.  birth[v] = batch number of v's latest insertion, rowepoch[u] = batch number of
  // the latest write of row u; an entry with birth[v] > rowepoch[u] predates v's present vector, so its
  // cached distance and its place in the pruned run are void.
  uint32_t* birth;
  uint32_t* rowepoch;
  uint32_t epoch;  // number of the running batch
  uint32_t R;
  uint64_t cap;
};

struct SearchArgs {
  Layout lay;
  GraphView g;
  uint32_t entry;
  const void* queries;   // packed nq x dim elements (used when qids == nullptr)
  const uint32_t* qids;  // queries are the store rows of these ids
  uint64_t nq;
  uint32_t L, vmax, k;
  uint32_t* out_ids;     // nq x k (nullable)
  void* out_dists;       // nq x k int32/float (nullable)
  unsigned long long* out_beam;  // nq x beam_stride clean keys, ascending (nullable)
  uint32_t* out_beam_n;
  uint32_t beam_stride;
  unsigned long long* out_vis;   // nq x vis_stride clean keys in expansion order (nullable)
  uint32_t* out_vis_n;
  uint32_t vis_stride;
  const uint32_t* boot_ids;  // bootstrap: scan these ids (all batch-mates) instead of walking the graph
  uint32_t boot_n;
  uint32_t hash_bits;
  uint32_t cache_ways;  // tags per bucket of the visited cache: 8 or 12 (set by the launcher)
  uint32_t auto_cache;  // the caller left hash_bits at its default: the launcher may enlarge the cache
  uint32_t* work_ctr;  // zeroed by the caller before the launch; nullptr = static striding
  uint32_t check_live; // 1: skip neighbours that are not live (rows may hold dangling edges)
  uint32_t mips;       // 1: rows are MIPS -> L2 augmented; reported distances go back to negated inner products
  float mips_M2;       // M^2 of that reduction
  DevState* state;
};
cudaError_t launch_beam_search(const SearchArgs& a, cudaStream_t s);
size_t beam_search_smem_per_warp(uint32_t L, uint32_t R, uint32_t hash_bits, uint32_t cache_ways);

struct PruneArgs {
  Layout lay;
  GraphView g;
  long long A_fix;
  float alpha;
  const uint32_t* ids;  // batch ids, n
  uint64_t n;
  const unsigned long long* cand;  // n x cand_stride keys (visited lists)
  const uint32_t* cand_n;
  uint32_t cand_stride;
  uint32_t fixed_mode;  // 1: no prune, row = first R candidates in key order (Alg. 7)
  // outputs: adjacency row + request tuples (target = selected neighbour, key = (dist, new id))
  uint32_t* req_tgt;             // n x R
  unsigned long long* req_key;   // n x R
  DevState* state;
};
cudaError_t launch_forward_prune(const PruneArgs& a, cudaStream_t s);

struct GroupArgs {
  const uint32_t* req_tgt;
  const unsigned long long* req_key;
  uint64_t nreq;
  uint32_t* cnt;    // per node, zero between calls
  uint32_t* fill;   // per node, zero between calls
  uint32_t* start;  // per node
  uint32_t* flag;   // per node dirty flag, zero between calls
  uint32_t* dirty;  // dirty list
  unsigned long long* seg_keys;  // grouped keys
  DevState* state;
  // Optional split of the dirty list for the Vamana rebuild (work == nullptr: no split).  A node whose row cannot
  // overflow (deg + requests <= R) with at most light_max requests only needs its requests appended (and, in a delete
  // batch, its row compacted): such nodes are listed from the back of `work`, all others from the front.
  uint32_t* work;
  uint32_t work_cap;
  uint32_t light_max;
  const uint32_t* deg;
  uint32_t R;
};
cudaError_t launch_group_requests(const GroupArgs& a, cudaStream_t s);

struct RebuildArgs {
  Layout lay;
  GraphView g;
  long long A_fix;
  float alpha;
  uint32_t P;
  const uint32_t* delmap;  // bitmap of the delete batch, or nullptr on insert
  const uint32_t* livemap; // visited-set delete mode: kept neighbours must be live ...
  const uint32_t* newmap;  // ... or members of the running insert batch (not published yet)
  uint32_t* cnt; uint32_t* fill; uint32_t* start; uint32_t* flag;
  const uint32_t* dirty;   // the nodes to rebuild: state->ndirty entries, or, with `split`, the work list
  uint32_t split;          // 1: `dirty` is a work list (heavy nodes from the front, light nodes from the back, dirty_cap entries)
  uint32_t dirty_cap;
  unsigned long long* seg_keys;
  uint32_t max_blocks;
  DevState* state;
};
cudaError_t launch_rebuild(const RebuildArgs& a, cudaStream_t s);

// fixed-degree reverse edges (Alg. 7): one owner per target, detour find-and-replace
struct FixedReverseArgs {
  GraphView g;
  const uint32_t* slot_of;   // id -> batch position
  const uint32_t* fwd_rows;  // batch position x R: forward rows as written (INVALID padded)
  uint32_t* cnt; uint32_t* fill; uint32_t* start; uint32_t* flag;
  const uint32_t* dirty;
  unsigned long long* seg_keys;
  uint32_t max_blocks;
  DevState* state;
};
cudaError_t launch_fixed_reverse(const FixedReverseArgs& a, cudaStream_t s);

// ---- reverse graph (Alg. 8): histogram -> exclusive scan -> scatter (-> sort rows)
struct TransposeArgs {
  GraphView g;
  uint32_t* indeg;  // cap+1 scratch (zeroed inside)
  uint32_t* off;    // cap+1
  uint32_t* fillc;  // cap scratch (zeroed inside)
  uint32_t* src;    // >= total edges (nullable: offsets only)
  uint32_t* scan_tmp;  // >= ceil((cap+1)/4096)+1
  bool sort_rows;
  const uint32_t* heads;  // optional bitmap: build only the rows of these nodes
  uint64_t src_capacity;  // entries `src` can hold; edges beyond it are dropped (the caller compares the total)
  uint32_t* bad;          // optional: set to 1 when a row names a neighbour id >= cap (such an edge is skipped)
  // optional (with `heads`, unsorted rows): list of the marked edges as (head << 32 | tail), its capacity in pairs
  // and a device word for its length; the rows are then scattered from the list instead of a second adjacency pass
  unsigned long long* pairs; uint64_t pairs_capacity; uint32_t* pair_count;
};
cudaError_t launch_transpose(const TransposeArgs& a, cudaStream_t s);
cudaError_t launch_exclusive_scan(const uint32_t* in, uint32_t* out, uint64_t n, uint32_t* tmp, cudaStream_t s);

// ---- delete repair (Alg. 6)
struct DeleteArgs {
  Layout lay;
  GraphView g;
  const uint32_t* ids; uint64_t n;   // delete batch
  const uint32_t* delmap;
  const unsigned long long* beam; const uint32_t* beam_n; uint32_t beam_stride;  // per-deleted search result
  unsigned long long* Ci; uint32_t* Ci_n; uint32_t k_repair;                    // repair candidates
  uint32_t c;
  const uint32_t* off; const uint32_t* src;   // reverse graph (exact mode): in-neighbours of p at src[off[p] ..]
  uint32_t src_stride;                        // visited-set mode: in-neighbours of batch member i at src[i * src_stride ..]
  const uint32_t* livemap;                    // visited-set mode: out-neighbours that are not live are skipped
  const unsigned long long* vis; const uint32_t* vis_n; uint32_t vis_stride;  // visited lists of the per-deleted searches
  uint32_t* in_cnt; uint32_t* pair_off;       // n+1
  uint32_t* unit_off;                         // n+1: work units (chunks of pairs) per deleted node, prefix
  uint32_t* unit_owner;                       // per unit: its batch member (wide-row picks only; at most (total_in + n*R) / 8 + n entries)
  uint32_t* scan_tmp;
  uint32_t* req_tgt; unsigned long long* req_key;   // (total_in + n*R) * c
  uint32_t* flag; uint32_t* dirty;
  DevState* state;
};
cudaError_t launch_delete_prepare(const DeleteArgs& a, cudaStream_t s);   // in-degree prefix, total_in
cudaError_t launch_delete_ci(const DeleteArgs& a, cudaStream_t s);        // repair candidates C_i
cudaError_t launch_delete_visited_in(const DeleteArgs& a, uint32_t* inlist, cudaStream_t s);  // Alg. 6 as printed: z in V_i with p_i in N_out(z)
// repair picks: the set-up kernels (dirty marks of the in-neighbours, work-unit prefix), then the pick kernel alone
cudaError_t launch_delete_picks_prepare(const DeleteArgs& a, uint64_t total_in, cudaStream_t s);
cudaError_t launch_delete_picks(const DeleteArgs& a, uint64_t total_in, cudaStream_t s);

struct FixedDeleteArgs {
  GraphView g;
  const uint32_t* ids; uint64_t n;
  const uint32_t* delmap;
  const uint32_t* off; uint32_t* src;  // in-neighbour rows of the batch (long rows are sorted in place)
  const uint32_t* pair_off;  // n+1 prefix of in-degrees
  uint32_t* flag; uint32_t* dirty;
  DevState* state;
};
cudaError_t launch_fixed_delete(const FixedDeleteArgs& a, uint64_t total_in, cudaStream_t s);

// ---- small kernels
cudaError_t launch_validate(const uint32_t* ids, uint64_t n, uint64_t cap, const uint32_t* live, uint32_t* mark,
                            int want_live, DevState* st, cudaStream_t s);
cudaError_t launch_clear_marks(const uint32_t* ids, uint64_t n, uint64_t cap, uint32_t* mark, cudaStream_t s);
cudaError_t launch_store_write(const Layout& lay, uint8_t* store, uint32_t* deg, uint32_t* slot_of, const uint32_t* ids,
                               const void* vecs, uint64_t n, cudaStream_t s);
cudaError_t launch_publish(const uint32_t* ids, uint64_t n, uint32_t* live, uint32_t* mark, DevState* st, cudaStream_t s);
cudaError_t launch_retire(const GraphView& g, const uint32_t* ids, uint64_t n, uint32_t* delmap,
                          const unsigned long long* Ci, const uint32_t* Ci_n, uint32_t k_repair, uint32_t fixed_mode,
                          DevState* st, cudaStream_t s);
cudaError_t launch_pick_medoid(const Layout& lay, const GraphView& g, const uint32_t* ids, uint64_t n, uint8_t* mean_row,
                               DevState* st, cudaStream_t s);
cudaError_t launch_count_live(const uint32_t* live, uint64_t cap, DevState* st, cudaStream_t s);
cudaError_t launch_pad_rows(const Layout& lay, uint8_t* store, const void* vecs, uint64_t n, cudaStream_t s);
// MIPS -> L2 reduction: norm check of a batch (status -1 above the bound) and the extra coordinate of stored rows
cudaError_t launch_check_norms(const Layout& lay, const void* vecs, uint64_t n, double M2, DevState* st, cudaStream_t s);
cudaError_t launch_augment_rows(const Layout& lay, uint8_t* store, const uint32_t* ids, uint64_t n, double M2, cudaStream_t s);
// dst[v][:] = src[v][:] for the listed rows v (ids >= cap are skipped)
cudaError_t launch_copy_rows(const uint32_t* src, uint32_t* dst, const uint32_t* ids, uint64_t n, uint32_t R, uint64_t cap, cudaStream_t s);
cudaError_t launch_pad_adjacency(uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R, cudaStream_t s);
cudaError_t launch_fill_u32(uint32_t* p, uint32_t v, uint64_t n, cudaStream_t s);
// status -1 when a degree exceeds R or a listed neighbour id is >= cap (caller-supplied graphs)
cudaError_t launch_check_graph(const uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R, DevState* st, cudaStream_t s);

}  // namespace grand

// ---- (G, CPL) dispatch table.  nchunk <= 2 -> (2,1); <= 8 -> (4,2); <= 16 -> (4,4); <= 24 -> (4,6) (teams of 4
// measured best for 128- and 384-byte rows); <= 32 -> (8,4); <= 64 -> (32,2); <= 128 -> (32,4); <= 256 -> (32,8).
#define GRAND_LAYOUT_SWITCH(code, FN, T, M, ...)            \
  switch (code) {                                           \
    case 0: return FN<T, M, 2, 1>(__VA_ARGS__);             \
    case 1: return FN<T, M, 4, 2>(__VA_ARGS__);             \
    case 2: return FN<T, M, 4, 4>(__VA_ARGS__);             \
    case 3: return FN<T, M, 4, 6>(__VA_ARGS__);             \
    case 4: return FN<T, M, 8, 4>(__VA_ARGS__);             \
    case 5: return FN<T, M, 32, 2>(__VA_ARGS__);            \
    case 6: return FN<T, M, 32, 4>(__VA_ARGS__);            \
    case 7: return FN<T, M, 32, 8>(__VA_ARGS__);            \
    default: return cudaErrorInvalidValue;                  \
  }
// all dtypes x both metrics
#define GRAND_DISPATCH_ALL(lay, FN, ...)                                                        \
  do {                                                                                          \
    if ((lay).dtype == 0) {                                                                     \
      if ((lay).metric == 0) { GRAND_LAYOUT_SWITCH((lay).code, FN, uint8_t, 0, __VA_ARGS__) }   \
      else { GRAND_LAYOUT_SWITCH((lay).code, FN, uint8_t, 1, __VA_ARGS__) }                     \
    } else if ((lay).dtype == 1) {                                                              \
      if ((lay).metric == 0) { GRAND_LAYOUT_SWITCH((lay).code, FN, int8_t, 0, __VA_ARGS__) }    \
      else { GRAND_LAYOUT_SWITCH((lay).code, FN, int8_t, 1, __VA_ARGS__) }                      \
    } else {                                                                                    \
      if ((lay).metric == 0) { GRAND_LAYOUT_SWITCH((lay).code, FN, float, 0, __VA_ARGS__) }     \
      else { GRAND_LAYOUT_SWITCH((lay).code, FN, float, 1, __VA_ARGS__) }                       \
    }                                                                                           \
  } while (0)
// L2 only (Vamana-mode kernels: alpha-pruning is defined for the L2 metric)
#define GRAND_DISPATCH_L2(lay, FN, ...)                                                         \
  do {                                                                                          \
    if ((lay).dtype == 0) { GRAND_LAYOUT_SWITCH((lay).code, FN, uint8_t, 0, __VA_ARGS__) }      \
    else if ((lay).dtype == 1) { GRAND_LAYOUT_SWITCH((lay).code, FN, int8_t, 0, __VA_ARGS__) }  \
    else { GRAND_LAYOUT_SWITCH((lay).code, FN, float, 0, __VA_ARGS__) }                         \
  } while (0)
