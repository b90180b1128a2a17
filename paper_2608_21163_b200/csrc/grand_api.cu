// C-ABI entry points (include/grand.h) and the host orchestration of each batch call: argument
// checks, workspace pool (allocated at creation, grow-only), the kernel sequence of one batch on
// the caller's stream, and the single status read-back that ends an update call.
#include <atomic>
#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/grand.h"
#include "grand_kernels.h"

namespace grand {

// Launch counting: the entry point that runs on this thread names its handle's counter.
static thread_local unsigned long long* tl_launches = nullptr;
void count_launches(unsigned n) {
  if (tl_launches) *tl_launches += n;
}
LaunchScope::LaunchScope(unsigned long long* counter) : prev(tl_launches) { tl_launches = counter; }
LaunchScope::~LaunchScope() { tl_launches = prev; }

// Per-device facts, looked up on first use on that device.
static std::atomic<int> g_sm_count[kMaxDevices];
static std::atomic<int> g_smem_optin[kMaxDevices];
static int current_device() {
  int dev = 0;
  cudaGetDevice(&dev);
  return dev >= 0 && dev < kMaxDevices ? dev : 0;
}
int sm_count() {
  const int dev = current_device();
  int n = g_sm_count[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 1;
    g_sm_count[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}
cudaError_t allow_full_dynamic_smem(const void* kernel, SmemOptIn* done) {
  const int dev = current_device();
  // (two threads may both find the slot empty; they then set the same value twice)
  if (__atomic_load_n(&done->done[dev], __ATOMIC_ACQUIRE)) return cudaSuccess;
  int most = g_smem_optin[dev].load(std::memory_order_relaxed);
  if (most == 0) {
    cudaDeviceGetAttribute(&most, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    g_smem_optin[dev].store(most, std::memory_order_relaxed);
  }
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
  if (e != cudaSuccess) return e;
  __atomic_store_n(&done->done[dev], 1, __ATOMIC_RELEASE);
  return cudaSuccess;
}

Layout make_layout(uint32_t dim, uint32_t dtype, uint32_t metric) {
  Layout l{};
  l.dim = dim; l.udim = dim; l.dtype = dtype; l.metric = metric;
  l.esize = dtype == GRAND_F32 ? 4 : 1;
  l.row_bytes = (uint32_t)(((uint64_t)dim * l.esize + 15) / 16 * 16);
  l.nchunk = l.row_bytes / 16;
  static const int Gs[8] = {2, 4, 4, 4, 8, 32, 32, 32};
  static const int Cs[8] = {1, 2, 4, 6, 4, 2, 4, 8};
  static const uint32_t lim[8] = {2, 8, 16, 24, 32, 64, 128, 256};
  l.code = -1;
  for (int i = 0; i < 8; ++i)
    if (l.nchunk <= lim[i]) { l.code = i; l.G = Gs[i]; l.CPL = Cs[i]; break; }
  return l;
}

}  // namespace grand

using namespace grand;

enum Phase { PH_SEARCH = 0, PH_PRUNE, PH_GROUP, PH_REBUILD, PH_TRANSPOSE, PH_PICKS, PH_OTHER, PH_COUNT };

struct Buf {
  void* p = nullptr;
  size_t bytes = 0;
};

struct grand_index {
  Layout lay;
  uint32_t R, L, P, c, k_repair, vmax, mode, hash_bits, full_transpose;
  uint32_t auto_cache = 0;  // hash_bits was left at its default
  bool approx = false; // visited-set delete mode (Alg. 6 as printed): rows may hold dangling edges
  unsigned long long* vis_keys = nullptr;  // max_batch x vmax visited lists of the per-deleted searches (that mode only)
  uint32_t *vis_n = nullptr, *vis_in = nullptr;
  uint32_t *birth = nullptr, *rowepoch = nullptr;  // per node: batch number of its insertion / of its row's last write
  uint32_t epoch = 0;                              // batches applied so far
  // snapshot mode: searches read the published adjacency buffer while an update batch works on the other one
  bool snap = false;
  uint32_t* adj_alt = nullptr;
  int pub = 0;                         // 0: adj is published, 1: adj_alt
  uint32_t* sync_ids = nullptr;        // ids of the last applied batch ...
  uint64_t sync_n = 0;
  Buf sync_dirty;                      // ... and its dirty list: the rows the unpublished buffer still lacks
  uint64_t sync_ndirty = 0;
  std::mutex pub_mu;                   // guards pub, entry and the reader lists against searches from other threads
  std::vector<cudaEvent_t> readers[2]; // end-of-search events of the searches launched on each buffer
  std::vector<cudaEvent_t> reader_pool;
  bool mips = false;   // MIPS -> L2 reduction active (Vamana mode, IP metric, fp32)
  double mips_M2 = 0.0;
  float alpha;
  long long A_fix;
  uint64_t cap, max_batch;
  int device;
  void* (*dev_alloc)(size_t, void*);
  void (*dev_free)(void*, void*);
  void* user;
  // index state
  uint8_t* store = nullptr;
  uint32_t *adj = nullptr, *deg = nullptr, *live = nullptr;
  uint8_t* rowpfx = nullptr;
  uint32_t* rowd = nullptr;
  DevState* d_state = nullptr;
  DevState* h_state = nullptr;  // pinned mirror
  uint32_t entry = GRAND_INVALID_ID;
  uint64_t nlive = 0;
  // workspace pool
  uint32_t *mark = nullptr, *cnt = nullptr, *fill = nullptr, *start = nullptr, *flag = nullptr, *slot_of = nullptr;
  unsigned long long* wk_keys = nullptr;  // max_batch x max(vmax, L): visited lists / worklists of update searches
  uint32_t* wk_n = nullptr;
  uint32_t wk_stride = 0;
  unsigned long long* Ci = nullptr;
  uint32_t *Ci_n = nullptr, *in_cnt = nullptr, *pair_off = nullptr, *unit_off = nullptr, *scan_tmp = nullptr;
  uint32_t* pair_count = nullptr;  // length of the marked-edge list of a delete batch's reverse graph
  uint8_t* mean_row = nullptr;
  // Work counters of the search launches.  Slot 0 serves the searches inside update calls (each such call ends
  // with a stream synchronisation, so its launch is over before the next one starts).  grand_search is
  // asynchronous: it takes a ring slot whose previous launch has completed (an event per slot tells), and runs
  // with static query striding when none is free.
  static constexpr int kCtrSlots = 64;
  uint32_t* search_ctrs = nullptr;  // 1 + kCtrSlots counters
  cudaEvent_t ctr_done[kCtrSlots] = {};
  bool ctr_used[kCtrSlots] = {};
  uint32_t ctr_next = 0;             // (ring state is touched only under pub_mu)
  uint64_t max_requests = 0;       // request tuples a batch may emit (buffers below are sized for it at creation)
  uint64_t max_delete_edges = 0;   // in-neighbour entries a delete batch may touch
  Buf req_tgt, req_key, seg_keys, dirty;              // sized at creation for max_requests
  Buf work;                                           // the dirty list split by the kind of rebuild a node needs (Vamana mode)
  Buf t_indeg, t_off, t_fill, t_src;                  // reverse graph of a delete batch, sized at creation
  Buf x_indeg, x_off, x_fill, x_src;                  // full reverse graph for grand_reverse_graph (introspection; grown on demand)
  Buf st_ids, st_vecs, st_out_ids, st_out_d;          // staging of the *_host entry points (updates: sized at creation)
  std::vector<void*> owned;
  // stats
  unsigned long long launches = 0;
  grand_stats stats{};
  bool profiling = false;
  std::vector<cudaEvent_t> ev_pool;
  struct Span { int phase; cudaEvent_t a, b; };
  std::vector<Span> spans;
  size_t ev_used = 0;
  std::string last_error;
};

namespace {

int fail(const grand_index* idx, int code, const std::string& msg) {
  if (idx) const_cast<grand_index*>(idx)->last_error = msg;
  return code;
}
int cuda_fail(const grand_index* idx, cudaError_t e, const char* what) {
  return fail(idx, GRAND_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define CK(call)                                                        \
  do {                                                                  \
    cudaError_t e__ = (call);                                           \
    if (e__ != cudaSuccess) return cuda_fail(idx, e__, #call);          \
  } while (0)

void* default_alloc(size_t bytes, void*) {
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) return nullptr;
  return p;
}
void default_free(void* p, void*) { cudaFree(p); }

template <typename T>
int alloc_dev(grand_index* idx, T** out, size_t count, bool zero) {
  const size_t bytes = (count ? count : 1) * sizeof(T);
  void* p = idx->dev_alloc(bytes, idx->user);
  if (!p) return fail(idx, GRAND_ERR_NOMEM, "device allocation of " + std::to_string(bytes) + " bytes failed");
  idx->owned.push_back(p);
  if (zero) CK(cudaMemset(p, 0, bytes));
  *out = reinterpret_cast<T*>(p);
  return GRAND_OK;
}
int ensure(grand_index* idx, Buf& b, size_t bytes, cudaStream_t s) {
  if (b.bytes >= bytes && b.p) return GRAND_OK;
  const bool regrow = b.p != nullptr;
  if (b.p) {
    CK(cudaStreamSynchronize(s));
    idx->dev_free(b.p, idx->user);
    b.p = nullptr;
    b.bytes = 0;
  }
  size_t want = regrow ? bytes + bytes / 4 : bytes;  // first allocation: exact; regrowth: with headroom
  if (want == 0) want = 16;
  void* p = idx->dev_alloc(want, idx->user);
  if (!p) return fail(idx, GRAND_ERR_NOMEM, "workspace allocation of " + std::to_string(want) + " bytes failed");
  b.p = p;
  b.bytes = want;
  return GRAND_OK;
}

// work = true: the buffer an update batch reads and writes; false: the published one
uint32_t* adj_of(const grand_index* idx, bool work) {
  if (!idx->snap) return idx->adj;
  const int b = work ? 1 - idx->pub : idx->pub;
  return b == 0 ? idx->adj : idx->adj_alt;
}
GraphView view(const grand_index* idx, bool work) {
  GraphView g;
  g.store = idx->store; g.adj = adj_of(idx, work); g.deg = idx->deg; g.live = idx->live; g.rowpfx = idx->rowpfx; g.rowd = idx->rowd; g.R = idx->R; g.cap = idx->cap;
  g.birth = idx->birth; g.rowepoch = idx->rowepoch; g.epoch = idx->epoch;
  return g;
}

struct PhaseTimer {
  grand_index* idx;
  cudaStream_t s;
  int phase;
  cudaEvent_t a = nullptr, b = nullptr;
  PhaseTimer(grand_index* i, cudaStream_t st, int ph) : idx(i), s(st), phase(ph) {
    if (!idx->profiling) return;
    while (idx->ev_pool.size() < idx->ev_used + 2) {
      cudaEvent_t e;
      cudaEventCreate(&e);
      idx->ev_pool.push_back(e);
    }
    a = idx->ev_pool[idx->ev_used++];
    b = idx->ev_pool[idx->ev_used++];
    cudaEventRecord(a, s);
  }
  ~PhaseTimer() {
    if (!a) return;
    cudaEventRecord(b, s);
    idx->spans.push_back({phase, a, b});
  }
};
// after the stream is synchronised: fold recorded spans into the stats
void collect_spans(grand_index* idx) {
  for (auto& sp : idx->spans) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, sp.a, sp.b) != cudaSuccess) continue;
    double* slot[PH_COUNT] = {&idx->stats.ms_search, &idx->stats.ms_prune, &idx->stats.ms_group, &idx->stats.ms_rebuild,
                              &idx->stats.ms_transpose, &idx->stats.ms_picks, &idx->stats.ms_other};
    *slot[sp.phase] += ms;
  }
  idx->spans.clear();
  idx->ev_used = 0;
}

int read_state(grand_index* idx, cudaStream_t s) {
  CK(cudaMemcpyAsync(idx->h_state, idx->d_state, sizeof(DevState), cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  return GRAND_OK;
}
int write_state_head(grand_index* idx, cudaStream_t s) {
  // status, entry, ndirty, cursor, nlive, total_in: reset per call, counters untouched
  idx->h_state->status = 0;
  idx->h_state->entry = idx->entry;
  idx->h_state->ndirty = 0;
  idx->h_state->cursor = 0;
  idx->h_state->work = 0;
  idx->h_state->nheavy = 0;
  idx->h_state->nlight = 0;
  idx->h_state->nlive = idx->nlive;
  idx->h_state->total_in = 0;
  CK(cudaMemcpyAsync(idx->d_state, idx->h_state, offsetof(DevState, medoid_key), cudaMemcpyHostToDevice, s));
  return GRAND_OK;
}

// slot < 0: the counter of the update calls; otherwise a ring slot taken by take_ctr_slot (or -2: none free)
SearchArgs search_args(grand_index* idx, cudaStream_t s, bool work, int slot = -1) {
  SearchArgs a{};
  a.work_ctr = slot == -2 ? nullptr : idx->search_ctrs + (slot < 0 ? 0 : 1 + slot);
  if (a.work_ctr) cudaMemsetAsync(a.work_ctr, 0, 4, s);
  a.lay = idx->lay;
  a.g = view(idx, work);
  a.entry = idx->entry;
  a.hash_bits = idx->hash_bits;
  a.auto_cache = idx->auto_cache;
  a.check_live = idx->approx ? 1u : 0u;
  a.mips = idx->mips ? 1u : 0u;
  a.mips_M2 = (float)idx->mips_M2;
  a.state = idx->d_state;
  return a;
}

// A ring slot whose last launch is over, or -2.  Caller holds pub_mu until the launch's end event is recorded.
int take_ctr_slot(grand_index* idx) {
  for (int tries = 0; tries < grand_index::kCtrSlots; ++tries) {
    const int slot = (int)(idx->ctr_next++ % grand_index::kCtrSlots);
    if (!idx->ctr_used[slot] || cudaEventQuery(idx->ctr_done[slot]) == cudaSuccess) {
      idx->ctr_used[slot] = true;
      return slot;
    }
    if (tries >= 3) break;  // a few probes, then static striding: the ring is full of running launches
  }
  return -2;
}

int ensure_requests(grand_index* idx, uint64_t nreq, cudaStream_t s) {
  int rc;
  if ((rc = ensure(idx, idx->req_tgt, nreq * 4, s))) return rc;
  if ((rc = ensure(idx, idx->req_key, nreq * 8, s))) return rc;
  if ((rc = ensure(idx, idx->seg_keys, nreq * 8, s))) return rc;
  if ((rc = ensure(idx, idx->dirty, nreq * 4, s))) return rc;
  if (idx->mode == GRAND_MODE_VAMANA && !idx->approx && (rc = ensure(idx, idx->work, nreq * 4, s))) return rc;
  return GRAND_OK;
}

// Snapshot mode, start of an update batch: the batch works on the unpublished buffer.  Searches that were
// launched while that buffer was the published one must have finished, and the rows the previous batch
// changed are carried over from the published buffer first.
int begin_update(grand_index* idx, const uint32_t* ids, uint64_t n, cudaStream_t s) {
  if (!idx->snap) return GRAND_OK;
  const int w = 1 - idx->pub;
  {
    std::lock_guard<std::mutex> lk(idx->pub_mu);
    for (cudaEvent_t ev : idx->readers[w]) {
      CK(cudaStreamWaitEvent(s, ev, 0));
      idx->reader_pool.push_back(ev);
    }
    idx->readers[w].clear();
  }
  const uint32_t* from = adj_of(idx, false);
  uint32_t* to = adj_of(idx, true);
  if (idx->sync_n) CK(launch_copy_rows(from, to, idx->sync_ids, idx->sync_n, idx->R, idx->cap, s));
  if (idx->sync_ndirty) CK(launch_copy_rows(from, to, (const uint32_t*)idx->sync_dirty.p, idx->sync_ndirty, idx->R, idx->cap, s));
  idx->sync_n = idx->sync_ndirty = 0;
  CK(cudaMemcpyAsync(idx->sync_ids, ids, n * 4, cudaMemcpyDeviceToDevice, s));  // the caller's array need not outlive the call
  return GRAND_OK;
}
// End of a successful batch (its kernels have completed): remember which rows the other buffer lacks, publish.
// A batch that failed after it had started to write (a device loop hit its limit) is not published; the same
// lists then bring its buffer back to the published state at the start of the next batch.
void end_update(grand_index* idx, uint64_t n) {
  const bool ok = idx->h_state->status == 0;
  std::lock_guard<std::mutex> lk(idx->pub_mu);
  idx->entry = idx->h_state->entry;
  idx->nlive = idx->h_state->nlive;
  if (!idx->snap) return;
  std::swap(idx->dirty, idx->sync_dirty);
  idx->sync_ndirty = idx->h_state->ndirty;
  idx->sync_n = n;
  if (ok) idx->pub = 1 - idx->pub;
}

}  // namespace

extern "C" {

const char* grand_strerror(int st) {
  switch (st) {
    case GRAND_OK: return "ok";
    case GRAND_ERR_INVALID_ARG: return "invalid argument";
    case GRAND_ERR_CAPACITY: return "id or batch size beyond capacity";
    case GRAND_ERR_DUPLICATE_ID: return "duplicate id in batch";
    case GRAND_ERR_ALREADY_LIVE: return "id is already live";
    case GRAND_ERR_NOT_LIVE: return "id is not live";
    case GRAND_ERR_UNSUPPORTED: return "unsupported configuration";
    case GRAND_ERR_CUDA: return "CUDA error";
    case GRAND_ERR_NOMEM: return "device memory allocation failed";
    default: return "unknown status";
  }
}
const char* grand_last_error(const grand_index* idx) { return idx ? idx->last_error.c_str() : ""; }

int grand_create(uint32_t dim, uint32_t dtype, uint32_t metric, uint32_t R, uint32_t L, float alpha, grand_index** out) {
  return grand_create_ex(dim, dtype, metric, R, L, alpha, nullptr, out);
}

int grand_create_ex(uint32_t dim, uint32_t dtype, uint32_t metric, uint32_t R, uint32_t L, float alpha,
                    const grand_options* o, grand_index** out) {
  if (!out) return GRAND_ERR_INVALID_ARG;
  *out = nullptr;
  grand_options z{};
  if (!o) o = &z;
  if (dim == 0 || dtype > GRAND_F32 || metric > GRAND_IP || R == 0 || R > GRAND_MAX_R || L == 0 || L > GRAND_MAX_L ||
      o->mode > GRAND_MODE_FIXED_DEGREE || !(alpha >= 1.0f))
    return GRAND_ERR_INVALID_ARG;
  const bool mips = o->mode == GRAND_MODE_VAMANA && metric == GRAND_IP && o->mips_max_norm > 0.0f && dtype == GRAND_F32;
  if (o->mode == GRAND_MODE_VAMANA && metric == GRAND_IP && !mips) return GRAND_ERR_UNSUPPORTED;
  if (o->snapshot_search && o->visited_set_delete) return GRAND_ERR_UNSUPPORTED;  // those searches read the live bitmap, which has one copy
  if (o->mode == GRAND_MODE_FIXED_DEGREE && R > L) return GRAND_ERR_INVALID_ARG;  // Alg. 7 keeps the R closest of a search result of L entries
  // MIPS -> L2 reduction: rows carry one extra coordinate and the index works on squared L2
  Layout lay = mips ? make_layout(dim + 1, dtype, GRAND_L2) : make_layout(dim, dtype, metric);
  lay.udim = dim;
  if (lay.code < 0 || lay.row_bytes > GRAND_MAX_ROW_BYTES) return GRAND_ERR_INVALID_ARG;
  grand_index* idx = new grand_index();
  idx->lay = lay;
  idx->R = R; idx->L = L; idx->alpha = alpha;
  idx->A_fix = (long long)llround((double)alpha * 65536.0);
  idx->cap = o->capacity ? o->capacity : (1ull << 20);
  idx->max_batch = o->max_batch ? o->max_batch : (1ull << 17);
  if (idx->max_batch > idx->cap) idx->max_batch = idx->cap;  // a batch names distinct ids
  idx->P = o->P ? o->P : 64;
  idx->c = o->c ? o->c : 2;
  idx->k_repair = o->k_repair ? o->k_repair : (L < 50 ? L : 50);
  idx->vmax = o->vmax ? o->vmax : 2 * L;
  idx->mode = o->mode;
  idx->hash_bits = o->hash_bits ? o->hash_bits : 10;
  idx->auto_cache = o->hash_bits == 0;
  idx->full_transpose = o->full_transpose;
  idx->approx = o->visited_set_delete != 0 && o->mode == GRAND_MODE_VAMANA;
  idx->snap = o->snapshot_search != 0;
  idx->mips = mips;
  idx->mips_M2 = (double)o->mips_max_norm * (double)o->mips_max_norm;
  idx->dev_alloc = o->dev_alloc ? o->dev_alloc : default_alloc;
  idx->dev_free = o->dev_free ? o->dev_free : default_free;
  idx->user = o->user;
  if (idx->cap >= (1ull << 31) || idx->cap * R >= (1ull << 32) || idx->P > 256 || idx->c > 8 || idx->k_repair > 128 ||
      idx->k_repair > L || idx->vmax > 1024 || idx->vmax == 0 || idx->hash_bits < 8 || idx->hash_bits > 13 ||
      (4u << idx->hash_bits) < lay.row_bytes ||
      idx->max_batch * R >= (1ull << 32)) {
    delete idx;
    return GRAND_ERR_INVALID_ARG;
  }
  cudaGetDevice(&idx->device);
  const uint64_t cap = idx->cap, mb = idx->max_batch;
  // Request tuples of one batch: an insert emits n*R; a Vamana delete c per (deleted node, surviving in- or
  // out-neighbour) pair; a fixed-degree delete one per in-neighbour entry.  The in-neighbour entries of a delete
  // batch are bounded by max_delete_edges (default: three times the out-edges of a full batch, or every edge of
  // the graph if that is less).
  idx->max_delete_edges = o->max_delete_edges ? o->max_delete_edges : std::min<uint64_t>(3 * mb * R, cap * R);
  idx->max_requests = std::max<uint64_t>(mb * R, idx->mode == GRAND_MODE_FIXED_DEGREE ? idx->max_delete_edges + 1
                                                                                          : (idx->max_delete_edges + mb * R) * idx->c);
  if (idx->max_requests >= (1ull << 32) || idx->max_delete_edges >= (1ull << 32)) {
    delete idx;
    return GRAND_ERR_INVALID_ARG;
  }
  const size_t words = (cap + 31) / 32;
  int rc = GRAND_OK;
  auto A = [&](int r) { if (rc == GRAND_OK) rc = r; };
  A(alloc_dev(idx, &idx->store, (size_t)cap * lay.row_bytes, true));
  A(alloc_dev(idx, &idx->adj, (size_t)cap * R, false));
  if (idx->snap) {
    A(alloc_dev(idx, &idx->adj_alt, (size_t)cap * R, false));
    A(alloc_dev(idx, &idx->sync_ids, mb, false));
  }
  A(alloc_dev(idx, &idx->deg, cap, true));
  A(alloc_dev(idx, &idx->live, words, true));
  A(alloc_dev(idx, &idx->rowpfx, cap, true));
  if (idx->mode == GRAND_MODE_VAMANA) A(alloc_dev(idx, &idx->rowd, (size_t)cap * R, false));
  A(alloc_dev(idx, &idx->d_state, 1, true));
  A(alloc_dev(idx, &idx->mark, words, true));
  A(alloc_dev(idx, &idx->cnt, cap, true));
  A(alloc_dev(idx, &idx->fill, cap, true));
  A(alloc_dev(idx, &idx->start, cap, true));
  A(alloc_dev(idx, &idx->flag, cap, true));
  if (idx->mode == GRAND_MODE_FIXED_DEGREE) A(alloc_dev(idx, &idx->slot_of, cap, true));
  idx->wk_stride = idx->vmax > L ? idx->vmax : L;
  A(alloc_dev(idx, &idx->wk_keys, (size_t)mb * idx->wk_stride, false));
  A(alloc_dev(idx, &idx->wk_n, mb, true));
  A(alloc_dev(idx, &idx->Ci, (size_t)mb * idx->k_repair, false));
  A(alloc_dev(idx, &idx->Ci_n, mb, true));
  A(alloc_dev(idx, &idx->in_cnt, mb + 1, true));
  A(alloc_dev(idx, &idx->pair_off, mb + 1, true));
  A(alloc_dev(idx, &idx->unit_off, mb + 1, true));
  A(alloc_dev(idx, &idx->scan_tmp, (cap + 1) / 2048 + mb / 2048 + 8, true));
  A(alloc_dev(idx, &idx->mean_row, lay.row_bytes, true));
  A(alloc_dev(idx, &idx->pair_count, 1, true));
  if (idx->approx) {
    A(alloc_dev(idx, &idx->vis_keys, (size_t)mb * idx->vmax, false));
    A(alloc_dev(idx, &idx->vis_n, mb, true));
    A(alloc_dev(idx, &idx->vis_in, (size_t)mb * idx->vmax, false));
    A(alloc_dev(idx, &idx->birth, cap, true));
    A(alloc_dev(idx, &idx->rowepoch, cap, true));
  }
  A(alloc_dev(idx, &idx->search_ctrs, 1 + grand_index::kCtrSlots, true));
  if (rc == GRAND_OK && cudaMemset(idx->adj, 0xFF, (size_t)cap * R * 4) != cudaSuccess) rc = GRAND_ERR_CUDA;
  if (rc == GRAND_OK && idx->snap && cudaMemset(idx->adj_alt, 0xFF, (size_t)cap * R * 4) != cudaSuccess) rc = GRAND_ERR_CUDA;
  if (rc == GRAND_OK && idx->rowd && cudaMemset(idx->rowd, 0xFF, (size_t)cap * R * 4) != cudaSuccess) rc = GRAND_ERR_CUDA;
  if (rc == GRAND_OK && cudaMallocHost(&idx->h_state, sizeof(DevState)) != cudaSuccess) rc = GRAND_ERR_CUDA;
  if (rc == GRAND_OK) {
    memset(idx->h_state, 0, sizeof(DevState));
    idx->h_state->entry = GRAND_INVALID_ID;
    if (cudaMemcpy(idx->d_state, idx->h_state, sizeof(DevState), cudaMemcpyHostToDevice) != cudaSuccess) rc = GRAND_ERR_CUDA;
  }
  // everything an update batch can need is allocated here: no allocation happens on the update path
  if (rc == GRAND_OK) rc = ensure_requests(idx, idx->max_requests, 0);
  if (rc == GRAND_OK && idx->snap) rc = ensure(idx, idx->sync_dirty, idx->max_requests * 4, 0);  // trades places with `dirty`
  if (rc == GRAND_OK) rc = ensure(idx, idx->t_indeg, (cap + 1) * 4, 0);
  if (rc == GRAND_OK) rc = ensure(idx, idx->t_off, (cap + 1) * 4, 0);
  if (rc == GRAND_OK) rc = ensure(idx, idx->t_fill, cap * 4, 0);
  if (rc == GRAND_OK) rc = ensure(idx, idx->t_src, (idx->full_transpose ? cap * R : idx->max_delete_edges) * 4, 0);
  if (rc == GRAND_OK) rc = ensure(idx, idx->st_ids, mb * 4, 0);
  if (rc == GRAND_OK) rc = ensure(idx, idx->st_vecs, mb * (size_t)lay.udim * lay.esize, 0);
  for (int i = 0; rc == GRAND_OK && i < grand_index::kCtrSlots; ++i)
    if (cudaEventCreateWithFlags(&idx->ctr_done[i], cudaEventDisableTiming) != cudaSuccess) rc = GRAND_ERR_CUDA;
  if (rc != GRAND_OK) {
    grand_destroy(idx);
    return rc;
  }
  *out = idx;
  return GRAND_OK;
}

int grand_destroy(grand_index* idx) {
  if (!idx) return GRAND_OK;
  cudaDeviceSynchronize();
  for (void* p : idx->owned) idx->dev_free(p, idx->user);
  for (Buf* b : {&idx->req_tgt, &idx->req_key, &idx->seg_keys, &idx->dirty, &idx->work, &idx->sync_dirty, &idx->t_indeg, &idx->t_off, &idx->t_fill, &idx->t_src,
                 &idx->x_indeg, &idx->x_off, &idx->x_fill, &idx->x_src, &idx->st_ids, &idx->st_vecs, &idx->st_out_ids, &idx->st_out_d})
    if (b->p) idx->dev_free(b->p, idx->user);
  for (auto e : idx->ctr_done)
    if (e) cudaEventDestroy(e);
  if (idx->h_state) cudaFreeHost(idx->h_state);
  for (auto e : idx->ev_pool) cudaEventDestroy(e);
  for (auto e : idx->reader_pool) cudaEventDestroy(e);
  for (auto& rd : idx->readers) for (auto e : rd) cudaEventDestroy(e);
  delete idx;
  return GRAND_OK;
}

// Vamana mode (exact delete): the dirty list is split into nodes that need the full rebuild and nodes whose row
// cannot overflow; the rebuild then reads the split list.
static void split_group_args(const grand_index* idx, GroupArgs& a) {
  if (!idx->work.p) return;
  a.work = (uint32_t*)idx->work.p;
  a.work_cap = (uint32_t)(idx->work.bytes / 4);
  a.light_max = 8;
  a.deg = idx->deg;
  a.R = idx->R;
}
static void split_rebuild_args(const grand_index* idx, RebuildArgs& a) {
  if (!idx->work.p) return;
  a.dirty = (const uint32_t*)idx->work.p;
  a.split = 1;
  a.dirty_cap = (uint32_t)(idx->work.bytes / 4);
}

// An update call that gives up after validation has marked its ids: clear the marks, drain the stream, report.
// Nothing of the index has been changed at the points where this is used, or the failure is a CUDA error.
static int abandon_batch(grand_index* idx, const uint32_t* ids, uint64_t n, cudaStream_t s, int code, const std::string& msg) {
  launch_clear_marks(ids, n, idx->cap, idx->mark, s);
  cudaStreamSynchronize(s);
  collect_spans(idx);
  return fail(idx, code, msg);
}
#define CKB(call)                                                                                           \
  do {                                                                                                      \
    cudaError_t e__ = (call);                                                                               \
    if (e__ != cudaSuccess)                                                                                 \
      return abandon_batch(idx, ids, n, s, GRAND_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__)); \
  } while (0)

int grand_insert_batch(grand_index* idx, const uint32_t* ids, const void* vecs, uint64_t n, grand_stream stream) {
  if (!idx || (n && (!ids || !vecs))) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (n == 0) return GRAND_OK;
  if (n > idx->max_batch) return fail(idx, GRAND_ERR_CAPACITY, "batch larger than max_batch");
  LaunchScope scope(&idx->launches);
  cudaStream_t s = (cudaStream_t)stream;
  const bool fixed = idx->mode == GRAND_MODE_FIXED_DEGREE;
  const uint32_t R = idx->R;
  int rc;
  if ((rc = write_state_head(idx, s))) return rc;
  {
    PhaseTimer pt(idx, s, PH_OTHER);
    CKB(launch_validate(ids, n, idx->cap, idx->live, idx->mark, 0, idx->d_state, s));
    if (idx->mips) CKB(launch_check_norms(idx->lay, vecs, n, idx->mips_M2, idx->d_state, s));
  }
  if ((rc = read_state(idx, s))) return abandon_batch(idx, ids, n, s, rc, idx->last_error);
  if (idx->h_state->status != 0) return abandon_batch(idx, ids, n, s, idx->h_state->status, grand_strerror(idx->h_state->status));
  if ((rc = begin_update(idx, ids, n, s))) return abandon_batch(idx, ids, n, s, rc, idx->last_error);
  ++idx->epoch;
  GraphView g = view(idx, true);
  {
    PhaseTimer pt(idx, s, PH_OTHER);
    CKB(launch_store_write(idx->lay, idx->store, idx->deg, idx->slot_of, ids, vecs, n, s));
    if (idx->mips) CKB(launch_augment_rows(idx->lay, idx->store, ids, n, idx->mips_M2, s));
  }
  const bool bootstrap = idx->nlive == 0;
  {
    // forward candidates: snapshot search (Alg. 5: visited list; Alg. 7: worklist) or bootstrap scan
    PhaseTimer pt(idx, s, PH_SEARCH);
    SearchArgs a = search_args(idx, s, true);
    a.qids = ids;
    a.nq = n;
    a.L = idx->L;
    a.vmax = idx->vmax;
    if (bootstrap) {
      a.boot_ids = ids;
      a.boot_n = (uint32_t)n;
      a.out_vis = idx->wk_keys; a.out_vis_n = idx->wk_n; a.vis_stride = idx->wk_stride;
    } else if (fixed) {
      a.out_beam = idx->wk_keys; a.out_beam_n = idx->wk_n; a.beam_stride = idx->wk_stride;
    } else {
      a.out_vis = idx->wk_keys; a.out_vis_n = idx->wk_n; a.vis_stride = idx->wk_stride;
    }
    CKB(launch_beam_search(a, s));
    idx->stats.n_search_launches++;
  }
  {
    PhaseTimer pt(idx, s, PH_PRUNE);
    PruneArgs a{};
    a.lay = idx->lay; a.g = g; a.A_fix = idx->A_fix; a.alpha = idx->alpha;
    a.ids = ids; a.n = n;
    a.cand = idx->wk_keys; a.cand_n = idx->wk_n; a.cand_stride = idx->wk_stride;
    a.fixed_mode = fixed;
    a.req_tgt = (uint32_t*)idx->req_tgt.p; a.req_key = (unsigned long long*)idx->req_key.p;
    a.state = idx->d_state;
    CKB(launch_forward_prune(a, s));
    idx->stats.n_prune_launches++;
  }
  {
    PhaseTimer pt(idx, s, PH_GROUP);
    GroupArgs a{};
    a.req_tgt = (uint32_t*)idx->req_tgt.p; a.req_key = (unsigned long long*)idx->req_key.p; a.nreq = n * R;
    a.cnt = idx->cnt; a.fill = idx->fill; a.start = idx->start; a.flag = idx->flag;
    a.dirty = (uint32_t*)idx->dirty.p; a.seg_keys = (unsigned long long*)idx->seg_keys.p; a.state = idx->d_state;
    split_group_args(idx, a);
    CKB(launch_group_requests(a, s));
  }
  {
    PhaseTimer pt(idx, s, PH_REBUILD);
    const uint64_t most = (uint64_t)sm_count() * 16u;
    const uint64_t mbk = n * R < most ? n * R : most;
    if (fixed) {
      FixedReverseArgs a{};
      a.g = g; a.slot_of = idx->slot_of; a.fwd_rows = (uint32_t*)idx->req_tgt.p;
      a.cnt = idx->cnt; a.fill = idx->fill; a.start = idx->start; a.flag = idx->flag;
      a.dirty = (uint32_t*)idx->dirty.p; a.seg_keys = (unsigned long long*)idx->seg_keys.p;
      a.max_blocks = (uint32_t)mbk; a.state = idx->d_state;
      CKB(launch_fixed_reverse(a, s));
    } else {
      RebuildArgs a{};
      a.lay = idx->lay; a.g = g; a.A_fix = idx->A_fix; a.alpha = idx->alpha; a.P = idx->P; a.delmap = nullptr;
      if (idx->approx) { a.livemap = idx->live; a.newmap = idx->mark; }  // rows may hold dangling edges: drop them
      a.cnt = idx->cnt; a.fill = idx->fill; a.start = idx->start; a.flag = idx->flag;
      a.dirty = (uint32_t*)idx->dirty.p; a.seg_keys = (unsigned long long*)idx->seg_keys.p;
      a.max_blocks = (uint32_t)mbk; a.state = idx->d_state;
      split_rebuild_args(idx, a);
      CKB(launch_rebuild(a, s));
      idx->stats.n_rebuild_launches++;
    }
  }
  {
    PhaseTimer pt(idx, s, PH_OTHER);
    CKB(launch_publish(ids, n, idx->live, idx->mark, idx->d_state, s));
    if (idx->entry == GRAND_INVALID_ID) CKB(launch_pick_medoid(idx->lay, g, ids, n, idx->mean_row, idx->d_state, s));
  }
  if ((rc = read_state(idx, s))) return rc;
  collect_spans(idx);
  end_update(idx, n);
  if (idx->h_state->status != 0) return fail(idx, idx->h_state->status, grand_strerror(idx->h_state->status));
  return GRAND_OK;
}

// Reverse graph of the current adjacency (Alg. 8, first loops).  heads != nullptr: only the rows of the marked nodes,
// into the buffers sized at creation (an update batch); heads == nullptr and !work: the whole graph for
// grand_reverse_graph, into buffers that grow on demand (introspection is the only caller that may allocate).
static int build_reverse(grand_index* idx, bool sort_rows, const uint32_t* heads, bool work, bool introspection, cudaStream_t s) {
  int rc;
  const uint64_t cap = idx->cap;
  Buf *indeg = &idx->t_indeg, *off = &idx->t_off, *fillc = &idx->t_fill, *src = &idx->t_src;
  if (introspection) {
    indeg = &idx->x_indeg; off = &idx->x_off; fillc = &idx->x_fill; src = &idx->x_src;
    if ((rc = ensure(idx, *indeg, (cap + 1) * 4, s))) return rc;
    if ((rc = ensure(idx, *off, (cap + 1) * 4, s))) return rc;
    if ((rc = ensure(idx, *fillc, cap * 4, s))) return rc;
    if ((rc = ensure(idx, *src, cap * idx->R * 4, s))) return rc;
  }
  TransposeArgs t{};
  t.g = view(idx, work);
  t.indeg = (uint32_t*)indeg->p; t.off = (uint32_t*)off->p; t.fillc = (uint32_t*)fillc->p;
  t.src = (uint32_t*)src->p; t.scan_tmp = idx->scan_tmp; t.sort_rows = sort_rows; t.heads = heads;
  t.src_capacity = src->bytes / 4;
  if (!introspection && heads && !sort_rows) {
    // the request buffer is idle until the picks are written: it holds the batch's marked edges meanwhile
    t.pairs = (unsigned long long*)idx->req_key.p; t.pairs_capacity = idx->req_key.bytes / 8; t.pair_count = idx->pair_count;
  }
  CK(launch_transpose(t, s));
  return GRAND_OK;
}

int grand_delete_batch(grand_index* idx, const uint32_t* ids, uint64_t n, grand_stream stream) {
  if (!idx || (n && !ids)) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (n == 0) return GRAND_OK;
  if (n > idx->max_batch) return fail(idx, GRAND_ERR_CAPACITY, "batch larger than max_batch");
  LaunchScope scope(&idx->launches);
  cudaStream_t s = (cudaStream_t)stream;
  const bool fixed = idx->mode == GRAND_MODE_FIXED_DEGREE;
  const uint32_t R = idx->R;
  int rc;
  if ((rc = write_state_head(idx, s))) return rc;
  {
    PhaseTimer pt(idx, s, PH_OTHER);
    CKB(launch_validate(ids, n, idx->cap, idx->live, idx->mark, 1, idx->d_state, s));
  }
  // (the status of the validation is read back together with the in-degree total below: what runs in between
  // only reads the graph and writes scratch, and skips ids beyond the capacity)
  if ((rc = begin_update(idx, ids, n, s))) return abandon_batch(idx, ids, n, s, rc, idx->last_error);
  ++idx->epoch;
  GraphView g = view(idx, true);
  DeleteArgs d{};
  d.lay = idx->lay; d.g = g; d.ids = ids; d.n = n; d.delmap = idx->mark;
  d.beam = idx->wk_keys; d.beam_n = idx->wk_n; d.beam_stride = idx->wk_stride;
  d.Ci = idx->Ci; d.Ci_n = idx->Ci_n; d.k_repair = idx->k_repair; d.c = idx->c;
  d.in_cnt = idx->in_cnt; d.pair_off = idx->pair_off; d.unit_off = idx->unit_off; d.scan_tmp = idx->scan_tmp;
  d.flag = idx->flag; d.state = idx->d_state;
  const bool approx = idx->approx && !fixed;
  if (!approx) {
    // reverse graph of the snapshot: exact in-neighbours, rebuilt per batch and not kept
    PhaseTimer pt(idx, s, PH_TRANSPOSE);
    // only the in-neighbour rows of the batch are read below, so only those are materialised
    if ((rc = build_reverse(idx, false, idx->full_transpose ? nullptr : idx->mark, true, false, s)))
      return abandon_batch(idx, ids, n, s, rc, idx->last_error);
    idx->stats.n_transpose_launches++;
    d.off = (uint32_t*)idx->t_off.p; d.src = (uint32_t*)idx->t_src.p;
    CKB(launch_delete_prepare(d, s));
  }
  if ((rc = read_state(idx, s))) return abandon_batch(idx, ids, n, s, rc, idx->last_error);
  if (idx->h_state->status != 0) return abandon_batch(idx, ids, n, s, idx->h_state->status, grand_strerror(idx->h_state->status));
  if (approx) {
    // Alg. 6 as printed: the searches come first, their visited sets are the only place where
    // in-neighbours are looked for
    {
      PhaseTimer pt(idx, s, PH_SEARCH);
      SearchArgs a = search_args(idx, s, true);
      a.qids = ids; a.nq = n; a.L = idx->L; a.vmax = idx->vmax;
      a.out_beam = idx->wk_keys; a.out_beam_n = idx->wk_n; a.beam_stride = idx->wk_stride;
      a.out_vis = idx->vis_keys; a.out_vis_n = idx->vis_n; a.vis_stride = idx->vmax;
      CKB(launch_beam_search(a, s));
      idx->stats.n_search_launches++;
    }
    {
      PhaseTimer pt(idx, s, PH_TRANSPOSE);
      d.vis = idx->vis_keys; d.vis_n = idx->vis_n; d.vis_stride = idx->vmax;
      d.src = idx->vis_in; d.src_stride = idx->vmax; d.livemap = idx->live;
      CKB(launch_delete_visited_in(d, idx->vis_in, s));
    }
    if ((rc = read_state(idx, s))) return abandon_batch(idx, ids, n, s, rc, idx->last_error);
  }
  const uint64_t total_in = idx->h_state->total_in;
  const uint64_t nreq = fixed ? total_in + 1 : (total_in + n * R) * idx->c;
  // nothing of the index has been written so far: a batch that touches more edges than the workspace was sized
  // for is refused as a whole
  if (total_in > idx->max_delete_edges || nreq > idx->max_requests)
    return abandon_batch(idx, ids, n, s, GRAND_ERR_CAPACITY,
                         "delete batch touches " + std::to_string(total_in) + " in-neighbour entries; the workspace holds " +
                             std::to_string(idx->max_delete_edges) + " (option max_delete_edges)");
  d.req_tgt = (uint32_t*)idx->req_tgt.p; d.req_key = (unsigned long long*)idx->req_key.p; d.dirty = (uint32_t*)idx->dirty.p;
  d.unit_owner = (uint32_t*)idx->seg_keys.p;  // the grouped-request buffer is idle until the picks have been written
  if (fixed) {
    PhaseTimer pt(idx, s, PH_REBUILD);
    FixedDeleteArgs f{};
    f.g = g; f.ids = ids; f.n = n; f.delmap = idx->mark; f.off = d.off; f.src = (uint32_t*)idx->t_src.p; f.pair_off = idx->pair_off;
    f.flag = idx->flag; f.dirty = (uint32_t*)idx->dirty.p; f.state = idx->d_state;
    CKB(launch_fixed_delete(f, total_in, s));
  } else {
    if (!approx) {
      PhaseTimer pt(idx, s, PH_SEARCH);
      SearchArgs a = search_args(idx, s, true);
      a.qids = ids; a.nq = n; a.L = idx->L; a.vmax = idx->vmax;
      a.out_beam = idx->wk_keys; a.out_beam_n = idx->wk_n; a.beam_stride = idx->wk_stride;
      CKB(launch_beam_search(a, s));
      idx->stats.n_search_launches++;
    }
    {
      PhaseTimer pt(idx, s, PH_GROUP);  // set-up of the picks: C_i, dirty marks of the in-neighbours, work units
      CKB(launch_delete_ci(d, s));
      CKB(launch_delete_picks_prepare(d, total_in, s));
    }
    {
      PhaseTimer pt(idx, s, PH_PICKS);
      CKB(launch_delete_picks(d, total_in, s));
      idx->stats.n_picks_launches++;
    }
    {
      PhaseTimer pt(idx, s, PH_GROUP);
      GroupArgs a{};
      a.req_tgt = d.req_tgt; a.req_key = d.req_key; a.nreq = nreq;
      a.cnt = idx->cnt; a.fill = idx->fill; a.start = idx->start; a.flag = idx->flag;
      a.dirty = d.dirty; a.seg_keys = (unsigned long long*)idx->seg_keys.p; a.state = idx->d_state;
      split_group_args(idx, a);
      CKB(launch_group_requests(a, s));
    }
    {
      PhaseTimer pt(idx, s, PH_REBUILD);
      RebuildArgs a{};
      a.lay = idx->lay; a.g = g; a.A_fix = idx->A_fix; a.alpha = idx->alpha; a.P = idx->P; a.delmap = idx->mark;
      if (approx) a.livemap = idx->live;
      a.cnt = idx->cnt; a.fill = idx->fill; a.start = idx->start; a.flag = idx->flag;
      a.dirty = d.dirty; a.seg_keys = (unsigned long long*)idx->seg_keys.p;
      const uint64_t most = (uint64_t)sm_count() * 16u;
      a.max_blocks = (uint32_t)(nreq < most ? nreq : most); a.state = idx->d_state;
      split_rebuild_args(idx, a);
      CKB(launch_rebuild(a, s));
      idx->stats.n_rebuild_launches++;
    }
  }
  {
    PhaseTimer pt(idx, s, PH_OTHER);
    CKB(launch_retire(g, ids, n, idx->mark, idx->Ci, idx->Ci_n, idx->k_repair, fixed, idx->d_state, s));
  }
  if ((rc = read_state(idx, s))) return rc;
  collect_spans(idx);
  end_update(idx, n);
  if (idx->h_state->status != 0) return fail(idx, idx->h_state->status, grand_strerror(idx->h_state->status));
  return GRAND_OK;
}

int grand_search(const grand_index* cidx, const void* queries, uint64_t nq, uint32_t k, uint32_t L, uint32_t* out_ids,
                 void* out_dists, grand_stream stream) {
  grand_index* idx = const_cast<grand_index*>(cidx);
  if (!idx || (nq && (!queries || !out_ids))) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (k == 0 || k > L || L > GRAND_MAX_L) return fail(idx, GRAND_ERR_INVALID_ARG, "need 1 <= k <= L <= GRAND_MAX_L");
  if (nq == 0) return GRAND_OK;
  cudaStream_t s = (cudaStream_t)stream;
  {
    // the lock keeps the choice of the published buffer, the launch and the registration of the launch's end
    // as a reader of that buffer together (an update batch on another host thread may publish at any time)
    std::lock_guard<std::mutex> lk(idx->pub_mu);
    LaunchScope scope(&idx->launches);
    PhaseTimer pt(idx, s, PH_SEARCH);
    const int slot = take_ctr_slot(idx);
    SearchArgs a = search_args(idx, s, false, slot);
    a.queries = queries; a.nq = nq; a.L = L; a.vmax = 2 * L; a.k = k;
    a.out_ids = out_ids; a.out_dists = out_dists;
    CK(launch_beam_search(a, s));
    if (slot >= 0) CK(cudaEventRecord(idx->ctr_done[slot], s));
    idx->stats.n_search_launches++;
    if (idx->snap) {
      std::vector<cudaEvent_t>& rd = idx->readers[idx->pub];
      if (rd.size() >= 256) {  // searches only, no update in between: recycle the events that have completed
        size_t w = 0;
        for (cudaEvent_t ev : rd) {
          if (cudaEventQuery(ev) == cudaSuccess) idx->reader_pool.push_back(ev);
          else rd[w++] = ev;
        }
        rd.resize(w);
      }
      cudaEvent_t ev = nullptr;
      if (!idx->reader_pool.empty()) {
        ev = idx->reader_pool.back();
        idx->reader_pool.pop_back();
      } else {
        CK(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
      }
      CK(cudaEventRecord(ev, s));
      rd.push_back(ev);
    }
  }
  if (idx->profiling) {
    CK(cudaStreamSynchronize(s));
    collect_spans(idx);
  }
  return GRAND_OK;
}

// ---- host-buffer variants: copies inside the call
int grand_insert_batch_host(grand_index* idx, const uint32_t* ids, const void* vecs, uint64_t n, grand_stream stream) {
  if (!idx || (n && (!ids || !vecs))) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (n == 0) return GRAND_OK;
  if (n > idx->max_batch) return fail(idx, GRAND_ERR_CAPACITY, "batch larger than max_batch");
  cudaStream_t s = (cudaStream_t)stream;
  int rc;
  const size_t vb = (size_t)n * idx->lay.udim * idx->lay.esize;
  if ((rc = ensure(idx, idx->st_ids, n * 4, s))) return rc;  // (sized for max_batch at creation: no allocation here)
  if ((rc = ensure(idx, idx->st_vecs, vb, s))) return rc;
  CK(cudaMemcpyAsync(idx->st_ids.p, ids, n * 4, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(idx->st_vecs.p, vecs, vb, cudaMemcpyHostToDevice, s));
  return grand_insert_batch(idx, (const uint32_t*)idx->st_ids.p, idx->st_vecs.p, n, stream);
}
int grand_delete_batch_host(grand_index* idx, const uint32_t* ids, uint64_t n, grand_stream stream) {
  if (!idx || (n && !ids)) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (n == 0) return GRAND_OK;
  if (n > idx->max_batch) return fail(idx, GRAND_ERR_CAPACITY, "batch larger than max_batch");
  cudaStream_t s = (cudaStream_t)stream;
  int rc;
  if ((rc = ensure(idx, idx->st_ids, n * 4, s))) return rc;
  CK(cudaMemcpyAsync(idx->st_ids.p, ids, n * 4, cudaMemcpyHostToDevice, s));
  return grand_delete_batch(idx, (const uint32_t*)idx->st_ids.p, n, stream);
}
int grand_search_host(grand_index* idx, const void* queries, uint64_t nq, uint32_t k, uint32_t L, uint32_t* out_ids,
                      void* out_dists, grand_stream stream) {
  if (!idx || (nq && (!queries || !out_ids))) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  if (nq == 0) return GRAND_OK;
  cudaStream_t s = (cudaStream_t)stream;
  int rc;
  const size_t qb = (size_t)nq * idx->lay.udim * idx->lay.esize;
  if ((rc = ensure(idx, idx->st_vecs, qb, s))) return rc;
  if ((rc = ensure(idx, idx->st_out_ids, nq * k * 4, s))) return rc;
  if ((rc = ensure(idx, idx->st_out_d, nq * k * 4, s))) return rc;
  CK(cudaMemcpyAsync(idx->st_vecs.p, queries, qb, cudaMemcpyHostToDevice, s));
  if ((rc = grand_search(idx, idx->st_vecs.p, nq, k, L, (uint32_t*)idx->st_out_ids.p, idx->st_out_d.p, stream))) return rc;
  CK(cudaMemcpyAsync(out_ids, idx->st_out_ids.p, nq * k * 4, cudaMemcpyDeviceToHost, s));
  if (out_dists) CK(cudaMemcpyAsync(out_dists, idx->st_out_d.p, nq * k * 4, cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  return GRAND_OK;
}

// ---- introspection
int grand_export_graph(const grand_index* idx, uint32_t* adj, uint32_t* deg, uint32_t* live, uint32_t* entry_out, grand_stream stream) {
  if (!idx) return GRAND_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (adj) CK(cudaMemcpyAsync(adj, adj_of(idx, false), (size_t)idx->cap * idx->R * 4, cudaMemcpyDeviceToDevice, s));
  if (deg) CK(cudaMemcpyAsync(deg, idx->deg, idx->cap * 4, cudaMemcpyDeviceToDevice, s));
  if (live) CK(cudaMemcpyAsync(live, idx->live, (idx->cap + 31) / 32 * 4, cudaMemcpyDeviceToDevice, s));
  if (entry_out) *entry_out = idx->entry;
  return GRAND_OK;
}
int grand_import_graph(grand_index* idx, const uint32_t* adj, const uint32_t* deg, const uint32_t* live, uint32_t entry,
                       const void* vecs, grand_stream stream) {
  if (!idx || !adj || !deg || !live || !vecs) return fail(idx, GRAND_ERR_INVALID_ARG, "null argument");
  cudaStream_t s = (cudaStream_t)stream;
  LaunchScope scope(&idx->launches);
  int rc;
  // the caller's graph is checked before anything is replaced: degrees <= R, listed neighbour ids < capacity
  if ((rc = write_state_head(idx, s))) return rc;
  CK(launch_check_graph(adj, deg, idx->cap, idx->R, idx->d_state, s));
  if ((rc = read_state(idx, s))) return rc;
  if (idx->h_state->status != 0) return fail(idx, GRAND_ERR_INVALID_ARG, "imported graph: a degree above R or a neighbour id beyond the capacity");
  CK(cudaMemcpyAsync(idx->adj, adj, (size_t)idx->cap * idx->R * 4, cudaMemcpyDeviceToDevice, s));
  idx->sync_n = idx->sync_ndirty = 0;  // both buffers are rewritten below
  CK(cudaMemcpyAsync(idx->deg, deg, idx->cap * 4, cudaMemcpyDeviceToDevice, s));
  CK(cudaMemcpyAsync(idx->live, live, (idx->cap + 31) / 32 * 4, cudaMemcpyDeviceToDevice, s));
  CK(launch_pad_rows(idx->lay, idx->store, vecs, idx->cap, s));
  if (idx->mips) CK(launch_augment_rows(idx->lay, idx->store, nullptr, idx->cap, idx->mips_M2, s));
  CK(cudaMemsetAsync(idx->rowpfx, 0, idx->cap, s));
  if (idx->birth) {
    CK(cudaMemsetAsync(idx->birth, 0, idx->cap * 4, s));
    CK(cudaMemsetAsync(idx->rowepoch, 0, idx->cap * 4, s));
  }
  if (idx->rowd) CK(cudaMemsetAsync(idx->rowd, 0xFF, (size_t)idx->cap * idx->R * 4, s));
  CK(launch_pad_adjacency(idx->adj, idx->deg, idx->cap, idx->R, s));
  if (idx->snap) CK(cudaMemcpyAsync(idx->adj_alt, idx->adj, (size_t)idx->cap * idx->R * 4, cudaMemcpyDeviceToDevice, s));
  idx->entry = entry;
  idx->nlive = 0;
  if ((rc = write_state_head(idx, s))) return rc;
  CK(launch_count_live(idx->live, idx->cap, idx->d_state, s));
  if ((rc = read_state(idx, s))) return rc;
  idx->nlive = idx->h_state->nlive;
  return GRAND_OK;
}
int grand_reverse_graph(grand_index* idx, uint32_t* off, uint32_t* src, uint64_t* E_out, grand_stream stream) {
  if (!idx) return GRAND_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  LaunchScope scope(&idx->launches);
  int rc;
  if ((rc = build_reverse(idx, true, nullptr, false, true, s))) return rc;
  uint32_t E = 0;
  CK(cudaMemcpyAsync(&E, (uint32_t*)idx->x_off.p + idx->cap, 4, cudaMemcpyDeviceToHost, s));
  CK(cudaStreamSynchronize(s));
  if (off) CK(cudaMemcpyAsync(off, idx->x_off.p, (idx->cap + 1) * 4, cudaMemcpyDeviceToDevice, s));
  if (src && E) CK(cudaMemcpyAsync(src, idx->x_src.p, (size_t)E * 4, cudaMemcpyDeviceToDevice, s));
  if (E_out) *E_out = E;
  CK(cudaStreamSynchronize(s));
  return GRAND_OK;
}

int grand_get_entry(const grand_index* idx, uint32_t* e) {
  if (!idx || !e) return GRAND_ERR_INVALID_ARG;
  *e = idx->entry;
  return GRAND_OK;
}
int grand_set_entry(grand_index* idx, uint32_t e) {
  if (!idx || (e != GRAND_INVALID_ID && e >= idx->cap)) return GRAND_ERR_INVALID_ARG;
  idx->entry = e;
  return GRAND_OK;
}
int grand_live_count(const grand_index* idx, uint64_t* n) {
  if (!idx || !n) return GRAND_ERR_INVALID_ARG;
  *n = idx->nlive;
  return GRAND_OK;
}
int grand_row_bytes(const grand_index* idx, uint32_t* rb) {
  if (!idx || !rb) return GRAND_ERR_INVALID_ARG;
  *rb = idx->lay.row_bytes;
  return GRAND_OK;
}

int grand_get_stats(const grand_index* cidx, grand_stats* out) {
  grand_index* idx = const_cast<grand_index*>(cidx);
  if (!idx || !out) return GRAND_ERR_INVALID_ARG;
  DevState st;
  CK(cudaMemcpy(&st, idx->d_state, sizeof(DevState), cudaMemcpyDeviceToHost));
  idx->stats.expansions = st.counters[CTR_EXP];
  idx->stats.dist_evals = st.counters[CTR_DIST];
  idx->stats.pair_dists = st.counters[CTR_PAIR];
  idx->stats.dirty_nodes = st.counters[CTR_DIRTY];
  idx->stats.prunes = st.counters[CTR_PRUNE];
  idx->stats.requests = st.counters[CTR_REQ];
  idx->stats.rebuild_bytes = st.counters[CTR_RB_BYTES];
  idx->stats.picks_bytes = st.counters[CTR_PK_BYTES];
  idx->stats.prune_bytes = st.counters[CTR_FP_BYTES];
  idx->stats.rebuild_prunes = st.counters[CTR_RB_PRUNED];
  idx->stats.picks_pair_dists = st.counters[CTR_PK_PAIRS];
  idx->stats.prune_pair_dists = st.counters[CTR_FP_PAIRS];
  idx->stats.kernel_launches = idx->launches;
  *out = idx->stats;
  return GRAND_OK;
}
int grand_reset_stats(grand_index* idx) {
  if (!idx) return GRAND_ERR_INVALID_ARG;
  CK(cudaMemset(idx->d_state->counters, 0, sizeof(idx->d_state->counters)));
  idx->stats = grand_stats{};  // (kernel_launches is refilled from the handle's running count)
  return GRAND_OK;
}
int grand_set_profiling(grand_index* idx, int on) {
  if (!idx) return GRAND_ERR_INVALID_ARG;
  idx->profiling = on != 0;
  return GRAND_OK;
}

}  // extern "C"
