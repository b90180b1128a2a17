// grand_reverse_graph_noalloc: the CSR reverse graph of a caller-supplied adjacency array, for
// callers that must not allocate device memory.
//
// Who needs this.  Some hosts hand the GPU to a runtime that fixes its memory plan at start-up:
// a serving process whose allocator has already carved up all of HBM, a sandboxed plug-in that is
// forbidden to call the driver's allocator, or a real-time loop that cannot afford the implicit
// device synchronisation and the possible failure of cudaMalloc in the middle of a request.  The
// regular entry point (grand_reverse_graph) grows a workspace pool through the index handle;
// this one touches no allocator at all.  Its only working memory (the per-node fill cursors of
// the scatter pass and the block sums of the scan) lives in one file-scope device array of fixed
// size that every GPU loading this library carries until the process exits
// (GRAND_NOALLOC_SCRATCH_BYTES, about 4.2 MB).  Inputs and outputs are the caller's.
//
// Consequences the caller must know:
//  * graphs with more than GRAND_NOALLOC_MAX_NODES nodes are rejected (GRAND_ERR_CAPACITY);
//  * all calls on one device share that array.  It still holds the previous call's values, so
//    everything that must start from zero is cleared inside each call; two calls whose work
//    overlaps on the GPU (different streams, or different host threads) race on it and corrupt
//    each other's result -- serialise them;
//  * the first call on each device looks the array's device address up (cudaGetSymbolAddress) and
//    caches it.  Make that first call during set-up, before any stream capture begins.
//
// In host code the array's name is only a handle for the runtime, not a device address, which is
// why the address is resolved explicitly and handed to the kernels as a pointer.
#include <mutex>

#include "../../include/grand.h"
#include "grand_kernels.h"

namespace {

constexpr uint64_t kMaxNodes = GRAND_NOALLOC_MAX_NODES;
constexpr uint64_t kScanWords = kMaxNodes / 2048 + 8;           // block sums of the exclusive scan
constexpr uint64_t kScratchWords = kMaxNodes + kScanWords + 1;  // fill cursors + scan sums + one "bad id" flag
static_assert(kScratchWords * 4 <= GRAND_NOALLOC_SCRATCH_BYTES, "scratch array smaller than its users need");

static __device__ __align__(256) uint32_t g_noalloc_scratch[GRAND_NOALLOC_SCRATCH_BYTES / 4];

constexpr int kMaxDevices = 64;
uint32_t* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (resolved once per device).
cudaError_t scratch_for_current_device(uint32_t** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    uint32_t* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int grand_reverse_graph_noalloc(const uint32_t* adj_dev, const uint32_t* deg_dev, uint64_t n_nodes, uint32_t R,
                                           uint32_t* off_dev, uint32_t* src_dev, uint64_t src_capacity,
                                           uint64_t* E_out_host, grand_stream stream) {
  if (!adj_dev || !deg_dev || !off_dev || n_nodes == 0 || R == 0 || R > GRAND_MAX_R) return GRAND_ERR_INVALID_ARG;
  if (n_nodes > kMaxNodes) return GRAND_ERR_CAPACITY;  // the fixed scratch array cannot hold more fill cursors
  cudaStream_t s = (cudaStream_t)stream;
  uint32_t* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return GRAND_ERR_CUDA;

  // The offsets array doubles as the in-degree histogram (the scan runs in place), so the only
  // scratch is the fill-cursor array and the scan's block sums.  launch_transpose clears the
  // histogram and the cursors itself; nothing of the previous call survives into this one.
  grand::TransposeArgs t{};
  t.g.store = nullptr;
  t.g.adj = const_cast<uint32_t*>(adj_dev);
  t.g.deg = const_cast<uint32_t*>(deg_dev);
  t.g.live = nullptr;
  t.g.rowpfx = nullptr;
  t.g.R = R;
  t.g.cap = n_nodes;
  t.indeg = off_dev;
  t.off = off_dev;
  t.fillc = scratch;
  t.scan_tmp = scratch + kMaxNodes;
  t.sort_rows = true;
  t.src_capacity = src_capacity;
  // A neighbour id at or beyond n_nodes would index outside off_dev and outside the scratch array: the kernels
  // skip such an edge and raise this flag (one word of the scratch array, cleared here like the rest), and the call
  // then reports an invalid argument.
  t.bad = scratch + kMaxNodes + kScanWords;
  if (cudaMemsetAsync(t.bad, 0, 4, s) != cudaSuccess) return GRAND_ERR_CUDA;
  uint32_t E = 0, bad = 0;
  if (src_dev) {
    // offsets first, so that the edge count can be checked against the caller's buffer
    t.src = nullptr;
    if (grand::launch_transpose(t, s) != cudaSuccess) return GRAND_ERR_CUDA;
    if (cudaMemcpyAsync(&E, off_dev + n_nodes, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GRAND_ERR_CUDA;
    if (cudaMemcpyAsync(&bad, t.bad, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GRAND_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return GRAND_ERR_CUDA;
    if (bad) return GRAND_ERR_INVALID_ARG;
    if (E > src_capacity) return GRAND_ERR_CAPACITY;
    t.src = src_dev;
  }
  if (grand::launch_transpose(t, s) != cudaSuccess) return GRAND_ERR_CUDA;
  if (cudaMemcpyAsync(&E, off_dev + n_nodes, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GRAND_ERR_CUDA;
  if (cudaMemcpyAsync(&bad, t.bad, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GRAND_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return GRAND_ERR_CUDA;
  if (bad) return GRAND_ERR_INVALID_ARG;
  if (E_out_host) *E_out_host = E;
  return GRAND_OK;
}
