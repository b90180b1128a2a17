// Integer plumbing kernels: grouping of reverse-edge / repair requests by target (the stand-in for
// the per-node scratch buffers of Alg. 5/6), the on-demand reverse graph (Alg. 8: histogram ->
// exclusive scan -> scatter, CSR), batch validation, store writes and live-set bookkeeping.
#include "grand_common.cuh"
#include "grand_kernels.h"

namespace grand {

constexpr int kThreads = 256;
static inline unsigned grid_for(uint64_t n, int threads = kThreads) {
  const uint64_t maxb = (uint64_t)sm_count() * 32u;
  uint64_t b = (n + threads - 1) / threads;
  if (b < 1) b = 1;
  return (unsigned)(b > maxb ? maxb : b);
}


// ---- request grouping: count per target (first touch appends to the dirty list), allocate one
// segment per dirty target from a global cursor, scatter keys into the segments.
__global__ void group_count_kernel(const GroupArgs a) {
  unsigned long long nv = 0;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  // warp-uniform trip count: every lane takes part in the aggregated append
  for (uint64_t b = blockIdx.x * (uint64_t)blockDim.x + (threadIdx.x & ~31u); b < a.nreq; b += stride) {
    const uint64_t i = b + (threadIdx.x & 31);
    const uint32_t tg = i < a.nreq ? a.req_tgt[i] : kInvalid;
    bool first = false;
    if (tg != kInvalid) {
      ++nv;
      // first request of this target in the batch, and not already listed by a repair touch
      first = atomicAdd(&a.cnt[tg], 1u) == 0u && atomicExch(&a.flag[tg], 1u) == 0u;
    }
    warp_append(a.dirty, &a.state->ndirty, first, tg);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) nv += __shfl_xor_sync(0xFFFFFFFFu, nv, o);
  if ((threadIdx.x & 31) == 0 && nv) atomicAdd(&a.state->counters[CTR_REQ], nv);
}
__global__ void group_alloc_kernel(const GroupArgs a) {
  const uint32_t nd = a.state->ndirty;
  const int lane = threadIdx.x & 31;
  // one cursor bump per warp: segment sizes are prefix-summed across the lanes
  for (uint32_t b = blockIdx.x * blockDim.x + (threadIdx.x & ~31u); b < nd; b += gridDim.x * blockDim.x) {
    const uint32_t k = b + lane;
    const uint32_t u = k < nd ? a.dirty[k] : 0u;
    const uint32_t c = k < nd ? a.cnt[u] : 0u;
    uint32_t inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if (lane >= o) inc += y;
    }
    uint32_t base = 0;
    if (lane == 31) base = atomicAdd(&a.state->cursor, inc);
    base = __shfl_sync(0xFFFFFFFFu, base, 31);
    if (k < nd) a.start[u] = base + inc - c;
    if (a.work) {
      const bool light = k < nd && c <= a.light_max && a.deg[u] + c <= a.R;
      const unsigned lb = __ballot_sync(0xFFFFFFFFu, light), hb = __ballot_sync(0xFFFFFFFFu, k < nd && !light);
      uint32_t lbase = 0, hbase = 0;
      if (lane == 0) {
        if (lb) lbase = atomicAdd(&a.state->nlight, (uint32_t)__popc(lb));
        if (hb) hbase = atomicAdd(&a.state->nheavy, (uint32_t)__popc(hb));
      }
      lbase = __shfl_sync(0xFFFFFFFFu, lbase, 0);
      hbase = __shfl_sync(0xFFFFFFFFu, hbase, 0);
      const uint32_t lt = (1u << lane) - 1u;
      if (light) a.work[a.work_cap - 1u - (lbase + __popc(lb & lt))] = u;
      else if (k < nd) a.work[hbase + __popc(hb & lt)] = u;
    }
  }
}
__global__ void group_scatter_kernel(const GroupArgs a) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < a.nreq; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t tg = a.req_tgt[i];
    if (tg == kInvalid) continue;
    a.seg_keys[a.start[tg] + atomicAdd(&a.fill[tg], 1u)] = a.req_key[i];
  }
}
cudaError_t launch_group_requests(const GroupArgs& a, cudaStream_t s) {
  if (a.nreq) group_count_kernel<<<grid_for(a.nreq), kThreads, 0, s>>>(a);
  group_alloc_kernel<<<grid_for(a.nreq ? a.nreq : 1), kThreads, 0, s>>>(a);
  if (a.nreq) group_scatter_kernel<<<grid_for(a.nreq), kThreads, 0, s>>>(a);
  count_launches(a.nreq ? 3 : 1);
  return cudaGetLastError();
}

// ---- exclusive scan of uint32 (three phases; 2048 elements per block)
constexpr int kScanThreads = 256, kScanPer = 8, kScanBlock = kScanThreads * kScanPer;

__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* sh, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) sh[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = lane < (int)(blockDim.x >> 5) ? sh[lane] : 0u;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, o);
      if (lane >= o) winc += y;
    }
    sh[32 + lane] = winc - w;
    if (lane == 31) sh[64] = winc;
  }
  __syncthreads();
  const uint32_t r = sh[32 + warp] + inc - v;
  *total = sh[64];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kScanThreads) scan_sums_kernel(const uint32_t* in, uint64_t n, uint32_t* sums) {
  __shared__ uint32_t sh[65];
  const uint64_t base = (uint64_t)blockIdx.x * kScanBlock + (uint64_t)threadIdx.x * kScanPer;
  uint32_t s = 0;
#pragma unroll
  for (int j = 0; j < kScanPer; ++j) s += base + j < n ? in[base + j] : 0u;
  uint32_t total;
  block_exclusive_scan(s, sh, &total);
  if (threadIdx.x == 0) sums[blockIdx.x] = total;
}
__global__ void __launch_bounds__(kScanThreads) scan_top_kernel(uint32_t* sums, uint32_t nblocks) {
  __shared__ uint32_t sh[65];
  uint32_t carry = 0;
  for (uint32_t b0 = 0; b0 < nblocks; b0 += kScanThreads) {
    const uint32_t i = b0 + threadIdx.x;
    const uint32_t v = i < nblocks ? sums[i] : 0u;
    uint32_t total;
    const uint32_t ex = block_exclusive_scan(v, sh, &total);
    if (i < nblocks) sums[i] = carry + ex;
    carry += total;
  }
}
__global__ void __launch_bounds__(kScanThreads) scan_final_kernel(const uint32_t* in, uint32_t* out, uint64_t n, const uint32_t* sums) {
  __shared__ uint32_t sh[65];
  const uint64_t base = (uint64_t)blockIdx.x * kScanBlock + (uint64_t)threadIdx.x * kScanPer;
  uint32_t v[kScanPer];
  uint32_t s = 0;
#pragma unroll
  for (int j = 0; j < kScanPer; ++j) {
    v[j] = base + j < n ? in[base + j] : 0u;
    s += v[j];
  }
  uint32_t total;
  uint32_t ex = block_exclusive_scan(s, sh, &total) + sums[blockIdx.x];
#pragma unroll
  for (int j = 0; j < kScanPer; ++j) {
    if (base + j < n) out[base + j] = ex;
    ex += v[j];
  }
}
cudaError_t launch_exclusive_scan(const uint32_t* in, uint32_t* out, uint64_t n, uint32_t* tmp, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const uint32_t nblocks = (uint32_t)((n + kScanBlock - 1) / kScanBlock);
  scan_sums_kernel<<<nblocks, kScanThreads, 0, s>>>(in, n, tmp);
  scan_top_kernel<<<1, kScanThreads, 0, s>>>(tmp, nblocks);
  scan_final_kernel<<<nblocks, kScanThreads, 0, s>>>(in, out, n, tmp);
  count_launches(3);
  return cudaGetLastError();
}

// ---- reverse graph
// `heads` (optional bitmap): only edges whose head is marked are counted / scattered, i.e. only the
// in-neighbour rows of the marked nodes are materialised (the delete path reads no other row).
// One warp per adjacency row (a coalesced read of the row, its degree fetched once, no index arithmetic per edge),
// four rows in flight per warp: degree -> row -> bitmap word is a chain of dependent loads, and one row at a time
// left the kernels waiting on it at a fifth of the memory bandwidth.
constexpr int kTransposeRows = 4;
// A neighbour id at or beyond the node count is never followed (a caller-supplied graph may hold one); `bad`, when
// given, records that one was met.
template <typename F>
__device__ __forceinline__ void for_each_marked_edge(const GraphView& g, const uint32_t* heads, uint32_t* bad, F&& f) {
  const int lane = threadIdx.x & 31;
  const uint64_t wglobal = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5;
  const uint64_t wtotal = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t v0 = wglobal; v0 < g.cap; v0 += kTransposeRows * wtotal) {
    uint32_t dv[kTransposeRows];
#pragma unroll
    for (int k = 0; k < kTransposeRows; ++k) {
      const uint64_t v = v0 + k * wtotal;
      dv[k] = v < g.cap ? min(g.deg[v], g.R) : 0u;
    }
    for (uint32_t sb = 0; sb < g.R; sb += 32) {
      uint32_t z[kTransposeRows];
#pragma unroll
      for (int k = 0; k < kTransposeRows; ++k) z[k] = sb + lane < dv[k] ? g.adj[(v0 + k * wtotal) * g.R + sb + lane] : 0xFFFFFFFFu;
      bool hit[kTransposeRows];
#pragma unroll
      for (int k = 0; k < kTransposeRows; ++k) {
        hit[k] = z[k] < g.cap && (!heads || bit_test(heads, z[k]));
        if (bad && z[k] != 0xFFFFFFFFu && z[k] >= g.cap) *bad = 1u;
      }
#pragma unroll
      for (int k = 0; k < kTransposeRows; ++k) f(hit[k], z[k], (uint32_t)(v0 + k * wtotal));  // (all lanes, converged)
    }
  }
}
__global__ void transpose_hist_kernel(const GraphView g, uint32_t* indeg, const uint32_t* heads, uint32_t* bad) {
  for_each_marked_edge(g, heads, bad, [&](bool hit, uint32_t z, uint32_t) {
    if (hit) atomicAdd(&indeg[z], 1u);
  });
}
// The same pass, which also writes the marked edges out as (head, tail) pairs: the heads of a delete batch catch a
// percent or so of the edges, and scattering them from the list spares the second pass over the adjacency.
// Pairs collect in a per-warp buffer and leave in runs (one bump of the list's counter per run, not per edge);
// pairs beyond the list's capacity are dropped and still counted, like entries beyond the capacity of `src`.
constexpr uint32_t kPairRun = 64;
__global__ void __launch_bounds__(kThreads) transpose_hist_pairs_kernel(const GraphView g, uint32_t* indeg, const uint32_t* heads,
                                                                        uint32_t* bad, unsigned long long* pairs,
                                                                        const uint64_t pairs_capacity, uint32_t* pair_count) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  __shared__ unsigned long long buf_s[kThreads / 32][kPairRun + 32];
  const int lane = threadIdx.x & 31;
  unsigned long long* buf = buf_s[threadIdx.x >> 5];
  const uint32_t lt_mask = (1u << lane) - 1u;
  uint32_t cnt = 0;  // (uniform over the warp)
  auto flush = [&] {
    __syncwarp();
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(pair_count, cnt);
    base = __shfl_sync(FULL, base, 0);
    for (uint32_t j = lane; j < cnt; j += 32)
      if ((uint64_t)base + j < pairs_capacity) pairs[(uint64_t)base + j] = buf[j];
    __syncwarp();
    cnt = 0;
  };
  for_each_marked_edge(g, heads, bad, [&](bool hit, uint32_t z, uint32_t v) {
    const unsigned bal = __ballot_sync(FULL, hit);
    if (!bal) return;
    if (hit) {
      atomicAdd(&indeg[z], 1u);
      buf[cnt + __popc(bal & lt_mask)] = ((unsigned long long)z << 32) | v;
    }
    cnt += __popc(bal);
    if (cnt >= kPairRun) flush();
  });
  if (cnt) flush();
}
__global__ void transpose_scatter_pairs_kernel(const unsigned long long* pairs, const uint64_t pairs_capacity, const uint32_t* pair_count,
                                               const uint32_t* off, uint32_t* fillc, uint32_t* src, const uint64_t src_capacity) {
  const uint64_t n = min((uint64_t)*pair_count, pairs_capacity);
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const unsigned long long pr = pairs[i];
    const uint32_t z = (uint32_t)(pr >> 32);
    const uint64_t at = (uint64_t)off[z] + atomicAdd(&fillc[z], 1u);
    if (at < src_capacity) src[at] = (uint32_t)pr;
  }
}
__global__ void transpose_scatter_kernel(const GraphView g, const uint32_t* off, uint32_t* fillc, uint32_t* src, const uint32_t* heads,
                                         const uint64_t src_capacity) {
  for_each_marked_edge(g, heads, nullptr, [&](bool hit, uint32_t z, uint32_t v) {
    if (!hit) return;
    const uint64_t at = (uint64_t)off[z] + atomicAdd(&fillc[z], 1u);
    if (at < src_capacity) src[at] = v;
  });
}
// ascending rows: shared-memory sort for short rows, in place in global memory for long ones
__global__ void __launch_bounds__(128) transpose_sort_rows_kernel(uint64_t cap, const uint32_t* off, uint32_t* src, const uint64_t src_capacity) {
  constexpr uint32_t kRowCap = 4096;
  __shared__ uint32_t sh[kRowCap];
  auto sync = [] { __syncthreads(); };
  for (uint64_t z = blockIdx.x; z < cap; z += gridDim.x) {
    const uint32_t b = off[z], n = off[z + 1] - b;
    if (n < 2 || (uint64_t)b + n > src_capacity) continue;
    if (n <= kRowCap) {
      for (uint32_t j = threadIdx.x; j < n; j += blockDim.x) sh[j] = src[b + j];
      __syncthreads();
      bitonic_sort_any(sh, n, threadIdx.x, blockDim.x, sync);
      for (uint32_t j = threadIdx.x; j < n; j += blockDim.x) src[b + j] = sh[j];
      __syncthreads();
    } else {
      bitonic_sort_any(src + b, n, threadIdx.x, blockDim.x, sync);
    }
  }
}
cudaError_t launch_transpose(const TransposeArgs& a, cudaStream_t s) {
  const uint64_t cap = a.g.cap;
  cudaMemsetAsync(a.indeg, 0, (cap + 1) * 4, s);
  const bool listed = a.heads && a.src && a.pairs && a.pair_count && !a.sort_rows;
  if (listed) {
    cudaMemsetAsync(a.pair_count, 0, 4, s);
    transpose_hist_pairs_kernel<<<grid_for(cap * 32), kThreads, 0, s>>>(a.g, a.indeg, a.heads, a.bad, a.pairs, a.pairs_capacity, a.pair_count);
  } else {
    transpose_hist_kernel<<<grid_for(cap * 32), kThreads, 0, s>>>(a.g, a.indeg, a.heads, a.bad);
  }
  count_launches(1);
  cudaError_t e = launch_exclusive_scan(a.indeg, a.off, cap + 1, a.scan_tmp, s);
  if (e != cudaSuccess) return e;
  if (listed) {
    cudaMemsetAsync(a.fillc, 0, cap * 4, s);
    transpose_scatter_pairs_kernel<<<(unsigned)sm_count() * 8u, kThreads, 0, s>>>(a.pairs, a.pairs_capacity, a.pair_count, a.off, a.fillc,
                                                                              a.src, a.src_capacity);
    count_launches(1);
    return cudaGetLastError();
  }
  if (a.src) {
    cudaMemsetAsync(a.fillc, 0, cap * 4, s);
    transpose_scatter_kernel<<<grid_for(cap * 32), kThreads, 0, s>>>(a.g, a.off, a.fillc, a.src, a.heads, a.src_capacity);
    count_launches(a.sort_rows ? 2 : 1);
    const uint64_t sort_blocks = (uint64_t)sm_count() * 16u;
    if (a.sort_rows) transpose_sort_rows_kernel<<<(unsigned)(cap < sort_blocks ? cap : sort_blocks), 128, 0, s>>>(cap, a.off, a.src, a.src_capacity);
  }
  return cudaGetLastError();
}

// ---- validation: ids < capacity, liveness as required, no repeated id (bitmap atomics)
__device__ __forceinline__ void set_status(DevState* st, int code) { atomicMin(&st->status, code); }

__global__ void validate_range_kernel(const uint32_t* ids, uint64_t n, uint64_t cap, DevState* st) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
    if (ids[i] >= cap) set_status(st, -2);
}
__global__ void validate_mark_kernel(const uint32_t* ids, uint64_t n, uint64_t cap, const uint32_t* live, uint32_t* mark,
                                     int want_live, DevState* st) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t v = ids[i];
    if (v >= cap) continue;
    const uint32_t bit = 1u << (v & 31);
    if (atomicOr(&mark[v >> 5], bit) & bit) set_status(st, -3);
  }
}
__global__ void validate_live_kernel(const uint32_t* ids, uint64_t n, uint64_t cap, const uint32_t* live, int want_live, DevState* st) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t v = ids[i];
    if (v >= cap) continue;
    const bool is_live = bit_test(live, v);
    // error precedence (capacity, duplicate, liveness) mirrors a sequential check of the whole batch
    if (want_live && !is_live) atomicCAS(&st->status, 0, -5);
    if (!want_live && is_live) atomicCAS(&st->status, 0, -4);
  }
}
cudaError_t launch_validate(const uint32_t* ids, uint64_t n, uint64_t cap, const uint32_t* live, uint32_t* mark, int want_live,
                            DevState* st, cudaStream_t s) {
  validate_range_kernel<<<grid_for(n), kThreads, 0, s>>>(ids, n, cap, st);
  validate_mark_kernel<<<grid_for(n), kThreads, 0, s>>>(ids, n, cap, live, mark, want_live, st);
  validate_live_kernel<<<grid_for(n), kThreads, 0, s>>>(ids, n, cap, live, want_live, st);
  count_launches(3);
  return cudaGetLastError();
}
__global__ void clear_marks_kernel(const uint32_t* ids, uint64_t n, uint64_t cap, uint32_t* mark) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t v = ids[i];
    if (v < cap) atomicAnd(&mark[v >> 5], ~(1u << (v & 31)));
  }
}
cudaError_t launch_clear_marks(const uint32_t* ids, uint64_t n, uint64_t cap, uint32_t* mark, cudaStream_t s) {
  clear_marks_kernel<<<grid_for(n), kThreads, 0, s>>>(ids, n, cap, mark);
  count_launches(1);
  return cudaGetLastError();
}

// ---- store write: re-stride packed vectors into 16-byte padded rows, zero the padding, deg <- 0
template <typename T>
__global__ void store_write_kernel(uint8_t* store, uint32_t* deg, uint32_t* slot_of, const uint32_t* ids, const T* vecs,
                                   uint64_t n, uint32_t dim, uint32_t row_bytes) {
  const uint32_t per_row = row_bytes / sizeof(T);
  const uint64_t total = n * per_row;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < total; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t r = i / per_row;
    const uint32_t j = (uint32_t)(i - r * per_row);
    const uint64_t dst_row = ids ? ids[r] : r;
    reinterpret_cast<T*>(store + dst_row * row_bytes)[j] = j < dim ? vecs[r * dim + j] : T(0);
    if (j == 0 && ids) {
      if (deg) deg[dst_row] = 0;
      if (slot_of) slot_of[dst_row] = (uint32_t)r;
    }
  }
}
cudaError_t launch_store_write(const Layout& lay, uint8_t* store, uint32_t* deg, uint32_t* slot_of, const uint32_t* ids,
                               const void* vecs, uint64_t n, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const uint64_t total = n * (lay.row_bytes / lay.esize);
  if (lay.esize == 4)
    store_write_kernel<float><<<grid_for(total), kThreads, 0, s>>>(store, deg, slot_of, ids, (const float*)vecs, n, lay.udim, lay.row_bytes);
  else
    store_write_kernel<uint8_t><<<grid_for(total), kThreads, 0, s>>>(store, deg, slot_of, ids, (const uint8_t*)vecs, n, lay.udim, lay.row_bytes);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_pad_rows(const Layout& lay, uint8_t* store, const void* vecs, uint64_t n, cudaStream_t s) {
  return launch_store_write(lay, store, nullptr, nullptr, nullptr, vecs, n, s);
}

// ---- MIPS -> L2 reduction (Sec. 5.3): one warp per vector sums the squares in double
__device__ __forceinline__ double warp_sq_norm(const float* v, uint32_t d) {
  double s = 0.0;
  for (uint32_t j = threadIdx.x & 31; j < d; j += 32) s += (double)v[j] * (double)v[j];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  return s;
}
__global__ void check_norms_kernel(const float* vecs, uint64_t n, uint32_t udim, double M2, DevState* st) {
  const uint64_t w = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5, nw = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t i = w; i < n; i += nw)
    if (warp_sq_norm(vecs + i * udim, udim) > M2 * (1.0 + 1e-6) && (threadIdx.x & 31) == 0) atomicMin(&st->status, -1);
}
__global__ void augment_rows_kernel(uint8_t* store, const uint32_t* ids, uint64_t n, uint32_t udim, uint32_t row_bytes, double M2) {
  const uint64_t w = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5, nw = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t i = w; i < n; i += nw) {
    float* row = reinterpret_cast<float*>(store + (size_t)(ids ? ids[i] : i) * row_bytes);
    const double n2 = warp_sq_norm(row, udim);
    if ((threadIdx.x & 31) == 0) row[udim] = (float)sqrt(fmax(M2 - n2, 0.0));
  }
}
cudaError_t launch_check_norms(const Layout& lay, const void* vecs, uint64_t n, double M2, DevState* st, cudaStream_t s) {
  check_norms_kernel<<<grid_for(n * 32), kThreads, 0, s>>>((const float*)vecs, n, lay.udim, M2, st);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_augment_rows(const Layout& lay, uint8_t* store, const uint32_t* ids, uint64_t n, double M2, cudaStream_t s) {
  augment_rows_kernel<<<grid_for(n * 32), kThreads, 0, s>>>(store, ids, n, lay.udim, lay.row_bytes, M2);
  count_launches(1);
  return cudaGetLastError();
}

// ---- publish (insert epilogue): live bits on, batch marks off
__global__ void publish_kernel(const uint32_t* ids, uint64_t n, uint32_t* live, uint32_t* mark, DevState* st) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t v = ids[i];
    atomicOr(&live[v >> 5], 1u << (v & 31));
    atomicAnd(&mark[v >> 5], ~(1u << (v & 31)));
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) st->nlive += n;
}
cudaError_t launch_publish(const uint32_t* ids, uint64_t n, uint32_t* live, uint32_t* mark, DevState* st, cudaStream_t s) {
  publish_kernel<<<grid_for(n), kThreads, 0, s>>>(ids, n, live, mark, st);
  count_launches(1);
  return cudaGetLastError();
}

// ---- retire (delete epilogue): choose a new medoid if the old one is deleted, clear rows and bits
__global__ void __launch_bounds__(256) new_entry_kernel(const GraphView g, const uint32_t* ids, uint64_t n, const uint32_t* delmap,
                                                        const unsigned long long* Ci, const uint32_t* Ci_n, uint32_t k_repair,
                                                        uint32_t fixed_mode, DevState* st) {
  const uint32_t m = st->entry;
  if (m == kInvalid || !bit_test(delmap, m)) return;
  __shared__ uint32_t found;
  if (threadIdx.x == 0) found = kInvalid;
  __syncthreads();
  if (fixed_mode) {  // first surviving out-neighbour of the old medoid (rows are nearest-first)
    if (threadIdx.x == 0) {
      const uint32_t d = min(g.deg[m], g.R);
      for (uint32_t s = 0; s < d; ++s) {
        const uint32_t v = g.adj[(size_t)m * g.R + s];
        if (!bit_test(delmap, v)) {
          found = v;
          break;
        }
      }
    }
  } else {  // first repair candidate of the deleted medoid
    for (uint64_t i = threadIdx.x; i < n; i += blockDim.x)
      if (ids[i] == m && Ci_n[i] > 0) found = key_id(Ci[i * k_repair]);
  }
  __syncthreads();
  if (threadIdx.x == 0) st->entry = found;  // kInvalid -> smallest live id, resolved after the bits are cleared
}
__global__ void retire_kernel(const GraphView g, const uint32_t* ids, uint64_t n, uint32_t* delmap, DevState* st) {
  const uint64_t total = n * g.R;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < total; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t r = i / g.R;
    const uint32_t s = (uint32_t)(i - r * g.R);
    const uint32_t p = ids[r];
    g.adj[(size_t)p * g.R + s] = kInvalid;
    if (s == 0) {
      g.deg[p] = 0;
      atomicAnd(&g.live[p >> 5], ~(1u << (p & 31)));
      atomicAnd(&delmap[p >> 5], ~(1u << (p & 31)));
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) st->nlive -= n;
}
__global__ void fallback_entry_kernel(const uint32_t* live, uint64_t nwords, DevState* st, uint32_t* scratch_min) {
  // runs only when the medoid was deleted without a replacement candidate
  for (uint64_t w = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; w < nwords; w += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t x = live[w];
    if (x) atomicMin(scratch_min, (uint32_t)(w * 32 + __ffs(x) - 1));
  }
}
__global__ void fallback_entry_begin(DevState* st, uint32_t* scratch_min) {
  scratch_min[0] = kInvalid;
  scratch_min[1] = st->entry == kInvalid ? 1u : 0u;
}
__global__ void fallback_entry_end(DevState* st, const uint32_t* scratch_min) {
  if (scratch_min[1]) st->entry = scratch_min[0];
}
cudaError_t launch_retire(const GraphView& g, const uint32_t* ids, uint64_t n, uint32_t* delmap, const unsigned long long* Ci,
                          const uint32_t* Ci_n, uint32_t k_repair, uint32_t fixed_mode, DevState* st, cudaStream_t s) {
  new_entry_kernel<<<1, 256, 0, s>>>(g, ids, n, delmap, Ci, Ci_n, k_repair, fixed_mode, st);
  retire_kernel<<<grid_for(n * g.R), kThreads, 0, s>>>(g, ids, n, delmap, st);
  // smallest live id as the last resort (cheap: one pass over the bitmap); scratch = medoid_key words
  uint32_t* scratch = reinterpret_cast<uint32_t*>(&st->medoid_key);
  fallback_entry_begin<<<1, 1, 0, s>>>(st, scratch);
  fallback_entry_kernel<<<grid_for((g.cap + 31) / 32), kThreads, 0, s>>>(g.live, (g.cap + 31) / 32, st, scratch);
  fallback_entry_end<<<1, 1, 0, s>>>(st, scratch);
  count_launches(5);
  return cudaGetLastError();
}

__global__ void count_live_kernel(const uint32_t* live, uint64_t nwords, DevState* st) {
  unsigned long long c = 0;
  for (uint64_t w = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; w < nwords; w += (uint64_t)gridDim.x * blockDim.x) c += __popc(live[w]);
  if (c) atomicAdd(&st->nlive, c);
}
cudaError_t launch_count_live(const uint32_t* live, uint64_t cap, DevState* st, cudaStream_t s) {
  count_live_kernel<<<grid_for((cap + 31) / 32), kThreads, 0, s>>>(live, (cap + 31) / 32, st);
  count_launches(1);
  return cudaGetLastError();
}

// rows are read whole by the search kernel: every slot at or beyond deg must hold the invalid id
__global__ void pad_adjacency_kernel(uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R) {
  const uint64_t total = cap * R;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < total; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t v = i / R;
    if ((uint32_t)(i - v * R) >= deg[v]) adj[i] = kInvalid;
  }
}
__global__ void copy_rows_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst, const uint32_t* __restrict__ ids,
                                 const uint64_t n, const uint32_t R, const uint64_t cap) {
  const int lane = threadIdx.x & 31;
  const uint64_t wglobal = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5;
  const uint64_t wtotal = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t i = wglobal; i < n; i += wtotal) {
    const uint32_t v = ids[i];
    if (v >= cap) continue;
    for (uint32_t s = lane; s < R; s += 32) dst[(size_t)v * R + s] = src[(size_t)v * R + s];
  }
}
cudaError_t launch_copy_rows(const uint32_t* src, uint32_t* dst, const uint32_t* ids, uint64_t n, uint32_t R, uint64_t cap, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  uint64_t blocks = (n + 7) / 8;
  if (blocks > (uint64_t)sm_count() * 32u) blocks = (uint64_t)sm_count() * 32u;
  copy_rows_kernel<<<(unsigned)blocks, 256, 0, s>>>(src, dst, ids, n, R, cap);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_pad_adjacency(uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R, cudaStream_t s) {
  pad_adjacency_kernel<<<grid_for(cap * R), kThreads, 0, s>>>(adj, deg, cap, R);
  count_launches(1);
  return cudaGetLastError();
}

__global__ void check_graph_kernel(const uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R, DevState* st) {
  const uint64_t total = cap * R;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < total; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t v = i / R;
    const uint32_t s = (uint32_t)(i - v * R), d = deg[v];
    if ((s == 0 && d > R) || (s < d && adj[i] >= cap)) atomicMin(&st->status, -1);
  }
}
cudaError_t launch_check_graph(const uint32_t* adj, const uint32_t* deg, uint64_t cap, uint32_t R, DevState* st, cudaStream_t s) {
  check_graph_kernel<<<grid_for(cap * R), kThreads, 0, s>>>(adj, deg, cap, R, st);
  count_launches(1);
  return cudaGetLastError();
}

__global__ void fill_u32_kernel(uint32_t* p, uint32_t v, uint64_t n) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) p[i] = v;
}
cudaError_t launch_fill_u32(uint32_t* p, uint32_t v, uint64_t n, cudaStream_t s) {
  if (n) { fill_u32_kernel<<<grid_for(n), kThreads, 0, s>>>(p, v, n); count_launches(1); }
  return cudaGetLastError();
}

}  // namespace grand
