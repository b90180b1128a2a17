// Delete-repair kernels (Alg. 6 with exact in-neighbours, Alg. 8 in fixed-degree mode) and the
// initial-medoid choice.  The work is flattened over (deleted node, in-neighbour) and (deleted
// node, out-slot) pairs so that hubs with a long in-neighbour row do not serialise a block.
#include "grand_common.cuh"
#include "grand_kernels.h"

namespace grand {

constexpr int kPickWarps = 4;
constexpr uint32_t kMaxKRepair = 128;


// start of the in-neighbour list of batch member i (reverse-graph row, or its slice of the visited-set list)
__device__ __forceinline__ uint32_t in_base(const DeleteArgs& a, uint64_t i) {
  return a.src_stride ? (uint32_t)i * a.src_stride : a.off[a.ids[i]];
}

// in_cnt[i] = in-degree of p_i in the reverse graph (0 for an id that fails validation), then the
// prefix over the batch and the total number of (deleted node, in-neighbour) pairs.
__global__ void delete_incnt_kernel(const DeleteArgs a) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i <= a.n; i += (uint64_t)gridDim.x * blockDim.x) {
    uint32_t c = 0;
    if (i < a.n) {
      const uint32_t p = a.ids[i];
      if (p < a.g.cap) c = a.off[p + 1] - a.off[p];
    }
    a.in_cnt[i] = c;
  }
}
__global__ void delete_total_kernel(const uint32_t* pair_off, uint64_t n, DevState* st) { st->total_in = pair_off[n]; }

cudaError_t launch_delete_prepare(const DeleteArgs& a, cudaStream_t s) {
  const uint64_t cap16 = (uint64_t)sm_count() * 16u;
  const unsigned blocks = (unsigned)((a.n + 256) / 256 > cap16 ? cap16 : (a.n + 256) / 256);
  delete_incnt_kernel<<<blocks, 256, 0, s>>>(a);
  cudaError_t e = launch_exclusive_scan(a.in_cnt, a.pair_off, a.n + 1, a.scan_tmp, s);
  if (e != cudaSuccess) return e;
  delete_total_kernel<<<1, 1, 0, s>>>(a.pair_off, a.n, a.state);
  count_launches(2);
  return cudaGetLastError();
}

// Alg. 6 as printed: the in-neighbours of p_i are the visited nodes z whose row holds p_i.  One warp per
// (batch member, visited entry); hits are appended to the member's slice of `inlist` (order is irrelevant:
// requests are grouped and sorted later) and counted in in_cnt, whose prefix then drives the pair loop.
__global__ void delete_visited_in_kernel(const DeleteArgs a, uint32_t* inlist) {
  const int lane = threadIdx.x & 31;
  const uint32_t R = a.g.R;
  const uint64_t total = a.n * a.vis_stride;
  const uint64_t wglobal = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5;
  const uint64_t wtotal = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t e = wglobal; e < total; e += wtotal) {
    const uint64_t i = e / a.vis_stride;
    const uint32_t j = (uint32_t)(e - i * a.vis_stride);
    if (j >= min(a.vis_n[i], a.vis_stride)) continue;
    const uint32_t z = key_id(a.vis[i * a.vis_stride + j]);
    if (bit_test(a.delmap, z)) continue;
    const uint32_t p = a.ids[i];
    const uint32_t dz = min(a.g.deg[z], R);
    bool hit = false;
    for (uint32_t sb = 0; sb < dz; sb += 32) hit |= sb + lane < dz && a.g.adj[(size_t)z * R + sb + lane] == p;
    if (__any_sync(0xFFFFFFFFu, hit) && lane == 0) inlist[i * a.vis_stride + atomicAdd(&a.in_cnt[i], 1u)] = z;
  }
}
cudaError_t launch_delete_visited_in(const DeleteArgs& a, uint32_t* inlist, cudaStream_t s) {
  cudaMemsetAsync(a.in_cnt, 0, (a.n + 1) * 4, s);
  uint64_t blocks = (a.n * a.vis_stride + 3) / 4;
  if (blocks > (uint64_t)sm_count() * 32u) blocks = (uint64_t)sm_count() * 32u;
  delete_visited_in_kernel<<<(unsigned)blocks, 128, 0, s>>>(a, inlist);
  cudaError_t e = launch_exclusive_scan(a.in_cnt, a.pair_off, a.n + 1, a.scan_tmp, s);
  if (e != cudaSuccess) return e;
  delete_total_kernel<<<1, 1, 0, s>>>(a.pair_off, a.n, a.state);
  count_launches(2);
  return cudaGetLastError();
}

// C_i = first k_repair worklist entries of the per-deleted search that are not in the batch.
__global__ void delete_ci_kernel(const DeleteArgs a) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  const int lane = threadIdx.x & 31;
  const uint64_t wglobal = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5;
  const uint64_t wtotal = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  unsigned long long ncand = 0;
  for (uint64_t i = wglobal; i < a.n; i += wtotal) {
    const uint32_t nb = min(a.beam_n[i], a.beam_stride);
    uint32_t nc = 0;
    for (uint32_t jb = 0; jb < nb && nc < a.k_repair; jb += 32) {
      const uint32_t j = jb + lane;
      unsigned long long k = 0;
      bool ok = false;
      if (j < nb) {
        k = a.beam[i * a.beam_stride + j];
        ok = !bit_test(a.delmap, key_id(k));
      }
      const unsigned bal = __ballot_sync(FULL, ok);
      const uint32_t pos = nc + __popc(bal & ((1u << lane) - 1u));
      if (ok && pos < a.k_repair) a.Ci[i * a.k_repair + pos] = k;
      nc += __popc(bal);
    }
    if (lane == 0) {
      a.Ci_n[i] = min(nc, a.k_repair);
      ncand += min(nc, a.k_repair);
    }
  }
  // the repair has to fetch every candidate row once per deleted node
  if (lane == 0 && ncand) atomicAdd(&a.state->counters[CTR_PK_BYTES], ncand * a.lay.row_bytes);
}
cudaError_t launch_delete_ci(const DeleteArgs& a, cudaStream_t s) {
  const uint64_t cap16 = (uint64_t)sm_count() * 16u;
  const unsigned blocks = (unsigned)((a.n + 3) / 4 > cap16 ? cap16 : (a.n + 3) / 4);
  delete_ci_kernel<<<blocks ? blocks : 1, 128, 0, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

// One warp per pair.  In-pair (p_i, z): z gets the c members of C_i \ {z} closest to z (requests
// z <- y).  Out-pair (p_i, w): the c members y of C_i \ {w} closest to w each get w (requests y <- w).
template <typename T, int METRIC, int G, int CPL>
__global__ void __launch_bounds__(kPickWarps * 32) delete_picks_kernel(const DeleteArgs a, const uint64_t total_in) {
  using Dist = typename Elem<T>::Dist;
  constexpr int NT = 32 / G;
  __shared__ unsigned long long keys_s[kPickWarps][kMaxKRepair];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = lane % G, team = lane / G;
  unsigned long long* keys = keys_s[warp];
  const uint32_t R = a.g.R, c = a.c;
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint64_t total = total_in + a.n * R;
  const uint64_t wglobal = (uint64_t)blockIdx.x * kPickWarps + warp, wtotal = (uint64_t)gridDim.x * kPickWarps;
  unsigned long long npair = 0, nrows = 0;
  for (uint64_t pair = wglobal; pair < total; pair += wtotal) {
    const bool is_in = pair < total_in;
    uint64_t i;
    uint32_t x = kInvalid;
    if (is_in) {
      uint64_t lo = 0, hi = a.n;  // largest i with pair_off[i] <= pair
      while (hi - lo > 1) {
        const uint64_t mid = (lo + hi) >> 1;
        if (a.pair_off[mid] <= pair) lo = mid; else hi = mid;
      }
      i = lo;
      x = a.src[in_base(a, i) + (uint32_t)(pair - a.pair_off[i])];
    } else {
      const uint64_t o = pair - total_in;
      i = o / R;
      const uint32_t s = (uint32_t)(o - i * R);
      const uint32_t p = a.ids[i];
      if (s < a.g.deg[p]) x = a.g.adj[(size_t)p * R + s];
    }
    const bool act = x != kInvalid && !bit_test(a.delmap, x) && (!a.livemap || bit_test(a.livemap, x));
    const uint64_t rbase = pair * c;
    if (!act) {
      if (lane < c) a.req_tgt[rbase + lane] = kInvalid;
      continue;
    }
    uint4 xr[CPL];
    load_row<G, CPL>(a.g.store + (size_t)x * row_bytes, nchunk, t, xr);
    const uint32_t nc = a.Ci_n[i];
    if (lane == 0) ++nrows;  // rows the method has to fetch here: x once per pair (C_i is charged where it is formed)
    constexpr int U = CPL == 1 ? 4 : (CPL == 2 ? 2 : 1);  // candidate rows in flight per team
    for (uint32_t jb = 0; jb < nc; jb += NT * U) {
      uint4 v[U][CPL];
      uint32_t yv[U];
#pragma unroll
      for (int uu = 0; uu < U; ++uu) {
        const uint32_t j = jb + uu * NT + team;
        yv[uu] = j < nc ? key_id(a.Ci[i * a.k_repair + j]) : kInvalid;
        if (yv[uu] != kInvalid && yv[uu] != x) {
          load_row<G, CPL>(a.g.store + (size_t)yv[uu] * row_bytes, nchunk, t, v[uu]);
        } else {
#pragma unroll
          for (int cc = 0; cc < CPL; ++cc) v[uu][cc] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int uu = 0; uu < U; ++uu) {
        const uint32_t j = jb + uu * NT + team;
        const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(xr, v[uu]);
        if (t == 0 && j < nc) {
          const bool go = yv[uu] != x;
          keys[j] = go ? make_key(d, yv[uu]) : kKeyMax;
          npair += go;
        }
      }
    }
    __syncwarp();
    for (uint32_t r = 0; r < c; ++r) {  // r-th smallest (dist, id)
      unsigned long long best = kKeyMax;
      for (uint32_t j = lane; j < nc; j += 32) best = min(best, keys[j]);
      best = warp_min_key(best);
      if (best != kKeyMax) {
        for (uint32_t j = lane; j < nc; j += 32)
          if (keys[j] == best) keys[j] = kKeyMax;
      }
      if (lane == 0) {
        if (best == kKeyMax) {
          a.req_tgt[rbase + r] = kInvalid;
        } else if (is_in) {
          a.req_tgt[rbase + r] = x;
          a.req_key[rbase + r] = best;
        } else {
          a.req_tgt[rbase + r] = key_id(best);
          a.req_key[rbase + r] = (best & 0xFFFFFFFF00000000ull) | x;
        }
      }
      __syncwarp();
    }
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_PK_PAIRS], npair);
  }
  if (nrows) atomicAdd(&a.state->counters[CTR_PK_BYTES], nrows * row_bytes);
}
// Every surviving in-neighbour of a deleted node is dirty even if it receives no candidate.
__global__ void delete_touch_kernel(const DeleteArgs a, const uint64_t total_in) {
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t b = blockIdx.x * (uint64_t)blockDim.x + (threadIdx.x & ~31u); b < total_in; b += stride) {
    const uint64_t pair = b + (threadIdx.x & 31);
    bool first = false;
    uint32_t z = kInvalid;
    if (pair < total_in) {
      uint64_t lo = 0, hi = a.n;
      while (hi - lo > 1) {
        const uint64_t mid = (lo + hi) >> 1;
        if (a.pair_off[mid] <= pair) lo = mid; else hi = mid;
      }
      z = a.src[in_base(a, lo) + (uint32_t)(pair - a.pair_off[lo])];
      first = !bit_test(a.delmap, z) && atomicExch(&a.flag[z], 1u) == 0u;
    }
    warp_append(a.dirty, &a.state->ndirty, first, z);
  }
}

// ---- staged variant: C_i is shared by every pair of deleted node i, so a block copies its rows into
// shared memory once and its warps run the pairs of that node against the copy.  Work units are
// chunks of kUnitPairs pairs of one node (hubs with long in-neighbour rows are split over blocks).
constexpr uint32_t kUnitPairs = 256;
__global__ void delete_units_kernel(const DeleteArgs a, const uint32_t unit_pairs) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i <= a.n; i += (uint64_t)gridDim.x * blockDim.x) {
    uint32_t units = 0;
    if (i < a.n) units = (a.pair_off[i + 1] - a.pair_off[i] + a.g.R + unit_pairs - 1) / unit_pairs;
    a.in_cnt[i] = units;  // the in-degree counts are not needed once their prefix exists
  }
}

template <typename T, int METRIC, int G, int CPL>
__global__ void __launch_bounds__(kPickWarps * 32) delete_picks_staged_kernel(const DeleteArgs a, const uint64_t total_in) {
  using Dist = typename Elem<T>::Dist;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int NT = 32 / G;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = lane % G, team = lane / G;
  const uint32_t R = a.g.R, c = a.c, kr = a.k_repair;
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  // staged rows sit on an odd number of 16-byte chunks, so that lanes reading the same chunk of 32 different
  // rows fall on different banks
  const uint32_t rs = (nchunk | 1u) * 16u;
  uint8_t* crow = smem_raw;                                                    // k_repair staged rows
  unsigned long long* ckeys = reinterpret_cast<unsigned long long*>(smem_raw + (size_t)kr * rs);  // their keys
  unsigned long long* keys = ckeys + kr + (size_t)warp * kMaxKRepair;          // per-warp pick scratch
  uint4* xb = reinterpret_cast<uint4*>(ckeys + ((kr + 1u) & ~1u) + (size_t)kPickWarps * kMaxKRepair) + (size_t)warp * nchunk;  // x's row
  int* cnorm = reinterpret_cast<int*>(reinterpret_cast<uint4*>(ckeys + ((kr + 1u) & ~1u) + (size_t)kPickWarps * kMaxKRepair) +
                                      (size_t)kPickWarps * nchunk);  // |y|^2 of the staged rows (integer rows only)
  uint32_t* xid = reinterpret_cast<uint32_t*>(cnorm + kr);  // the unit's x ids (invalid id = nothing to do for the pair)
  const uint32_t nunits = a.unit_off[a.n];
  unsigned long long npair = 0, nrows = 0;
  for (uint32_t unit = blockIdx.x; unit < nunits; unit += gridDim.x) {
    uint32_t lo = 0, hi = (uint32_t)a.n;  // largest i with unit_off[i] <= unit
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (a.unit_off[mid] <= unit) lo = mid; else hi = mid;
    }
    const uint32_t i = lo, p = a.ids[i];
    const uint32_t nin = a.pair_off[i + 1] - a.pair_off[i];
    const uint32_t q0 = (unit - a.unit_off[i]) * kUnitPairs, q1 = min(nin + R, q0 + kUnitPairs);
    const uint32_t nc = a.Ci_n[i];
    __syncthreads();  // the previous unit's readers are done with the staged rows
    for (uint32_t j = threadIdx.x; j < nc; j += blockDim.x) ckeys[j] = a.Ci[(size_t)i * kr + j];
    for (uint32_t e = threadIdx.x; e < nc * nchunk; e += blockDim.x) {
      const uint32_t j = e / nchunk, ch = e - j * nchunk;
      const uint32_t y = key_id(a.Ci[(size_t)i * kr + j]);
      reinterpret_cast<uint4*>(crow + (size_t)j * rs)[ch] = __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)y * row_bytes) + ch);
    }
    // the unit's x ids, resolved by the whole block at once (id, batch and liveness bits are dependent loads that a
    // warp would otherwise wait for pair by pair), and their vectors requested towards L2
    for (uint32_t j = threadIdx.x; j < q1 - q0; j += blockDim.x) {
      const uint32_t q = q0 + j;
      uint32_t x = kInvalid;
      if (q < nin) {
        x = a.src[in_base(a, i) + q];
      } else if (q - nin < a.g.deg[p]) {
        x = a.g.adj[(size_t)p * R + (q - nin)];
      }
      if (x != kInvalid && (bit_test(a.delmap, x) || (a.livemap && !bit_test(a.livemap, x)))) x = kInvalid;
      xid[j] = x;
      if (x != kInvalid)
        for (uint32_t b = 0; b < row_bytes; b += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.g.store + (size_t)x * row_bytes + b));
    }
    __syncthreads();
    if constexpr (sizeof(T) == 1) {
      // |x - y|^2 = |x|^2 + |y|^2 - 2 x.y in exact integers: the pair loop then needs one dp4a per word, not two
      for (uint32_t j = threadIdx.x; j < nc; j += blockDim.x) {
        const uint4* cr = reinterpret_cast<const uint4*>(crow + (size_t)j * rs);
        int acc = 0;
        for (uint32_t ch = 0; ch < nchunk; ++ch) acc_chunk<T, kMetricIP>(cr[ch], cr[ch], acc);
        cnorm[j] = acc;
      }
      __syncthreads();
    }
    for (uint32_t q = q0 + warp; q < q1; q += kPickWarps) {
      const bool is_in = q < nin;
      const uint32_t x = xid[q - q0];
      const uint64_t rbase = is_in ? ((uint64_t)a.pair_off[i] + q) * c : (total_in + (uint64_t)i * R + (q - nin)) * c;
      if (x == kInvalid) {
        if (lane < c) a.req_tgt[rbase + lane] = kInvalid;
        continue;
      }
      if (lane == 0) ++nrows;  // x's row, fetched once per pair
      if constexpr (sizeof(T) == 1) {
        // integer rows: any summation order gives the same distance, so one lane takes one candidate and walks
        // its staged row against x's row (a broadcast read); the keys stay in registers
        int xn = 0;
        for (uint32_t ch = lane; ch < nchunk; ch += 32) {
          const uint4 xv = __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)x * row_bytes) + ch);
          xb[ch] = xv;
          acc_chunk<T, kMetricIP>(xv, xv, xn);
        }
        xn = __reduce_add_sync(FULL, xn);
        __syncwarp();
        unsigned long long k[kMaxKRepair / 32];
#pragma unroll
        for (int ps = 0; ps < (int)(kMaxKRepair / 32); ++ps) {
          k[ps] = kKeyMax;
          if ((uint32_t)ps * 32u < nc) {
            const uint32_t j = (uint32_t)ps * 32u + lane;
            const uint4* cr = reinterpret_cast<const uint4*>(crow + (size_t)min(j, nc - 1u) * rs);
            int dot = 0;
#pragma unroll 2
            for (uint32_t ch = 0; ch < nchunk; ++ch) acc_chunk<T, kMetricIP>(xb[ch], cr[ch], dot);
            if (j < nc) {
              const uint32_t y = key_id(ckeys[j]);
              if (y != x) {
                k[ps] = make_key(xn + cnorm[j] - 2 * dot, y);
                ++npair;
              }
            }
          }
        }
        __syncwarp();
        for (uint32_t r = 0; r < c; ++r) {  // r-th smallest (dist, id)
          unsigned long long mine = k[0];
#pragma unroll
          for (int ps = 1; ps < (int)(kMaxKRepair / 32); ++ps) mine = min(mine, k[ps]);
          const unsigned long long best = warp_min_key(mine);
#pragma unroll
          for (int ps = 0; ps < (int)(kMaxKRepair / 32); ++ps)
            if (k[ps] == best) k[ps] = kKeyMax;
          if (lane == 0) {
            if (best == kKeyMax) {
              a.req_tgt[rbase + r] = kInvalid;
            } else if (is_in) {
              a.req_tgt[rbase + r] = x;
              a.req_key[rbase + r] = best;
            } else {
              a.req_tgt[rbase + r] = key_id(best);
              a.req_key[rbase + r] = (best & 0xFFFFFFFF00000000ull) | x;
            }
          }
        }
        continue;
      }
      uint4 xr[CPL];
      load_row<G, CPL>(a.g.store + (size_t)x * row_bytes, nchunk, t, xr);
      for (uint32_t jb = 0; jb < nc; jb += NT) {
        const uint32_t j = jb + team;
        unsigned long long kc = 0;
        uint4 v[CPL];
        if (j < nc) {
          kc = ckeys[j];
#pragma unroll
          for (int cc = 0; cc < CPL; ++cc) {
            const uint32_t ch = t + cc * G;
            v[cc] = ch < nchunk ? reinterpret_cast<const uint4*>(crow + (size_t)j * rs)[ch] : make_uint4(0, 0, 0, 0);
          }
        } else {
#pragma unroll
          for (int cc = 0; cc < CPL; ++cc) v[cc] = make_uint4(0, 0, 0, 0);
        }
        const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(xr, v);
        if (t == 0 && j < nc) {
          const uint32_t y = key_id(kc);
          keys[j] = y != x ? make_key(d, y) : kKeyMax;
          npair += y != x;
        }
      }
      __syncwarp();
      for (uint32_t r = 0; r < c; ++r) {  // r-th smallest (dist, id)
        unsigned long long best = kKeyMax;
        for (uint32_t j = lane; j < nc; j += 32) best = min(best, keys[j]);
        best = warp_min_key(best);
        if (best != kKeyMax) {
          for (uint32_t j = lane; j < nc; j += 32)
            if (keys[j] == best) keys[j] = kKeyMax;
        }
        if (lane == 0) {
          if (best == kKeyMax) {
            a.req_tgt[rbase + r] = kInvalid;
          } else if (is_in) {
            a.req_tgt[rbase + r] = x;
            a.req_key[rbase + r] = best;
          } else {
            a.req_tgt[rbase + r] = key_id(best);
            a.req_key[rbase + r] = (best & 0xFFFFFFFF00000000ull) | x;
          }
        }
        __syncwarp();
      }
    }
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_PK_PAIRS], npair);
  }
  if (nrows) atomicAdd(&a.state->counters[CTR_PK_BYTES], nrows * row_bytes);
}

// ---- tensor-core variant for integer rows.  All pairs (x, y) of one deleted node, x among its surviving in- and
// out-neighbours and y in C_i, need dist(x, y): a dense cross-distance block.  With
// |x - y|^2 = |x|^2 + |y|^2 - 2 x.y the cross term is an integer matrix product X * C_i^T, exact in int32, which
// the tensor cores take as 8-bit mma tiles (m16n8k32).  A work unit is up to kMmaUnitPairs rows of X for one node:
// the block stages the unit's x rows and the candidate rows (zero-padded to 32-byte steps, on a stride that keeps
// the fragment loads free of bank conflicts), each warp multiplies 16-row tiles against all candidate tiles and
// then picks the c smallest (dist, id) per row out of the accumulators.
constexpr uint32_t kMmaUnitPairs = 128;
constexpr int kMmaNTiles = 7;  // candidate tiles of 8: k_repair <= 56
constexpr int kMmaWarps = 4;

static size_t delete_picks_mma_smem(uint32_t row_bytes) {
  const size_t rs = ((row_bytes + 31u) & ~31u) + 16u;
  return (size_t)(kMmaUnitPairs + kMmaNTiles * 8) * rs + (size_t)kMmaNTiles * 8 * 12 + (size_t)kMmaUnitPairs * 8;
}

template <typename T>
__global__ void __launch_bounds__(kMmaWarps * 32) delete_picks_mma_kernel(const DeleteArgs a, const uint64_t total_in) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr uint32_t NC = kMmaNTiles * 8;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const uint32_t R = a.g.R, c = a.c, kr = a.k_repair;
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint32_t kb = (row_bytes + 31u) & ~31u, rs = kb + 16u, kch = kb / 16u, ksteps = kb / 32u;
  uint8_t* xrow = smem_raw;                                   // kMmaUnitPairs rows of X
  uint8_t* crow = xrow + (size_t)kMmaUnitPairs * rs;          // NC candidate rows
  unsigned long long* ckeys = reinterpret_cast<unsigned long long*>(crow + (size_t)NC * rs);
  int* cnorm = reinterpret_cast<int*>(ckeys + NC);
  int* xnorm = cnorm + NC;
  uint32_t* xid = reinterpret_cast<uint32_t*>(xnorm + kMmaUnitPairs);
  const uint32_t nunits = a.unit_off[a.n];
  unsigned long long npair = 0, nrows = 0;
  for (uint32_t unit = blockIdx.x; unit < nunits; unit += gridDim.x) {
    uint32_t lo = 0, hi = (uint32_t)a.n;  // largest i with unit_off[i] <= unit
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (a.unit_off[mid] <= unit) lo = mid; else hi = mid;
    }
    const uint32_t i = lo, p = a.ids[i];
    const uint32_t nin = a.pair_off[i + 1] - a.pair_off[i];
    const uint32_t q0 = (unit - a.unit_off[i]) * kMmaUnitPairs, q1 = min(nin + R, q0 + kMmaUnitPairs);
    const uint32_t M = q1 - q0, nc = min(a.Ci_n[i], NC);
    __syncthreads();  // the previous unit's readers are done with the staged rows
    for (uint32_t j = threadIdx.x; j < NC; j += blockDim.x) ckeys[j] = j < nc ? a.Ci[(size_t)i * kr + j] : kKeyMax;
    for (uint32_t e = threadIdx.x; e < NC * kch; e += blockDim.x) {
      const uint32_t j = e / kch, ch = e - j * kch;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (j < nc && ch < nchunk)
        v = __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)key_id(a.Ci[(size_t)i * kr + j]) * row_bytes) + ch);
      reinterpret_cast<uint4*>(crow + (size_t)j * rs)[ch] = v;
    }
    for (uint32_t j = threadIdx.x; j < kMmaUnitPairs; j += blockDim.x) {
      const uint32_t q = q0 + j;
      uint32_t x = kInvalid;
      if (j < M) {
        if (q < nin) {
          x = a.src[in_base(a, i) + q];
        } else if (q - nin < a.g.deg[p]) {
          x = a.g.adj[(size_t)p * R + (q - nin)];
        }
        if (x != kInvalid && (bit_test(a.delmap, x) || (a.livemap && !bit_test(a.livemap, x)))) x = kInvalid;
      }
      xid[j] = x;
    }
    __syncthreads();
    for (uint32_t e = threadIdx.x; e < kMmaUnitPairs * kch; e += blockDim.x) {
      const uint32_t j = e / kch, ch = e - j * kch;
      const uint32_t x = xid[j];
      uint4 v = make_uint4(0, 0, 0, 0);
      if (x != kInvalid && ch < nchunk) v = __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)x * row_bytes) + ch);
      reinterpret_cast<uint4*>(xrow + (size_t)j * rs)[ch] = v;
    }
    __syncthreads();
    for (uint32_t j = threadIdx.x; j < kMmaUnitPairs + NC; j += blockDim.x) {  // squared norms of all staged rows
      const uint4* rp = reinterpret_cast<const uint4*>(j < kMmaUnitPairs ? xrow + (size_t)j * rs : crow + (size_t)(j - kMmaUnitPairs) * rs);
      int acc = 0;
      for (uint32_t ch = 0; ch < nchunk; ++ch) acc_chunk<T, kMetricIP>(rp[ch], rp[ch], acc);
      if (j < kMmaUnitPairs) xnorm[j] = acc; else cnorm[j - kMmaUnitPairs] = acc;
    }
    __syncthreads();
    for (uint32_t mt = warp; mt * 16u < M; mt += kMmaWarps) {
      int acc[kMmaNTiles][4];
#pragma unroll
      for (int nt = 0; nt < kMmaNTiles; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0;
      const uint8_t* xr0 = xrow + (size_t)(mt * 16u + gid) * rs + tig * 4;
      const uint8_t* xr1 = xr0 + 8 * (size_t)rs;
      const uint8_t* cr = crow + (size_t)gid * rs + tig * 4;
      for (uint32_t ks = 0; ks < ksteps; ++ks) {
        uint32_t xa[4];
        xa[0] = *reinterpret_cast<const uint32_t*>(xr0 + ks * 32);
        xa[1] = *reinterpret_cast<const uint32_t*>(xr1 + ks * 32);
        xa[2] = *reinterpret_cast<const uint32_t*>(xr0 + ks * 32 + 16);
        xa[3] = *reinterpret_cast<const uint32_t*>(xr1 + ks * 32 + 16);
#pragma unroll
        for (int nt = 0; nt < kMmaNTiles; ++nt) {
          uint32_t yb[2];
          yb[0] = *reinterpret_cast<const uint32_t*>(cr + (size_t)nt * 8 * rs + ks * 32);
          yb[1] = *reinterpret_cast<const uint32_t*>(cr + (size_t)nt * 8 * rs + ks * 32 + 16);
          mma_m16n8k32<T>(acc[nt], xa, yb);
        }
      }
      // accumulator element (nt, h * 2 + jj) of this lane: row mt * 16 + gid + 8 h, candidate nt * 8 + tig * 2 + jj
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t r = mt * 16u + gid + 8u * h;
        const uint32_t x = xid[r];
        const int xn = xnorm[r];
        const uint32_t q = q0 + r;
        const bool is_in = q < nin;
        const uint64_t rbase = is_in ? ((uint64_t)a.pair_off[i] + q) * c : (total_in + (uint64_t)i * R + (q - nin)) * c;
        unsigned long long prev = 0;  // every key is larger (order-preserving distance bits are non-zero)
        for (uint32_t round = 0; round < c; ++round) {
          unsigned long long best = kKeyMax;  // smallest key above the previous round's pick
#pragma unroll
          for (int nt = 0; nt < kMmaNTiles; ++nt) {
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
              const uint32_t n = nt * 8 + tig * 2 + jj;
              const unsigned long long kc = ckeys[n];
              const uint32_t y = key_id(kc);
              if (kc != kKeyMax && y != x) {
                const unsigned long long key = make_key(xn + cnorm[n] - 2 * acc[nt][h * 2 + jj], y);
                if (key > prev && key < best) best = key;
              }
            }
          }
          best = min(best, __shfl_xor_sync(FULL, best, 1));
          best = min(best, __shfl_xor_sync(FULL, best, 2));
          if (tig == 0 && r < M) {
            if (x == kInvalid || best == kKeyMax) {
              a.req_tgt[rbase + round] = kInvalid;
            } else if (is_in) {
              a.req_tgt[rbase + round] = x;
              a.req_key[rbase + round] = best;
            } else {
              a.req_tgt[rbase + round] = key_id(best);
              a.req_key[rbase + round] = (best & 0xFFFFFFFF00000000ull) | x;
            }
          }
          prev = best;
        }
        if (tig == 0 && r < M && x != kInvalid) {
          npair += nc;
          ++nrows;  // x's row, fetched once per pair
        }
      }
    }
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_PK_PAIRS], npair);
  }
  if (nrows) atomicAdd(&a.state->counters[CTR_PK_BYTES], nrows * row_bytes);
}

// ---- register-tiled variant for fp32 rows of at most 384 bytes (teams of at most 4 lanes).  The pairs (x, y) of one
// deleted node form a dense block of distances, x among its surviving in- and out-neighbours and y in C_i.  A work
// unit stages up to kTileUnitPairs x rows and the candidate rows in shared memory; a thread owns a tile of 2 x rows by
// 4 candidates, so six 16-byte shared-memory loads feed 64 arithmetic instructions, where a team per pair needs one
// load per eight (the staged kernel spends its time on the shared-memory pipe and on per-pair bookkeeping).
// Every distance is summed in exactly the order a team of G lanes uses (lane t of a team takes chunks t, t + G, ...
// in sequence, then the lanes' partial sums fold pairwise), so the keys are bit for bit the ones the other kernels
// compute for the same pair.  Each thread keeps the c smallest keys of its part of a row; the four threads that share
// a row then merge their heads.
// 16 bytes global -> shared without a round trip through registers; the copies of one thread complete in order of
// issue and are awaited together
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  const unsigned sa = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gsrc));
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr uint32_t kTileUnitPairs = 64;
constexpr int kTileWarps = 4;
constexpr int kTileMaxC = 4;

static size_t delete_picks_tile_smem(uint32_t nchunk, uint32_t k_repair) {
  const size_t rs = (size_t)(nchunk | 1u) * 16u, kr16 = (k_repair + 15u) & ~15u;
  return (kTileUnitPairs + kr16) * rs + kr16 * 8 + kTileUnitPairs * 4;
}

template <int G, int CPL>
__global__ void __launch_bounds__(kTileWarps * 32) delete_picks_tile_kernel(const DeleteArgs a, const uint64_t total_in) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int xr = lane >> 2, cg = lane & 3;
  const uint32_t R = a.g.R, c = a.c, kr = a.k_repair, kr16 = (kr + 15u) & ~15u;
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint32_t rs = (nchunk | 1u) * 16u;  // odd number of chunks: rows of neighbouring lanes fall on different banks
  uint8_t* xrow = smem_raw;
  uint8_t* crow = xrow + (size_t)kTileUnitPairs * rs;
  unsigned long long* ckeys = reinterpret_cast<unsigned long long*>(crow + (size_t)kr16 * rs);
  uint32_t* xid = reinterpret_cast<uint32_t*>(ckeys + kr16);
  const uint32_t nunits = a.unit_off[a.n];
  unsigned long long npair = 0, nrows = 0;
  for (uint32_t unit = blockIdx.x; unit < nunits; unit += gridDim.x) {
    uint32_t lo = 0, hi = (uint32_t)a.n;  // largest i with unit_off[i] <= unit
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (a.unit_off[mid] <= unit) lo = mid; else hi = mid;
    }
    const uint32_t i = lo, p = a.ids[i];
    const uint32_t nin = a.pair_off[i + 1] - a.pair_off[i];
    const uint32_t q0 = (unit - a.unit_off[i]) * kTileUnitPairs, q1 = min(nin + R, q0 + kTileUnitPairs);
    const uint32_t M = q1 - q0, nc = min(a.Ci_n[i], kr);
    __syncthreads();  // the previous unit's readers are done with the staged rows
    for (uint32_t j = threadIdx.x; j < kr16; j += blockDim.x) ckeys[j] = j < nc ? a.Ci[(size_t)i * kr + j] : kKeyMax;
    // the candidate rows are on their way (asynchronous copies) while the x ids are resolved
    for (uint32_t e = threadIdx.x; e < kr16 * nchunk; e += blockDim.x) {
      const uint32_t j = e / nchunk, ch = e - j * nchunk;
      uint4* dst = reinterpret_cast<uint4*>(crow + (size_t)j * rs) + ch;
      if (j < nc) cp_async16(dst, reinterpret_cast<const uint4*>(a.g.store + (size_t)key_id(a.Ci[(size_t)i * kr + j]) * row_bytes) + ch);
      else *dst = make_uint4(0, 0, 0, 0);
    }
    for (uint32_t j = threadIdx.x; j < kTileUnitPairs; j += blockDim.x) {
      const uint32_t q = q0 + j;
      uint32_t x = kInvalid;
      if (j < M) {
        if (q < nin) {
          x = a.src[in_base(a, i) + q];
        } else if (q - nin < a.g.deg[p]) {
          x = a.g.adj[(size_t)p * R + (q - nin)];
        }
        if (x != kInvalid && (bit_test(a.delmap, x) || (a.livemap && !bit_test(a.livemap, x)))) x = kInvalid;
      }
      xid[j] = x;
    }
    __syncthreads();
    for (uint32_t e = threadIdx.x; e < kTileUnitPairs * nchunk; e += blockDim.x) {
      const uint32_t j = e / nchunk, ch = e - j * nchunk;
      const uint32_t x = xid[j];
      uint4* dst = reinterpret_cast<uint4*>(xrow + (size_t)j * rs) + ch;
      if (x != kInvalid) cp_async16(dst, reinterpret_cast<const uint4*>(a.g.store + (size_t)x * row_bytes) + ch);
      else *dst = make_uint4(0, 0, 0, 0);
    }
    cp_async_wait_all();
    __syncthreads();
    // this thread's two x rows and its running picks for them
    const uint32_t r0 = (uint32_t)warp * 16u + (uint32_t)xr * 2u;
    const uint4* xp0 = reinterpret_cast<const uint4*>(xrow + (size_t)r0 * rs);
    const uint4* xp1 = reinterpret_cast<const uint4*>(xrow + (size_t)(r0 + 1) * rs);
    const uint32_t x0 = xid[r0], x1 = xid[r0 + 1];
    unsigned long long best[2][kTileMaxC];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int r = 0; r < kTileMaxC; ++r) best[h][r] = kKeyMax;
    if ((uint32_t)warp * 16u < M) {  // (uniform per warp: a warp without pairs only keeps the barriers company)
      for (uint32_t cb = 0; cb < nc; cb += 16) {
        float acc[2][4][G];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int t = 0; t < G; ++t) acc[h][jj][t] = 0.0f;
        const uint4* cp = reinterpret_cast<const uint4*>(crow + (size_t)(cb + cg) * rs);
        const uint32_t cstep = 4u * (rs / 16u);  // candidate cb + cg + 4 jj
        // (candidate rows beyond nc are staged as zeros and carry the invalid key: a block is always swept whole -
        // skipping the empty groups of the last block was measured and is slower)
#pragma unroll
        for (int cc = 0; cc < CPL; ++cc) {
#pragma unroll
          for (int t = 0; t < G; ++t) {
            const uint32_t ch = (uint32_t)(t + cc * G);
            if (ch < nchunk) {  // (uniform)
              const uint4 xa = xp0[ch], xb = xp1[ch];
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                const uint4 yv = cp[(size_t)jj * cstep + ch];
                acc_chunk<float, kMetricL2>(xa, yv, acc[0][jj][t]);
                acc_chunk<float, kMetricL2>(xb, yv, acc[1][jj][t]);
              }
            }
          }
        }
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const unsigned long long kc = ckeys[cb + cg + 4 * jj];
          const uint32_t y = key_id(kc);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float d;
            if constexpr (G == 4) d = (acc[h][jj][0] + acc[h][jj][2]) + (acc[h][jj][1] + acc[h][jj][3]);
            else if constexpr (G == 2) d = acc[h][jj][0] + acc[h][jj][1];
            else d = acc[h][jj][0];
            const uint32_t x = h ? x1 : x0;
            unsigned long long key = (kc != kKeyMax && y != x) ? make_key(d, y) : kKeyMax;
            // keep the c smallest seen so far, ascending
#pragma unroll
            for (int r = 0; r < kTileMaxC; ++r) {
              if ((uint32_t)r < c && key < best[h][r]) {
                const unsigned long long tmp = best[h][r];
                best[h][r] = key;
                key = tmp;
              }
            }
          }
        }
      }
      // ---- the four threads that share a row merge their heads: round r takes the smallest head, its owner pops
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t r = r0 + h, x = h ? x1 : x0;
        const uint32_t q = q0 + r;
        const bool is_in = q < nin;
        const uint64_t rbase = is_in ? ((uint64_t)a.pair_off[i] + q) * c : (total_in + (uint64_t)i * R + (q - nin)) * c;
        for (uint32_t round = 0; round < c; ++round) {
          unsigned long long m = best[h][0];
          m = min(m, __shfl_xor_sync(FULL, m, 1));
          m = min(m, __shfl_xor_sync(FULL, m, 2));
          if (m != kKeyMax && best[h][0] == m) {  // keys are distinct (one id per candidate): exactly one owner
#pragma unroll
            for (int rr = 0; rr + 1 < kTileMaxC; ++rr) best[h][rr] = best[h][rr + 1];
            best[h][kTileMaxC - 1] = kKeyMax;
          }
          if (cg == 0 && r < M) {
            if (x == kInvalid || m == kKeyMax) {
              a.req_tgt[rbase + round] = kInvalid;
            } else if (is_in) {
              a.req_tgt[rbase + round] = x;
              a.req_key[rbase + round] = m;
            } else {
              a.req_tgt[rbase + round] = key_id(m);
              a.req_key[rbase + round] = (m & 0xFFFFFFFF00000000ull) | x;
            }
          }
        }
        if (cg == 0 && r < M && x != kInvalid) {
          npair += nc;
          ++nrows;  // x's row, fetched once per pair
        }
      }
    }
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_PK_PAIRS], npair);
  }
  if (nrows) atomicAdd(&a.state->counters[CTR_PK_BYTES], nrows * row_bytes);
}

// unit_owner[u] = the batch member whose rows unit u covers (largest i with unit_off[i] <= u)
__global__ void delete_unit_owner_kernel(const DeleteArgs a) {
  const uint32_t nunits = a.unit_off[a.n];
  for (uint32_t u = blockIdx.x * blockDim.x + threadIdx.x; u < nunits; u += gridDim.x * blockDim.x) {
    uint32_t lo = 0, hi = (uint32_t)a.n;
    while (hi - lo > 1) {
      const uint32_t mid = (lo + hi) >> 1;
      if (a.unit_off[mid] <= u) lo = mid; else hi = mid;
    }
    a.unit_owner[u] = lo;
  }
}

// ---- register-tiled variant for wide fp32 rows (teams of 32 lanes: a warp is one team).  Neither the candidate
// rows nor a useful number of x rows fit shared memory at 2 to 4 KB a row, and a team per pair re-reads a candidate
// row from L2 for every pair.  Here a warp owns a tile of 8 x rows by 8 candidates: lane t walks its chunks t, t + 32,
// ... of all sixteen rows (coalesced 512-byte slices straight from L2) and carries 64 partial sums, so a row slice is
// loaded once per eight pairs.  The 64 per-lane partials then fold across the lanes in the order a team uses (offsets
// 16, 8, 4, 2, 1): at each step a lane keeps the half of the sums that its bit selects and trades the other half, which
// gives every lane the same bits the butterfly gives it, for two of the 64 pairs, in 62 shuffles instead of 320.
// The c smallest keys per x row are kept per lane and merged over the four lanes that share a row.
constexpr uint32_t kWideRows = 8;
constexpr int kWideCands = 8;
template <int CPL>
__global__ void __launch_bounds__(kPickWarps * 32, 3) delete_picks_wide_kernel(const DeleteArgs a, const uint64_t total_in) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int XT = (int)kWideRows, CT = kWideCands;
  __shared__ uint32_t xid_s[kPickWarps][XT];
  __shared__ unsigned long long ck_s[kPickWarps][kMaxKRepair];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t R = a.g.R, c = a.c, kr = a.k_repair;
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint32_t nunits = a.unit_off[a.n];
  unsigned long long npair = 0, nrows = 0;
  // Neighbouring warps take neighbouring units, i.e. tiles of the same deleted node: its candidate rows are then in
  // use by many warps at once and stay in L2 (a contiguous run of units per warp was measured: every warp then
  // works on another node, the candidate rows of all of them exceed L2, and the kernel is 1.4x slower).  The owner
  // of each unit comes from a table written by delete_unit_owner_kernel: a binary search over the prefix here is
  // a chain of dependent loads half as long as a unit's arithmetic.
  for (uint32_t unit = blockIdx.x * kPickWarps + warp; unit < nunits; unit += gridDim.x * kPickWarps) {
    const uint32_t i = a.unit_owner[unit];
    const uint32_t p = a.ids[i];
    const uint32_t nin = a.pair_off[i + 1] - a.pair_off[i];
    const uint32_t q0 = (unit - a.unit_off[i]) * kWideRows, q1 = min(nin + R, q0 + kWideRows);
    const uint32_t M = q1 - q0, nc = min(a.Ci_n[i], kr);
    __syncwarp();  // the previous unit's readers are done with the warp's lists
    if (lane < XT) {
      const uint32_t q = q0 + lane;
      uint32_t x = kInvalid;
      if ((uint32_t)lane < M) {
        if (q < nin) {
          x = a.src[in_base(a, i) + q];
        } else if (q - nin < a.g.deg[p]) {
          x = a.g.adj[(size_t)p * R + (q - nin)];
        }
        if (x != kInvalid && (bit_test(a.delmap, x) || (a.livemap && !bit_test(a.livemap, x)))) x = kInvalid;
      }
      xid_s[warp][lane] = x;
    }
    const uint32_t ncp = (nc + CT - 1) / CT * CT;
    for (uint32_t j = lane; j < ncp; j += 32) ck_s[warp][j] = j < nc ? a.Ci[(size_t)i * kr + j] : kKeyMax;
    __syncwarp();
    // (row ids rather than pointers are carried: 16 registers instead of 32, and the address is one multiply-add)
    uint32_t xi[XT];
#pragma unroll
    for (int h = 0; h < XT; ++h) xi[h] = xid_s[warp][h];
    const int myrow = lane >> 2, cg = lane & 3;
    const uint32_t myx = xid_s[warp][myrow];
    unsigned long long best[kTileMaxC];
#pragma unroll
    for (int r = 0; r < kTileMaxC; ++r) best[r] = kKeyMax;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    for (uint32_t cb = 0; cb < nc; cb += CT) {
      float acc[XT * CT];
#pragma unroll
      for (int e = 0; e < XT * CT; ++e) acc[e] = 0.0f;
      uint32_t yi[CT];
#pragma unroll
      for (int j = 0; j < CT; ++j) {
        const unsigned long long kc = ck_s[warp][cb + j];
        yi[j] = kc != kKeyMax ? key_id(kc) : kInvalid;
      }
#pragma unroll 1
      for (int cc = 0; cc < CPL; ++cc) {
        const uint32_t ch = (uint32_t)lane + 32u * (uint32_t)cc;
        const bool inb = ch < nchunk;
        // all sixteen slices are requested before the first is used: one round trip to L2 per step, not nine
        uint4 xv[XT], yv[CT];
#pragma unroll
        for (int h = 0; h < XT; ++h)
          xv[h] = inb && xi[h] != kInvalid ? __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)xi[h] * row_bytes) + ch) : zero4;
#pragma unroll
        for (int j = 0; j < CT; ++j)
          yv[j] = inb && yi[j] != kInvalid ? __ldg(reinterpret_cast<const uint4*>(a.g.store + (size_t)yi[j] * row_bytes) + ch) : zero4;
#pragma unroll
        for (int j = 0; j < CT; ++j)
#pragma unroll
          for (int h = 0; h < XT; ++h) acc_chunk<float, kMetricL2>(xv[h], yv[j], acc[h * CT + j]);
      }
      // ---- fold over the lanes; afterwards this lane holds the sums of pairs 2 * lane and 2 * lane + 1
      //      (pair e = row * 8 + candidate: row lane / 4, candidates 2 * (lane % 4) and + 1)
      float r32[32], r16[16], r8[8], r4[4], r2[2];
      {
        const bool up = lane & 16;
#pragma unroll
        for (int k = 0; k < 32; ++k) r32[k] = (up ? acc[k + 32] : acc[k]) + __shfl_xor_sync(FULL, up ? acc[k] : acc[k + 32], 16);
      }
      {
        const bool up = lane & 8;
#pragma unroll
        for (int k = 0; k < 16; ++k) r16[k] = (up ? r32[k + 16] : r32[k]) + __shfl_xor_sync(FULL, up ? r32[k] : r32[k + 16], 8);
      }
      {
        const bool up = lane & 4;
#pragma unroll
        for (int k = 0; k < 8; ++k) r8[k] = (up ? r16[k + 8] : r16[k]) + __shfl_xor_sync(FULL, up ? r16[k] : r16[k + 8], 4);
      }
      {
        const bool up = lane & 2;
#pragma unroll
        for (int k = 0; k < 4; ++k) r4[k] = (up ? r8[k + 4] : r8[k]) + __shfl_xor_sync(FULL, up ? r8[k] : r8[k + 4], 2);
      }
      {
        const bool up = lane & 1;
#pragma unroll
        for (int k = 0; k < 2; ++k) r2[k] = (up ? r4[k + 2] : r4[k]) + __shfl_xor_sync(FULL, up ? r4[k] : r4[k + 2], 1);
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const unsigned long long kc = ck_s[warp][cb + 2 * cg + k];
        const uint32_t y = key_id(kc);
        unsigned long long key = (kc != kKeyMax && y != myx) ? make_key(r2[k], y) : kKeyMax;
#pragma unroll
        for (int r = 0; r < kTileMaxC; ++r) {
          if ((uint32_t)r < c && key < best[r]) {
            const unsigned long long tmp = best[r];
            best[r] = key;
            key = tmp;
          }
        }
      }
    }
    // ---- the four lanes that share a row merge their heads: round r takes the smallest head, its owner pops
    {
      const uint32_t r = (uint32_t)myrow, x = myx;
      const uint32_t q = q0 + r;
      const bool is_in = q < nin;
      const uint64_t rbase = is_in ? ((uint64_t)a.pair_off[i] + q) * c : (total_in + (uint64_t)i * R + (q - nin)) * c;
      for (uint32_t round = 0; round < c; ++round) {
        unsigned long long m = best[0];
        m = min(m, __shfl_xor_sync(FULL, m, 1));
        m = min(m, __shfl_xor_sync(FULL, m, 2));
        if (m != kKeyMax && best[0] == m) {  // keys are distinct (one id per candidate): exactly one owner
#pragma unroll
          for (int rr = 0; rr + 1 < kTileMaxC; ++rr) best[rr] = best[rr + 1];
          best[kTileMaxC - 1] = kKeyMax;
        }
        if (cg == 0 && r < M) {
          if (x == kInvalid || m == kKeyMax) {
            a.req_tgt[rbase + round] = kInvalid;
          } else if (is_in) {
            a.req_tgt[rbase + round] = x;
            a.req_key[rbase + round] = m;
          } else {
            a.req_tgt[rbase + round] = key_id(m);
            a.req_key[rbase + round] = (m & 0xFFFFFFFF00000000ull) | x;
          }
        }
      }
      if (cg == 0 && r < M && x != kInvalid) {
        npair += nc;
        ++nrows;  // x's row, fetched once per pair
      }
    }
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_PK_PAIRS], npair);
  }
  if (nrows) atomicAdd(&a.state->counters[CTR_PK_BYTES], nrows * row_bytes);
}

// Which pick kernel serves this index: 4 = warp tiles straight from L2 (fp32 rows above 512 bytes, c <= 4),
// 3 = register tiles (fp32 rows up to 384 bytes, c <= 4), 2 = tensor-core tiles
// (integer rows up to 256 bytes, k_repair <= 56), 1 = candidate rows staged in shared memory, 0 = rows straight from L2.
template <typename T>
static int picks_variant(const DeleteArgs& a) {
#ifndef GRAND_NO_TILE_PICKS
  if (sizeof(T) == 4 && a.lay.G <= 4 && a.c <= (uint32_t)kTileMaxC && a.lay.metric == kMetricL2) return 3;
#endif
#ifndef GRAND_NO_WIDE_PICKS
  if (sizeof(T) == 4 && a.lay.G == 32 && a.c <= (uint32_t)kTileMaxC && a.k_repair <= kMaxKRepair && a.lay.metric == kMetricL2) return 4;
#endif
  if (sizeof(T) == 1 && a.k_repair <= (uint32_t)kMmaNTiles * 8u && a.lay.row_bytes <= 256u) return 2;
  const size_t stage = (size_t)a.k_repair * ((a.lay.nchunk | 1u) * 16u);
  return stage <= 64 * 1024 ? 1 : 0;
}

template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_delete_picks_prepare_t(const DeleteArgs& a, uint64_t total_in, cudaStream_t s) {
  const uint64_t total = total_in + a.n * a.g.R;
  if (total == 0) return cudaSuccess;
  if (total_in) {
    uint64_t tb = (total_in + 255) / 256;
    if (tb > (uint64_t)sm_count() * 32u) tb = (uint64_t)sm_count() * 32u;
    delete_touch_kernel<<<(unsigned)tb, 256, 0, s>>>(a, total_in);
    count_launches(1);
  }
  const int variant = picks_variant<T>(a);
  if (variant == 0) return cudaGetLastError();
  const uint64_t cap16 = (uint64_t)sm_count() * 16u;
  const unsigned ub = (unsigned)((a.n + 256) / 256 > cap16 ? cap16 : (a.n + 256) / 256);
  delete_units_kernel<<<ub, 256, 0, s>>>(a, variant == 4 ? kWideRows : variant == 3 ? kTileUnitPairs : variant == 2 ? kMmaUnitPairs : kUnitPairs);
  count_launches(1);
  cudaError_t e = launch_exclusive_scan(a.in_cnt, a.unit_off, a.n + 1, a.scan_tmp, s);
  if (e != cudaSuccess || variant != 4) return e;
  delete_unit_owner_kernel<<<(unsigned)sm_count() * 8u, 256, 0, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_delete_picks_t(const DeleteArgs& a, uint64_t total_in, cudaStream_t s) {
  const uint64_t total = total_in + a.n * a.g.R;
  if (total == 0) return cudaSuccess;
  const int variant = picks_variant<T>(a);
  const uint64_t sms = (uint64_t)sm_count();
  if constexpr (sizeof(T) == 1) {
    if (variant == 2) {
      const size_t smem = delete_picks_mma_smem(a.lay.row_bytes);
      auto kern = delete_picks_mma_kernel<T>;
      static SmemOptIn optin{};
      cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
      if (e != cudaSuccess) return e;
      uint64_t blocks = (total + kMmaUnitPairs - 1) / kMmaUnitPairs + a.n;  // upper bound on the number of units
      if (blocks > sms * 8u) blocks = sms * 8u;
      kern<<<(unsigned)blocks, kMmaWarps * 32, smem, s>>>(a, total_in);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  if constexpr (sizeof(T) == 4 && G <= 4) {
    if (variant == 3) {
      const size_t smem = delete_picks_tile_smem(a.lay.nchunk, a.k_repair);
      auto kern = delete_picks_tile_kernel<G, CPL>;
      static SmemOptIn optin{};
      cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
      if (e != cudaSuccess) return e;
      uint64_t blocks = (total + kTileUnitPairs - 1) / kTileUnitPairs + a.n;  // upper bound on the number of units
      if (blocks > sms * 8u) blocks = sms * 8u;
      kern<<<(unsigned)blocks, kTileWarps * 32, smem, s>>>(a, total_in);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  if constexpr (sizeof(T) == 4 && G == 32) {
    if (variant == 4) {
      uint64_t blocks = ((total + kWideRows - 1) / kWideRows + a.n + kPickWarps - 1) / kPickWarps;  // upper bound on the units
      if (blocks > sms * 3u) blocks = sms * 3u;
      delete_picks_wide_kernel<CPL><<<(unsigned)blocks, kPickWarps * 32, 0, s>>>(a, total_in);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  if (variant == 1) {
    // candidate rows fit shared memory: one staged copy per work unit
    const size_t stage = (size_t)a.k_repair * ((a.lay.nchunk | 1u) * 16u);
    const size_t smem = stage + ((size_t)((a.k_repair + 1u) & ~1u) + (size_t)kPickWarps * kMaxKRepair) * 8 +
                        (size_t)kPickWarps * a.lay.row_bytes + (size_t)a.k_repair * 4 + (size_t)kUnitPairs * 4;
    auto kern = delete_picks_staged_kernel<T, METRIC, G, CPL>;
    static SmemOptIn optin{};
    cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
    if (e != cudaSuccess) return e;
    uint64_t blocks = (total + kUnitPairs - 1) / kUnitPairs + a.n;  // upper bound on the number of units
    if (blocks > sms * 16u) blocks = sms * 16u;
    kern<<<(unsigned)blocks, kPickWarps * 32, smem, s>>>(a, total_in);
    count_launches(1);
    return cudaGetLastError();
  }
  uint64_t blocks = (total + kPickWarps - 1) / kPickWarps;
  if (blocks > sms * 16u) blocks = sms * 16u;
  delete_picks_kernel<T, METRIC, G, CPL><<<(unsigned)blocks, kPickWarps * 32, 0, s>>>(a, total_in);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_delete_picks_prepare(const DeleteArgs& a, uint64_t total_in, cudaStream_t s) {
  GRAND_DISPATCH_L2(a.lay, launch_delete_picks_prepare_t, a, total_in, s);
  return cudaErrorInvalidValue;
}
cudaError_t launch_delete_picks(const DeleteArgs& a, uint64_t total_in, cudaStream_t s) {
  GRAND_DISPATCH_L2(a.lay, launch_delete_picks_t, a, total_in, s);
  return cudaErrorInvalidValue;
}

// ---- fixed-degree delete (Alg. 8): mark every surviving in-neighbour of a deleted node dirty, then
// one warp per dirty node rewrites its deleted slots in slot order with PickOne.
__global__ void fixed_delete_mark_kernel(const FixedDeleteArgs a, const uint64_t total_in) {
  for (uint64_t pair = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; pair < total_in; pair += (uint64_t)gridDim.x * blockDim.x) {
    uint64_t lo = 0, hi = a.n;
    while (hi - lo > 1) {
      const uint64_t mid = (lo + hi) >> 1;
      if (a.pair_off[mid] <= pair) lo = mid; else hi = mid;
    }
    const uint32_t u = a.src[a.off[a.ids[lo]] + (uint32_t)(pair - a.pair_off[lo])];
    if (!bit_test(a.delmap, u) && atomicExch(&a.flag[u], 1u) == 0u) a.dirty[atomicAdd(&a.state->ndirty, 1u)] = u;
  }
}
// In-neighbour rows come out of the scatter in no particular order.  The rank of u in such a row is
// counted directly while the row is short; long rows (hubs: in-degrees are heavy-tailed, and every
// in-neighbour of a deleted hub asks for its own rank) are sorted once, so that the rank is a
// binary search instead of a pass over the row per in-neighbour.
constexpr uint32_t kRankLinear = 256;
constexpr uint32_t kSortRowSmem = 48 * 1024;  // entries of a long row sorted in shared memory
__global__ void __launch_bounds__(1024) fixed_delete_sort_rows_kernel(const FixedDeleteArgs a) {
  extern __shared__ uint32_t sort_sh[];  // kSortRowSmem entries, then the list of long rows and its length
  uint32_t* longrow = sort_sh + kSortRowSmem;
  uint32_t& nlong = sort_sh[kSortRowSmem + 1024];
  auto sync = [] { __syncthreads(); };
  const uint32_t tid = threadIdx.x;
  for (uint64_t base = (uint64_t)blockIdx.x * 1024u; base < a.n; base += (uint64_t)gridDim.x * 1024u) {
    if (tid == 0) nlong = 0;
    __syncthreads();
    if (base + tid < a.n) {
      const uint32_t p = a.ids[base + tid];
      if (a.off[p + 1] - a.off[p] > kRankLinear) longrow[atomicAdd(&nlong, 1u)] = p;
    }
    __syncthreads();
    const uint32_t nl = nlong;
    for (uint32_t r = 0; r < nl; ++r) {
      const uint32_t p = longrow[r];
      const uint32_t b = a.off[p], n = a.off[p + 1] - b;
      if (n <= kSortRowSmem) {
        for (uint32_t j = tid; j < n; j += 1024u) sort_sh[j] = a.src[b + j];
        __syncthreads();
        bitonic_sort_any(sort_sh, n, tid, 1024u, sync);
        for (uint32_t j = tid; j < n; j += 1024u) a.src[b + j] = sort_sh[j];
      } else {
        bitonic_sort_any(a.src + b, n, tid, 1024u, sync);
      }
      __syncthreads();
    }
  }
}
// The deleted slots of a row are found with one parallel bitmap test per 32 slots, and a deleted
// neighbour's row is staged once with its own parallel test, so that a dirty node costs a handful
// of dependent memory round trips instead of one per slot and per candidate.
__global__ void __launch_bounds__(128) fixed_delete_rewire_kernel(const FixedDeleteArgs a) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr uint32_t kMaxR = 128;
  __shared__ uint32_t rows[4][kMaxR];
  __shared__ uint32_t prows[4][kMaxR];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* row = rows[warp];
  uint32_t* prow = prows[warp];
  const uint32_t R = a.g.R;
  const uint32_t nd = a.state->ndirty;
  const uint64_t wglobal = (uint64_t)blockIdx.x * 4 + warp, wtotal = (uint64_t)gridDim.x * 4;
  uint32_t ndone = 0;
  for (uint64_t k = wglobal; k < nd; k += wtotal) {
    const uint32_t u = a.dirty[k];
    const uint32_t du = min(a.g.deg[u], R);
    uint32_t delw = 0;  // lane w: word w of the set of slots that hold a deleted neighbour
    for (uint32_t sb = 0; sb < du; sb += 32) {
      const uint32_t s = sb + lane;
      uint32_t v = kInvalid;
      if (s < du) {
        v = a.g.adj[(size_t)u * R + s];
        row[s] = v;
      }
      const unsigned bal = __ballot_sync(FULL, v != kInvalid && bit_test(a.delmap, v));
      if ((uint32_t)lane == (sb >> 5)) delw = bal;
    }
    __syncwarp();
    for (uint32_t w = 0; w * 32 < du; ++w) {
      uint32_t m = __shfl_sync(FULL, delw, w);
      while (m) {
        const uint32_t s = w * 32 + (uint32_t)__ffs(m) - 1u;
        m &= m - 1;
        const uint32_t p = row[s];
        // round-robin offset: rank of u among the in-neighbours of p
        const uint32_t b = a.off[p], e = a.off[p + 1];
        uint32_t rank = 0;
        if (e - b > kRankLinear) {  // sorted by fixed_delete_sort_rows_kernel
          uint32_t lo = b, hi = e;
          while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            if (a.src[mid] < u) lo = mid + 1; else hi = mid;
          }
          rank = lo - b;
        } else {
          for (uint32_t jb = b; jb < e; jb += 32) {
            const uint32_t j = jb + lane;
            rank += __popc(__ballot_sync(FULL, j < e && a.src[j] < u));
          }
        }
        const uint32_t np = min(a.g.deg[p], R);
        uint32_t okw = 0;  // lane x: word x of the set of p's neighbours that are alive and not u itself
        for (uint32_t ib = 0; ib < np; ib += 32) {
          const uint32_t i = ib + lane;
          bool ok = false;
          if (i < np) {
            const uint32_t c = a.g.adj[(size_t)p * R + i];
            prow[i] = c;
            ok = c != u && !bit_test(a.delmap, c);
          }
          const unsigned bal = __ballot_sync(FULL, ok);
          if ((uint32_t)lane == (ib >> 5)) okw = bal;
        }
        __syncwarp();
        uint32_t chosen = kInvalid;
        for (uint32_t tt = 0; tt < np && chosen == kInvalid; ++tt) {
          const uint32_t i = (rank + tt) % np;
          if (!((__shfl_sync(FULL, okw, i >> 5) >> (i & 31)) & 1u)) continue;
          const uint32_t cand = prow[i];
          bool inrow = false;
          for (uint32_t sb = 0; sb < du; sb += 32) inrow |= __any_sync(FULL, sb + lane < du && row[sb + lane] == cand);
          if (!inrow) chosen = cand;
        }
        __syncwarp();
        if (lane == 0) row[s] = chosen;
        __syncwarp();
      }
    }
    // stable compaction of the surviving slots
    uint32_t wr = 0;
    for (uint32_t sb = 0; sb < R; sb += 32) {
      const uint32_t s = sb + lane;
      const uint32_t v = s < du ? row[s] : kInvalid;
      const bool ok = v != kInvalid;
      const unsigned bal = __ballot_sync(FULL, ok);
      if (ok) a.g.adj[(size_t)u * R + wr + __popc(bal & ((1u << lane) - 1u))] = v;
      wr += __popc(bal);
    }
    for (uint32_t s = wr + lane; s < R; s += 32) a.g.adj[(size_t)u * R + s] = kInvalid;
    if (lane == 0) {
      a.g.deg[u] = wr;
      a.flag[u] = 0;
      ++ndone;
    }
    __syncwarp();
  }
  if (lane == 0 && ndone) atomicAdd(&a.state->counters[CTR_DIRTY], (unsigned long long)ndone);
}
cudaError_t launch_fixed_delete(const FixedDeleteArgs& a, uint64_t total_in, cudaStream_t s) {
  if (total_in) {
    uint64_t blocks = (total_in + 255) / 256;
    if (blocks > (uint64_t)sm_count() * 32u) blocks = (uint64_t)sm_count() * 32u;
    fixed_delete_mark_kernel<<<(unsigned)blocks, 256, 0, s>>>(a, total_in);
    count_launches(1);
  }
  if (total_in > kRankLinear) {  // otherwise no row is long
    auto kern = fixed_delete_sort_rows_kernel;
    static SmemOptIn optin{};
    cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
    if (e != cudaSuccess) return e;
    uint64_t blocks = (a.n + 1023) / 1024;
    if (blocks > (uint64_t)sm_count()) blocks = (uint64_t)sm_count();
    kern<<<(unsigned)blocks, 1024, (kSortRowSmem + 1024 + 1) * sizeof(uint32_t), s>>>(a);
    count_launches(1);
  }
  fixed_delete_rewire_kernel<<<(unsigned)sm_count() * 8u, 128, 0, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

// ---- initial medoid: the batch point closest to the per-dimension mean (ties by id)
template <typename T>
__global__ void medoid_mean_kernel(const uint8_t* store, const uint32_t* ids, uint64_t n, uint32_t dim, uint32_t row_bytes,
                                   uint8_t* mean_row) {
  const uint32_t per_row = row_bytes / sizeof(T);
  for (uint32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < per_row; j += gridDim.x * blockDim.x) {
    T m = T(0);
    if (j < dim) {
      if constexpr (sizeof(T) == 4) {
        double s = 0.0;
        for (uint64_t i = 0; i < n; ++i) s += (double)reinterpret_cast<const float*>(store + (size_t)ids[i] * row_bytes)[j];
        m = (float)(s / (double)n);
      } else {
        long long s = 0;
        for (uint64_t i = 0; i < n; ++i) s += (long long)reinterpret_cast<const T*>(store + (size_t)ids[i] * row_bytes)[j];
        const long long num = 2 * s + (long long)n, den = 2 * (long long)n;  // round-half-up via floor division
        long long q = num / den;
        if (num % den != 0 && num < 0) --q;
        m = (T)q;
      }
    }
    reinterpret_cast<T*>(mean_row)[j] = m;
  }
}
template <typename T, int METRIC, int G, int CPL>
__global__ void medoid_argmin_kernel(const uint8_t* store, const uint32_t* ids, uint64_t n, uint32_t row_bytes, uint32_t nchunk,
                                     const uint8_t* mean_row, DevState* st) {
  using Dist = typename Elem<T>::Dist;
  constexpr int NT = 32 / G;
  const int lane = threadIdx.x & 31;
  const int t = lane % G, team = lane / G;
  uint4 mr[CPL];
  load_row<G, CPL>(mean_row, nchunk, t, mr);
  const uint64_t wglobal = (blockIdx.x * (uint64_t)blockDim.x + threadIdx.x) >> 5;
  const uint64_t wtotal = ((uint64_t)gridDim.x * blockDim.x) >> 5;
  for (uint64_t b0 = wglobal * NT; b0 < n; b0 += wtotal * NT) {
    const uint64_t i = b0 + team;
    uint4 v[CPL];
    uint32_t id = kInvalid;
    if (i < n) {
      id = ids[i];
      load_row<G, CPL>(store + (size_t)id * row_bytes, nchunk, t, v);
    } else {
#pragma unroll
      for (int c = 0; c < CPL; ++c) v[c] = make_uint4(0, 0, 0, 0);
    }
    const Dist d = team_dist_regs<T, METRIC, G, CPL>(v, mr);
    if (t == 0 && id != kInvalid) atomicMin(&st->medoid_key, make_key(d, id));
  }
}
__global__ void medoid_begin_kernel(DevState* st) { st->medoid_key = kKeyMax; }
__global__ void medoid_end_kernel(DevState* st) {
  if (st->medoid_key != kKeyMax) st->entry = key_id(st->medoid_key);
}
template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_pick_medoid_t(const Layout& lay, const GraphView& g, const uint32_t* ids, uint64_t n, uint8_t* mean_row,
                                        DevState* st, cudaStream_t s) {
  medoid_begin_kernel<<<1, 1, 0, s>>>(st);
  medoid_mean_kernel<T><<<(lay.row_bytes / sizeof(T) + 127) / 128, 128, 0, s>>>(g.store, ids, n, lay.dim, lay.row_bytes, mean_row);
  uint64_t blocks = (n + 3) / 4;
  if (blocks > (uint64_t)sm_count() * 8u) blocks = (uint64_t)sm_count() * 8u;
  if (blocks < 1) blocks = 1;
  medoid_argmin_kernel<T, METRIC, G, CPL><<<(unsigned)blocks, 128, 0, s>>>(g.store, ids, n, lay.row_bytes, lay.nchunk, mean_row, st);
  medoid_end_kernel<<<1, 1, 0, s>>>(st);
  count_launches(4);
  return cudaGetLastError();
}
cudaError_t launch_pick_medoid(const Layout& lay, const GraphView& g, const uint32_t* ids, uint64_t n, uint8_t* mean_row,
                               DevState* st, cudaStream_t s) {
  GRAND_DISPATCH_ALL(lay, launch_pick_medoid_t, lay, g, ids, n, mean_row, st, s);
  return cudaErrorInvalidValue;
}

}  // namespace grand
