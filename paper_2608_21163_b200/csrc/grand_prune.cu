// Forward RobustPrune of new nodes (Alg. 5, first parallel loop; Alg. 4) and the fixed-degree detour
// find-and-replace (Alg. 7).  One thread block owns one node, so no two blocks ever write the same
// adjacency row.  (The rebuild of dirty nodes lives in grand_rebuild.cu.)
#include "grand_common.cuh"
#include "grand_kernels.h"

namespace grand {

constexpr int kPruneThreads = 128;
constexpr uint32_t kMaxCand = 1024;  // >= vmax limit
constexpr uint32_t kMaxR = 128;

// GrANDRobustPrune (Alg. 4) over candidate keys sorted ascending in shared memory.  The whole
// block takes part.  The candidates are taken in key order and each is asked the one question the
// sequential algorithm ever asks about it: does a member selected so far prune it
// (alpha * dist(s, c) <= D_p[c])?  If none does, it is selected.  That is the same result as "select
// the closest valid candidate, invalidate what it prunes", but a candidate costs at most as many
// tests as there are selected members, the first hit ends it, and nothing behind the R-th selected
// member is ever looked at.  A team of G lanes takes one selected member per pass.
// Selected candidate indices go to out_idx; returns how many were selected.
template <typename T, int G, int CPL>
__device__ uint32_t block_prune(const uint8_t* __restrict__ store, uint32_t row_bytes, uint32_t nchunk, const AlphaParam ap,
                                const unsigned long long* cand, uint32_t n, uint32_t R, uint32_t* out_idx,
                                unsigned long long& npair, unsigned long long& nrows) {
  using Dist = typename Elem<T>::Dist;
  const uint32_t tid = threadIdx.x, nthreads = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int t = lane % G;
  const uint32_t team_global = tid / G, nteams = nthreads / G, teams_per_warp = 32u / G;
  uint32_t cnt = 0;
  for (uint32_t c = 0; c < n && cnt < R; ++c) {
    const unsigned long long kc = cand[c];
    const Dist Dc = key_dist<Dist>(kc);
    bool pruned = false;
    if (tid == 0) ++nrows;  // every candidate the prune looks at has its row fetched once
    if (cnt) {
      uint4 rc[CPL];
      load_row<G, CPL>(store + (size_t)key_id(kc) * row_bytes, nchunk, t, rc);
      for (uint32_t sb = 0; sb < cnt && !pruned; sb += nteams) {
        bool hit = false;
        if (sb + (uint32_t)warp * teams_per_warp < cnt) {  // (a warp without a member to test only joins the vote)
          const uint32_t sidx = sb + team_global;
          const bool act = sidx < cnt;
          uint4 rs[CPL];
          if (act) {
            load_row<G, CPL>(store + (size_t)key_id(cand[out_idx[sidx]]) * row_bytes, nchunk, t, rs);
          } else {
#pragma unroll
            for (int cc = 0; cc < CPL; ++cc) rs[cc] = make_uint4(0, 0, 0, 0);
          }
          const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rs, rc);
          if (act && t == 0) ++npair;
          hit = act && alpha_test(ap, d, Dc);
        }
        pruned = __syncthreads_or(hit) != 0;
      }
    }
    if (!pruned) {
      if (tid == 0) out_idx[cnt] = c;
      ++cnt;
      __syncthreads();  // the new member is visible before the next candidate's tests read the list
    }
  }
  __syncthreads();
  return cnt;
}

template <typename T, int METRIC, int G, int CPL>
__global__ void __launch_bounds__(kPruneThreads) forward_prune_kernel(const PruneArgs a) {
  __shared__ unsigned long long cand[kMaxCand];
  __shared__ uint32_t out_idx[kMaxR];
  const uint32_t tid = threadIdx.x, nthreads = blockDim.x;
  const uint32_t R = a.g.R;
  const AlphaParam ap{a.A_fix, a.alpha};
  unsigned long long npair = 0, nrows = 0;
  uint32_t nprune = 0;
  auto sync = [] { __syncthreads(); };
  for (uint64_t i = blockIdx.x; i < a.n; i += gridDim.x) {
    const uint32_t p = a.ids[i];
    const uint32_t nc = min(min(a.cand_n[i], a.cand_stride), kMaxCand);
    for (uint32_t j = tid; j < nc; j += nthreads) {
      const unsigned long long k = a.cand[i * a.cand_stride + j];
      cand[j] = key_id(k) == p ? kKeyMax : k;
    }
    __syncthreads();
    bitonic_sort_any(cand, nc, tid, nthreads, sync);
    uint32_t n = nc;
    while (n > 0 && cand[n - 1] == kKeyMax) --n;
    uint32_t cnt;
    if (a.fixed_mode) {
      cnt = min(n, R);
      for (uint32_t j = tid; j < cnt; j += nthreads) out_idx[j] = j;
      __syncthreads();
    } else {
      cnt = block_prune<T, G, CPL>(a.g.store, a.lay.row_bytes, a.lay.nchunk, ap, cand, n, R, out_idx, npair, nrows);
      ++nprune;
    }
    for (uint32_t s = tid; s < R; s += nthreads) {
      uint32_t id = kInvalid;
      unsigned long long rk = 0;
      if (s < cnt) {
        const unsigned long long k = cand[out_idx[s]];
        id = key_id(k);
        rk = (k & 0xFFFFFFFF00000000ull) | p;  // dist(p, id) is symmetric: the request carries it
      }
      a.g.adj[(size_t)p * R + s] = id;
      if (a.g.rowd) a.g.rowd[(size_t)p * R + s] = s < cnt ? (uint32_t)(cand[out_idx[s]] >> 32) : kInvalid;
      a.req_tgt[i * R + s] = id;
      a.req_key[i * R + s] = rk;
    }
    if (tid == 0) {
      a.g.deg[p] = cnt;
      a.g.rowpfx[p] = a.fixed_mode ? 0 : (uint8_t)cnt;
      if (a.g.birth) {
        a.g.birth[p] = a.g.epoch;
        a.g.rowepoch[p] = a.g.epoch;
      }
    }
    __syncthreads();
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_FP_PAIRS], npair);
  }
  if (tid == 0 && nprune) atomicAdd(&a.state->counters[CTR_PRUNE], (unsigned long long)nprune);
  if (tid == 0 && nrows) atomicAdd(&a.state->counters[CTR_FP_BYTES], nrows * a.lay.row_bytes);
}

// The same candidate-ordered prune with one WARP per node: a short row keeps only a few lanes busy per test, the
// tests of one candidate are few, and a block would spend its time in barriers (measured on 384-byte rows:
// 12.8 -> 7.6 ms per 100,000 nodes against the block-per-node kernel; on 3,840-byte rows, where a warp is a single
// team, 28.7 -> 26.0 ms per 20,000 nodes with a tenth fewer tests - a block tests four members at once and the
// first hit wastes the others).  The block-per-node kernel keeps the candidate lists longer than 256.
constexpr uint32_t kWarpPruneCand = 256;  // candidates per node this kernel accepts (shared memory per warp)
constexpr int kWarpPruneWarps = 4;

template <typename T, int G, int CPL>
__global__ void __launch_bounds__(kWarpPruneWarps * 32) forward_prune_warp_kernel(const PruneArgs a) {
  using Dist = typename Elem<T>::Dist;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int NT = 32 / G;
  __shared__ unsigned long long cand_s[kWarpPruneWarps][kWarpPruneCand];
  __shared__ uint32_t out_s[kWarpPruneWarps][kMaxR];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = lane % G, team = lane / G;
  unsigned long long* cand = cand_s[warp];
  uint32_t* out_idx = out_s[warp];
  const uint32_t R = a.g.R, row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint8_t* __restrict__ store = a.g.store;
  const AlphaParam ap{a.A_fix, a.alpha};
  unsigned long long npair = 0, nrows = 0;
  uint32_t nprune = 0;
  auto wsync = [] { __syncwarp(); };
  // (handing the nodes out through a counter was measured and is slower than this fixed assignment)
  const uint64_t wglobal = (uint64_t)blockIdx.x * kWarpPruneWarps + warp, wtotal = (uint64_t)gridDim.x * kWarpPruneWarps;
  for (uint64_t i = wglobal; i < a.n; i += wtotal) {
    const uint32_t p = a.ids[i];
    const uint32_t nc = min(min(a.cand_n[i], a.cand_stride), kWarpPruneCand);
    for (uint32_t j = lane; j < nc; j += 32) {
      const unsigned long long k = a.cand[i * a.cand_stride + j];
      cand[j] = key_id(k) == p ? kKeyMax : k;
    }
    __syncwarp();
    bitonic_sort_any(cand, nc, (uint32_t)lane, 32u, wsync);
    uint32_t n = nc;
    while (n > 0 && cand[n - 1] == kKeyMax) --n;
    uint32_t cnt = 0;
    for (uint32_t c = 0; c < n && cnt < R; ++c) {
      const unsigned long long kc = cand[c];
      const Dist Dc = key_dist<Dist>(kc);
      bool pruned = false;
      ++nrows;  // every candidate the prune looks at has its row fetched once
      if (cnt) {
        uint4 rc[CPL];
        load_row<G, CPL>(store + (size_t)key_id(kc) * row_bytes, nchunk, t, rc);
        for (uint32_t sb = 0; sb < cnt && !pruned; sb += NT) {
          const uint32_t sidx = sb + team;
          const bool act = sidx < cnt;
          uint4 rs[CPL];
          if (act) {
            load_row<G, CPL>(store + (size_t)key_id(cand[out_idx[sidx]]) * row_bytes, nchunk, t, rs);
          } else {
#pragma unroll
            for (int cc = 0; cc < CPL; ++cc) rs[cc] = make_uint4(0, 0, 0, 0);
          }
          const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rs, rc);
          if (act && t == 0) ++npair;
          if (__any_sync(FULL, act && alpha_test(ap, d, Dc))) pruned = true;
        }
      }
      if (!pruned) {
        if (lane == 0) out_idx[cnt] = c;
        ++cnt;
        __syncwarp();
      }
    }
    ++nprune;
    for (uint32_t sl = lane; sl < R; sl += 32) {
      uint32_t id = kInvalid, db = kInvalid;
      unsigned long long rk = 0;
      if (sl < cnt) {
        const unsigned long long k = cand[out_idx[sl]];
        id = key_id(k);
        rk = (k & 0xFFFFFFFF00000000ull) | p;  // dist(p, id) is symmetric: the request carries it
        db = (uint32_t)(k >> 32);
      }
      a.g.adj[(size_t)p * R + sl] = id;
      if (a.g.rowd) a.g.rowd[(size_t)p * R + sl] = db;
      a.req_tgt[i * R + sl] = id;
      a.req_key[i * R + sl] = rk;
    }
    if (lane == 0) {
      a.g.deg[p] = cnt;
      a.g.rowpfx[p] = (uint8_t)cnt;
      if (a.g.birth) {
        a.g.birth[p] = a.g.epoch;
        a.g.rowepoch[p] = a.g.epoch;
      }
    }
    __syncwarp();
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_FP_PAIRS], npair);
  }
  if (lane == 0 && nprune) atomicAdd(&a.state->counters[CTR_PRUNE], (unsigned long long)nprune);
  if (lane == 0 && nrows) atomicAdd(&a.state->counters[CTR_FP_BYTES], nrows * row_bytes);
}

// The candidate-ordered prune on tensor cores, for integer rows of at most 128 bytes and R <= 64: one warp per
// node takes the sorted candidates 16 at a time.  With |s - c|^2 = |s|^2 + |c|^2 - 2 s.c and the threshold
// T_c = floor(D_p[c] * 65536 / A) (so that A * d <= D_p[c] * 65536 <=> d <= T_c, exact for integers), "member s
// prunes candidate c" is  |s|^2 - 2 s.c <= T_c - |c|^2: one integer product per pair, taken as 8-bit mma tiles of
// the block's 16 rows against the rows of the members selected so far and against the block itself.  The 16
// candidates are then resolved in order on bit masks (a candidate falls to a member selected before the block or
// to an earlier candidate of the block that was itself selected) and the selected ones join the member rows.
constexpr uint32_t kMmaPruneR = 64, kMmaPruneCand = 256;
constexpr int kMmaPruneWarps = 4;

static size_t forward_prune_mma_smem_per_warp(uint32_t row_bytes) {
  const size_t rs = ((row_bytes + 31u) & ~31u) + 16u;
  return (size_t)kMmaPruneCand * 8 + (size_t)(kMmaPruneR + 16) * rs + (size_t)(kMmaPruneR + 16 + 16) * 4 + (size_t)kMmaPruneR * 4;
}

template <typename T>
__global__ void __launch_bounds__(kMmaPruneWarps * 32) forward_prune_mma_kernel(const PruneArgs a, const uint32_t per_warp_bytes) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int gid = lane >> 2, tig = lane & 3;
  const uint32_t R = a.g.R, row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint32_t kb = (row_bytes + 31u) & ~31u, rs = kb + 16u, kch = kb / 16u, ksteps = kb / 32u;
  unsigned char* base = smem_raw + (size_t)warp * per_warp_bytes;
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(base);
  uint8_t* srow = base + (size_t)kMmaPruneCand * 8;            // rows of the selected members
  uint8_t* brow = srow + (size_t)kMmaPruneR * rs;              // rows of the block's 16 candidates
  int* sV = reinterpret_cast<int*>(brow + 16 * (size_t)rs);    // |s|^2 per selected member
  int* bU = sV + kMmaPruneR;                                   // T_c - |c|^2 per block candidate
  int* bN = bU + 16;                                           // |c|^2 per block candidate
  uint32_t* out_idx = reinterpret_cast<uint32_t*>(bN + 16);
  const uint8_t* __restrict__ store = a.g.store;
  unsigned long long npair = 0, nrows = 0;
  uint32_t nprune = 0;
  auto wsync = [] { __syncwarp(); };
  const uint64_t wglobal = (uint64_t)blockIdx.x * kMmaPruneWarps + warp, wtotal = (uint64_t)gridDim.x * kMmaPruneWarps;
  for (uint64_t i = wglobal; i < a.n; i += wtotal) {
    const uint32_t p = a.ids[i];
    const uint32_t nc = min(min(a.cand_n[i], a.cand_stride), kMmaPruneCand);
    for (uint32_t j = lane; j < nc; j += 32) {
      const unsigned long long k = a.cand[i * a.cand_stride + j];
      cand[j] = key_id(k) == p ? kKeyMax : k;
    }
    __syncwarp();
    bitonic_sort_any(cand, nc, (uint32_t)lane, 32u, wsync);
    uint32_t n = nc;
    while (n > 0 && cand[n - 1] == kKeyMax) --n;
    uint32_t cnt = 0;
    for (uint32_t c0 = 0; c0 < n && cnt < R; c0 += 16) {
      const uint32_t nb = min(16u, n - c0);
      // ---- the block's rows (zero beyond the row and beyond the block), their norms and thresholds
      for (uint32_t e = lane; e < 16 * kch; e += 32) {
        const uint32_t j = e / kch, ch = e - j * kch;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < nb && ch < nchunk) v = __ldg(reinterpret_cast<const uint4*>(store + (size_t)key_id(cand[c0 + j]) * row_bytes) + ch);
        reinterpret_cast<uint4*>(brow + (size_t)j * rs)[ch] = v;
      }
      __syncwarp();
      if (lane < 16) {
        const uint4* rp = reinterpret_cast<const uint4*>(brow + (size_t)lane * rs);
        int nrm = 0;
        for (uint32_t ch = 0; ch < nchunk; ++ch) acc_chunk<T, kMetricIP>(rp[ch], rp[ch], nrm);
        long long thr = 0;
        if ((uint32_t)lane < nb) thr = ((long long)key_dist<int>(cand[c0 + lane]) * 65536ll) / a.A_fix;
        if (thr > 0x7FFFFFFFll) thr = 0x7FFFFFFFll;  // no distance is larger: the clamp changes no test
        bN[lane] = nrm;
        bU[lane] = (int)(thr - (long long)nrm > -0x80000000ll ? thr - (long long)nrm : -0x80000000ll);
      }
      __syncwarp();
      // ---- tiles: the block against the selected members, and against itself
      uint32_t xa[4][4];  // the block's fragments for up to 4 steps of 32 bytes
      {
        const uint8_t* x0 = brow + (size_t)gid * rs + tig * 4;
        const uint8_t* x1 = x0 + 8 * (size_t)rs;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          if ((uint32_t)ks < ksteps) {
            xa[ks][0] = *reinterpret_cast<const uint32_t*>(x0 + ks * 32);
            xa[ks][1] = *reinterpret_cast<const uint32_t*>(x1 + ks * 32);
            xa[ks][2] = *reinterpret_cast<const uint32_t*>(x0 + ks * 32 + 16);
            xa[ks][3] = *reinterpret_cast<const uint32_t*>(x1 + ks * 32 + 16);
          } else {
            xa[ks][0] = xa[ks][1] = xa[ks][2] = xa[ks][3] = 0u;
          }
        }
      }
      const int u0 = bU[gid], u1 = bU[gid + 8];
      bool old0 = false, old1 = false;  // rows gid / gid + 8 fall to a member selected before this block
      for (uint32_t nt = 0; nt * 8 < cnt; ++nt) {
        int acc[4] = {0, 0, 0, 0};
        const uint8_t* yr = srow + (size_t)(nt * 8 + gid) * rs + tig * 4;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          if ((uint32_t)ks < ksteps) {
            uint32_t yb[2];
            yb[0] = *reinterpret_cast<const uint32_t*>(yr + ks * 32);
            yb[1] = *reinterpret_cast<const uint32_t*>(yr + ks * 32 + 16);
            mma_m16n8k32<T>(acc, xa[ks], yb);
          }
        }
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const uint32_t sidx = nt * 8 + tig * 2 + jj;
          if (sidx < cnt) {
            const int vs = sV[sidx];
            old0 |= vs - 2 * acc[jj] <= u0;
            old1 |= vs - 2 * acc[2 + jj] <= u1;
          }
        }
      }
      uint32_t rm0 = 0, rm1 = 0;  // bit j: candidate j of the block prunes candidate gid / gid + 8 of the block
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        int acc[4] = {0, 0, 0, 0};
        const uint8_t* yr = brow + (size_t)(nt * 8 + gid) * rs + tig * 4;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          if ((uint32_t)ks < ksteps) {
            uint32_t yb[2];
            yb[0] = *reinterpret_cast<const uint32_t*>(yr + ks * 32);
            yb[1] = *reinterpret_cast<const uint32_t*>(yr + ks * 32 + 16);
            mma_m16n8k32<T>(acc, xa[ks], yb);
          }
        }
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const uint32_t j = nt * 8 + tig * 2 + jj;
          const int vj = bN[j];
          if (vj - 2 * acc[jj] <= u0) rm0 |= 1u << j;
          if (vj - 2 * acc[2 + jj] <= u1) rm1 |= 1u << j;
        }
      }
      // a row's results are spread over the 4 lanes of its group
      {
        uint32_t o = (old0 ? 1u : 0u) | (old1 ? 2u : 0u);
        o |= __shfl_xor_sync(FULL, o, 1);
        o |= __shfl_xor_sync(FULL, o, 2);
        old0 = o & 1u;
        old1 = o & 2u;
        rm0 |= __shfl_xor_sync(FULL, rm0, 1);
        rm0 |= __shfl_xor_sync(FULL, rm0, 2);
        rm1 |= __shfl_xor_sync(FULL, rm1, 1);
        rm1 |= __shfl_xor_sync(FULL, rm1, 2);
      }
      const unsigned oldlo = __ballot_sync(FULL, old0), oldhi = __ballot_sync(FULL, old1);  // row r: bit 4 * (r & 7)
      // ---- the 16 candidates in order
      uint32_t sel = 0;
      uint32_t room = R - cnt;
      for (uint32_t r = 0; r < nb && room; ++r) {
        const uint32_t rm = __shfl_sync(FULL, r < 8 ? rm0 : rm1, 4 * (r & 7));
        const bool old = ((r < 8 ? oldlo : oldhi) >> (4 * (r & 7))) & 1u;
        if (!old && !(rm & sel)) {  // (sel holds only earlier candidates)
          sel |= 1u << r;
          --room;
        }
      }
      if (lane == 0) {
        npair += (unsigned long long)nb * cnt + (unsigned long long)nb * (nb - 1) / 2;
        nrows += nb;  // the block's candidate rows, fetched once
      }
      // ---- the selected candidates join the members: index, norm, row
      const uint32_t nsel = __popc(sel);
      if (lane < 16 && ((sel >> lane) & 1u)) {
        const uint32_t dst = cnt + __popc(sel & ((1u << lane) - 1u));
        out_idx[dst] = c0 + lane;
        sV[dst] = bN[lane];
      }
      for (uint32_t e = lane; e < 16 * kch; e += 32) {
        const uint32_t j = e / kch, ch = e - j * kch;
        if ((sel >> j) & 1u) {
          const uint32_t dst = cnt + __popc(sel & ((1u << j) - 1u));
          reinterpret_cast<uint4*>(srow + (size_t)dst * rs)[ch] = reinterpret_cast<const uint4*>(brow + (size_t)j * rs)[ch];
        }
      }
      cnt += nsel;
      __syncwarp();
    }
    ++nprune;
    for (uint32_t sl = lane; sl < R; sl += 32) {
      uint32_t id = kInvalid, db = kInvalid;
      unsigned long long rk = 0;
      if (sl < cnt) {
        const unsigned long long k = cand[out_idx[sl]];
        id = key_id(k);
        rk = (k & 0xFFFFFFFF00000000ull) | p;  // dist(p, id) is symmetric: the request carries it
        db = (uint32_t)(k >> 32);
      }
      a.g.adj[(size_t)p * R + sl] = id;
      if (a.g.rowd) a.g.rowd[(size_t)p * R + sl] = db;
      a.req_tgt[i * R + sl] = id;
      a.req_key[i * R + sl] = rk;
    }
    if (lane == 0) {
      a.g.deg[p] = cnt;
      a.g.rowpfx[p] = (uint8_t)cnt;
      if (a.g.birth) {
        a.g.birth[p] = a.g.epoch;
        a.g.rowepoch[p] = a.g.epoch;
      }
    }
    __syncwarp();
  }
  if (npair) {
    atomicAdd(&a.state->counters[CTR_PAIR], npair);
    atomicAdd(&a.state->counters[CTR_FP_PAIRS], npair);
  }
  if (lane == 0 && nprune) atomicAdd(&a.state->counters[CTR_PRUNE], (unsigned long long)nprune);
  if (lane == 0 && nrows) atomicAdd(&a.state->counters[CTR_FP_BYTES], nrows * row_bytes);
}

template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_forward_prune_t(const PruneArgs& a, cudaStream_t s) {
  if (a.n == 0) return cudaSuccess;
  if constexpr (sizeof(T) == 1) {
    if (!a.fixed_mode && a.lay.row_bytes <= 128u && a.g.R <= kMmaPruneR && a.cand_stride <= kMmaPruneCand && a.A_fix > 0) {
      const size_t per_warp = (forward_prune_mma_smem_per_warp(a.lay.row_bytes) + 15) / 16 * 16;
      const size_t smem = per_warp * kMmaPruneWarps;
      auto kern = forward_prune_mma_kernel<T>;
      static SmemOptIn optin{};
      cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
      if (e != cudaSuccess) return e;
      const uint64_t want = (a.n + kMmaPruneWarps - 1) / kMmaPruneWarps, most = (uint64_t)sm_count() * 8u;
      const unsigned blocks = (unsigned)(want < most ? want : most);
      kern<<<blocks, kMmaPruneWarps * 32, smem, s>>>(a, (uint32_t)per_warp);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  {
    if (!a.fixed_mode && a.cand_stride <= kWarpPruneCand) {
      const uint64_t want = (a.n + kWarpPruneWarps - 1) / kWarpPruneWarps, most = (uint64_t)sm_count() * 16u;
      const unsigned blocks = (unsigned)(want < most ? want : most);
      forward_prune_warp_kernel<T, G, CPL><<<blocks, kWarpPruneWarps * 32, 0, s>>>(a);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  const uint64_t most = (uint64_t)sm_count() * 16u;
  const unsigned blocks = (unsigned)(a.n < most ? a.n : most);
  forward_prune_kernel<T, METRIC, G, CPL><<<blocks, kPruneThreads, 0, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_forward_prune(const PruneArgs& a, cudaStream_t s) {
  GRAND_DISPATCH_ALL(a.lay, launch_forward_prune_t, a, s);
  return cudaErrorInvalidValue;
}

// Fixed-degree backward edges (Alg. 7): the owner of target q takes its requests in (dist, id)
// order; a request from new node p appends while deg(q) < R, else replaces the highest-index slot
// of N_out(q) that also occurs in N_out(p) and was not replaced earlier in this batch.
// One warp owns one target: almost every target of a batch receives a single request, so a
// block per target would leave three of its four warps at the barrier.  Short segments are
// sorted in the warp's shared-memory slice, long ones in place in global memory.
constexpr uint32_t kFixedSegWarp = 64;
__global__ void __launch_bounds__(kPruneThreads) fixed_reverse_kernel(const FixedReverseArgs a) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int kWarps = kPruneThreads / 32;
  __shared__ unsigned long long seg_s[kWarps][kFixedSegWarp];
  __shared__ uint32_t row_s[kWarps][kMaxR];
  __shared__ uint32_t prow_s[kWarps][kMaxR];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* row = row_s[warp];
  uint32_t* prow = prow_s[warp];
  auto wsync = [] { __syncwarp(); };
  const uint32_t R = a.g.R;
  uint32_t ndone = 0;
  const uint32_t ndirty = a.state->ndirty;
  const uint64_t wglobal = (uint64_t)blockIdx.x * kWarps + warp, wtotal = (uint64_t)gridDim.x * kWarps;
  for (uint64_t k = wglobal; k < ndirty; k += wtotal) {
    const uint32_t q = a.dirty[k];
    const uint32_t cntq = a.cnt[q];
    unsigned long long* seg = a.seg_keys + a.start[q];
    if (cntq <= kFixedSegWarp) {
      for (uint32_t j = lane; j < cntq; j += 32) seg_s[warp][j] = seg[j];
      seg = seg_s[warp];
    }
    for (uint32_t s = lane; s < R; s += 32) row[s] = a.g.adj[(size_t)q * R + s];
    __syncwarp();
    bitonic_sort_any(seg, cntq, (uint32_t)lane, 32u, wsync);
    uint32_t repl = 0;  // lane w: word w of the set of slots replaced in this batch
    uint32_t nrepl = 0;
    uint32_t dq = min(a.g.deg[q], R);
    unsigned long long prev = kKeyMax;
    for (uint32_t j = 0; j < cntq; ++j) {
      if (nrepl == R) break;  // every slot already replaced once: no later request can change the row
      const unsigned long long kk = seg[j];
      if (kk == prev) continue;
      prev = kk;
      const uint32_t p = key_id(kk);
      // already linked?
      bool present = false;
      for (uint32_t sb = 0; sb < dq; sb += 32) {
        const uint32_t s = sb + lane;
        present |= __any_sync(FULL, s < dq && row[s] == p);
      }
      if (present) continue;
      if (dq < R) {
        if (lane == 0) row[dq] = p;
        ++dq;
        __syncwarp();
        continue;
      }
      const uint32_t* pg = a.fwd_rows + (size_t)a.slot_of[p] * R;
      for (uint32_t y = lane; y < R; y += 32) prow[y] = pg[y];
      __syncwarp();
      int pick = -1;
      for (uint32_t sb = 0; sb < dq; sb += 32) {
        const uint32_t s = sb + lane;
        const uint32_t rw = __shfl_sync(FULL, repl, sb >> 5);
        bool hit = false;
        if (s < dq && !((rw >> lane) & 1u)) {
          const uint32_t x = row[s];
          for (uint32_t y = 0; y < R; ++y) hit |= prow[y] == x;   // INVALID padding never equals a live id
        }
        const unsigned bal = __ballot_sync(FULL, hit);
        if (bal) pick = (int)sb + 31 - __clz(bal);
      }
      if (pick >= 0) {
        if (lane == 0) row[pick] = p;
        if (lane == (pick >> 5)) repl |= 1u << (pick & 31);
        ++nrepl;
      }
      __syncwarp();
    }
    for (uint32_t s = lane; s < R; s += 32) a.g.adj[(size_t)q * R + s] = s < dq ? row[s] : kInvalid;
    if (lane == 0) {
      a.g.deg[q] = dq;
      a.cnt[q] = 0;
      a.fill[q] = 0;
      a.flag[q] = 0;
      ++ndone;
    }
    __syncwarp();
  }
  if (lane == 0 && ndone) atomicAdd(&a.state->counters[CTR_DIRTY], (unsigned long long)ndone);
}

cudaError_t launch_fixed_reverse(const FixedReverseArgs& a, cudaStream_t s) {
  fixed_reverse_kernel<<<a.max_blocks, kPruneThreads, 0, s>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace grand
