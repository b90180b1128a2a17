// Rebuild of dirty nodes (Alg. 5 dirty loop, Alg. 6 rebuild loop): one WARP owns one dirty node.
//
// C = (N_out(u) \ B) ++ (scratch_u \ N_out(u) \ {u}); if |C| <= R the row is stored as is, else D_u is
// computed for the kept neighbours (requests already carry dist(u, id)) and GrANDRobustPrune
// (Alg. 4) runs on C.  The prune is restructured for the GPU without changing its result:
//
//  * Rows carry the cached distances dist(u, v) of their entries (rowd), so D_u of a kept neighbour
//    costs no gather.
//  * Every row remembers how long its leading run of prune output is (rowpfx).  Two members of
//    that run both survived an earlier prune of this very node, which means the earlier one does
//    not prune the later one; distances and D_u are recomputed to the same bits, so those tests
//    are known to be false and the sequential prune can only change at an "uncertain" member
//    (appended since the last prune, or fresh).
//  * The uncertain members are walked in key order: does a valid member of the run in front of it
//    prune it (the first hit ends it)?  If not it is selected and prunes among the valid candidates
//    behind it; the walk stops once R valid candidates stand in front.  Only tests the sequential
//    algorithm needs are evaluated.  A full, entirely pruned row that receives one candidate takes a
//    two-phase shortcut of the same walk.  Candidate lists with more than 2P uncertain members
//    (possible only for R > P, or rows without a trusted run) fall back to evaluating every test
//    alpha * dist(c_i, c_j) <= D_u[c_j], i < j, into a bit matrix and replaying the selection on masks.
//
// Dirty nodes are handed out through an atomic work counter because a node that prunes costs far
// more than one that only appends.
#include "grand_common.cuh"
#include "grand_kernels.h"

namespace grand {

constexpr int kRebuildWarps = 4;
constexpr uint32_t kSegSmem = 128;       // request segments up to this length are sorted in shared memory

static inline uint32_t even_up_h(uint32_t x) { return (x + 1u) & ~1u; }
static size_t rebuild_smem_per_warp(uint32_t R, uint32_t P) {
  const size_t NM = R + P, W = (NM + 31) / 32, Rp = even_up_h(R);
  size_t b = (size_t)kSegSmem * 8 + (size_t)P * 8 + NM * 8 + Rp * 4 * 3 + (NM + 1) * W * 4;
  return (b + 15) / 16 * 16;
}

// Resident blocks per SM the register allocation must leave room for.  On rows of at most 512 bytes the kernel waits
// on memory with few warps to hide it (103 registers allowed only 4 blocks on 128-byte rows, 93 only 5 on 384-byte
// rows): 7 blocks took 7% off the launch on 384-byte rows and 4% on 128-byte rows (on 384-byte rows 5 / 6 / 7 / 8
// blocks measure 56.5 / 52.5 / 50.6 / 59.9 ms per step on the Deep-shaped stream); 8 spills and is slower.
// Whole-warp teams keep their registers (no gain measured there).
template <int G, int CPL>
constexpr int rebuild_min_blocks() {
  return G == 32 ? 1 : 7;
}

// The P smallest distinct keys of a long request segment, ascending, into `best` (shared memory); returns how many.
// Kept out of line: a rare path whose code would otherwise sit in the middle of the per-node loop.
__device__ __forceinline__ uint32_t stream_best_keys_impl(const unsigned long long* seg, uint32_t cntu, unsigned long long* scratch,
                                                          uint32_t P, int lane) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  uint32_t ns = 0;
      for (uint32_t jb0 = 0; jb0 < cntu; jb0 += 128) {
       unsigned long long k4[4];  // four chunks requested together: the stream is a chain of dependent steps otherwise
#pragma unroll
       for (int q = 0; q < 4; ++q) k4[q] = jb0 + q * 32 + lane < cntu ? seg[jb0 + q * 32 + lane] : kKeyMax;
#pragma unroll
       for (int q = 0; q < 4; ++q) {
        const unsigned long long kk = k4[q];
        const unsigned long long thr = ns == P ? scratch[P - 1] : kKeyMax;
        unsigned bal = __ballot_sync(FULL, kk < thr);
        while (bal) {  // (uniform)
          const int srcl = __ffs(bal) - 1;
          bal &= bal - 1u;
          const unsigned long long key = ((unsigned long long)__shfl_sync(FULL, (uint32_t)(kk >> 32), srcl) << 32) |
                                         __shfl_sync(FULL, (uint32_t)kk, srcl);
          if (ns == P && !(key < scratch[P - 1])) continue;  // the list has tightened since the ballot
          uint32_t pos = 0;
          unsigned dup = 0;
          for (uint32_t cb = 0; cb < ns; cb += 32) {
            const uint32_t i = cb + lane;
            const unsigned long long e = i < ns ? scratch[i] : kKeyMax;
            pos += __popc(__ballot_sync(FULL, e < key));
            dup |= __ballot_sync(FULL, e == key);
          }
          if (dup) continue;
          const uint32_t last = min(ns, P - 1u);  // entries [pos, last) move up by one; a full list drops its last entry
          if (last > pos) {
            for (int ch = (int)((last - 1u) >> 5); ch >= (int)(pos >> 5); --ch) {
              const uint32_t i = (uint32_t)ch * 32u + lane;
              const bool mv = i >= pos && i < last;
              const unsigned long long e = mv ? scratch[i] : 0ull;
              __syncwarp();
              if (mv) scratch[i + 1] = e;
            }
          }
          __syncwarp();
          if (lane == 0) scratch[pos] = key;
          __syncwarp();
          ns = min(ns + 1u, P);
        }
       }
      }
  return ns;
}
__device__ __noinline__ uint32_t stream_best_keys_ool(const unsigned long long* seg, uint32_t cntu, unsigned long long* scratch,
                                                      uint32_t P, int lane) {
  return stream_best_keys_impl(seg, cntu, scratch, P, lane);
}
// Whether the rare paths of the rebuild sit out of line.  Out of line they shorten the per-node loop, which pays on
// rows of at most 128 bytes, where the kernel is bound by instruction issue and fetch (rebuild 1.79 -> 1.60 ms per
// step, alternating runs of both builds on one GPU).  Elsewhere they stay inline: the calls cost the 6-chunk layout,
// which runs at its register bound, a few more spills (53.3 against 51.8 ms per step), and on wide rows with reused
// ids and strong hubs these paths are not rare at all (GIST-shaped rebuild 41 against 55 ms per step).
template <int G, int CPL>
constexpr bool rebuild_cold_paths_out_of_line() { return G * CPL <= 8; }

// Fallback of the prune for candidate lists without a trusted run: every test alpha * dist(c_i, c_j) <= D_u[c_j],
// i < j, goes into a bit matrix (row i, bit j = "c_i prunes c_j"), and the sequential selection is replayed on
// masks.  Lane w holds word w of the set of still-valid candidates; the updated word is returned.  Out of line: rare.
template <typename T, int G, int CPL>
__device__ __forceinline__ uint32_t prune_all_pairs_impl(const uint8_t* __restrict__ store, uint32_t row_bytes, uint32_t nchunk,
                                                         const unsigned long long* cs, uint32_t nC, uint32_t W, uint32_t* prune, uint32_t* hasp,
                                                         AlphaParam ap, uint32_t valid, unsigned long long& npair, int lane) {
  using Dist = typename Elem<T>::Dist;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int NT = 32 / G;
  const int t = lane % G, team = lane / G;
  for (uint32_t w = lane; w < nC * W; w += 32) prune[w] = 0u;
  __syncwarp();
  uint32_t jprev = kInvalid;
  uint4 rj[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) rj[c] = make_uint4(0, 0, 0, 0);
  const uint32_t npairs = nC * (nC - 1) / 2;
  for (uint32_t pb = 0; pb < npairs; pb += NT) {
    const uint32_t p = pb + team;
    const bool act = p < npairs;
    uint32_t i = 0, j = 1;
    if (act) {
      j = (uint32_t)((1.0f + sqrtf(1.0f + 8.0f * (float)p)) * 0.5f);
      while (j * (j - 1) / 2 > p) --j;
      while ((j + 1) * j / 2 <= p) ++j;
      i = p - j * (j - 1) / 2;
    }
    uint4 ri[CPL];
    if (act) {
      if (j != jprev) {
        load_row<G, CPL>(store + (size_t)key_id(cs[j]) * row_bytes, nchunk, t, rj);
        jprev = j;
      }
      load_row<G, CPL>(store + (size_t)key_id(cs[i]) * row_bytes, nchunk, t, ri);
    } else {
#pragma unroll
      for (int c = 0; c < CPL; ++c) ri[c] = make_uint4(0, 0, 0, 0);
    }
    const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(ri, rj);
    if (act && t == 0) {
      ++npair;
      if (alpha_test(ap, d, key_dist<Dist>(cs[j]))) {
        atomicOr(&prune[i * W + (j >> 5)], 1u << (j & 31));
        atomicOr(&hasp[i >> 5], 1u << (i & 31));
      }
    }
  }
  __syncwarp();
  // the valid set only changes when a still-valid candidate with a non-zero matrix row is reached, so only those
  // candidates are visited, in ascending order; everything valid in between is selected
  for (uint32_t w = 0; w < W; ++w) {
    uint32_t hw = hasp[w];
    while (hw) {
      const uint32_t b = __ffs(hw) - 1;
      hw &= hw - 1;
      const uint32_t vw = __shfl_sync(FULL, valid, w);
      if (((vw >> b) & 1u) && (uint32_t)lane < W) valid &= ~prune[(w * 32 + b) * W + lane];
    }
  }
  return valid;
}
template <typename T, int G, int CPL>
__device__ __noinline__ uint32_t prune_all_pairs_ool(const uint8_t* __restrict__ store, uint32_t row_bytes, uint32_t nchunk,
                                                     const unsigned long long* cs, uint32_t nC, uint32_t W, uint32_t* prune, uint32_t* hasp,
                                                     AlphaParam ap, uint32_t valid, unsigned long long& npair, int lane) {
  return prune_all_pairs_impl<T, G, CPL>(store, row_bytes, nchunk, cs, nC, W, prune, hasp, ap, valid, npair, lane);
}

// D_u for kept neighbours whose distance is not cached in the row (rows of an imported graph, ids that have come
// back since the row was written): dist(u, keep[j]) into cand[j], tagged uncertain behind the pruned run.
template <typename T, int G, int CPL>
__device__ __forceinline__ void fill_uncached_dists_impl(const uint8_t* __restrict__ store, uint32_t row_bytes, uint32_t nchunk, uint32_t u,
                                                         const uint32_t* keep, const uint32_t* keepd, uint32_t nk, uint32_t kp,
                                                         unsigned long long* cand, unsigned long long& npair, int lane) {
  using Dist = typename Elem<T>::Dist;
  constexpr int NT = 32 / G;
  const int t = lane % G, team = lane / G;
  uint4 ur[CPL];
  load_row<G, CPL>(store + (size_t)u * row_bytes, nchunk, t, ur);
  for (uint32_t jb = 0; jb < nk; jb += NT) {
    const uint32_t j = jb + team;
    const bool act = j < nk && keepd[j] == kInvalid;
    uint4 v[CPL];
    if (act) {
      load_row<G, CPL>(store + (size_t)keep[j] * row_bytes, nchunk, t, v);
    } else {
#pragma unroll
      for (int c = 0; c < CPL; ++c) v[c] = make_uint4(0, 0, 0, 0);
    }
    const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(ur, v);
    if (act && t == 0) {
      cand[j] = make_key(d, keep[j]) | (j >= kp ? kExpandedBit : 0ull);
      ++npair;
    }
  }
}
template <typename T, int G, int CPL>
__device__ __noinline__ void fill_uncached_dists_ool(const uint8_t* __restrict__ store, uint32_t row_bytes, uint32_t nchunk, uint32_t u,
                                                     const uint32_t* keep, const uint32_t* keepd, uint32_t nk, uint32_t kp,
                                                     unsigned long long* cand, unsigned long long& npair, int lane) {
  fill_uncached_dists_impl<T, G, CPL>(store, row_bytes, nchunk, u, keep, keepd, nk, kp, cand, npair, lane);
}

template <typename T, int METRIC, int G, int CPL>
__global__ void __launch_bounds__(kRebuildWarps * 32, rebuild_min_blocks<G, CPL>()) rebuild_kernel(const RebuildArgs a, const uint32_t per_warp_bytes) {
  using Dist = typename Elem<T>::Dist;
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int NT = 32 / G;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = lane % G, team = lane / G;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const uint32_t R = a.g.R, P = a.P, NM = R + P, W = (NM + 31) >> 5, Rp = (R + 1u) & ~1u;
  unsigned char* base = smem_raw + (size_t)warp * per_warp_bytes;
  unsigned long long* seg_s = reinterpret_cast<unsigned long long*>(base);
  unsigned long long* scratch = seg_s + kSegSmem;
  unsigned long long* cand = scratch + P;
  uint32_t* keep = reinterpret_cast<uint32_t*>(cand + NM);
  uint32_t* keepd = keep + Rp;     // cached dist(u, keep[j]) bits (0xFFFFFFFF = not cached)
  uint32_t* out_idx = keepd + Rp;
  uint32_t* prune = out_idx + Rp;  // NM rows x W words: bit j of row i = "c_i prunes c_j"
  uint32_t* hasp = prune + NM * W;  // W words: bit i = row i of the matrix is non-zero (c_i prunes something)
  uint32_t* upos = reinterpret_cast<uint32_t*>(scratch);  // positions of uncertain candidates (2P entries; scratch is free by then)
  unsigned long long* cs = cand;  // C in key order: cand itself, or the segment buffer after a rank merge
  const AlphaParam ap{a.A_fix, a.alpha};
  const uint32_t row_bytes = a.lay.row_bytes, nchunk = a.lay.nchunk;
  const uint8_t* __restrict__ store = a.g.store;
  auto wsync = [] { __syncwarp(); };
  unsigned long long npair = 0, nbytes = 0;  // nbytes: what the method has to move for the rows this warp rebuilds
  uint32_t nprune = 0, ndone = 0;
  const uint32_t ndirty = a.split ? a.state->nheavy : a.state->ndirty;  // (split: the front of the work list)

  // One counter serves every warp of the grid.  The ticket for the node after this one is drawn while this one
  // is processed, so the atomic's round trip is never waited for.
  uint32_t ticket = 0;
  if (lane == 0) ticket = atomicAdd(&a.state->work, 1u);
  for (;;) {
    const uint32_t k = __shfl_sync(FULL, ticket, 0);
    if (k >= ndirty) break;
    if (lane == 0) ticket = atomicAdd(&a.state->work, 1u);
    const uint32_t u = a.dirty[k];
    // the node some warp will take about one generation of warps from now: its id is fetched here and its row,
    // cached distances and counters are pulled towards L2 once this node is done
    const uint32_t k_ahead = k + gridDim.x * kRebuildWarps;
    const uint32_t u_ahead = k_ahead < ndirty ? a.dirty[k_ahead] : kInvalid;
    // Everything the node needs from global memory is requested up front, in two rounds (what depends only on
    // u; then the request segment and the batch-membership bits of the row's entries), so that the latencies
    // overlap instead of following one another through the phases below.
    const uint32_t cntu = a.cnt[u];
    const uint32_t startu = a.start[u];
    const uint32_t du = min(a.g.deg[u], R);
    uint32_t pfx = min((uint32_t)a.g.rowpfx[u], du);
    const uint32_t rowep = a.g.birth ? a.g.rowepoch[u] : 0u;
    uint32_t* row = a.g.adj + (size_t)u * R;
    uint32_t vrow[4], vrd[4];  // the row and its cached distances, spread over the lanes (R <= 128)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint32_t sl = (uint32_t)c * 32u + lane;
      vrow[c] = sl < R ? row[sl] : kInvalid;
      vrd[c] = a.g.rowd && sl < R ? a.g.rowd[(size_t)u * R + sl] : kInvalid;
    }
    // ---- scratch_u: sort the request segment by (dist, id), keep the first P distinct entries
    unsigned long long* seg = a.seg_keys + startu;
    if (cntu <= kSegSmem) {
      for (uint32_t j = lane; j < cntu; j += 32) seg_s[j] = seg[j];
      seg = seg_s;
    }
    uint32_t okbits = 0;  // bit c: entry c * 32 + lane of the row stays
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint32_t sl = (uint32_t)c * 32u + lane, v = vrow[c];
      if (sl < du) {
        bool ok = !(a.delmap && bit_test(a.delmap, v));
        if (ok && a.livemap) ok = bit_test(a.livemap, v) || (a.newmap && bit_test(a.newmap, v));  // drops dangling edges
        okbits |= (uint32_t)ok << c;
      }
    }
    __syncwarp();
    uint32_t ns = 0;
    if (cntu > kSegSmem) {
      // A hub can be the target of a large part of a batch's requests (hundreds of thousands on data with strong
      // hubness), and only the P smallest distinct keys are wanted: the segment is streamed once against a sorted
      // list of the best P so far instead of being sorted.  After the first few chunks almost every key fails the
      // comparison with the list's last entry.  Same list as sort + drop repeats + cut at P.
      if constexpr (rebuild_cold_paths_out_of_line<G, CPL>()) ns = stream_best_keys_ool(seg, cntu, scratch, P, lane);
      else ns = stream_best_keys_impl(seg, cntu, scratch, P, lane);
    } else {
    bitonic_sort_any(seg, cntu, (uint32_t)lane, 32u, wsync);
    for (uint32_t jb = 0; jb < cntu && ns < P; jb += 32) {
      const uint32_t j = jb + lane;
      bool ok = j < cntu;
      unsigned long long kk = 0;
      if (ok) {
        kk = seg[j];
        if (j > 0 && seg[j - 1] == kk) ok = false;  // equal requests are adjacent after the sort
      }
      const unsigned bal = __ballot_sync(FULL, ok);
      const uint32_t pos = ns + __popc(bal & lt_mask);
      if (ok && pos < P) scratch[pos] = kk;
      ns += __popc(bal);
    }
    ns = min(ns, P);
    }
    // ---- keep = N_out(u) \ B, stable; kp = how many kept entries come from the pruned prefix
    uint32_t nk = 0, kp = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint32_t sb = (uint32_t)c * 32u;
      if (sb < du) {
        const uint32_t v = vrow[c];
        const bool ok = (okbits >> c) & 1u;
        // an old edge to an id that has come back since this row was written: a legal edge to the new node, but
        // nothing cached about it holds, and the pruned run ends in front of it
        const bool reborn = ok && a.g.birth && a.g.birth[v] > rowep;
        const unsigned bal = __ballot_sync(FULL, ok);
        if (a.g.birth) {
          const unsigned rbal = __ballot_sync(FULL, reborn);
          if (rbal) pfx = min(pfx, sb + (uint32_t)__ffs(rbal) - 1u);
        }
        if (ok) {
          const uint32_t pos = nk + __popc(bal & lt_mask);
          keep[pos] = v;
          keepd[pos] = reborn ? kInvalid : vrd[c];
        }
        nk += __popc(bal);
        kp += __popc(bal & (pfx > sb ? (pfx - sb >= 32u ? FULL : (1u << (pfx - sb)) - 1u) : 0u));
      }
    }
    __syncwarp();
    // ---- fresh = scratch \ keep \ {u}, stable, placed after the keep slots of cand (tagged uncertain)
    uint32_t nf = 0;
    {
      uint32_t kreg[4];  // the kept ids, spread over the lanes (R <= 128); the invalid id never matches
#pragma unroll
      for (int c = 0; c < 4; ++c) kreg[c] = (uint32_t)(c * 32 + lane) < nk ? keep[c * 32 + lane] : kInvalid;
      for (uint32_t j = 0; j < ns; ++j) {
        const unsigned long long kk = scratch[j];
        const uint32_t id = key_id(kk);
        const bool hit = kreg[0] == id || kreg[1] == id || kreg[2] == id || kreg[3] == id;
        if (__any_sync(FULL, hit) || id == u) continue;
        if (lane == 0) cand[nk + nf] = kk | kExpandedBit;
        ++nf;
      }
    }
    __syncwarp();
    const uint32_t nC = nk + nf;
    // the row read and written back, the node's request tuples, and (below) the candidates' vectors when a prune runs
    nbytes += 2ull * R * 4u + (unsigned long long)cntu * 12u;
    if (nC <= R) {
      for (uint32_t s = lane; s < R; s += 32) {
        row[s] = s < nk ? keep[s] : (s < nC ? key_id(cand[s]) : kInvalid);
        if (a.g.rowd) a.g.rowd[(size_t)u * R + s] = s < nk ? keepd[s] : (s < nC ? (uint32_t)(cand[s] >> 32) : kInvalid);
      }
      if (lane == 0) {
        a.g.deg[u] = nC;
        a.g.rowpfx[u] = (uint8_t)kp;  // the surviving part of the pruned run still leads the row
      }
    } else {
      nbytes += (unsigned long long)nC * row_bytes;
      // ---- D_u for the kept neighbours (those appended after the last prune are tagged uncertain)
      bool all_cached = true;
      for (uint32_t jb = 0; jb < nk; jb += 32) {
        const uint32_t j = jb + lane;
        bool miss = false;
        if (j < nk) {
          miss = keepd[j] == kInvalid;
          if (!miss) cand[j] = ((unsigned long long)keepd[j] << 32) | keep[j] | (j >= kp ? kExpandedBit : 0ull);
        }
        if (__any_sync(FULL, miss)) all_cached = false;
      }
      if (!all_cached) {
        if constexpr (rebuild_cold_paths_out_of_line<G, CPL>()) {
          unsigned long long tested = 0;
          fill_uncached_dists_ool<T, G, CPL>(store, row_bytes, nchunk, u, keep, keepd, nk, kp, cand, tested, lane);
          npair += tested;
        } else {
          fill_uncached_dists_impl<T, G, CPL>(store, row_bytes, nchunk, u, keep, keepd, nk, kp, cand, npair, lane);
        }
      }
      __syncwarp();
      if (kp == nk && nf == 1) {
        // ---- the common case of an insert batch: a full row that is entirely prune output receives one
        //      fresh candidate p.  Kept members never prune each other, so the sequential prune reduces to:
        //      (1) does a kept member closer than p prune p?  then nothing changes;  (2) otherwise p enters
        //      at its rank and the only other tests that can fire are p against the members behind it.
        const unsigned long long kf = key_clean(cand[nk]);
        const Dist Dp = key_dist<Dist>(kf);
        uint32_t pos = 0;
        for (uint32_t jb = 0; jb < nk; jb += 32) pos += __popc(__ballot_sync(FULL, jb + lane < nk && cand[jb + lane] < kf));
        uint4 rf[CPL];
        load_row<G, CPL>(store + (size_t)key_id(kf) * row_bytes, nchunk, t, rf);
        bool pruned = false;
        for (uint32_t ib = 0; ib < pos && !pruned; ib += NT) {
          const uint32_t i = ib + team;
          const bool act = i < pos;
          uint4 rx[CPL];
          if (act) {
            load_row<G, CPL>(store + (size_t)key_id(cand[i]) * row_bytes, nchunk, t, rx);
          } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) rx[c] = make_uint4(0, 0, 0, 0);
          }
          const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rf, rx);
          if (act && t == 0) ++npair;
          if (__any_sync(FULL, act && alpha_test(ap, d, Dp))) pruned = true;
        }
        if (!pruned) {
          for (uint32_t w = lane; w < W; w += 32) prune[w] = 0u;  // bit j: kept member j is pruned by p
          __syncwarp();
          for (uint32_t jb = pos; jb < nk; jb += NT) {
            const uint32_t j = jb + team;
            const bool act = j < nk;
            uint4 rx[CPL];
            if (act) {
              load_row<G, CPL>(store + (size_t)key_id(cand[j]) * row_bytes, nchunk, t, rx);
            } else {
#pragma unroll
              for (int c = 0; c < CPL; ++c) rx[c] = make_uint4(0, 0, 0, 0);
            }
            const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rf, rx);
            if (act && t == 0) {
              ++npair;
              if (alpha_test(ap, d, key_dist<Dist>(cand[j]))) atomicOr(&prune[j >> 5], 1u << (j & 31));
            }
          }
          __syncwarp();
          // new row: kept[0..pos), p, surviving kept[pos..), cut at R
          uint32_t wpos = 0;
          for (uint32_t sb = 0; sb <= nk; sb += 32) {
            const uint32_t q = sb + lane;
            bool ok = false;
            unsigned long long key = 0;
            if (q <= nk) {
              if (q < pos) {
                key = cand[q];
                ok = true;
              } else if (q == pos) {
                key = kf;
                ok = true;
              } else {
                key = cand[q - 1];
                ok = !((prune[(q - 1) >> 5] >> ((q - 1) & 31)) & 1u);
              }
            }
            const unsigned bal = __ballot_sync(FULL, ok);
            const uint32_t o = wpos + __popc(bal & lt_mask);
            if (ok && o < R) {
              row[o] = key_id(key);
              if (a.g.rowd) a.g.rowd[(size_t)u * R + o] = (uint32_t)(key >> 32);
            }
            wpos += __popc(bal);
          }
          const uint32_t cnt = min(wpos, R);
          for (uint32_t sl = cnt + lane; sl < R; sl += 32) {
            row[sl] = kInvalid;
            if (a.g.rowd) a.g.rowd[(size_t)u * R + sl] = kInvalid;
          }
          if (lane == 0) {
            a.g.deg[u] = cnt;
            a.g.rowpfx[u] = (uint8_t)cnt;
          }
        }
        ++nprune;
      } else {
      // ---- C in key order.  The kept prefix is prune output and therefore already ascending: sort
      //      only the uncertain tail and merge the two runs by rank (checked, with a full sort as the
      //      fallback); long candidate lists take the full sort as well.
      uint32_t kpe = kp;
      bool merged = false;
      if (nC <= kSegSmem && kp > 0) {
        bool asc = true;
        for (uint32_t ib = 0; ib + 1 < kp; ib += 32) {
          const uint32_t i = ib + lane;
          const bool bad = i + 1 < kp && !(cand[i] < cand[i + 1]);
          if (__any_sync(FULL, bad)) asc = false;
        }
        if (asc) {
          const uint32_t nt = nC - kp;
          bitonic_sort_clean(cand + kp, nt, (uint32_t)lane, 32u, wsync);
          for (uint32_t i = lane; i < kp; i += 32) {
            const unsigned long long e = cand[i];
            uint32_t sft = 0;
            if (nt <= 8) {
              for (uint32_t r = 0; r < nt; ++r) sft += key_clean(cand[kp + r]) < e;
            } else {
              sft = lower_bound_clean(cand + kp, nt, e);
            }
            seg_s[i + sft] = e;
          }
          for (uint32_t r = lane; r < nt; r += 32) {
            const unsigned long long tk = cand[kp + r];
            seg_s[r + lower_bound_clean(cand, kp, key_clean(tk))] = tk;
          }
          __syncwarp();
          cs = seg_s;
          merged = true;
        } else {
          kpe = 0;  // not the expected order: trust nothing, test the whole triangle
        }
      }
      if (!merged) {
        bitonic_sort_clean(cand, nC, (uint32_t)lane, 32u, wsync);
        cs = cand;
      }
      if ((uint32_t)lane < W) hasp[lane] = 0u;
      // lane w holds word w of the set of candidates that are still valid
      uint32_t valid = 0;
      if ((uint32_t)lane < W) {
        const uint32_t lo = lane * 32;
        valid = nC >= lo + 32 ? 0xFFFFFFFFu : (nC > lo ? (1u << (nC - lo)) - 1u : 0u);
      }
      const uint32_t nu = nC - kpe;
      if (nu <= 2 * P && kpe == kp) {  // (the list of uncertain positions holds 2P entries; the tags must be trusted)
        // ---- few uncertain members among a pruned run.  Members of the run never prune each other, so the
        //      sequential prune only ever changes at an uncertain member f, and those are taken in key order:
        //      (a) does a valid member of the run in front of f prune it (earlier uncertain survivors have
        //      already had their say in their own step b)?  then f is gone;  (b) otherwise f is selected and
        //      prunes among the valid candidates behind it.  Only tests the sequential algorithm needs are
        //      evaluated, and (a) stops at the first hit.
        uint32_t nfound = 0;
        for (uint32_t jb = 0; jb < nC; jb += 32) {
          const uint32_t j = jb + lane;
          const bool un = j < nC && (cs[j] & kExpandedBit);
          const unsigned bal = __ballot_sync(FULL, un);
          if (un) upos[nfound + __popc(bal & lt_mask)] = j;
          nfound += __popc(bal);
        }
        __syncwarp();
        for (uint32_t fi = 0; fi < nfound; ++fi) {
          const uint32_t f = upos[fi];
          const uint32_t fw = __shfl_sync(FULL, valid, f >> 5);
          if (!((fw >> (f & 31)) & 1u)) continue;  // pruned by an earlier uncertain survivor
          // once R valid candidates stand in front of f, neither f nor anything behind it reaches the row
          uint32_t before = 0;
          if ((uint32_t)lane < (f >> 5)) before = __popc(valid);
          else if ((uint32_t)lane == (f >> 5)) before = __popc(valid & ((1u << (f & 31)) - 1u));
          if (__reduce_add_sync(FULL, before) >= R) break;
          const unsigned long long kf = cs[f];
          const Dist Df = key_dist<Dist>(kf);
          uint4 rf[CPL];
          load_row<G, CPL>(store + (size_t)key_id(kf) * row_bytes, nchunk, t, rf);
          bool pruned = false;
          for (uint32_t xb = 0; xb < f && !pruned; xb += NT) {
            const uint32_t x = xb + team;
            const unsigned long long kx = x < f ? cs[x] : 0ull;
            const uint32_t xw = __shfl_sync(FULL, valid, min(x, nC - 1u) >> 5);
            const bool act = x < f && !(kx & kExpandedBit) && ((xw >> (x & 31)) & 1u);
            uint4 rx[CPL];
            if (act) {
              load_row<G, CPL>(store + (size_t)key_id(kx) * row_bytes, nchunk, t, rx);
            } else {
#pragma unroll
              for (int c = 0; c < CPL; ++c) rx[c] = make_uint4(0, 0, 0, 0);
            }
            const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rf, rx);  // bitwise symmetric in its operands
            if (act && t == 0) ++npair;
            if (__any_sync(FULL, act && alpha_test(ap, d, Df))) pruned = true;
          }
          if (pruned) {
            if ((uint32_t)lane == (f >> 5)) valid &= ~(1u << (f & 31));
            continue;
          }
          for (uint32_t xb = f + 1; xb < nC; xb += NT) {
            const uint32_t x = xb + team;
            const unsigned long long kx = x < nC ? cs[x] : 0ull;
            const uint32_t xw = __shfl_sync(FULL, valid, min(x, nC - 1u) >> 5);
            const bool act = x < nC && ((xw >> (x & 31)) & 1u);
            uint4 rx[CPL];
            if (act) {
              load_row<G, CPL>(store + (size_t)key_id(kx) * row_bytes, nchunk, t, rx);
            } else {
#pragma unroll
              for (int c = 0; c < CPL; ++c) rx[c] = make_uint4(0, 0, 0, 0);
            }
            const Dist d = team_dist_regs<T, kMetricL2, G, CPL>(rf, rx);
            if (act && t == 0) {
              ++npair;
              if (alpha_test(ap, d, key_dist<Dist>(kx))) atomicOr(&hasp[x >> 5], 1u << (x & 31));
            }
          }
          __syncwarp();
          if ((uint32_t)lane < W) {
            valid &= ~hasp[lane];
            hasp[lane] = 0u;
          }
          __syncwarp();
        }
      } else {
        if constexpr (rebuild_cold_paths_out_of_line<G, CPL>()) {
          unsigned long long tested = 0;  // (a local of this branch: the loop's own counter stays in a register)
          valid = prune_all_pairs_ool<T, G, CPL>(store, row_bytes, nchunk, cs, nC, W, prune, hasp, ap, valid, tested, lane);
          npair += tested;
        } else {
          valid = prune_all_pairs_impl<T, G, CPL>(store, row_bytes, nchunk, cs, nC, W, prune, hasp, ap, valid, npair, lane);
        }
      }
      __syncwarp();
      // the first R members of the final valid set, in key order, are the new row
      uint32_t base_rank = 0;
      for (uint32_t sb = 0; sb < nC; sb += 32) {
        const uint32_t word = __shfl_sync(FULL, valid, sb >> 5);
        const uint32_t rank = base_rank + __popc(word & lt_mask);
        if (((word >> lane) & 1u) && rank < R) {
          const unsigned long long ks = cs[sb + lane];
          row[rank] = key_id(ks);
          if (a.g.rowd) a.g.rowd[(size_t)u * R + rank] = (uint32_t)(ks >> 32);
        }
        base_rank += __popc(word);
      }
      const uint32_t cnt = min(base_rank, R);
      for (uint32_t sl = cnt + lane; sl < R; sl += 32) {
        row[sl] = kInvalid;
        if (a.g.rowd) a.g.rowd[(size_t)u * R + sl] = kInvalid;
      }
      if (lane == 0) {
        a.g.deg[u] = cnt;
        a.g.rowpfx[u] = (uint8_t)cnt;
      }
      ++nprune;
      }  // general prune
    }
    if (lane == 0) {
      a.cnt[u] = 0;
      a.fill[u] = 0;
      a.flag[u] = 0;
      if (a.g.birth) a.g.rowepoch[u] = a.g.epoch;  // every kept entry now refers to its target's present vector
    }
    ++ndone;
    if (u_ahead != kInvalid) {
      const uint32_t lines = (R + 31u) >> 5;  // 128-byte lines of a row
      const void* pa = nullptr;
      if ((uint32_t)lane < lines) pa = a.g.adj + (size_t)u_ahead * R + lane * 32;
      else if ((uint32_t)lane < 2 * lines) pa = a.g.rowd ? a.g.rowd + (size_t)u_ahead * R + (lane - lines) * 32 : nullptr;
      else if ((uint32_t)lane == 2 * lines) pa = a.cnt + u_ahead;
      else if ((uint32_t)lane == 2 * lines + 1) pa = a.start + u_ahead;
      else if ((uint32_t)lane == 2 * lines + 2) pa = a.g.deg + u_ahead;
      else if ((uint32_t)lane == 2 * lines + 3) pa = a.g.rowpfx + u_ahead;
      if (pa) asm volatile("prefetch.global.L2 [%0];" ::"l"(pa));
    }
    __syncwarp();
  }
  if (npair) atomicAdd(&a.state->counters[CTR_PAIR], npair);
  if (lane == 0) {
    if (nprune) {
      atomicAdd(&a.state->counters[CTR_PRUNE], (unsigned long long)nprune);
      atomicAdd(&a.state->counters[CTR_RB_PRUNED], (unsigned long long)nprune);
    }
    if (ndone) atomicAdd(&a.state->counters[CTR_DIRTY], (unsigned long long)ndone);
    if (nbytes) atomicAdd(&a.state->counters[CTR_RB_BYTES], nbytes);
  }
}

// ---- dirty nodes whose row cannot overflow (deg + requests <= R, at most kLightReq requests): nothing is pruned,
// the requests are appended in key order behind the kept part of the row, and in a delete batch the row is
// compacted first.  A team of 8 lanes owns one node (four nodes per warp); the row travels through registers
// (R <= 128: 16 slots per lane), the requests sit one per lane and are ranked against each other with shuffles.
// The result is exactly what rebuild_kernel's "|C| <= R" branch stores.
constexpr uint32_t kLightReq = 8;
constexpr int kLightWarps = 4;

__global__ void __launch_bounds__(kLightWarps * 32) rebuild_light_kernel(const RebuildArgs a) {
  constexpr unsigned FULL = 0xFFFFFFFFu;
  constexpr int TS = 8, SL = 16;  // team size, row slots per lane
  const int lane = threadIdx.x & 31, t = lane & (TS - 1), tsh = lane & ~(TS - 1);
  const uint32_t R = a.g.R, nlight = a.state->nlight;
  const uint32_t below = (1u << t) - 1u;
  const uint64_t team0 = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) / TS, nteams = ((uint64_t)gridDim.x * blockDim.x) / TS;
  unsigned long long nbytes = 0;
  uint32_t ndone = 0;
  // warp-uniform trip count: the four teams of a warp run in lockstep (team votes are bytes of warp ballots)
  for (uint64_t k0 = team0 - (uint64_t)(lane / TS); k0 < nlight; k0 += nteams) {
    const uint64_t k = k0 + (uint64_t)(lane / TS);
    const bool act = k < nlight;
    const uint32_t u = act ? a.dirty[a.dirty_cap - 1u - (uint32_t)k] : 0u;
    const uint32_t cntu = act ? a.cnt[u] : 0u;
    const uint32_t startu = act ? a.start[u] : 0u;
    const uint32_t du = act ? min(a.g.deg[u], R) : 0u;
    const uint32_t pfx = act ? min((uint32_t)a.g.rowpfx[u], du) : 0u;
    uint32_t* row = a.g.adj + (size_t)u * R;
    uint32_t* rowd = a.g.rowd ? a.g.rowd + (size_t)u * R : nullptr;
    // the request of this lane
    unsigned long long key = kKeyMax;
    if ((uint32_t)t < cntu) key = a.seg_keys[startu + t];
    // the row, slot j * 8 + t in register j
    uint32_t rv[SL], rd[SL];
#pragma unroll
    for (int j = 0; j < SL; ++j) {
      const uint32_t sl = (uint32_t)j * TS + t;
      rv[j] = sl < du ? row[sl] : kInvalid;
      rd[j] = (rowd && sl < du) ? rowd[sl] : kInvalid;
    }
    // ---- keep = N_out(u) \ B, stable, written straight back (every slot is in a register by now)
    uint32_t nk = 0, kp = 0, okbits = 0;
#pragma unroll
    for (int j = 0; j < SL; ++j) {
      if ((uint32_t)j * TS < R) {  // (uniform)
        const uint32_t sl = (uint32_t)j * TS + t;
        const bool ok = sl < du && !(a.delmap && bit_test(a.delmap, rv[j]));
        const unsigned tb = (__ballot_sync(FULL, ok) >> tsh) & 0xFFu;
        if (ok) {
          const uint32_t pos = nk + __popc(tb & below);
          okbits |= 1u << j;
          if (a.delmap) {  // (an insert batch leaves the kept part where it is)
            row[pos] = rv[j];
            if (rowd) rowd[pos] = rd[j];
          }
        }
        const uint32_t inpfx = pfx > (uint32_t)j * TS ? min(pfx - (uint32_t)j * TS, (uint32_t)TS) : 0u;
        kp += __popc(tb & ((1u << inpfx) - 1u));
        nk += __popc(tb);
      }
    }
    // ---- requests: rank by key, drop repeats, keep the first P, drop what the row already holds and u itself
    uint32_t less = 0, eqb = 0;  // bit s: request s has a smaller key / the same key and a lower lane
    const uint32_t klo = (uint32_t)key, khi = (uint32_t)(key >> 32);
    const uint32_t cmax = __reduce_max_sync(FULL, cntu);  // most requests of any of the warp's four nodes
#pragma unroll
    for (int s2 = 0; s2 < TS; ++s2) {
      if ((uint32_t)s2 >= cmax) break;
      const unsigned long long ks = ((unsigned long long)__shfl_sync(FULL, khi, s2, TS) << 32) | __shfl_sync(FULL, klo, s2, TS);
      if (ks < key) less |= 1u << s2;
      if (ks == key && s2 < t) eqb |= 1u << s2;
    }
    const bool have = (uint32_t)t < cntu;
    const bool first = have && eqb == 0;  // not a repeat of an earlier lane's request
    const unsigned firstb = (__ballot_sync(FULL, first) >> tsh) & 0xFFu;
    const uint32_t id = key_id(key);
    bool inrow = false;
#pragma unroll
    for (int s2 = 0; s2 < TS; ++s2) {
      if ((uint32_t)s2 >= cmax) break;
      const uint32_t ids = __shfl_sync(FULL, id, s2, TS);
      bool hit = false;
#pragma unroll
      for (int j = 0; j < SL; ++j) hit |= ((okbits >> j) & 1u) && rv[j] == ids;
      const unsigned hb = (__ballot_sync(FULL, hit) >> tsh) & 0xFFu;
      if (s2 == t) inrow = hb != 0;
    }
    const bool fresh = first && __popc(less & firstb) < a.P && id != u && !inrow;
    const unsigned freshb = (__ballot_sync(FULL, fresh) >> tsh) & 0xFFu;
    const uint32_t nC = nk + __popc(freshb);
    if (fresh) {
      const uint32_t pos = nk + __popc(less & freshb);
      row[pos] = id;
      if (rowd) rowd[pos] = khi;
    }
    // a compacted row ends earlier than before: the slots behind it go back to the invalid id
    for (uint32_t sl = nC + t; sl < du; sl += TS) {
      row[sl] = kInvalid;
      if (rowd) rowd[sl] = kInvalid;
    }
    if (act && t == 0) {
      a.g.deg[u] = nC;
      a.g.rowpfx[u] = (uint8_t)kp;
      a.cnt[u] = 0;
      a.fill[u] = 0;
      a.flag[u] = 0;
      nbytes += 2ull * R * 4u + (unsigned long long)cntu * 12u;
      ++ndone;
    }
  }
  if (ndone) {
    atomicAdd(&a.state->counters[CTR_DIRTY], (unsigned long long)ndone);
    atomicAdd(&a.state->counters[CTR_RB_BYTES], nbytes);
  }
}

template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_rebuild_t(const RebuildArgs& a, cudaStream_t s) {
  const size_t per_warp = rebuild_smem_per_warp(a.g.R, a.P);
  const size_t smem = per_warp * kRebuildWarps;
  auto kern = rebuild_kernel<T, METRIC, G, CPL>;
  static SmemOptIn optin{};
  cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
  if (e != cudaSuccess) return e;
  int occ = 1;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kRebuildWarps * 32, smem);
  if (occ < 1) occ = 1;
  uint32_t blocks = (uint32_t)sm_count() * occ;
  if (blocks > a.max_blocks && a.max_blocks) blocks = a.max_blocks;
  if (a.split) {
    // the light nodes first (their launch is short); neither kernel touches a node of the other's list
    uint32_t lb = (uint32_t)sm_count() * 8u;
    if (lb > a.max_blocks && a.max_blocks) lb = a.max_blocks;
    rebuild_light_kernel<<<lb, kLightWarps * 32, 0, s>>>(a);
    count_launches(1);
  }
  kern<<<blocks, kRebuildWarps * 32, smem, s>>>(a, (uint32_t)per_warp);
  count_launches(1);
  return cudaGetLastError();
}
cudaError_t launch_rebuild(const RebuildArgs& a, cudaStream_t s) {
  GRAND_DISPATCH_L2(a.lay, launch_rebuild_t, a, s);
  return cudaErrorInvalidValue;
}

}  // namespace grand
