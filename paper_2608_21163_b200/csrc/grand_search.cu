// Batched greedy beam search (BeamSearch, Alg. 1): one warp per query.
//
// Per warp, in shared memory: the sorted worklist C (L keys; the expanded flag rides in bit 31 of
// the id word), a visited cache that may forget but never lies, and the candidate staging arrays
// of one expansion.  One expansion = read the adjacency row of the best unexpanded entry, drop ids
// the cache has seen, gather the surviving neighbours' vectors with 128-bit loads (a team of G
// lanes per vector, several vectors in flight per lane), reduce the distances with shuffles, and
// merge the survivors into the worklist in parallel.
//
// The worklist always equals the L smallest (dist, id) keys seen so far, so the result does not
// depend on what the cache forgets: a re-evaluated node either matches an entry exactly (dropped
// as a duplicate by key equality) or fails the comparison with the worst entry.
//
// Visited cache.  When every id fits 16 + (bucket bits) bits, the cache stores 16-bit tags in
// buckets of 8: an odd multiplier is a bijection on that id range, its high bits pick the bucket
// and its low 16 bits are the tag, so (bucket, tag) identifies the id exactly and a hit is never
// false.  That doubles the entries per byte and makes forgetting rare.  Larger capacities fall
// back to a direct-mapped table of full 32-bit ids.
#include "grand_common.cuh"
#include "grand_kernels.h"

namespace grand {

constexpr int kSearchWarps = 4;

static inline uint32_t even_up(uint32_t x) { return (x + 1u) & ~1u; }

size_t beam_search_smem_per_warp(uint32_t L, uint32_t R, uint32_t hash_bits, uint32_t cache_ways) {
  const size_t Lp = even_up(L), Rp = even_up(R);
  return Lp * 8 + Rp * 8 + Rp * 8 + Rp * 4 + Rp * 4 + ((size_t)(cache_ways == 12 ? 6 : 4) << hash_bits);
}

// Hint: bring one adjacency row (R ids) towards L2; lanes cover its 128-byte lines.
__device__ __forceinline__ void prefetch_row(const uint32_t* row, uint32_t R, int lane) {
  if ((uint32_t)lane * 32u < R) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + lane * 32));
}

// Visited cache probe: returns true if v was not known (and records it).
// (ways12: buckets of twelve tags in 24 bytes instead of eight in 16 - the same number of buckets, half as many tags
// again; taken on long rows, where a re-evaluated node costs a row of HBM traffic and shared memory is left over)
__device__ __forceinline__ bool visit_fresh(uint32_t* hash, uint32_t hash_bits, bool tags16, bool ways12, uint32_t v) {
  if (tags16) {
    const uint32_t ub = hash_bits + 14;  // bucket bits (hash_bits - 2) + 16 tag bits
    const uint32_t h = (v * 0x9E3779B1u) & ((1u << ub) - 1u);
    const uint32_t bucket = h >> 16, tag = h & 0xFFFFu;
    if (tag == 0xFFFFu) return true;  // the empty marker cannot be stored: always re-evaluate
    if (ways12) {
      uint2* bp = reinterpret_cast<uint2*>(hash) + (size_t)bucket * 3u;
      const uint2 b0 = bp[0], b1 = bp[1], b2 = bp[2];
      const uint32_t t2 = tag | (tag << 16);
      auto z = [](uint32_t x) { return (x - 0x00010001u) & ~x & 0x80008000u; };
      if (z(b0.x ^ t2) | z(b0.y ^ t2) | z(b1.x ^ t2) | z(b1.y ^ t2) | z(b2.x ^ t2) | z(b2.y ^ t2)) return false;
      uint2 n0, n1, n2;
      n2.y = __funnelshift_l(b2.x, b2.y, 16);
      n2.x = __funnelshift_l(b1.y, b2.x, 16);
      n1.y = __funnelshift_l(b1.x, b1.y, 16);
      n1.x = __funnelshift_l(b0.y, b1.x, 16);
      n0.y = __funnelshift_l(b0.x, b0.y, 16);
      n0.x = (b0.x << 16) | tag;
      bp[0] = n0; bp[1] = n1; bp[2] = n2;
      return true;
    }
    const uint4 b = reinterpret_cast<const uint4*>(hash)[bucket];
    const uint32_t t2 = tag | (tag << 16);
    // zero-halfword test: z(x) has bit 15 / 31 set where the low / high half of x is zero
    auto z = [](uint32_t x) { return (x - 0x00010001u) & ~x & 0x80008000u; };
    if (z(b.x ^ t2) | z(b.y ^ t2) | z(b.z ^ t2) | z(b.w ^ t2)) return false;
    // the bucket is a queue: the new tag enters in front and the oldest one (or an empty marker) falls out
    uint4 nb;
    nb.w = __funnelshift_l(b.z, b.w, 16);
    nb.z = __funnelshift_l(b.y, b.z, 16);
    nb.y = __funnelshift_l(b.x, b.y, 16);
    nb.x = (b.x << 16) | tag;
    reinterpret_cast<uint4*>(hash)[bucket] = nb;
    return true;
  }
  const uint32_t h = (v * 2654435761u) >> (32 - hash_bits);
  if (hash[h] == v) return false;
  hash[h] = v;
  return true;
}

// Resident blocks per SM that the register allocation must leave room for, per layout (measured: the 6-chunk
// layout gains a sixth block from its bound; the widest rows keep so many loads in flight per lane that a tighter
// bound than 3 blocks means spills; short rows run best at 7 blocks of the 8 their shared memory allows).
template <int G, int CPL>
constexpr int search_min_blocks() {
  return G == 32 ? (CPL >= 8 ? 3 : CPL >= 4 ? 5 : 8) : (CPL >= 6 ? 6 : 7);
}

// RC / LC: degree bound and worklist size as compile-time constants (0 = taken from the arguments).  On short rows
// the kernel is bound by instruction issue, and the common parameter pairs get an instantiation whose loops over the
// row and over the worklist are unrolled, whose worklist chunks travel through registers during a merge, and which
// loads the adjacency row of the next expansion into registers one expansion ahead.
template <typename T, int METRIC, int G, int CPL, int RC, int LC>
__global__ void __launch_bounds__(kSearchWarps * 32, search_min_blocks<G, CPL>()) beam_search_kernel(const SearchArgs a, const uint32_t per_warp_bytes) {
  using Dist = typename Elem<T>::Dist;
  constexpr int RW = RC ? (RC + 31) / 32 : 4;   // 32-id words of an adjacency row per lane
  constexpr int LW = LC ? (LC + 31) / 32 : 1;   // worklist chunks (used only when LC is given)
  constexpr int NT = 32 / G;                                   // teams per warp
  constexpr int U = CPL == 1 ? 4 : ((CPL == 2 || G == 32) ? 2 : 1);  // vectors in flight per team
  constexpr unsigned FULL = 0xFFFFFFFFu;
  extern __shared__ __align__(16) unsigned char smem_raw[];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = lane % G, team = lane / G;
  const uint32_t lt_mask = (1u << lane) - 1u;
  const uint32_t L = LC ? (uint32_t)LC : a.L, R = RC ? (uint32_t)RC : a.g.R, HB = a.hash_bits, H = 1u << HB;
  const uint32_t Lp = (L + 1u) & ~1u, Rp = (R + 1u) & ~1u;
  unsigned char* base = smem_raw + (size_t)warp * per_warp_bytes;
  unsigned long long* beam = reinterpret_cast<unsigned long long*>(base);
  unsigned long long* ckey = beam + Lp;     // candidate keys of this expansion, then the compacted survivors
  unsigned long long* cskey = ckey + Rp;    // surviving candidate keys, ascending
  uint32_t* cid = reinterpret_cast<uint32_t*>(cskey + Rp);  // candidate ids, later the survivors' worklist ranks
  uint32_t* csb = cid + Rp;                 // worklist rank of each sorted survivor
  uint32_t* hash = csb + Rp;                // visited cache (also query staging)

  const uint32_t nchunk = a.lay.nchunk, row_bytes = a.lay.row_bytes;
  const uint8_t* __restrict__ store = a.g.store;
  const bool tags16 = a.g.cap <= (1ull << (a.hash_bits + 14));
  const bool ways12 = tags16 && a.cache_ways == 12;
  const uint32_t Hw = ways12 ? H + (H >> 1) : H;  // words of the visited cache
  unsigned long long n_exp = 0, n_dist = 0;

  const uint64_t wglobal = (uint64_t)blockIdx.x * kSearchWarps + warp;
  const uint64_t wtotal = (uint64_t)gridDim.x * kSearchWarps;
  uint64_t qi_static = wglobal;
  for (;;) {
    // queries are handed out through an atomic counter when the caller provides one (search times
    // vary, and the last partial round would otherwise leave most warps idle)
    uint64_t qi;
    if (a.work_ctr) {
      unsigned k = 0;
      if (lane == 0) k = atomicAdd(a.work_ctr, 1u);
      qi = __shfl_sync(FULL, k, 0);
    } else {
      qi = qi_static;
      qi_static += wtotal;
    }
    if (qi >= a.nq) break;
    // ---- query into registers: lane t of each team holds chunks t, t+G, ...
    uint4 q[CPL];
    uint32_t self = kInvalid;
    if (a.qids) {
      self = a.qids[qi];
      load_row<G, CPL>(store + (size_t)self * row_bytes, nchunk, t, q);
    } else {
      T* stage = reinterpret_cast<T*>(hash);
      const T* src = reinterpret_cast<const T*>(a.queries) + qi * a.lay.udim;
      const uint32_t npad = row_bytes / sizeof(T);
      for (uint32_t j = lane; j < npad; j += 32) stage[j] = j < a.lay.udim ? src[j] : T(0);  // extra coordinate of a query: 0
      __syncwarp();
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        const uint32_t ch = t + c * G;
        q[c] = ch < nchunk ? reinterpret_cast<const uint4*>(stage)[ch] : make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
    }
    for (uint32_t j = lane; j < Hw; j += 32) hash[j] = kInvalid;
    __syncwarp();

    uint32_t beam_n = 0, nvis = 0, cursor = 0;
    unsigned long long alt_key = kKeyMax;  // best unexpanded entry besides the one being expanded
    uint32_t nrow[RW];              // (RC given) adjacency row loaded ahead for the likeliest next expansion
    uint32_t nrow_id = kInvalid;
#pragma unroll
    for (int c = 0; c < RW; ++c) nrow[c] = kInvalid;
    auto load_adj_row = [&](uint32_t id, uint32_t (&dst)[RW]) {
      const uint32_t* __restrict__ rp = a.g.adj + (size_t)id * R;
#pragma unroll
      for (int c = 0; c < RW; ++c) dst[c] = (uint32_t)(c * 32 + lane) < R ? __ldg(rp + c * 32 + lane) : kInvalid;
    };

    // Evaluate cid[0..n) against the query and merge the survivors into the worklist.
    auto process = [&](uint32_t n) {
      // 1. distances: NT teams, U vectors in flight per team; only keys below the worst entry are kept
      const unsigned long long worst = beam_n == L ? key_clean(beam[L - 1]) : kKeyMax;
      uint32_t nkept = 0;
      for (uint32_t b0 = 0; b0 < n; b0 += NT * U) {
        uint4 v[U][CPL];
        uint32_t idv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const uint32_t idx = b0 + u * NT + team;
          idv[u] = kInvalid;
          // warp-uniform: this slice of the pass is empty (whole-warp teams keep both rows' loads back to back)
          if (G < 32 && u > 0 && b0 + u * NT >= n) continue;
          if (idx < n) idv[u] = cid[idx];            // (no per-team early exit here: it would serialise the loads)
          if (idv[u] != kInvalid) {
            load_row<G, CPL>(store + (size_t)idv[u] * row_bytes, nchunk, t, v[u]);
          } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) v[u][c] = make_uint4(0, 0, 0, 0);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          if (G < 32 && u > 0 && b0 + u * NT >= n) continue;
          const Dist d = team_dist_regs<T, METRIC, G, CPL>(q, v[u]);
          const unsigned long long key = make_key(d, idv[u]);
          const bool below = t == 0 && idv[u] != kInvalid && key < worst;
          const unsigned bal = __ballot_sync(FULL, below);
          if (below) ckey[nkept + __popc(bal & lt_mask)] = key;
          nkept += __popc(bal);
        }
      }
      n_dist += n;
      if (nkept == 0) return;  // the common case late in a search: nothing enters the worklist
      __syncwarp();
      if constexpr (LC > 0) {
        if (nkept == 1) {
          // one key: its rank is a count over the worklist chunks, which then move up by one through registers
          const unsigned long long key = ckey[0];
          unsigned long long e[LW];
          uint32_t b = 0;
          unsigned dup = 0;
#pragma unroll
          for (int c = 0; c < LW; ++c) {
            const uint32_t i = (uint32_t)c * 32 + lane;
            const bool in = i < beam_n;
            e[c] = in ? beam[i] : 0ull;
            const unsigned long long ec = key_clean(e[c]);
            b += __popc(__ballot_sync(FULL, in && ec < key));
            dup |= __ballot_sync(FULL, in && ec == key);
          }
          if (dup) return;  // already in the worklist
          if (!a.boot_ids && key < key_clean(alt_key)) {  // it will be expanded next
            if constexpr (RC > 0) {
              nrow_id = key_id(key);
              load_adj_row(nrow_id, nrow);
            } else {
              prefetch_row(a.g.adj + (size_t)key_id(key) * R, R, lane);
            }
          }
          __syncwarp();
#pragma unroll
          for (int c = 0; c < LW; ++c) {
            const uint32_t i = (uint32_t)c * 32 + lane;
            if (i < beam_n && i >= b && i + 1 < L) beam[i + 1] = e[c];
          }
          if (lane == 0) beam[b] = key;
          __syncwarp();
          beam_n = min(L, beam_n + 1);
          cursor = min(cursor, b);
          return;
        }
      }
      // 2. drop keys that are already in the worklist; compact the rest in place (a write never passes the
      //    reader of its own chunk) and remember their ranks
      uint32_t m = 0;
      unsigned long long best = kKeyMax;
      for (uint32_t jb = 0; jb < nkept; jb += 32) {
        const uint32_t j = jb + lane;
        bool pass = false;
        unsigned long long key = 0;
        uint32_t b = 0;
        if (j < nkept) {
          key = ckey[j];
          b = lower_bound_clean(beam, beam_n, key);
          pass = !(b < beam_n && key_clean(beam[b]) == key);
        }
        const unsigned bal = __ballot_sync(FULL, pass);
        if (pass) {
          const uint32_t pos = m + __popc(bal & lt_mask);
          ckey[pos] = key;
          cid[pos] = b;
          best = min(best, key);
        }
        m += __popc(bal);
      }
      __syncwarp();
      if (m == 0) return;
      if (!a.boot_ids) {  // a new entry closer than every unexpanded one will be expanded next
        best = warp_min_key(best);
        if (best < key_clean(alt_key)) {
          if constexpr (RC > 0) {
            nrow_id = key_id(best);
            load_adj_row(nrow_id, nrow);
          } else {
            prefetch_row(a.g.adj + (size_t)key_id(best) * R, R, lane);
          }
        }
      }
      // rank the survivors among themselves (m is small)
      for (uint32_t j = lane; j < m; j += 32) {
        const unsigned long long key = ckey[j];
        uint32_t r = 0;
        for (uint32_t i = 0; i < m; ++i) r += ckey[i] < key;
        cskey[r] = key;
        csb[r] = cid[j];
      }
      __syncwarp();
      // 3. shift worklist entries to their final places, highest chunk first (a move never goes
      //    down, so an entry that is still unread is never overwritten).  Entry i moves up by the
      //    number of survivors whose rank is <= i.
      const uint32_t minb = csb[0];
      if constexpr (LC > 0) {
        // every chunk is read into registers before any entry is written: no ordering between chunks is needed
        unsigned long long e[LW];
        uint32_t np[LW];
#pragma unroll
        for (int c = 0; c < LW; ++c) {
          const uint32_t i = (uint32_t)c * 32 + lane;
          np[c] = kInvalid;
          e[c] = 0ull;
          if (i < beam_n && i >= minb) {
            e[c] = beam[i];
            uint32_t sft = 0;
            if (m <= 8) {
              for (uint32_t r = 0; r < m; ++r) sft += csb[r] <= i;
            } else {
              uint32_t lo = 0, hi = m;  // first r with csb[r] > i
              while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (csb[mid] <= i) lo = mid + 1; else hi = mid;
              }
              sft = lo;
            }
            np[c] = i + sft;
          }
        }
        __syncwarp();
#pragma unroll
        for (int c = 0; c < LW; ++c)
          if (np[c] < L) beam[np[c]] = e[c];
        __syncwarp();
      } else if (beam_n > minb) {
        const int top = (int)((beam_n - 1) >> 5), low = (int)(minb >> 5);
        for (int ch = top; ch >= low; --ch) {
          const uint32_t i = (uint32_t)ch * 32 + lane;
          unsigned long long e = 0;
          uint32_t np = kInvalid;
          if (i < beam_n && i >= minb) {
            e = beam[i];
            uint32_t s = 0;
            if (m <= 8) {
              for (uint32_t r = 0; r < m; ++r) s += csb[r] <= i;
            } else {
              uint32_t lo = 0, hi = m;  // first r with csb[r] > i
              while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (csb[mid] <= i) lo = mid + 1; else hi = mid;
              }
              s = lo;
            }
            np = i + s;
          }
          __syncwarp();  // every read of this chunk precedes its writes; lower chunks are not written from here
          if (np < L) beam[np] = e;
        }
        __syncwarp();
      }
      // 4. drop the survivors in
      for (uint32_t r = lane; r < m; r += 32) {
        const uint32_t np = r + csb[r];
        if (np < L) beam[np] = cskey[r];
      }
      __syncwarp();
      beam_n = min(L, beam_n + m);
      cursor = min(cursor, minb);
    };

    if (a.boot_ids) {
      // bootstrap batch: no graph yet, scan every batch-mate (brute force through the same merge)
      for (uint32_t c0 = 0; c0 < a.boot_n; c0 += R) {
        uint32_t n = 0;
        for (uint32_t sb = 0; sb < R; sb += 32) {
          const uint32_t s = sb + lane;
          uint32_t v = kInvalid;
          if (s < R && c0 + s < a.boot_n) v = a.boot_ids[c0 + s];
          const bool ok = v != kInvalid && v != self;
          const unsigned bal = __ballot_sync(FULL, ok);
          if (ok) cid[n + __popc(bal & lt_mask)] = v;
          n += __popc(bal);
        }
        __syncwarp();
        if (n) process(n);
      }
    } else if (a.entry != kInvalid) {
      if (lane == 0) {
        cid[0] = a.entry;
        visit_fresh(hash, HB, tags16, ways12, a.entry);
      }
      __syncwarp();
      process(1);
      while (nvis < a.vmax) {
        // closest unexpanded entry; everything before `cursor` is expanded
        // ... and the one after it, the likeliest next expansion
        uint32_t pos = kInvalid, apos = kInvalid;
        for (uint32_t cb = cursor & ~31u; cb < beam_n; cb += 32) {
          const uint32_t i = cb + lane;
          const bool un = i < beam_n && i >= cursor && !(beam[i] & kExpandedBit);
          unsigned bal = __ballot_sync(FULL, un);
          if (pos == kInvalid && bal) {
            pos = cb + __ffs(bal) - 1;
            bal &= bal - 1u;
          }
          if (pos != kInvalid && bal) {
            apos = cb + __ffs(bal) - 1;
            break;
          }
        }
        if (pos == kInvalid) break;
        const unsigned long long ek = beam[pos];
        alt_key = apos != kInvalid ? beam[apos] : kKeyMax;
        __syncwarp();
        if (lane == 0) {
          beam[pos] = ek | kExpandedBit;
          if (a.out_vis) a.out_vis[qi * a.vis_stride + nvis] = ek;
        }
        cursor = pos + 1;
        ++nvis;
        const uint32_t u = key_id(ek);
        // Rows are padded with the invalid id, so the whole row is read without waiting for deg[u].
        uint32_t vrow[RW];
        if constexpr (RC > 0) {
          if (u == nrow_id) {
#pragma unroll
            for (int c = 0; c < RW; ++c) vrow[c] = nrow[c];
          } else {
            load_adj_row(u, vrow);
          }
          // the row of the likeliest next expansion is loaded ahead (process() replaces it when a closer candidate turns up)
          nrow_id = kInvalid;
          if (alt_key != kKeyMax) {
            nrow_id = key_id(alt_key);
            load_adj_row(nrow_id, nrow);
          }
        } else {
          load_adj_row(u, vrow);
          // While that load is in flight: pull the adjacency row of the likeliest next expansion towards L2
          // (process() does the same for a closer new candidate).
          if (alt_key != kKeyMax) prefetch_row(a.g.adj + (size_t)key_id(alt_key) * R, R, lane);
        }
        uint32_t n = 0;
#pragma unroll
        for (int c = 0; c < RW; ++c) {
          if ((uint32_t)(c * 32) < R) {
            const uint32_t v = vrow[c];
            const bool fresh = v != kInvalid && (!a.check_live || bit_test(a.g.live, v)) && visit_fresh(hash, HB, tags16, ways12, v);
            const unsigned bal = __ballot_sync(FULL, fresh);
            if (fresh) cid[n + __popc(bal & lt_mask)] = v;
            n += __popc(bal);
          }
        }
        __syncwarp();
        if (n) process(n);
      }
      n_exp += nvis;
    }

    // ---- outputs
    float qn = 0.0f;  // |q|^2, needed to turn augmented L2 back into a negated inner product
    if constexpr (sizeof(T) == 4) {
      if (a.mips && a.out_dists) {
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
          const float* qf = reinterpret_cast<const float*>(&q[c]);
          qn = fmaf(qf[0], qf[0], fmaf(qf[1], qf[1], fmaf(qf[2], qf[2], fmaf(qf[3], qf[3], qn))));
        }
        qn = team_sum<G>(qn);
      }
    }
    if (a.out_ids) {
      for (uint32_t j = lane; j < a.k; j += 32) {
        const bool have = j < beam_n;
        const unsigned long long key = have ? beam[j] : 0ull;
        a.out_ids[qi * a.k + j] = have ? key_id(key) : kInvalid;
        if (a.out_dists) {
          if constexpr (sizeof(T) == 4) {
            float dv = have ? key_dist<float>(key) : __int_as_float(0x7f800000);
            if (a.mips && have) dv = (dv - qn - a.mips_M2) * 0.5f;
            reinterpret_cast<float*>(a.out_dists)[qi * a.k + j] = dv;
          } else {
            reinterpret_cast<int*>(a.out_dists)[qi * a.k + j] = have ? key_dist<int>(key) : 0x7fffffff;
          }
        }
      }
    }
    if (a.out_beam) {
      for (uint32_t j = lane; j < beam_n; j += 32) a.out_beam[qi * a.beam_stride + j] = key_clean(beam[j]);
      if (lane == 0) a.out_beam_n[qi] = beam_n;
    }
    if (a.out_vis) {
      if (a.boot_ids) {  // bootstrap: the candidate list handed to the prune is the sorted worklist
        const uint32_t nv = min(beam_n, a.vis_stride);
        for (uint32_t j = lane; j < nv; j += 32) a.out_vis[qi * a.vis_stride + j] = key_clean(beam[j]);
        if (lane == 0) a.out_vis_n[qi] = nv;
      } else if (lane == 0) {
        a.out_vis_n[qi] = nvis;
      }
    }
    __syncwarp();
  }
  if (lane == 0 && a.state) {
    if (n_exp) atomicAdd(&a.state->counters[CTR_EXP], n_exp);
    if (n_dist) atomicAdd(&a.state->counters[CTR_DIST], n_dist);
  }
}

template <typename T, int METRIC, int G, int CPL, int RC, int LC>
static cudaError_t launch_beam_search_rl(const SearchArgs& a0, cudaStream_t s) {
  SearchArgs a = a0;
  auto kern = beam_search_kernel<T, METRIC, G, CPL, RC, LC>;
  static SmemOptIn optin{};
  cudaError_t e = allow_full_dynamic_smem((const void*)kern, &optin);
  if (e != cudaSuccess) return e;
  a.cache_ways = 8;
  size_t per_warp = beam_search_smem_per_warp(a.L, a.g.R, a.hash_bits, 8);
  size_t smem = per_warp * kSearchWarps;
  int occ = 1;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kSearchWarps * 32, smem);
  if (occ < 1) occ = 1;
  if constexpr (G == 32) {
    // Rows above 512 bytes: the kernel is bound by HBM traffic, a re-evaluated node costs a whole row of it, and
    // registers limit the resident blocks to a few - so the visited cache takes what shared memory those blocks
    // leave over: buckets of twelve tags, and twice the buckets when the caller left the size to the library.
    // (Not on 384-byte rows: six resident blocks with the larger cache take 210 KB of the SM's 256 KB, what is left
    // as L1 no longer holds the loads in flight, and the search slows from 84.7 to 112.5 ms per step although it
    // gathers 5% fewer bytes.)
#ifndef GRAND_NO_WAYS12
    const uint32_t hb0 = a.hash_bits;
    const uint32_t try_hb[4] = {hb0 + 1, hb0 + 1, hb0, hb0}, try_ways[4] = {12, 8, 12, 8};
    for (int k = a.auto_cache ? 0 : 2; k < 3; ++k) {
      if (try_hb[k] > 13 || a.g.cap > (1ull << (try_hb[k] + 14))) continue;  // (the tag layout must hold every id)
      const size_t pw = beam_search_smem_per_warp(a.L, a.g.R, try_hb[k], try_ways[k]);
      int o2 = 0;
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, kern, kSearchWarps * 32, pw * kSearchWarps);
      if (o2 >= occ) {
        a.hash_bits = try_hb[k];
        a.cache_ways = try_ways[k];
        per_warp = pw;
        smem = per_warp * kSearchWarps;
        break;
      }
    }
#endif
  }
  uint64_t blocks = (a.nq + kSearchWarps - 1) / kSearchWarps;
  const uint64_t cap = (uint64_t)sm_count() * occ;
  if (blocks > cap) blocks = cap;
  if (blocks == 0) return cudaSuccess;
  kern<<<(unsigned)blocks, kSearchWarps * 32, smem, s>>>(a, (uint32_t)per_warp);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T, int METRIC, int G, int CPL>
static cudaError_t launch_beam_search_t(const SearchArgs& a, cudaStream_t s) {
  // short rows (teams of at most 8 lanes) with the usual parameter pairs take the unrolled instantiations
  if constexpr (G <= 8) {
    if (a.g.R == 64 && a.L == 128) return launch_beam_search_rl<T, METRIC, G, CPL, 64, 128>(a, s);
    if (a.g.R == 64 && a.L == 32) return launch_beam_search_rl<T, METRIC, G, CPL, 64, 32>(a, s);  // query searches at a small L
    if (a.g.R == 32 && a.L == 64) return launch_beam_search_rl<T, METRIC, G, CPL, 32, 64>(a, s);
  }
  return launch_beam_search_rl<T, METRIC, G, CPL, 0, 0>(a, s);
}

cudaError_t launch_beam_search(const SearchArgs& a, cudaStream_t s) {
  GRAND_DISPATCH_ALL(a.lay, launch_beam_search_t, a, s);
  return cudaErrorInvalidValue;
}

}  // namespace grand
