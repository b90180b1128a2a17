// GrAND oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-file CPU restatement of the batched dynamic update and search of a
// Vamana-style proximity graph (GrAND: Alg. 1 BeamSearch, Alg. 2/4 RobustPrune, Alg. 5
// BatchInsert, Alg. 6 BatchDelete with in-neighbours taken from the exact on-demand reverse
// graph of Alg. 8, and the fixed-degree find-and-replace mode of Alg. 7/8).
// It shares no code with the CUDA library and must never be imported by the product path:
// only the test-suite, the smoke check and the CPU-baseline leg of the benchmark call it.
//
// Deterministic batch semantics (one legal outcome of the races the paper's lock-free scheme
// allows): every search of a batch runs on the batch-start snapshot; reverse-edge candidates
// of one target merge in (distance, id) order; every tie breaks by id.
//
// Distances: L2 = squared Euclidean, IP = negated dot product.  uint8/int8 vectors use exact
// integer arithmetic; fp32 vectors accumulate in double in index order and round once to
// float.  All distances are carried as double (both cases are exactly representable).
//
// Parity pins (see tests/test_oracle_*.py): every function below is pinned by closed forms,
// hand-worked examples, brute force or invariants; nothing here is "parity unpinned" except
// the paper-level absolute numbers, which the paper does not print.

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <limits>
#include <thread>
#include <unordered_set>
#include <vector>

namespace {

constexpr uint32_t INVALID = 0xFFFFFFFFu;
enum { DT_U8 = 0, DT_I8 = 1, DT_F32 = 2 };
enum { M_L2 = 0, M_IP = 1 };
enum { MODE_VAMANA = 0, MODE_FIXED = 1 };
enum {
  OK = 0, ERR_INVALID_ARG = -1, ERR_CAPACITY = -2, ERR_DUPLICATE_ID = -3, ERR_ALREADY_LIVE = -4,
  ERR_NOT_LIVE = -5, ERR_UNSUPPORTED = -6
};

// key(v) = (dist, id), compared lexicographically: the total order behind every "closest",
// "argmin", "sort" and "first c" of the method.
struct Key {
  double d;
  uint32_t id;
};
inline bool key_less(const Key& a, const Key& b) { return a.d < b.d || (a.d == b.d && a.id < b.id); }

struct BeamEntry {
  Key k;
  bool expanded;
};

struct Stats {
  std::atomic<uint64_t> expansions{0}, dist_evals{0}, dead_edges_seen{0}, prunes{0}, dirty{0};
};

struct Index {
  uint32_t dim, dtype, metric, R, L;  // dim / metric as used internally (see `augment`)
  uint32_t udim = 0;                  // dimension of the caller's vectors
  bool augment = false;               // MIPS -> L2 reduction (Sec. 5.3): x -> [x, sqrt(M^2 - |x|^2)], q -> [q, 0]
  double M2 = 0.0;                    // M^2, M = bound on the base vectors' norms
  bool approx_delete = false;         // Alg. 6 as printed: in-neighbours of a deleted node are looked for in the
                                      // visited set of its search only; edges from other nodes stay behind
                                      // ("dangling") and every traversal skips neighbours that are not live
  float alpha;
  int64_t A_fix;  // round(alpha * 65536): fixed-point alpha for integer vectors
  uint64_t cap;
  uint32_t P, c, k_repair, vmax, mode, nthreads;
  size_t esize;
  std::vector<uint8_t> store;  // cap * dim elements, row-major
  std::vector<uint32_t> adj;   // cap * R, ordered rows
  std::vector<uint32_t> deg;   // cap
  std::vector<uint8_t> live;   // cap
  uint64_t nlive = 0;
  uint32_t entry = INVALID;  // medoid m
  Stats st;

  const void* vec(uint32_t id) const { return store.data() + (size_t)id * dim * esize; }
  uint32_t* row(uint32_t id) { return adj.data() + (size_t)id * R; }
  const uint32_t* row(uint32_t id) const { return adj.data() + (size_t)id * R; }
};

// Static partition of [0,n) over the index's threads; each item is independent per-node work.
void parallel_for(const Index& ix, size_t n, const std::function<void(size_t)>& fn) {
  size_t T = std::max<size_t>(1, std::min<size_t>(ix.nthreads, n));
  if (T == 1) {
    for (size_t i = 0; i < n; ++i) fn(i);
    return;
  }
  std::vector<std::thread> th;
  for (size_t t = 0; t < T; ++t) {
    size_t lo = n * t / T, hi = n * (t + 1) / T;
    th.emplace_back([lo, hi, &fn]() {
      for (size_t i = lo; i < hi; ++i) fn(i);
    });
  }
  for (auto& t : th) t.join();
}

// dist(a,b): L2 -> sum_j (a_j-b_j)^2 (squared, no root); IP -> -sum_j a_j*b_j.
double dist_raw(const Index& ix, const void* a, const void* b) {
  const uint32_t d = ix.dim;
  if (ix.dtype == DT_F32) {
    const float* x = (const float*)a;
    const float* y = (const float*)b;
    double acc = 0.0;
    if (ix.metric == M_L2) {
      for (uint32_t j = 0; j < d; ++j) {
        double t = (double)x[j] - (double)y[j];
        acc += t * t;
      }
    } else {
      for (uint32_t j = 0; j < d; ++j) acc += (double)x[j] * (double)y[j];
      acc = -acc;
    }
    return (double)(float)acc;  // rounded once to float
  }
  int64_t acc = 0;
  for (uint32_t j = 0; j < d; ++j) {
    int64_t xv, yv;
    if (ix.dtype == DT_U8) {
      xv = ((const uint8_t*)a)[j];
      yv = ((const uint8_t*)b)[j];
    } else {
      xv = ((const int8_t*)a)[j];
      yv = ((const int8_t*)b)[j];
    }
    if (ix.metric == M_L2) acc += (xv - yv) * (xv - yv);
    else acc -= xv * yv;
  }
  return (double)acc;
}

// Store one caller vector as an internal row.  With the MIPS->L2 reduction the extra coordinate is
// sqrt(M^2 - |x|^2) for base vectors and 0 for queries; squared L2 between such rows orders candidates
// exactly like the negated inner product does.
void to_row(const Index& ix, const void* src, void* dst, bool is_query) {
  std::memcpy(dst, src, (size_t)ix.udim * ix.esize);
  if (!ix.augment) return;
  double n2 = 0.0;
  for (uint32_t j = 0; j < ix.udim; ++j) n2 += (double)((const float*)src)[j] * (double)((const float*)src)[j];
  ((float*)dst)[ix.udim] = is_query ? 0.0f : (float)std::sqrt(std::max(ix.M2 - n2, 0.0));
}
double sq_norm(const Index& ix, const void* v) {
  double n2 = 0.0;
  for (uint32_t j = 0; j < ix.udim; ++j) n2 += (double)((const float*)v)[j] * (double)((const float*)v)[j];
  return n2;
}

// alpha test of GrANDRobustPrune (Alg. 4): alpha * dist(p*,p') <= D_p[p'].
bool alpha_test(const Index& ix, double d_star_cand, double d_p_cand) {
  if (ix.dtype == DT_F32) {
    float t = ix.alpha * (float)d_star_cand;  // one correctly rounded fp32 multiply
    return t <= (float)d_p_cand;
  }
  int64_t lhs = ix.A_fix * (int64_t)d_star_cand;
  int64_t rhs = (int64_t)d_p_cand * 65536;
  return lhs <= rhs;
}

// BeamSearch (Alg. 1) from `entry` on the current adjacency.  C: sorted worklist of capacity L
// with expanded flags; V: expanded nodes with their distances, in expansion order, at most vmax.
// use_seen_set adds a full visited set (as in the paper's prose); the result must not depend on
// it, because under a strict total order an evicted node can never re-enter the worklist.
void greedy_search(const Index& ix, uint32_t entry, const void* q, uint32_t L, uint32_t vmax,
                   bool use_seen_set, std::vector<BeamEntry>& C, std::vector<Key>& V, Stats* st) {
  C.clear();
  V.clear();
  if (entry == INVALID || L == 0) return;
  std::unordered_set<uint32_t> seen;
  C.push_back({{dist_raw(ix, q, ix.vec(entry)), entry}, false});
  if (use_seen_set) seen.insert(entry);
  uint64_t nd = 1, ne = 0, dead = 0;
  while (V.size() < vmax) {
    size_t ui = C.size();
    for (size_t i = 0; i < C.size(); ++i)
      if (!C[i].expanded) {
        ui = i;
        break;
      }
    if (ui == C.size()) break;
    C[ui].expanded = true;
    const uint32_t u = C[ui].k.id;
    V.push_back(C[ui].k);
    ++ne;
    const uint32_t* nb = ix.row(u);
    const uint32_t du = ix.deg[u];
    for (uint32_t s = 0; s < du; ++s) {
      const uint32_t v = nb[s];
      if (!ix.live[v]) {  // defensive; exact deletes make it unreachable (counted, tests assert 0)
        ++dead;
        continue;
      }
      if (use_seen_set) {
        if (!seen.insert(v).second) continue;
      }
      bool inC = false;
      for (const auto& e : C)
        if (e.k.id == v) {
          inC = true;
          break;
        }
      if (inC) continue;
      Key kv{dist_raw(ix, q, ix.vec(v)), v};
      ++nd;
      if (C.size() >= L && !key_less(kv, C.back().k)) continue;
      auto pos = std::lower_bound(C.begin(), C.end(), kv,
                                  [](const BeamEntry& e, const Key& k) { return key_less(e.k, k); });
      C.insert(pos, BeamEntry{kv, false});
      if (C.size() > L) C.pop_back();
    }
  }
  if (st) {
    st->expansions += ne;
    st->dist_evals += nd;
    st->dead_edges_seen += dead;
  }
}

// GrANDRobustPrune (Alg. 4 / Alg. 2): cand holds (D_p[v], v).  Returns the selected ids in
// selection order (ascending key) together with their cached distances.
std::vector<Key> robust_prune(const Index& ix, uint32_t p, std::vector<Key> cand, uint32_t R,
                              Stats* st) {
  cand.erase(std::remove_if(cand.begin(), cand.end(), [p](const Key& k) { return k.id == p; }),
             cand.end());
  std::sort(cand.begin(), cand.end(), key_less);
  {  // drop repeated ids, keeping the first in key order
    std::unordered_set<uint32_t> ids;
    std::vector<Key> u;
    for (const auto& k : cand)
      if (ids.insert(k.id).second) u.push_back(k);
    cand.swap(u);
  }
  std::vector<char> valid(cand.size(), 1);
  std::vector<Key> out;
  uint64_t nd = 0;
  for (;;) {
    size_t s = 0;
    while (s < cand.size() && !valid[s]) ++s;
    if (s == cand.size()) break;
    out.push_back(cand[s]);
    valid[s] = 0;
    if (out.size() == R) break;
    for (size_t j = 0; j < cand.size(); ++j) {
      if (!valid[j]) continue;
      double dpp = dist_raw(ix, ix.vec(cand[s].id), ix.vec(cand[j].id));
      ++nd;
      if (alpha_test(ix, dpp, cand[j].d)) valid[j] = 0;
    }
  }
  if (st) {
    st->dist_evals += nd;
    st->prunes += 1;
  }
  return out;
}

// Exact transpose of the live adjacency in CSR (Alg. 8, reverse-neighbour computation): row z lists
// every live v with z in N_out(v), ascending v.
void transpose(const Index& ix, std::vector<uint64_t>& off, std::vector<uint32_t>& src) {
  off.assign(ix.cap + 1, 0);
  for (uint64_t v = 0; v < ix.cap; ++v) {
    if (!ix.live[v]) continue;
    for (uint32_t s = 0; s < ix.deg[v]; ++s) off[ix.row((uint32_t)v)[s] + 1]++;
  }
  for (uint64_t z = 0; z < ix.cap; ++z) off[z + 1] += off[z];
  src.assign(off[ix.cap], 0);
  std::vector<uint64_t> fill(off.begin(), off.end() - 1);
  for (uint64_t v = 0; v < ix.cap; ++v) {  // ascending v => rows come out sorted
    if (!ix.live[v]) continue;
    for (uint32_t s = 0; s < ix.deg[v]; ++s) src[fill[ix.row((uint32_t)v)[s]]++] = (uint32_t)v;
  }
}

// One reverse-edge / repair request: target u receives candidate (dist(u,id), id).
struct Request {
  uint32_t target;
  Key k;
};

// Groups requests by target; each group sorted by (dist,id), repeated ids dropped, first `cap_p`
// kept (cap_p == 0: no cap).  Emulates the per-node scratch buffers of capacity P (Alg. 5/6).
struct Grouped {
  std::vector<uint32_t> targets;          // distinct, ascending
  std::vector<std::vector<Key>> scratch;  // parallel to targets
};
Grouped group_requests(std::vector<Request>& rq, uint32_t cap_p) {
  std::sort(rq.begin(), rq.end(), [](const Request& a, const Request& b) {
    if (a.target != b.target) return a.target < b.target;
    return key_less(a.k, b.k);
  });
  Grouped g;
  size_t i = 0;
  while (i < rq.size()) {
    size_t j = i;
    std::vector<Key> s;
    std::unordered_set<uint32_t> ids;
    while (j < rq.size() && rq[j].target == rq[i].target) {
      if (ids.insert(rq[j].k.id).second && (cap_p == 0 || s.size() < cap_p)) s.push_back(rq[j].k);
      ++j;
    }
    g.targets.push_back(rq[i].target);
    g.scratch.push_back(std::move(s));
    i = j;
  }
  return g;
}

// Rebuild of one dirty node u (Alg. 5 dirty loop / Alg. 6 rebuild loop): C = (N_out(u) u scratch_u) \ B;
// if |C| <= R store it (old order, then new in key order), else compute D_u and prune.
void rebuild_dirty(Index& ix, uint32_t u, const std::vector<Key>& scratch, const std::vector<uint8_t>* inB,
                   const std::vector<uint8_t>* alive = nullptr) {
  std::vector<uint32_t> keep;
  uint32_t* r = ix.row(u);
  for (uint32_t s = 0; s < ix.deg[u]; ++s)
    if ((!inB || !(*inB)[r[s]]) && (!alive || (*alive)[r[s]])) keep.push_back(r[s]);  // `alive`: drops dangling edges
  std::vector<Key> fresh;
  for (const auto& k : scratch) {
    if (k.id == u) continue;
    if (std::find(keep.begin(), keep.end(), k.id) != keep.end()) continue;
    fresh.push_back(k);
  }
  ix.st.dirty += 1;
  if (keep.size() + fresh.size() <= ix.R) {
    uint32_t n = 0;
    for (uint32_t v : keep) r[n++] = v;
    for (const auto& k : fresh) r[n++] = k.id;
    ix.deg[u] = n;
    return;
  }
  std::vector<Key> cand;
  uint64_t nd = 0;
  for (uint32_t v : keep) {
    cand.push_back({dist_raw(ix, ix.vec(u), ix.vec(v)), v});
    ++nd;
  }
  ix.st.dist_evals += nd;
  for (const auto& k : fresh) cand.push_back(k);  // request distances are dist(u, id) already
  std::vector<Key> out = robust_prune(ix, u, cand, ix.R, &ix.st);
  for (size_t s = 0; s < out.size(); ++s) r[s] = out[s].id;
  ix.deg[u] = (uint32_t)out.size();
}

// Initial medoid: the bootstrap-batch point minimising (dist(x, mean), id).
uint32_t pick_medoid(const Index& ix, const std::vector<uint32_t>& ids_sorted) {
  const uint32_t d = ix.dim;
  const int64_t B = (int64_t)ids_sorted.size();
  std::vector<uint8_t> mean(d * ix.esize);
  if (ix.dtype == DT_F32) {
    for (uint32_t j = 0; j < d; ++j) {
      double s = 0.0;
      for (uint32_t id : ids_sorted) s += (double)((const float*)ix.vec(id))[j];
      ((float*)mean.data())[j] = (float)(s / (double)B);
    }
  } else {
    for (uint32_t j = 0; j < d; ++j) {
      int64_t s = 0;
      for (uint32_t id : ids_sorted)
        s += ix.dtype == DT_U8 ? (int64_t)((const uint8_t*)ix.vec(id))[j] : (int64_t)((const int8_t*)ix.vec(id))[j];
      int64_t num = 2 * s + B, den = 2 * B;  // round-half-up mean via floor division
      int64_t m = num / den;
      if (num % den != 0 && num < 0) --m;
      if (ix.dtype == DT_U8) mean[j] = (uint8_t)m;
      else ((int8_t*)mean.data())[j] = (int8_t)m;
    }
  }
  Key best{0.0, INVALID};
  for (uint32_t id : ids_sorted) {
    Key k{dist_raw(ix, ix.vec(id), mean.data()), id};
    if (best.id == INVALID || key_less(k, best)) best = k;
  }
  return best.id;
}

int validate_insert(const Index& ix, const uint32_t* ids, uint64_t n) {
  std::unordered_set<uint32_t> s;
  for (uint64_t i = 0; i < n; ++i) {
    if (ids[i] >= ix.cap) return ERR_CAPACITY;
    if (!s.insert(ids[i]).second) return ERR_DUPLICATE_ID;
  }
  for (uint64_t i = 0; i < n; ++i)
    if (ix.live[ids[i]]) return ERR_ALREADY_LIVE;
  return OK;
}

// Brute-force nearest batch-mates for the bootstrap batch (empty snapshot; the paper starts from
// an offline-built seed graph instead).
std::vector<Key> nearest_batchmates(const Index& ix, const uint32_t* ids, uint64_t n, uint64_t i, uint32_t want) {
  std::vector<Key> all;
  for (uint64_t j = 0; j < n; ++j)
    if (j != i) all.push_back({dist_raw(ix, ix.vec(ids[i]), ix.vec(ids[j])), ids[j]});
  std::sort(all.begin(), all.end(), key_less);
  if (all.size() > want) all.resize(want);
  return all;
}

int insert_batch(Index& ix, const uint32_t* ids, const void* vecs, uint64_t n) {
  if (n == 0) return OK;
  int rc = validate_insert(ix, ids, n);
  if (rc != OK) return rc;
  const size_t rb = (size_t)ix.dim * ix.esize, urb = (size_t)ix.udim * ix.esize;
  if (ix.augment)
    for (uint64_t i = 0; i < n; ++i)
      if (sq_norm(ix, (const uint8_t*)vecs + i * urb) > ix.M2 * (1.0 + 1e-6)) return ERR_INVALID_ARG;  // norm above the stated bound
  for (uint64_t i = 0; i < n; ++i) {  // write vector, deg <- 0 (Alg. 5 first loop)
    to_row(ix, (const uint8_t*)vecs + i * urb, ix.store.data() + (size_t)ids[i] * rb, false);
    ix.deg[ids[i]] = 0;
  }
  const bool bootstrap = ix.nlive == 0;
  const bool fixed = ix.mode == MODE_FIXED;
  std::vector<std::vector<Key>> fwd(n);  // selected forward neighbours with dist(p_i, .)
  parallel_for(ix, n, [&](size_t i) {
    std::vector<Key> cand;
    if (bootstrap) {
      cand = nearest_batchmates(ix, ids, n, i, fixed ? ix.R : ix.L);
    } else {
      std::vector<BeamEntry> C;
      std::vector<Key> V;
      greedy_search(ix, ix.entry, ix.vec(ids[i]), ix.L, ix.vmax, false, C, V, &ix.st);
      if (fixed) {
        for (const auto& e : C) cand.push_back(e.k);  // final worklist, ascending key
      } else {
        cand = V;  // visited (expanded) list feeds the prune (Alg. 5)
      }
    }
    if (fixed) {  // Alg. 7: forward edges = R nearest found, no prune
      cand.erase(std::remove_if(cand.begin(), cand.end(), [&](const Key& k) { return k.id == ids[i]; }), cand.end());
      if (cand.size() > ix.R) cand.resize(ix.R);
      fwd[i] = cand;
    } else {
      fwd[i] = robust_prune(ix, ids[i], cand, ix.R, &ix.st);
    }
  });
  for (uint64_t i = 0; i < n; ++i) {  // forward rows: each new node writes only its own list
    uint32_t* r = ix.row(ids[i]);
    for (size_t s = 0; s < fwd[i].size(); ++s) r[s] = fwd[i][s].id;
    ix.deg[ids[i]] = (uint32_t)fwd[i].size();
  }
  std::vector<Request> rq;
  for (uint64_t i = 0; i < n; ++i)
    for (const auto& k : fwd[i]) rq.push_back({k.id, {k.d, ids[i]}});  // dist is symmetric: reuse D_{p_i}[u]
  if (!fixed) {
    Grouped g = group_requests(rq, ix.P);
    std::vector<uint8_t> alive;  // visited-set delete mode: rows may hold dangling edges; batch members count as alive
    if (ix.approx_delete) {
      alive = ix.live;
      for (uint64_t i = 0; i < n; ++i) alive[ids[i]] = 1;
    }
    parallel_for(ix, g.targets.size(), [&](size_t t) {
      rebuild_dirty(ix, g.targets[t], g.scratch[t], nullptr, ix.approx_delete ? &alive : nullptr);
    });
  } else {
    // Alg. 7 backward edges: detour find-and-replace, one owner per target, requests in key order.
    Grouped g = group_requests(rq, 0);
    std::vector<uint8_t> isnew(ix.cap, 0);
    std::vector<uint64_t> which(ix.cap, 0);
    for (uint64_t i = 0; i < n; ++i) {
      isnew[ids[i]] = 1;
      which[ids[i]] = i;
    }
    // rows of the new nodes as they stood after the forward phase (a bootstrap target is itself new)
    std::vector<std::vector<uint32_t>> frow(n);
    for (uint64_t i = 0; i < n; ++i)
      for (const auto& k : fwd[i]) frow[i].push_back(k.id);
    parallel_for(ix, g.targets.size(), [&](size_t t) {
      const uint32_t q = g.targets[t];
      uint32_t* r = ix.row(q);
      std::vector<char> replaced(ix.R, 0);
      for (const auto& k : g.scratch[t]) {
        const uint32_t p = k.id;
        uint32_t dq = ix.deg[q];
        if (std::find(r, r + dq, p) != r + dq) continue;  // already linked (bootstrap only)
        if (dq < ix.R) {
          r[dq] = p;
          ix.deg[q] = dq + 1;
          continue;
        }
        const std::vector<uint32_t>& np = frow[which[p]];
        int pick = -1;
        for (uint32_t j = 0; j < dq; ++j)
          if (!replaced[j] && std::find(np.begin(), np.end(), r[j]) != np.end()) pick = (int)j;
        if (pick >= 0) {
          r[pick] = p;
          replaced[pick] = 1;
        }
      }
    });
  }
  for (uint64_t i = 0; i < n; ++i) ix.live[ids[i]] = 1;
  ix.nlive += n;
  if (ix.entry == INVALID) {
    std::vector<uint32_t> s(ids, ids + n);
    std::sort(s.begin(), s.end());
    ix.entry = pick_medoid(ix, s);
  }
  return OK;
}

int delete_batch(Index& ix, const uint32_t* ids, uint64_t n) {
  if (n == 0) return OK;
  {
    std::unordered_set<uint32_t> s;
    for (uint64_t i = 0; i < n; ++i) {
      if (ids[i] >= ix.cap) return ERR_CAPACITY;
      if (!s.insert(ids[i]).second) return ERR_DUPLICATE_ID;
    }
    for (uint64_t i = 0; i < n; ++i)
      if (!ix.live[ids[i]]) return ERR_NOT_LIVE;
  }
  std::vector<uint8_t> inB(ix.cap, 0);
  for (uint64_t i = 0; i < n; ++i) inB[ids[i]] = 1;
  std::vector<uint64_t> off;
  std::vector<uint32_t> src;
  const bool approx = ix.approx_delete && ix.mode == MODE_VAMANA;
  if (!approx) transpose(ix, off, src);  // exact in-neighbours, rebuilt per delete batch and not kept

  uint32_t new_entry = INVALID;  // replacement medoid, used only if the medoid is in B
  if (ix.mode == MODE_FIXED) {
    // medoid deleted: its first surviving out-neighbour (rows are nearest-first)
    if (inB[ix.entry])
      for (uint32_t s = 0; s < ix.deg[ix.entry] && new_entry == INVALID; ++s)
        if (!inB[ix.row(ix.entry)[s]]) new_entry = ix.row(ix.entry)[s];
    // Alg. 8 rewire: every surviving in-neighbour u replaces each deleted slot by PickOne.
    std::vector<uint32_t> affected;
    for (uint64_t i = 0; i < n; ++i)
      for (uint64_t e = off[ids[i]]; e < off[ids[i] + 1]; ++e)
        if (!inB[src[e]]) affected.push_back(src[e]);
    std::sort(affected.begin(), affected.end());
    affected.erase(std::unique(affected.begin(), affected.end()), affected.end());
    parallel_for(ix, affected.size(), [&](size_t a) {
      const uint32_t u = affected[a];
      uint32_t* r = ix.row(u);
      const uint32_t du = ix.deg[u];
      for (uint32_t s = 0; s < du; ++s) {
        const uint32_t p = r[s];
        if (p == INVALID || !inB[p]) continue;
        const uint32_t* in0 = src.data() + off[p];
        const uint32_t* in1 = src.data() + off[p + 1];
        const uint64_t j = (uint64_t)(std::lower_bound(in0, in1, u) - in0);  // round-robin offset
        const uint32_t np = ix.deg[p];
        uint32_t chosen = INVALID;
        for (uint32_t t = 0; t < np && chosen == INVALID; ++t) {
          const uint32_t cand = ix.row(p)[(j + t) % np];
          if (inB[cand] || cand == u) continue;
          if (std::find(r, r + du, cand) != r + du) continue;
          chosen = cand;
        }
        r[s] = chosen;  // INVALID marks a slot to be removed
      }
      uint32_t w = 0;
      for (uint32_t s = 0; s < du; ++s)
        if (r[s] != INVALID) r[w++] = r[s];
      ix.deg[u] = w;
    });
  } else {
    // Alg. 6: per-deleted search on the snapshot; C_i = first k_r of the final worklist minus B.
    std::vector<std::vector<Key>> Ci(n);
    std::vector<std::vector<uint32_t>> Vi(n);  // visited sets, used by the visited-set variant only
    parallel_for(ix, n, [&](size_t i) {
      std::vector<BeamEntry> C;
      std::vector<Key> V;
      greedy_search(ix, ix.entry, ix.vec(ids[i]), ix.L, ix.vmax, false, C, V, &ix.st);
      if (approx)
        for (const auto& k : V) Vi[i].push_back(k.id);
      for (const auto& e : C) {
        if (inB[e.k.id]) continue;
        if (Ci[i].size() == ix.k_repair) break;
        Ci[i].push_back(e.k);
      }
    });
    // c members of C_i \ {x} closest to x, by (dist(x,y), y)
    auto closest_c = [&](uint32_t x, const std::vector<Key>& C) {
      std::vector<Key> t;
      for (const auto& k : C)
        if (k.id != x) t.push_back({dist_raw(ix, ix.vec(x), ix.vec(k.id)), k.id});
      ix.st.dist_evals += t.size();
      std::sort(t.begin(), t.end(), key_less);
      if (t.size() > ix.c) t.resize(ix.c);
      return t;
    };
    std::vector<std::vector<Request>> per(n);
    std::vector<std::vector<uint32_t>> touched(n);
    parallel_for(ix, n, [&](size_t i) {
      const uint32_t p = ids[i];
      if (approx) {  // Alg. 6 as printed: z in V_i where p_i in N_out(z)
        for (uint32_t z : Vi[i]) {
          if (inB[z]) continue;
          const uint32_t* zr = ix.row(z);
          if (std::find(zr, zr + ix.deg[z], p) == zr + ix.deg[z]) continue;
          touched[i].push_back(z);
          for (const auto& k : closest_c(z, Ci[i])) per[i].push_back({z, k});
        }
      } else {
        for (uint64_t e = off[p]; e < off[p + 1]; ++e) {  // in-neighbour repair: z -> y
          const uint32_t z = src[e];
          if (inB[z]) continue;
          touched[i].push_back(z);
          for (const auto& k : closest_c(z, Ci[i])) per[i].push_back({z, k});
        }
      }
      for (uint32_t s = 0; s < ix.deg[p]; ++s) {  // out-neighbour repair: y -> w
        const uint32_t w = ix.row(p)[s];
        if (inB[w] || !ix.live[w]) continue;  // (a dangling edge of p itself: nothing to reconnect)
        for (const auto& k : closest_c(w, Ci[i])) per[i].push_back({k.id, {k.d, w}});
      }
    });
    std::vector<Request> rq;
    for (uint64_t i = 0; i < n; ++i) {
      rq.insert(rq.end(), per[i].begin(), per[i].end());
      for (uint32_t z : touched[i]) rq.push_back({z, {0.0, INVALID}});  // dirty without a candidate
    }
    Grouped g = group_requests(rq, 0);
    for (auto& s : g.scratch) {  // drop the marker, then cap at P
      s.erase(std::remove_if(s.begin(), s.end(), [](const Key& k) { return k.id == INVALID; }), s.end());
      if (s.size() > ix.P) s.resize(ix.P);
    }
    parallel_for(ix, g.targets.size(), [&](size_t t) {
      rebuild_dirty(ix, g.targets[t], g.scratch[t], &inB, approx ? &ix.live : nullptr);
    });
    if (inB[ix.entry]) {  // medoid deleted: first repair candidate of the old medoid
      for (uint64_t i = 0; i < n; ++i)
        if (ids[i] == ix.entry && !Ci[i].empty()) new_entry = Ci[i][0].id;
    }
  }
  for (uint64_t i = 0; i < n; ++i) {  // remove p_i
    ix.deg[ids[i]] = 0;
    ix.live[ids[i]] = 0;
  }
  ix.nlive -= n;
  if (inB[ix.entry]) {
    ix.entry = new_entry;
    if (ix.entry == INVALID)  // no candidate: fall back to the smallest live id
      for (uint64_t v = 0; v < ix.cap; ++v)
        if (ix.live[v]) {
          ix.entry = (uint32_t)v;
          break;
        }
  }
  return OK;
}

}  // namespace

extern "C" {

int grand_oracle_create(uint32_t dim, uint32_t dtype, uint32_t metric, uint32_t R, uint32_t L, float alpha,
                        uint64_t capacity, uint32_t P, uint32_t c, uint32_t k_repair, uint32_t vmax,
                        uint32_t mode, uint32_t nthreads, float max_norm, uint32_t approx_delete, void** out) {
  if (!out || dim == 0 || R == 0 || L == 0 || dtype > 2 || metric > 1 || mode > 1 || capacity == 0) return ERR_INVALID_ARG;
  const bool augment = mode == MODE_VAMANA && metric == M_IP && max_norm > 0.0f && dtype == DT_F32;
  if (mode == MODE_VAMANA && metric == M_IP && !augment) return ERR_UNSUPPORTED;
  if (mode == MODE_FIXED && R > L) return ERR_INVALID_ARG;  // Alg. 7: the forward row is the R closest of a search result of L entries
  Index* ix = new Index();
  ix->udim = dim;
  ix->approx_delete = approx_delete != 0 && mode == MODE_VAMANA;
  ix->augment = augment;
  ix->M2 = (double)max_norm * (double)max_norm;
  if (augment) {
    dim += 1;
    metric = M_L2;
  }
  ix->dim = dim; ix->dtype = dtype; ix->metric = metric; ix->R = R; ix->L = L; ix->alpha = alpha;
  ix->A_fix = std::llround((double)alpha * 65536.0);
  ix->cap = capacity;
  ix->P = P ? P : 64;
  ix->c = c ? c : 2;
  ix->k_repair = k_repair ? k_repair : std::min<uint32_t>(50, L);
  ix->vmax = vmax ? vmax : 2 * L;
  ix->mode = mode;
  ix->nthreads = nthreads ? nthreads : 1;
  ix->esize = dtype == DT_F32 ? 4 : 1;
  ix->store.assign((size_t)capacity * dim * ix->esize, 0);
  ix->adj.assign((size_t)capacity * R, INVALID);
  ix->deg.assign(capacity, 0);
  ix->live.assign(capacity, 0);
  *out = ix;
  return OK;
}

void grand_oracle_destroy(void* h) { delete (Index*)h; }

int grand_oracle_insert_batch(void* h, const uint32_t* ids, const void* vecs, uint64_t n) {
  return insert_batch(*(Index*)h, ids, vecs, n);
}
int grand_oracle_delete_batch(void* h, const uint32_t* ids, uint64_t n) { return delete_batch(*(Index*)h, ids, n); }

// Search (Alg. 1): first k worklist entries, padded with id 0xFFFFFFFF / +inf.  Expansion cap 2*L.
int grand_oracle_search(void* h, const void* queries, uint64_t nq, uint32_t k, uint32_t L, uint32_t use_seen_set,
                        uint32_t* out_ids, double* out_dists) {
  Index& ix = *(Index*)h;
  if (k == 0 || k > L) return ERR_INVALID_ARG;
  const size_t urb = (size_t)ix.udim * ix.esize;
  parallel_for(ix, nq, [&](size_t i) {
    std::vector<BeamEntry> C;
    std::vector<Key> V;
    std::vector<uint8_t> qrow((size_t)ix.dim * ix.esize);
    const uint8_t* qsrc = (const uint8_t*)queries + i * urb;
    to_row(ix, qsrc, qrow.data(), true);
    greedy_search(ix, ix.entry, qrow.data(), L, 2 * L, use_seen_set != 0, C, V, &ix.st);
    const double qn = ix.augment ? sq_norm(ix, qsrc) : 0.0;
    for (uint32_t j = 0; j < k; ++j) {
      out_ids[i * k + j] = j < C.size() ? C[j].k.id : INVALID;
      double d = j < C.size() ? C[j].k.d : std::numeric_limits<double>::infinity();
      if (ix.augment && j < C.size()) d = (d - qn - ix.M2) * 0.5;  // back to the negated inner product
      out_dists[i * k + j] = d;
    }
  });
  return OK;
}

// One search exposing worklist and visited list (unit-level pin access).
int grand_oracle_greedy(void* h, const void* q, uint32_t L, uint32_t vmax, uint32_t use_seen_set,
                        uint32_t* beam_ids, double* beam_d, uint32_t* nbeam, uint32_t* vis_ids, double* vis_d,
                        uint32_t* nvis) {
  Index& ix = *(Index*)h;
  std::vector<BeamEntry> C;
  std::vector<Key> V;
  std::vector<uint8_t> qrow((size_t)ix.dim * ix.esize);
  to_row(ix, q, qrow.data(), true);
  greedy_search(ix, ix.entry, qrow.data(), L, vmax, use_seen_set != 0, C, V, &ix.st);
  for (size_t i = 0; i < C.size(); ++i) {
    beam_ids[i] = C[i].k.id;
    beam_d[i] = C[i].k.d;
  }
  for (size_t i = 0; i < V.size(); ++i) {
    vis_ids[i] = V[i].id;
    vis_d[i] = V[i].d;
  }
  *nbeam = (uint32_t)C.size();
  *nvis = (uint32_t)V.size();
  return OK;
}

double grand_oracle_dist(void* h, const void* a, const void* b) { return dist_raw(*(Index*)h, a, b); }

// RobustPrune on explicit candidates (ids must have vectors in the store); D given by caller.
int grand_oracle_prune(void* h, uint32_t p, const uint32_t* cand_ids, const double* cand_d, uint32_t n, uint32_t R,
                       uint32_t* out_ids, uint32_t* nout) {
  Index& ix = *(Index*)h;
  std::vector<Key> c;
  for (uint32_t i = 0; i < n; ++i) c.push_back({cand_d[i], cand_ids[i]});
  std::vector<Key> o = robust_prune(ix, p, c, R, &ix.st);
  for (size_t i = 0; i < o.size(); ++i) out_ids[i] = o[i].id;
  *nout = (uint32_t)o.size();
  return OK;
}

int grand_oracle_export_graph(void* h, uint32_t* adj, uint32_t* deg, uint32_t* live_bitmap, uint32_t* entry) {
  Index& ix = *(Index*)h;
  if (adj) std::memcpy(adj, ix.adj.data(), ix.adj.size() * 4);
  if (deg) std::memcpy(deg, ix.deg.data(), ix.deg.size() * 4);
  if (live_bitmap) {
    std::memset(live_bitmap, 0, ((ix.cap + 31) / 32) * 4);
    for (uint64_t v = 0; v < ix.cap; ++v)
      if (ix.live[v]) live_bitmap[v >> 5] |= 1u << (v & 31);
  }
  if (entry) *entry = ix.entry;
  return OK;
}

// Replace the whole state (tests build tiny graphs by hand).  vecs: capacity x dim, packed.
int grand_oracle_import_graph(void* h, const uint32_t* adj, const uint32_t* deg, const uint32_t* live_bitmap,
                              uint32_t entry, const void* vecs) {
  Index& ix = *(Index*)h;
  std::memcpy(ix.adj.data(), adj, ix.adj.size() * 4);
  std::memcpy(ix.deg.data(), deg, ix.deg.size() * 4);
  ix.nlive = 0;
  for (uint64_t v = 0; v < ix.cap; ++v) {
    ix.live[v] = (live_bitmap[v >> 5] >> (v & 31)) & 1;
    ix.nlive += ix.live[v];
  }
  ix.entry = entry;
  for (uint64_t v = 0; v < ix.cap; ++v)
    to_row(ix, (const uint8_t*)vecs + v * ix.udim * ix.esize, ix.store.data() + v * ix.dim * ix.esize, false);
  return OK;
}

// off: capacity+1 entries (uint64); src: at least *E entries (call with src == NULL to size it).
int grand_oracle_reverse_graph(void* h, uint64_t* off, uint32_t* src, uint64_t* E) {
  Index& ix = *(Index*)h;
  std::vector<uint64_t> o;
  std::vector<uint32_t> s;
  transpose(ix, o, s);
  if (off) std::memcpy(off, o.data(), o.size() * 8);
  if (src) std::memcpy(src, s.data(), s.size() * 4);
  if (E) *E = s.size();
  return OK;
}

uint32_t grand_oracle_get_entry(void* h) { return ((Index*)h)->entry; }
void grand_oracle_set_entry(void* h, uint32_t e) { ((Index*)h)->entry = e; }
uint64_t grand_oracle_live_count(void* h) { return ((Index*)h)->nlive; }

// stats: expansions, dist_evals, dead_edges_seen, prunes, dirty
void grand_oracle_get_stats(void* h, uint64_t* out5) {
  Index& ix = *(Index*)h;
  out5[0] = ix.st.expansions;
  out5[1] = ix.st.dist_evals;
  out5[2] = ix.st.dead_edges_seen;
  out5[3] = ix.st.prunes;
  out5[4] = ix.st.dirty;
}

}  // extern "C"
