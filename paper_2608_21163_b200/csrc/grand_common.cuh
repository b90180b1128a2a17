// Device-side building blocks shared by all kernels of the library: the (distance, id) key
// encoding, the per-dtype distance accumulation over 16-byte chunks, team reductions, and a
// direction-free bitonic sort that works for any length.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace grand {

constexpr uint32_t kInvalid = 0xFFFFFFFFu;
constexpr unsigned long long kKeyMax = 0xFFFFFFFFFFFFFFFFull;
constexpr unsigned long long kExpandedBit = 1ull << 31;  // worklist flag, lives in the id word
constexpr int kMetricL2 = 0, kMetricIP = 1;

// ---- key(v) = (dist, id): one 64-bit integer whose unsigned order is the lexicographic order.
__device__ __forceinline__ uint32_t order_bits(int d) { return (uint32_t)d ^ 0x80000000u; }
__device__ __forceinline__ uint32_t order_bits(float f) {
  uint32_t b = __float_as_uint(f);
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ int unorder_int(uint32_t o) { return (int)(o ^ 0x80000000u); }
__device__ __forceinline__ float unorder_float(uint32_t o) {
  uint32_t b = (o >> 31) ? (o ^ 0x80000000u) : ~o;
  return __uint_as_float(b);
}
template <typename D>
__device__ __forceinline__ unsigned long long make_key(D d, uint32_t id) {
  return ((unsigned long long)order_bits(d) << 32) | id;
}
__device__ __forceinline__ uint32_t key_id(unsigned long long k) { return (uint32_t)k & 0x7FFFFFFFu; }
__device__ __forceinline__ unsigned long long key_clean(unsigned long long k) { return k & ~kExpandedBit; }

// ---- element traits: accumulator type and the per-chunk update for each (dtype, metric).
template <typename T> struct Elem;
template <> struct Elem<uint8_t> { using Acc = int; using Dist = int; };
template <> struct Elem<int8_t> { using Acc = int; using Dist = int; };
template <> struct Elem<float> { using Acc = float; using Dist = float; };

template <typename T, int METRIC>
__device__ __forceinline__ void acc_chunk(const uint4& a, const uint4& b, typename Elem<T>::Acc& acc) {
  if constexpr (sizeof(T) == 4) {
    const float* x = reinterpret_cast<const float*>(&a);
    const float* y = reinterpret_cast<const float*>(&b);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if constexpr (METRIC == kMetricL2) {
        float t = x[j] - y[j];
        acc = fmaf(t, t, acc);
      } else {
        acc = fmaf(x[j], y[j], acc);
      }
    }
  } else {
    const uint32_t* x = reinterpret_cast<const uint32_t*>(&a);
    const uint32_t* y = reinterpret_cast<const uint32_t*>(&b);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if constexpr (METRIC == kMetricL2) {
        // |a-b| per byte fits 8 unsigned bits for both signed and unsigned inputs
        uint32_t df = (T(-1) < T(0)) ? __vabsdiffs4(x[j], y[j]) : __vabsdiffu4(x[j], y[j]);
        acc = (int)__dp4a(df, df, (uint32_t)acc);
      } else {
        if constexpr (T(-1) < T(0)) acc = __dp4a((int)x[j], (int)y[j], acc);
        else acc = (int)__dp4a(x[j], y[j], (uint32_t)acc);
      }
    }
  }
}

// Sum over the G lanes of a team (G a power of two, teams are aligned lane groups).
template <int G, typename A>
__device__ __forceinline__ A team_sum(A v) {
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

template <typename T, int METRIC>
__device__ __forceinline__ typename Elem<T>::Dist finish_dist(typename Elem<T>::Acc acc) {
  if constexpr (METRIC == kMetricL2) return acc;
  else if constexpr (sizeof(T) == 4) return __fadd_rn(-acc, 0.0f);  // no negative zero
  else return -acc;
}

// Lane t of a team owns chunks t, t+G, ... (CPL per lane) of a padded row.
template <int G, int CPL>
__device__ __forceinline__ void load_row(const uint8_t* row, uint32_t nchunk, int t, uint4 (&r)[CPL]) {
#pragma unroll
  for (int c = 0; c < CPL; ++c) {
    const uint32_t ch = t + c * G;
    r[c] = ch < nchunk ? __ldg(reinterpret_cast<const uint4*>(row) + ch) : make_uint4(0, 0, 0, 0);
  }
}

// dist between a row held in registers (a) and a row in memory, over one team; every lane of the
// team returns the full distance.  All distance evaluations of the library go through this
// function (or team_dist_regs on the same layout), so a pair of rows always yields the same bits.
template <typename T, int METRIC, int G, int CPL>
__device__ __forceinline__ typename Elem<T>::Dist team_dist_regs(const uint4 (&a)[CPL], const uint4 (&b)[CPL]) {
  typename Elem<T>::Acc acc = 0;
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc_chunk<T, METRIC>(a[c], b[c], acc);
  acc = team_sum<G>(acc);
  return finish_dist<T, METRIC>(acc);
}

// ---- tensor-core tile for integer rows: D (16 x 8, int32) += X (16 x 32 bytes, row-major) * Y^T (8 rows of 32 bytes).
// Lane l (g = l / 4, t = l % 4) holds x[0] = X[g][4t..], x[1] = X[g + 8][4t..], x[2] = X[g][16 + 4t..],
// x[3] = X[g + 8][16 + 4t..]; y[0] = Y[g][4t..], y[1] = Y[g][16 + 4t..]; d[0..1] = D[g][2t, 2t + 1],
// d[2..3] = D[g + 8][2t, 2t + 1].
template <typename T>
__device__ __forceinline__ void mma_m16n8k32(int (&d)[4], const uint32_t (&x)[4], const uint32_t (&y)[2]) {
  if constexpr (T(-1) < T(0)) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(x[0]), "r"(x[1]), "r"(x[2]), "r"(x[3]), "r"(y[0]), "r"(y[1]));
  } else {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(x[0]), "r"(x[1]), "r"(x[2]), "r"(x[3]), "r"(y[0]), "r"(y[1]));
  }
}

// ---- sorting: bitonic network with min-to-lower-index comparators only, so any length works
// (indices >= n behave as +inf and are never touched).  `sync` separates the stages.
template <typename K, typename SyncFn>
__device__ __forceinline__ void bitonic_sort_any(K* a, uint32_t n, uint32_t tid, uint32_t nthreads, SyncFn sync) {
  if (n < 2) return;
  uint32_t m = 1;
  while (m < n) m <<= 1;
  for (uint32_t k = 2; k <= m; k <<= 1) {
    for (uint32_t i = tid; i < n; i += nthreads) {
      uint32_t p = i ^ (k - 1);
      if (p > i && p < n) {
        K x = a[i], y = a[p];
        if (y < x) { a[i] = y; a[p] = x; }
      }
    }
    sync();
    for (uint32_t j = k >> 2; j > 0; j >>= 1) {
      for (uint32_t i = tid; i < n; i += nthreads) {
        uint32_t p = i ^ j;
        if (p > i && p < n) {
          K x = a[i], y = a[p];
          if (y < x) { a[i] = y; a[p] = x; }
        }
      }
      sync();
    }
  }
}

// the same network ordering 64-bit keys by their clean value (bit 31 of the id word rides along as a tag)
template <typename SyncFn>
__device__ __forceinline__ void bitonic_sort_clean(unsigned long long* a, uint32_t n, uint32_t tid, uint32_t nthreads, SyncFn sync) {
  if (n < 2) return;
  uint32_t m = 1;
  while (m < n) m <<= 1;
  for (uint32_t k = 2; k <= m; k <<= 1) {
    for (uint32_t i = tid; i < n; i += nthreads) {
      uint32_t p = i ^ (k - 1);
      if (p > i && p < n) {
        unsigned long long x = a[i], y = a[p];
        if (key_clean(y) < key_clean(x)) { a[i] = y; a[p] = x; }
      }
    }
    sync();
    for (uint32_t j = k >> 2; j > 0; j >>= 1) {
      for (uint32_t i = tid; i < n; i += nthreads) {
        uint32_t p = i ^ j;
        if (p > i && p < n) {
          unsigned long long x = a[i], y = a[p];
          if (key_clean(y) < key_clean(x)) { a[i] = y; a[p] = x; }
        }
      }
      sync();
    }
  }
}

// first index in sorted a[0..n) whose clean key is >= k
__device__ __forceinline__ uint32_t lower_bound_clean(const unsigned long long* a, uint32_t n, unsigned long long k) {
  uint32_t lo = 0, hi = n;
  while (lo < hi) {
    uint32_t mid = (lo + hi) >> 1;
    if (key_clean(a[mid]) < k) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Smallest 64-bit key over the warp (all lanes call this): two 32-bit min reductions, high word first.
__device__ __forceinline__ unsigned long long warp_min_key(unsigned long long k) {
  const uint32_t hi = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(k >> 32));
  const uint32_t lo = __reduce_min_sync(0xFFFFFFFFu, (uint32_t)(k >> 32) == hi ? (uint32_t)k : 0xFFFFFFFFu);
  return ((unsigned long long)hi << 32) | lo;
}

// Append `value` to list[*counter ...] for every lane with `need`: one atomic per warp instead of one
// per lane (all 32 lanes must call this together).  Counters hit by every dirty node or request would
// otherwise serialise on a single address.
__device__ __forceinline__ void warp_append(uint32_t* list, uint32_t* counter, bool need, uint32_t value) {
  const unsigned bal = __ballot_sync(0xFFFFFFFFu, need);
  if (!bal) return;
  const int lane = threadIdx.x & 31, leader = __ffs(bal) - 1;
  uint32_t base = 0;
  if (lane == leader) base = atomicAdd(counter, (uint32_t)__popc(bal));
  base = __shfl_sync(0xFFFFFFFFu, base, leader);
  if (need) list[base + __popc(bal & ((1u << lane) - 1u))] = value;
}

__device__ __forceinline__ bool bit_test(const uint32_t* bm, uint32_t v) { return (bm[v >> 5] >> (v & 31)) & 1u; }

// alpha test of RobustPrune (Alg. 4): alpha * dist(p*,p') <= D_p[p'].
// Integer vectors: fixed point A = round(alpha * 65536).  fp32: one correctly rounded multiply.
struct AlphaParam {
  long long A_fix;
  float alpha;
};
__device__ __forceinline__ bool alpha_test(const AlphaParam& ap, int d_star, int d_p) {
  return ap.A_fix * (long long)d_star <= ((long long)d_p) * 65536ll;
}
__device__ __forceinline__ bool alpha_test(const AlphaParam& ap, float d_star, float d_p) {
  return __fmul_rn(ap.alpha, d_star) <= d_p;
}

template <typename D> __device__ __forceinline__ D key_dist(unsigned long long k);
template <> __device__ __forceinline__ int key_dist<int>(unsigned long long k) { return unorder_int((uint32_t)(k >> 32)); }
template <> __device__ __forceinline__ float key_dist<float>(unsigned long long k) { return unorder_float((uint32_t)(k >> 32)); }

}  // namespace grand
