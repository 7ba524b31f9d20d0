// Device-side building blocks of the lossy data-parallel step (sm_100a).
//
// Work decomposition shared by every kernel here: the bucket is walked in
// "chunks" of 256 contiguous elements (one warp, 8 elements = 16 or 32 bytes per
// lane) that never straddle a packet, so the delivery masks of a chunk are
// warp-uniform. Chunk q belongs to packet k = q / chunks_per_packet. Warps take
// chunks grid-stride, so at any moment the grid streams one contiguous window
// of every buffer.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lossy {

constexpr int kMaxW = 64;
#ifndef LOSSY_THREADS
#define LOSSY_THREADS 256
#endif
#ifndef LOSSY_MIN_BLOCKS
#define LOSSY_MIN_BLOCKS 1
#endif
constexpr int kThreads = LOSSY_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kChunk = 256;  // elements per warp-chunk

enum Phase : int { AGG = 1, STEP = 2, BCAST = 4, DRIFT = 8 };
// bits of Params::flags that the kernels look at (the values of the public flags of the same meaning)
constexpr uint32_t kSelfLossless = 1u, kZeroSkip = 2u, kSkipOwner = 8u;

struct Params {
  const void* grads[kMaxW];
  void* replicas[kMaxW];
  float* master;
  float* m;
  float* v;
  float* ghat;            // AGG: optional output; STEP without AGG: input
  float* ghat_prev;       // non-NULL: Algorithm 1's gradient half (last surviving aggregate, in/out)
  uint8_t* count;         // optional output (AGG)
  uint64_t* recv_bits;    // optional output (AGG)
  uint64_t* stale_bits;   // optional output (BCAST)
  const uint8_t* count_in;  // STEP without AGG and ZERO_SKIP: received counts
  double* partials;       // DRIFT: [gridDim.x][kMaxW] per-block squared sums
  // Drift finalisation inside the last block to finish (no second launch): `ticket` counts finished blocks
  // over all launches of one call; NULL = a separate finalize kernel follows.
  uint32_t* ticket;
  uint32_t total_rows;    // partial rows (= blocks) of the whole call
  float* norms;           // [W] or NULL
  double* sumsq;          // [W], added to, or NULL
  const uint64_t* reliable;  // [2][K] (row 0 gradient links, row 1 broadcast links): set bits are never lost; or NULL
  const uint64_t* burst_in;  // bursty loss: link states after the previous step, [2][K] (row 0 gradient links, row 1 broadcast links)
  uint64_t* burst_out;       // link states after this step, same layout (a different buffer)
  uint64_t n;
  uint64_t packet_base;
  uint64_t step_key;      // hash key of (seed, step), derived on the host
  uint32_t num_chunks;    // K * chunks_per_packet
  uint32_t chunk_begin;   // first chunk this launch covers (a bulk-copy launch may own the chunks before it)
  uint32_t partials_row0; // first row of `partials` this launch writes
  uint32_t chunks_per_packet;
  uint32_t pps;           // packets per shard (of the whole bucket)
  uint32_t k0;            // bucket packet index of this context's packet 0 (a context may cover a packet range)
  uint32_t P;
  uint32_t W;
  uint32_t Tg, Tp;        // drop iff hash < T
  uint32_t Tenter, Tstay; // bursty loss: a good link turns bad iff hash < Tenter, a bad one stays bad iff hash < Tstay
  uint32_t K;             // packets in the bucket
  uint32_t flags;
  uint32_t prefetch_next; // register kernel: L2-prefetch the warp's next chunk
  float lr, b1, b2, omb1, omb2, ibc1, ibc2, eps;
  // Owner-elided replicas (kSkipOwner): replica i stores this context's elements WITHOUT the packets worker i
  // owns, so everything behind worker i's shard sits rep_skip[i] elements lower in its array. All zero otherwise.
  uint64_t rep_skip[kMaxW];
  // Debug build (LOSSY_DEVCHECK): where a failed index check is recorded (4 words: site, element offset low and
  // high, length; the first failure wins) and the element count the checks hold a range against (n, or less when
  // the self-test shrinks it). Unused otherwise.
  uint32_t* check;
  uint64_t check_n;
};

// Owner-elided replicas: rep_skip[i] = elements of worker i's shard inside the context's packet range
// [k0, k0 + K) of a bucket cut into shards of pps packets (the last packet may be short: n elements in all).
__host__ inline void fill_rep_skip(Params& P, bool elide) {
  for (uint32_t i = 0; i < (uint32_t)kMaxW; ++i) P.rep_skip[i] = 0;
  if (!elide) return;
  for (uint32_t i = 0; i < P.W; ++i) {
    const uint64_t s0 = (uint64_t)i * P.pps, s1 = s0 + P.pps;          // shard i in bucket packets
    const uint64_t c0 = P.k0, c1 = (uint64_t)P.k0 + P.K;                // this context in bucket packets
    const uint64_t lo = s0 > c0 ? s0 : c0, hi = s1 < c1 ? s1 : c1;
    if (lo >= hi) continue;
    const uint64_t e0 = (lo - c0) * P.P, e1 = (hi - c0) * P.P;
    P.rep_skip[i] = (e1 < P.n ? e1 : P.n) - (e0 < P.n ? e0 : P.n);
  }
}
// Index of bucket element e, which lies in a packet owned by worker j, inside replica i's array (i != j when
// the replicas are owner-elided; with full replicas every rep_skip is 0 and the index is e).
__device__ __forceinline__ uint64_t rep_index(const Params& P, uint32_t i, uint32_t j, uint64_t e) {
  return e - (j > i ? P.rep_skip[i] : 0ull);
}
// Debug build (compiled with -DLOSSY_DEVCHECK, a library of its own): before a kernel of the step path touches
// memory for a chunk or tile it checks the element range and the packet index against the context's sizes, and
// every replica's range (through the owner-elided index map) against that replica's length. A range that fails
// is recorded in Params::check and not touched: the register kernel skips the chunk, a pipeline raises its abort
// flag and every role leaves through the bounded-wait exit. Nothing traps or asserts. In the normal build all of
// this compiles to nothing.
#ifdef LOSSY_DEVCHECK
constexpr bool kDevCheck = true;
#else
constexpr bool kDevCheck = false;
#endif
enum CheckSite : uint32_t { kSiteRegister = 1, kSiteFusedPacked = 2, kSiteFused = 3, kSitePhase = 4, kSiteGather = 5, kSiteReplica = 16 };
__device__ __forceinline__ void check_record(const Params& P, uint32_t site, uint64_t e0, uint64_t len) {
  if (atomicCAS(&P.check[0], 0u, site) == 0u) {
    P.check[1] = (uint32_t)e0;
    P.check[2] = (uint32_t)(e0 >> 32);
    P.check[3] = (uint32_t)len;
  }
}
// elements [e0, e0 + len) of packet k: inside the slab, and k a packet of it
__device__ __forceinline__ bool span_ok(const Params& P, uint32_t k, uint64_t e0, uint64_t len, uint32_t site) {
  if constexpr (!kDevCheck) return true;
  if (!P.check) return true;      // a caller without a context (the no-allocation entry point) has nowhere to record
  if (k < P.K && (len == 0 || (len <= P.check_n && e0 <= P.check_n - len))) return true;   // an empty range touches nothing
  check_record(P, site, e0, len);
  return false;
}
// the same elements inside replica i's array (owner j; the owner has no copy when the replicas are owner-elided)
__device__ __forceinline__ bool rep_span_ok(const Params& P, uint32_t i, uint32_t j, uint64_t e0, uint64_t len, uint32_t site) {
  if constexpr (!kDevCheck) return true;
  if (!P.check || len == 0 || ((P.flags & kSkipOwner) && i == j)) return true;
  const uint64_t limit = P.check_n - (P.rep_skip[i] < P.check_n ? P.rep_skip[i] : P.check_n);
  const uint64_t at = e0 - (j > i ? P.rep_skip[i] : 0ull);
  if (at <= e0 && len <= limit && at <= limit - len) return true;
  check_record(P, site | kSiteReplica, at, len);
  return false;
}
// every replica's range of a tile or chunk, the workers dealt over the lanes; warp-uniform result
__device__ __forceinline__ bool tile_ok(const Params& P, uint32_t k, uint32_t j, uint64_t e0, uint64_t len, uint32_t site, int lane) {
  if constexpr (!kDevCheck) return true;
  bool ok = span_ok(P, k, e0, len, site);
  for (uint32_t i = (uint32_t)lane; i < P.W; i += 32u) ok = rep_span_ok(P, i, j, e0, len, site) && ok;
  return __all_sync(0xFFFFFFFFu, ok);
}

// The replica that does not exist for a packet of owner j (as a bit), or 0 with full replicas.
__device__ __forceinline__ uint64_t own_bit(const Params& P, uint32_t j) {
  return (P.flags & kSkipOwner) ? 1ull << j : 0ull;
}

// ---- delivery-indicator hash (Section 3: s, r ~ Bernoulli(1-p)) -------------
// 64-bit finalizer of the splitmix64 generator; the constants of the keyed
// rounds are this library's own choice and are part of its documented contract.
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
  z ^= z >> 27; z *= 0x94D049BB133111EBULL;
  z ^= z >> 31;
  return z;
}
__host__ __device__ __forceinline__ uint64_t step_key_of(uint64_t seed, uint64_t step) {
  return mix64(mix64(seed ^ 0x6A09E667F3BCC908ULL) + step * 0x9E3779B97F4A7C15ULL);
}
__host__ __device__ __forceinline__ uint64_t packet_key_of(uint64_t step_key, uint64_t packet) {
  return mix64(step_key ^ (packet * 0xD6E8FEB86659FD93ULL));
}
__host__ __device__ __forceinline__ uint32_t pair_hash(uint64_t packet_key, uint32_t src, uint32_t dst) {
  const uint64_t pair = ((uint64_t)src << 32) | (uint64_t)dst;
  return (uint32_t)(mix64(packet_key + pair * 0xC2B2AE3D27D4EB4FULL) >> 32);
}

// ---- streaming 128-bit memory operations ------------------------------------
// Everything on this path is touched exactly once per step, so loads and stores
// carry the evict-first ("streaming") cache operator.
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ void st_stream(void* p, uint4 v) {
  __stcs(reinterpret_cast<uint4*>(p), v);
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// ---- element-type adapters ----------------------------------------------------
struct F32 { using raw = float; static constexpr int kVecs = 2; };       // 8 elements = 2 x 16 B
struct BF16 { using raw = uint16_t; static constexpr int kVecs = 1; };   // 8 elements = 1 x 16 B

template <class T> struct Vec8 { uint4 q[T::kVecs]; };

template <class T>
__device__ __forceinline__ Vec8<T> load8(const void* base, uint64_t e) {
  Vec8<T> r;
  const typename T::raw* p = reinterpret_cast<const typename T::raw*>(base) + e;
#pragma unroll
  for (int i = 0; i < T::kVecs; ++i) r.q[i] = ld_stream(reinterpret_cast<const uint4*>(p) + i);
  return r;
}
// Ragged tail of the bucket: the last vector may hold fewer than 8 elements.
template <class T>
__device__ __forceinline__ Vec8<T> load8_tail(const void* base, uint64_t e, int nvalid) {
  Vec8<T> r;
  typename T::raw tmp[8];
  const typename T::raw* p = reinterpret_cast<const typename T::raw*>(base) + e;
#pragma unroll
  for (int i = 0; i < 8; ++i) tmp[i] = i < nvalid ? p[i] : (typename T::raw)0;
  if constexpr (T::kVecs == 2) {
    r.q[0] = make_uint4(__float_as_uint(tmp[0]), __float_as_uint(tmp[1]), __float_as_uint(tmp[2]), __float_as_uint(tmp[3]));
    r.q[1] = make_uint4(__float_as_uint(tmp[4]), __float_as_uint(tmp[5]), __float_as_uint(tmp[6]), __float_as_uint(tmp[7]));
  } else {
    r.q[0] = make_uint4((uint32_t)tmp[0] | ((uint32_t)tmp[1] << 16), (uint32_t)tmp[2] | ((uint32_t)tmp[3] << 16),
                        (uint32_t)tmp[4] | ((uint32_t)tmp[5] << 16), (uint32_t)tmp[6] | ((uint32_t)tmp[7] << 16));
  }
  return r;
}
template <class T>
__device__ __forceinline__ void store8(void* base, uint64_t e, const Vec8<T>& v, int nvalid) {
  typename T::raw* p = reinterpret_cast<typename T::raw*>(base) + e;
  if (nvalid == 8) {
#pragma unroll
    for (int i = 0; i < T::kVecs; ++i) st_stream(reinterpret_cast<uint4*>(p) + i, v.q[i]);
  } else {
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&v.q[0]);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i < nvalid) {
        if constexpr (T::kVecs == 2) p[i] = __uint_as_float(w[i]);
        else p[i] = (uint16_t)(w[i >> 1] >> ((i & 1) * 16));
      }
    }
  }
}
template <class T>
__device__ __forceinline__ Vec8<T> load8_any(const void* base, uint64_t e, int nvalid) {
  return nvalid == 8 ? load8<T>(base, e) : load8_tail<T>(base, e, nvalid);
}

// widen 8 elements to fp32 (bf16 -> fp32 is a 16-bit shift, exact)
template <class T>
__device__ __forceinline__ void widen(const Vec8<T>& v, float (&f)[8]) {
  const uint32_t* w = reinterpret_cast<const uint32_t*>(&v.q[0]);
  if constexpr (T::kVecs == 2) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(w[i]);
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
}
// narrow 8 fp32 values to the wire type (bf16: IEEE round-to-nearest-even)
template <class T>
__device__ __forceinline__ Vec8<T> narrow(const float (&f)[8]) {
  Vec8<T> r;
  uint32_t* w = reinterpret_cast<uint32_t*>(&r.q[0]);
  if constexpr (T::kVecs == 2) {
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = __float_as_uint(f[i]);
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
  }
  return r;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = __fadd_rn(x, __shfl_xor_sync(0xFFFFFFFFu, x, o));
  return x;
}

// Warp totals of N (4 or 8) per-lane values at once. Each exchange (lane distance 16, 8, ...) halves the
// values a lane carries: the lanes whose bit is set keep the upper half and hand over the lower half. The
// one value left is then summed over the remaining lane bits, so every lane ends with the warp total of
// value number lane / (32 / N), in N + 1 (N = 8) or N + 2 (N = 4) shuffles instead of 5 N.
template <int N>
__device__ __forceinline__ float warp_sum_multi(float (&v)[N], int lane) {
  static_assert(N == 4 || N == 8, "4 or 8 values");
  constexpr unsigned kFull = 0xFFFFFFFFu;
  int o = 16;
#pragma unroll
  for (int h = N / 2; h >= 1; h >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int x = 0; x < h; ++x) {
      const float keep = up ? v[x + h] : v[x];
      const float give = up ? v[x] : v[x + h];
      v[x] = __fadd_rn(keep, __shfl_xor_sync(kFull, give, o));
    }
    o >>= 1;
  }
#pragma unroll
  for (int r = 32 / N / 2; r >= 1; r >>= 1) v[0] = __fadd_rn(v[0], __shfl_xor_sync(kFull, v[0], r));
  return v[0];
}

}  // namespace lossy
