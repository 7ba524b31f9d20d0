// The kernels of the lossy data-parallel step: one template, specialised by the
// phases it runs. Fused = AGG|STEP|BCAST|DRIFT in a single pass over the bucket.
#pragma once
#include "lossy_device.cuh"

namespace lossy {

// acc / count as the IEEE fp32 quotient. A power-of-two count is an exact scaling, so the multiplication by
// its reciprocal gives the same correctly rounded value as the division (also in the subnormal range) at a
// tenth of the instructions; count 0 leaves the zeros in place.
template <int N>
__device__ __forceinline__ void divide_by_count(float (&a)[N], uint32_t cnt) {
  if (cnt <= 1) return;
  if ((cnt & (cnt - 1)) == 0) {
    const float inv = __uint_as_float((127u - (uint32_t)(__ffs(cnt) - 1)) << 23);   // 2^-log2(cnt)
#pragma unroll
    for (int x = 0; x < N; ++x) a[x] = __fmul_rn(a[x], inv);
  } else {
    const float fc = (float)cnt;
#pragma unroll
    for (int x = 0; x < N; ++x) a[x] = __fdiv_rn(a[x], fc);
  }
}

// One optimizer update of N elements, every operation rounded on its own
// (Section 3 step (3); Adam as bias-corrected Kingma-Ba with host-side corrections).
template <int OPT, int N>
__device__ __forceinline__ void optimizer_n(const Params& P, const float (&g)[N], float (&th)[N], float (&m)[N],
                                            float (&v)[N]) {
#pragma unroll
  for (int x = 0; x < N; ++x) {
    if constexpr (OPT == 0) {
      th[x] = __fsub_rn(th[x], __fmul_rn(P.lr, g[x]));
    } else {
      const float mn = __fadd_rn(__fmul_rn(P.b1, m[x]), __fmul_rn(P.omb1, g[x]));
      const float vn = __fadd_rn(__fmul_rn(P.b2, v[x]), __fmul_rn(__fmul_rn(P.omb2, g[x]), g[x]));
      const float mh = __fmul_rn(mn, P.ibc1);
      const float vh = __fmul_rn(vn, P.ibc2);
      const float den = __fadd_rn(__fsqrt_rn(vh), P.eps);
      th[x] = __fsub_rn(th[x], __fdiv_rn(__fmul_rn(P.lr, mh), den));
      m[x] = mn;
      v[x] = vn;
    }
  }
}
template <int OPT>
__device__ __forceinline__ void optimizer8(const Params& P, const float (&g)[8], float (&th)[8], float (&m)[8],
                                           float (&v)[8]) {
  optimizer_n<OPT, 8>(P, g, th, m, v);
}

// Last-block drift finalisation. Every block has stored its row of `partials`; the block that draws the
// last ticket sums the rows of each replica in a fixed order (lane l takes rows l, l+32, ..., then a shuffle
// tree), so the result does not depend on which block happens to be last. Nothing here waits on another
// block. Call with all threads of the block; `nwarps` warps share the replicas.
__device__ __forceinline__ void drift_last_block(const Params& P, int warp, int lane, int nwarps) {
  __shared__ uint32_t is_last;
  __threadfence();                       // this block's partial row is visible device-wide ...
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t prev = atomicAdd(P.ticket, 1u);   // ... before its ticket is
    is_last = prev + 1u == P.total_rows ? 1u : 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (uint32_t i = warp; i < P.W; i += nwarps) {
    double t = 0.0;
    for (uint32_t b = lane; b < P.total_rows; b += 32) t += __ldcg(&P.partials[(size_t)b * kMaxW + i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    if (lane == 0) {
      if (P.sumsq) P.sumsq[i] += t;
      if (P.norms) P.norms[i] = (float)sqrt(t);
    }
  }
  if (threadIdx.x == 0) *P.ticket = 0u;  // ready for the next call on this context
}

// Delivery indicators of packet k (owner j), evaluated one worker per lane and gathered by ballot:
// recv bit i = gradient piece of worker i reached the owner; stale bit i = replica i missed the broadcast.
// Independent loss: one threshold compare per link. Bursty loss (P.burst_in set): each link is a two-state
// chain on the same hash value, bad_t = bad_{t-1} ? (u < Tstay) : (u < Tenter), lost iff bad; the new states
// come back in gbad / pbad for the one caller that stores them.
template <int PH>
__device__ __forceinline__ void packet_masks(const Params& P, uint32_t k, uint32_t j, int lane, uint64_t& recv,
                                             uint64_t& stale, uint64_t& gbad, uint64_t& pbad) {
  const uint32_t W = P.W;
  const uint64_t pkey = packet_key_of(P.step_key, P.packet_base + k);
  const uint32_t i0 = lane, i1 = lane + 32;
  const bool bursty = P.burst_in != nullptr;
  gbad = 0;
  pbad = 0;
  if constexpr (PH & AGG) {
    // Algorithm 1's gradient half: the reduce is reliable and ONE draw (the owner's own link of the
    // hash) keeps or drops the packet's whole aggregate; otherwise one draw per contributing worker.
    const bool alg1 = P.ghat_prev != nullptr;
    const uint32_t src0 = alg1 ? j : i0, src1 = alg1 ? j : i1;
    const uint64_t gin = bursty ? P.burst_in[k] : 0ull;
    const uint32_t u0 = pair_hash(pkey, src0, j);
    const bool was0 = (gin >> (alg1 ? 0u : i0)) & 1ull;
    bool lost0 = bursty ? (was0 ? u0 < P.Tstay : u0 < P.Tenter) : u0 < P.Tg;
    if (!alg1 && (P.flags & 1u) && i0 == j) lost0 = false;
    uint32_t lo = __ballot_sync(0xFFFFFFFFu, i0 < W && !lost0), hi = 0;
    uint32_t blo = __ballot_sync(0xFFFFFFFFu, i0 < W && lost0), bhi = 0;
    if (W > 32) {
      const uint32_t u1 = pair_hash(pkey, src1, j);
      const bool was1 = (gin >> (alg1 ? 0u : i1)) & 1ull;
      bool lost1 = bursty ? (was1 ? u1 < P.Tstay : u1 < P.Tenter) : u1 < P.Tg;
      if (!alg1 && (P.flags & 1u) && i1 == j) lost1 = false;
      hi = __ballot_sync(0xFFFFFFFFu, i1 < W && !lost1);
      bhi = __ballot_sync(0xFFFFFFFFu, i1 < W && lost1);
    }
    recv = ((uint64_t)hi << 32) | lo;
    gbad = alg1 ? (uint64_t)(blo & 1u) : (((uint64_t)bhi << 32) | blo);
    if (P.reliable) {   // transmissions on the reliable channel always arrive
      const uint64_t all = W == 64 ? ~0ull : ((1ull << W) - 1ull);
      const uint64_t rel = P.reliable[k];
      if (alg1) { if (rel & 1ull) recv = all; }
      else recv |= rel & all;
    }
  }
  if constexpr (PH & BCAST) {
    const uint64_t pin = bursty ? P.burst_in[(size_t)P.K + k] : 0ull;
    const uint32_t u0 = pair_hash(pkey, j, i0);
    const bool was0 = (pin >> i0) & 1ull;
    const bool d0 = i0 < W && i0 != j && (bursty ? (was0 ? u0 < P.Tstay : u0 < P.Tenter) : u0 < P.Tp);
    uint32_t lo = __ballot_sync(0xFFFFFFFFu, d0), hi = 0;
    if (W > 32) {
      const uint32_t u1 = pair_hash(pkey, j, i1);
      const bool was1 = (pin >> i1) & 1ull;
      const bool d1 = i1 < W && i1 != j && (bursty ? (was1 ? u1 < P.Tstay : u1 < P.Tenter) : u1 < P.Tp);
      hi = __ballot_sync(0xFFFFFFFFu, d1);
    }
    stale = ((uint64_t)hi << 32) | lo;
    pbad = stale;
    if (P.reliable) stale &= ~P.reliable[(size_t)P.K + k];
  }
}
template <int PH>
__device__ __forceinline__ void packet_masks(const Params& P, uint32_t k, uint32_t j, int lane, uint64_t& recv,
                                             uint64_t& stale) {
  uint64_t gbad, pbad;
  packet_masks<PH>(P, k, j, lane, recv, stale, gbad, pbad);
}

// The same draws for several packets per ballot (W <= 32, not Algorithm 1's aggregate): the warp's lanes
// are split into 32 / Wp segments of Wp lanes (Wp = W rounded up to a power of two); a lane evaluates
// link `i` of the packet `k` (owner `j`) of its segment. One warp evaluating one packet at a time is a
// chain of dependent instructions (the hash) that bounds a producer warp when tiles carry few bytes.
struct BatchDraws {
  uint32_t recv_ok;     // bit = gradient piece delivered
  uint32_t grad_lost;   // bit = gradient link in its lossy state (before the reliable channel)
  uint32_t bcast_lost;  // bit = replica missed the broadcast (before the reliable channel)
};
template <int PH>
__device__ __forceinline__ BatchDraws batch_draws(const Params& P, uint32_t k, uint32_t j, uint32_t i, bool valid) {
  const uint64_t pkey = packet_key_of(P.step_key, P.packet_base + k);
  const bool bursty = P.burst_in != nullptr;
  BatchDraws d = {0u, 0u, 0u};
  if constexpr (PH & AGG) {
    const bool was = bursty && ((P.burst_in[k] >> i) & 1ull);
    const uint32_t u = pair_hash(pkey, i, j);
    bool lost = bursty ? (was ? u < P.Tstay : u < P.Tenter) : u < P.Tg;
    if ((P.flags & 1u) && i == j) lost = false;
    d.recv_ok = __ballot_sync(0xFFFFFFFFu, valid && !lost);
    d.grad_lost = __ballot_sync(0xFFFFFFFFu, valid && lost);
  }
  if constexpr (PH & BCAST) {
    const bool was = bursty && ((P.burst_in[(size_t)P.K + k] >> i) & 1ull);
    const uint32_t u = pair_hash(pkey, j, i);
    const bool lost = i != j && (bursty ? (was ? u < P.Tstay : u < P.Tenter) : u < P.Tp);
    d.bcast_lost = __ballot_sync(0xFFFFFFFFu, valid && lost);
  }
  return d;
}
// masks of the packet `k` whose segment starts at lane `src` (segment mask `wmask`), as packet_masks returns them
template <int PH>
__device__ __forceinline__ void batch_masks(const Params& P, const BatchDraws& d, uint32_t k, int src, uint32_t wmask,
                                            uint64_t& recv, uint64_t& stale, uint64_t& gbad, uint64_t& pbad) {
  recv = stale = gbad = pbad = 0;
  if constexpr (PH & AGG) {
    recv = (d.recv_ok >> src) & wmask;
    gbad = (d.grad_lost >> src) & wmask;
    if (P.reliable) recv |= P.reliable[k] & ((1ull << P.W) - 1ull);   // W <= 32 here
  }
  if constexpr (PH & BCAST) {
    stale = (d.bcast_lost >> src) & wmask;
    pbad = stale;
    if (P.reliable) stale &= ~P.reliable[(size_t)P.K + k];
  }
}

// ELIDE = owner-elided replicas: a build of its own, so that the index arithmetic of that layout costs the
// default layout nothing (this kernel is bound by its issue slots, not by memory).
template <int PH, class GT, class RT, int OPT, bool ELIDE = false>
__global__ void __launch_bounds__(kThreads, LOSSY_MIN_BLOCKS) lossy_kernel(const __grid_constant__ Params P) {
  auto rep_at = [&](uint32_t i, uint32_t j, uint64_t e) { return ELIDE ? rep_index(P, i, j, e) : e; };
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t W = P.W;

  // per-lane drift accumulators: lane l holds replicas l and l + 32
  double dacc0 = 0.0, dacc1 = 0.0;

  const uint32_t warps_in_grid = gridDim.x * kWarps;
  for (uint32_t q = P.chunk_begin + blockIdx.x * kWarps + warp; q < P.num_chunks; q += warps_in_grid) {
    const uint32_t k = q / P.chunks_per_packet;
    const uint32_t c = q - k * P.chunks_per_packet;
    const uint32_t j = (P.k0 + k) / P.pps;  // owner W_j of packet k
    const uint32_t in_pkt = c * kChunk + lane * 8;
    const uint64_t e = (uint64_t)k * P.P + in_pkt;
    int nvalid = 0;
    if (in_pkt < P.P && e < P.n) nvalid = (P.n - e >= 8) ? 8 : (int)(P.n - e);
    if constexpr (kDevCheck) {   // debug build: the chunk's range, in the slab and in every replica
      const uint64_t c0 = (uint64_t)k * P.P + (uint64_t)c * kChunk;
      const uint64_t in_packet = P.P - c * kChunk < (uint32_t)kChunk ? P.P - c * kChunk : (uint32_t)kChunk;   // a chunk ends with its packet
      const uint64_t cl = c0 < P.n ? (P.n - c0 < in_packet ? P.n - c0 : in_packet) : 0;
      if (!tile_ok(P, k, j, c0, cl, kSiteRegister, lane)) continue;
    }

    // ---- delivery indicators of this packet (warp-uniform) -------------------
    uint64_t recv = 0, stale = 0, gbad = 0, pbad = 0;
    packet_masks<PH>(P, k, j, lane, recv, stale, gbad, pbad);
    // Pull the NEXT chunk of this warp toward L2 while this one is processed. Worth its
    // instructions only in the fused kernel when few workers feed a chunk (measured: +3..13 % for W <= 8,
    // a loss above, and a loss in the single-phase kernels).
    if (P.prefetch_next) {
      const uint32_t qn = q + warps_in_grid;
      if (qn < P.num_chunks) {
        const uint32_t kn = qn / P.chunks_per_packet;
        const uint32_t cn = qn - kn * P.chunks_per_packet;
        const uint32_t inn = cn * kChunk + lane * 8;
        const uint64_t en = (uint64_t)kn * P.P + inn;
        uint64_t rn = 0, sn = 0;
        packet_masks<PH>(P, kn, (P.k0 + kn) / P.pps, lane, rn, sn);
        if (inn < P.P && en + 8 <= P.n) {
          if constexpr (PH & (STEP | BCAST | DRIFT)) prefetch_l2(P.master + en);
          if constexpr ((PH & STEP) && OPT == 1) { prefetch_l2(P.m + en); prefetch_l2(P.v + en); }
          if constexpr (PH & AGG) {
            while (rn) {
              const int i = __ffsll((long long)rn) - 1;
              rn &= rn - 1;
              prefetch_l2(reinterpret_cast<const typename GT::raw*>(P.grads[i]) + en);
            }
          }
          if constexpr ((PH & BCAST) && (PH & DRIFT)) {
            while (sn) {
              const int i = __ffsll((long long)sn) - 1;
              sn &= sn - 1;
              prefetch_l2(reinterpret_cast<const typename RT::raw*>(P.replicas[i]) + rep_at(i, (P.k0 + kn) / P.pps, en));
            }
          }
        }
      }
    }
    uint32_t cnt = __popcll(recv);
    if (c == 0 && lane == 0) {
      if constexpr (PH & AGG) {
        if (P.count) P.count[k] = (uint8_t)cnt;
        if (P.recv_bits) P.recv_bits[k] = recv;
      }
      if constexpr (PH & BCAST) {
        if (P.stale_bits) P.stale_bits[k] = stale;
      }
      if (P.burst_out) {   // the first chunk of a packet stores its links' new states
        if constexpr (PH & AGG) P.burst_out[k] = gbad;
        if constexpr (PH & BCAST) P.burst_out[(size_t)P.K + k] = pbad;
      }
    }
    // Lanes past a short packet or past the bucket end keep nvalid == 0: they stay in the
    // warp for the shuffles below and every load/store helper skips them.

    // stale copies are read late (for the drift term): start them toward L2 now
    if constexpr ((PH & BCAST) && (PH & DRIFT)) {
      uint64_t sm = nvalid > 0 ? stale : 0ull;
      while (sm) {
        const int i = __ffsll((long long)sm) - 1;
        sm &= sm - 1;
        prefetch_l2(reinterpret_cast<const typename RT::raw*>(P.replicas[i]) + rep_at(i, j, e));
      }
    }

    // ---- optimizer state: issue these loads before the gradient loop ---------
    Vec8<F32> rth, rm, rv;
    if constexpr (PH & (STEP | BCAST | DRIFT)) rth = load8_any<F32>(P.master, e, nvalid);
    if constexpr ((PH & STEP) && OPT == 1) {
      rm = load8_any<F32>(P.m, e, nvalid);
      rv = load8_any<F32>(P.v, e, nvalid);
    }

    // ---- (2) unbiased aggregate: masked sum in ascending worker order / count --
    float g[8];
    if constexpr (PH & AGG) {
#pragma unroll
      for (int x = 0; x < 8; ++x) g[x] = 0.0f;
      for (uint32_t g0 = 0; g0 < W; g0 += 8) {
        const uint32_t bits = (uint32_t)(recv >> g0) & 0xFFu;
        if (bits == 0) continue;
        Vec8<GT> raw[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if ((bits >> u) & 1u) raw[u] = load8_any<GT>(P.grads[g0 + u], e, nvalid);
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if ((bits >> u) & 1u) {
            float f[8];
            widen<GT>(raw[u], f);
#pragma unroll
            for (int x = 0; x < 8; ++x) g[x] = __fadd_rn(g[x], f[x]);
          }
      }
      divide_by_count<8>(g, cnt);
      if (P.ghat_prev) {
        // Algorithm 1: a dropped packet falls back to the saved aggregate, a surviving one is saved
        if (cnt == 0) {
          const Vec8<F32> pv = load8_any<F32>(P.ghat_prev, e, nvalid);
          widen<F32>(pv, g);
        } else {
          store8<F32>(P.ghat_prev, e, narrow<F32>(g), nvalid);
        }
      }
      if (P.ghat) {
        Vec8<F32> o = narrow<F32>(g);
        store8<F32>(P.ghat, e, o, nvalid);
      }
    } else if constexpr (PH & STEP) {
      Vec8<F32> r = load8_any<F32>(P.ghat, e, nvalid);
      widen<F32>(r, g);
      cnt = (P.flags & 2u) ? (uint32_t)P.count_in[k] : 1u;
    }

    // ---- (3) the owner's update ------------------------------------------------
    float th[8];
    if constexpr (PH & (STEP | BCAST | DRIFT)) widen<F32>(rth, th);
    if constexpr (PH & STEP) {
      if (!((P.flags & 2u) && cnt == 0)) {
        float m[8], v[8];
        if constexpr (OPT == 1) {
          widen<F32>(rm, m);
          widen<F32>(rv, v);
        }
        optimizer8<OPT>(P, g, th, m, v);
        store8<F32>(P.master, e, narrow<F32>(th), nvalid);
        if constexpr (OPT == 1) {
          store8<F32>(P.m, e, narrow<F32>(m), nvalid);
          store8<F32>(P.v, e, narrow<F32>(v), nvalid);
        }
      }
    }

    // ---- (4) broadcast with stale retention, and the drift of every copy -------
    if constexpr (PH & (BCAST | DRIFT)) {
      const Vec8<RT> wire = narrow<RT>(th);
      float xw[8];
      widen<RT>(wire, xw);
      const uint64_t own = ELIDE ? 1ull << j : 0ull;   // owner-elided replicas: worker j holds no copy of this packet
      if constexpr (PH & BCAST) {
        const uint64_t keep = stale | own;
        for (uint32_t i = 0; i < W; ++i)
          if (!((keep >> i) & 1ull)) store8<RT>(P.replicas[i], rep_at(i, j, e), wire, nvalid);
      }
      if constexpr (PH & DRIFT) {
        // copies that differ from the wire value: the stale ones after a broadcast, or (standalone) all
        uint64_t todo = (PH & BCAST) ? stale : ((W == 64 ? ~0ull : ((1ull << W) - 1ull)) & ~own);
        while (todo) {
          // up to four copies are fetched before the first is used
          int ids[4];
          Vec8<RT> old[4];
          int nb = 0;
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            ids[b] = -1;
            if (todo) {
              ids[b] = __ffsll((long long)todo) - 1;
              todo &= todo - 1;
              nb = b + 1;
              old[b] = load8_any<RT>(P.replicas[ids[b]], rep_at((uint32_t)ids[b], j, e), nvalid);
            }
          }
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            if (b < nb) {
              float fo[8];
              widen<RT>(old[b], fo);
              float s = 0.0f;
#pragma unroll
              for (int x = 0; x < 8; ++x) {
                const float d = x < nvalid ? __fsub_rn(fo[x], xw[x]) : 0.0f;
                s = __fadd_rn(s, __fmul_rn(d, d));
              }
              const float tot = warp_sum(s);
              if ((ids[b] & 31) == lane) {
                if (ids[b] < 32) dacc0 += (double)tot; else dacc1 += (double)tot;
              }
            }
          }
        }
      }
    }
  }

  // ---- per-block drift partials, fixed order ------------------------------------
  if constexpr (PH & DRIFT) {
    __shared__ double sh[kWarps][kMaxW];
    sh[warp][lane] = dacc0;
    sh[warp][lane + 32] = dacc1;
    __syncthreads();
    if (threadIdx.x < kMaxW) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) t += sh[w][threadIdx.x];
      P.partials[(size_t)(P.partials_row0 + blockIdx.x) * kMaxW + threadIdx.x] = t;
    }
    if (P.ticket) drift_last_block(P, warp, lane, kWarps);
  }
}

// Sum the per-block partials of replica blockIdx.x in a fixed order (lane l takes rows l, l+32, ...,
// then a shuffle tree); add to sumsq, write the norm. One warp per replica.
static __global__ void drift_finalize_kernel(const double* __restrict__ partials, uint32_t nblocks, uint32_t W,
                                      float* norms, double* sumsq) {
  const uint32_t i = blockIdx.x;
  if (i >= W) return;
  double t = 0.0;
  for (uint32_t b = threadIdx.x; b < nblocks; b += 32) t += partials[(size_t)b * kMaxW + i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
  if (threadIdx.x == 0) {
    if (sumsq) sumsq[i] += t;
    if (norms) norms[i] = (float)sqrt(t);
  }
}

// Squared norm of every (worker, packet) gradient piece: out[i * K + k]. One warp per piece.
struct SqnormArgs {
  const void* grads[kMaxW];
  float* out;
  uint64_t n;
  uint32_t W, P, K;
};
template <class GT>
static __global__ void __launch_bounds__(256) packet_sqnorms_kernel(const __grid_constant__ SqnormArgs A) {
  const int lane = threadIdx.x & 31;
  const uint64_t warps = (uint64_t)gridDim.x * (blockDim.x >> 5);
  const uint64_t tasks = (uint64_t)A.W * A.K;
  for (uint64_t task = (uint64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); task < tasks; task += warps) {
    const uint32_t i = (uint32_t)(task / A.K), k = (uint32_t)(task % A.K);
    const uint64_t e0 = (uint64_t)k * A.P;
    const uint64_t e1 = e0 + A.P < A.n ? e0 + A.P : A.n;
    float s = 0.0f;
    for (uint64_t e = e0 + (uint64_t)lane * 8; e < e1; e += 256) {
      const int nvalid = e1 - e >= 8 ? 8 : (int)(e1 - e);
      float f[8];
      widen<GT>(load8_any<GT>(A.grads[i], e, nvalid), f);
#pragma unroll
      for (int x = 0; x < 8; ++x) s = __fadd_rn(s, x < nvalid ? __fmul_rn(f[x], f[x]) : 0.0f);
    }
    s = warp_sum(s);
    if (lane == 0) A.out[(size_t)i * A.K + k] = s;
  }
}

// Pairwise drift, the theorem's own quantity: d2[i*W + k] += sum_e (replica_i[e] - replica_k[e])^2.
// blockIdx.y picks a pair of 4-replica blocks (I <= J); each lane keeps the 16 pair sums of its elements in
// fp64 and walks 8-element vectors grid-stride in x. Cross-block accumulation uses fp64 atomics, so the order
// of that last sum is not fixed (results agree to ~1e-15 relative). A diagnostic, not on the timed path.
struct PairwiseArgs {
  const void* replicas[kMaxW];
  double* d2;
  uint64_t n;
  uint32_t W;
  uint32_t nblk;   // ceil(W / 4)
  // owner-elided replicas (elide != 0): the owner of an element holds no copy of it, so the element adds only
  // to the pairs of the other workers; rep_skip as in Params
  uint32_t elide, P, pps, k0;
  uint64_t rep_skip[kMaxW];
};

template <class RT>
static __global__ void __launch_bounds__(256) drift_pairwise_kernel(const __grid_constant__ PairwiseArgs A) {
  // blockIdx.y -> (I, J) with I <= J
  uint32_t I = 0, rem = blockIdx.y;
  while (rem >= A.nblk - I) { rem -= A.nblk - I; ++I; }
  const uint32_t J = I + rem;
  double acc[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) acc[q] = 0.0;
  const uint64_t nvec = (A.n + 7) / 8;
  for (uint64_t vi = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; vi < nvec; vi += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t e = vi * 8;
    const int nvalid = A.n - e >= 8 ? 8 : (int)(A.n - e);
    float a[4][8], b[4][8];
    uint32_t owner = 0xFFFFFFFFu;          // the worker without a copy of this vector (a vector lies in one packet)
    uint64_t kb = 0;                       // its bucket packet
    if (A.elide) {
      kb = (uint64_t)A.k0 + e / A.P;
      owner = (uint32_t)(kb / A.pps);
    }
    auto at = [&](uint32_t i) { return (A.elide && kb >= (uint64_t)(i + 1u) * A.pps) ? e - A.rep_skip[i] : e; };
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t ia = I * 4 + u, ib = J * 4 + u;
      if (ia < A.W && ia != owner) widen<RT>(load8_any<RT>(A.replicas[ia], at(ia), nvalid), a[u]);
      if (ib < A.W && ib != owner) widen<RT>(load8_any<RT>(A.replicas[ib], at(ib), nvalid), b[u]);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        if (I * 4 + u < A.W && J * 4 + v < A.W && I * 4 + u != owner && J * 4 + v != owner) {
          float s = 0.0f;
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const float d = x < nvalid ? __fsub_rn(a[u][x], b[v][x]) : 0.0f;
            s = __fadd_rn(s, __fmul_rn(d, d));
          }
          acc[u * 4 + v] += (double)s;
        }
      }
  }
  __shared__ double sh[8][16];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    double t = acc[q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    if (lane == 0) sh[warp][q] = t;
  }
  __syncthreads();
  if (threadIdx.x < 16) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += sh[w][threadIdx.x];
    const uint32_t i = I * 4 + threadIdx.x / 4, k = J * 4 + threadIdx.x % 4;
    if (i < A.W && k < A.W) {
      atomicAdd(&A.d2[(size_t)i * A.W + k], t);
      if (I != J) atomicAdd(&A.d2[(size_t)k * A.W + i], t);   // mirror; a diagonal block already holds both orders
    }
  }
}

// Closed-loop stand-in for the local gradient computation (Section 3 step (1)): worker i's gradient of
// 1/2 sum a (theta - x*)^2 at ITS OWN replica plus its noise, g_i = cast(a * (replica_i - x*) + noise_i),
// each operation rounded on its own. One lane per 8 elements, workers four at a time.
struct ClosedLoopArgs {
  const void* noise[kMaxW];
  const void* replicas[kMaxW];
  void* grads[kMaxW];
  const float* curv;
  const float* target;
  uint64_t n;
  uint32_t W;
};

template <class GT, class RT>
static __global__ void __launch_bounds__(256) closed_loop_grads_kernel(const __grid_constant__ ClosedLoopArgs A) {
  const uint64_t nvec = (A.n + 7) / 8;
  for (uint64_t vi = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; vi < nvec; vi += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t e = vi * 8;
    const int nvalid = A.n - e >= 8 ? 8 : (int)(A.n - e);
    float a[8], xs[8];
    widen<F32>(load8_any<F32>(A.curv, e, nvalid), a);
    widen<F32>(load8_any<F32>(A.target, e, nvalid), xs);
    for (uint32_t i0 = 0; i0 < A.W; i0 += 4) {
      Vec8<RT> rep[4];
      Vec8<GT> nz[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + u < A.W) {
          rep[u] = load8_any<RT>(A.replicas[i0 + u], e, nvalid);
          nz[u] = load8_any<GT>(A.noise[i0 + u], e, nvalid);
        }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + u < A.W) {
          float r[8], z[8], g[8];
          widen<RT>(rep[u], r);
          widen<GT>(nz[u], z);
#pragma unroll
          for (int x = 0; x < 8; ++x) g[x] = __fadd_rn(__fmul_rn(a[x], __fsub_rn(r[x], xs[x])), z[x]);
          store8<GT>(A.grads[i0 + u], e, narrow<GT>(g), nvalid);
        }
    }
  }
}

// Delivery indicators on a dense grid of tuples (host/device agreement check).
static __global__ void mask_grid_kernel(uint64_t seed, uint64_t step, const uint32_t* src, const uint32_t* dst,
                                 const uint64_t* packet, uint64_t count, uint32_t T, uint8_t* out) {
  const uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= count) return;
  const uint64_t pkey = packet_key_of(step_key_of(seed, step), packet[q]);
  out[q] = pair_hash(pkey, src[q], dst[q]) >= T ? 1 : 0;
}

}  // namespace lossy
