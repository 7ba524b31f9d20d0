// Fused lossy step for packets SHORTER than a tile: the "gather" pipeline (sm_100a).
//
// A tile holds 2, 4 or 8 whole packets ("sub-packets"), each with delivery masks of its own, so every stream
// of the step has holes at sub-packet granularity: dropped gradient pieces are not read, replicas that miss
// a broadcast are not written, and their old copies are read for the drift term. Bulk copies of a few
// hundred bytes are bound by their issue rate, not by memory, and a worker's whole tile piece in one bulk
// copy reads the dropped sub-packets too. Here everything with holes moves as 16 bytes per lane (512 bytes per
// warp instruction, whole lines), each lane testing the sub-packet its bytes lie in; only theta / m / v, which
// have no holes, stay bulk copies. Roles of a CTA:
//   mask warp      evaluates the delivery draws of a tile's sub-packets several tiles ahead and publishes them
//                  in a ring of kGatherRing entries (also the optional count / bit-set outputs)
//   gather warps   per tile and group of up to eight workers: asynchronous copies (cp.async, global -> shared
//                  memory without passing through registers) of the DELIVERED pieces, completing on the stage's
//                  mbarrier (cp.async.mbarrier.arrive.noinc); theta / m / v ride along as bulk copies
//   compute warps  sum the pieces in ascending worker order, divide by the received count, run the optimizer
//                  in place in shared memory, and write the wire tile into a ring of its own
//   store warp     theta / m / v back with three bulk copies; releases the stage
//   replica warps  each owns a fixed share of the replicas: from the wire ring it stores every (replica,
//                  sub-packet) pair that takes the broadcast
//   drift norms    the old copy of every pair that misses the broadcast is read and its squared difference from
//                  the wire tile summed, by whichever of three the host picked: eight drift warps of their own
//                  (wide geometry, RD), the replica warps (twin geometry, RD), or the compute warps
// A compute warp's 128 elements lie inside one sub-packet (packets here are powers of two from 128 elements
// that divide the tile). Every wait is bounded as in the other pipelines. No cluster, no multicast.
#pragma once
#include "lossy_tma.cuh"

namespace lossy {

constexpr uint32_t kGatherRing = 8;     // tiles whose masks may be published ahead of the replica warps
constexpr uint32_t kWireRing = 4;       // wire tiles between the compute warps and the replica warps
// RD: the build in which the stale copies are read outside the compute warps (see the kernel): by the replica
// warps in the twin geometry, by drift warps of their own in the wide one
template <int CW, bool RD = false> struct GatherShape {
  static constexpr int kProducers = CW >= 16 ? 2 : 1;                     // gather warps
  static constexpr int kReplicaWarps = (CW >= 16 || RD) ? 4 : 2;
  static constexpr int kDriftWarps = (CW >= 16 && RD) ? 8 : 0;
  static constexpr int kRdBuffers = kDriftWarps ? 1 : 2;                  // scratch buffers per warp that reads stale copies
  static constexpr int kAccRows = RD ? (kDriftWarps ? kMaxSub : 1) : CW;  // rows of fp64 drift sums: per compute warp, or per part of a row (RD)
  static constexpr int kThreads = (CW + 2 + kProducers + kReplicaWarps + kDriftWarps) * 32;   // compute + mask + gather + store + replica (+ drift)
  static constexpr int kTile = CW * 32 * kEpl;
  static constexpr int kCtasPerSm = CW >= 16 ? 1 : 2;
};
constexpr uint32_t kRdTwinMaxWorkers = 4;   // twin RD builds serve at most this many workers: one replica per replica warp
constexpr uint32_t kGatherMaxStages = 8;    // a tile of few workers is small: more of them in flight
constexpr uint32_t kGatherBarBytes = 512;   // 3 barriers per stage, 2 per mask-ring and wire-ring entry (8 B each), the abort flag
static_assert((3 * kGatherMaxStages + 2 * kGatherRing + 2 * kWireRing) * 8 + 4 <= kGatherBarBytes, "barrier area too small");

struct __align__(16) TileMasks {        // one ring entry: what the mask warp publishes about a tile
  uint64_t recv[kMaxSub];               // per sub-packet: bit i = worker i's piece was delivered
  uint64_t stale[kMaxSub];              // per sub-packet: bit i = replica i misses the broadcast
  uint32_t j[kMaxSub];                  // per sub-packet: owner
  uint64_t e0;                          // first element of the tile
  uint32_t npk, len;                    // sub-packets and elements of the tile
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// the executing thread's earlier cp.async copies, once complete, count as one arrival on the barrier
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// One lane's arithmetic at the end of a tile: estimate = sum / count (Algorithm 1 mode: the saved aggregate
// on a drop), the optimizer in place in shared memory, the wire value written once into `wire_tile` and returned widened.
template <class RT, int OPT>
__device__ __forceinline__ void finish_tile_lane(const Params& P, float (&acc)[kEpl], uint32_t cnt, unsigned char* sb,
                                                 uint32_t off_th, uint32_t off_m, uint32_t off_v, unsigned char* wire_tile,
                                                 uint32_t idx, uint64_t e, float (&wire)[kEpl]) {
  divide_by_count<kEpl>(acc, cnt);
  if (P.ghat_prev) {
    uint32_t pw[4];
    if (cnt == 0) {
      load_words_stream<kEpl>(P.ghat_prev + e, pw);
      unpack_lane<F32>(pw, acc);
    } else {
#pragma unroll
      for (int x = 0; x < kEpl; ++x) pw[x] = __float_as_uint(acc[x]);
      __stcs(reinterpret_cast<uint4*>(P.ghat_prev + e), make_uint4(pw[0], pw[1], pw[2], pw[3]));
    }
  }
  if (P.ghat) {
    uint32_t gw[4];
#pragma unroll
    for (int x = 0; x < kEpl; ++x) gw[x] = __float_as_uint(acc[x]);
    store_words<kEpl>(P.ghat + e, gw);
  }
  float th[kEpl], m[kEpl], v[kEpl];
  lds_lane<F32>(sb + off_th, idx, th);
  if (!((P.flags & kZeroSkip) && cnt == 0)) {
    if constexpr (OPT == 1) {
      lds_lane<F32>(sb + off_m, idx, m);
      lds_lane<F32>(sb + off_v, idx, v);
    }
    optimizer_n<OPT, kEpl>(P, acc, th, m, v);
    sts_lane_f32(sb + off_th, idx, th);
    if constexpr (OPT == 1) {
      sts_lane_f32(sb + off_m, idx, m);
      sts_lane_f32(sb + off_v, idx, v);
    }
  }
  if constexpr (RT::kVecs == 2) {
    sts_lane_f32(wire_tile, idx, th);
#pragma unroll
    for (int x = 0; x < kEpl; ++x) wire[x] = th[x];
  } else {
    uint32_t ww[4];
    pack_bf16_lane(th, ww);
    store_words<kEpl / 2>(wire_tile + (size_t)idx * 2, ww);
    unpack_lane<BF16>(ww, wire);
  }
}

// RD (a way of computing the drift norms): the old copies of the stale (replica, sub-packet) pairs are read outside
// the compute warps, with asynchronous copies into a scratch of G.rd_cap 512-byte chunks per buffer, requested as
// soon as the tile's masks are known and used once its wire tile exists; chunks beyond the scratch are loaded
// directly. Twin geometry (few workers): the replica warps do it, one tile ahead in the second of two buffers.
// Wide geometry: eight drift warps of their own do nothing else (four were the step's bottleneck: 0.61 of the copy
// rate at W = 16, P = 256, p = 0.3, against 0.85 with eight); one buffer each is enough, because the masks run
// several tiles ahead of the wire tile.
template <class GT, class RT, int OPT, bool DRIFTK, int CW, bool RD = false>
__global__ void __launch_bounds__(GatherShape<CW, RD>::kThreads, GatherShape<CW, RD>::kCtasPerSm)
    lossy_fused_gather_kernel(const __grid_constant__ Params P, const __grid_constant__ TmaGeom G) {
  static_assert(!RD || DRIFTK, "RD is a way of computing the drift norms");
  constexpr bool kWarpDrift = DRIFTK && !RD;               // the compute warps read the stale copies
  constexpr int kTile = GatherShape<CW, RD>::kTile;
  constexpr int kNP = GatherShape<CW, RD>::kProducers;
  constexpr int kNR = GatherShape<CW, RD>::kReplicaWarps;
  constexpr int kND = GatherShape<CW, RD>::kDriftWarps;
  constexpr int kAccRows = GatherShape<CW, RD>::kAccRows;
  constexpr int kGroup = 8;
  constexpr uint32_t kGB = sizeof(typename GT::raw), kRB = sizeof(typename RT::raw);
  constexpr uint32_t kRowG = kTile * kGB, kRowR = kTile * kRB;          // bytes of one worker's / replica's row of a tile
  extern __shared__ __align__(128) unsigned char smem[];
  // layout: barriers | abort flag (kGatherBarBytes) | ring of tile masks | stage headers | fp64 drift sums per compute
  //         warp and replica | wire ring | stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kGatherBarBytes - 4);
  TileMasks* ring = reinterpret_cast<TileMasks*>(smem + kGatherBarBytes);
  StageHdr* hdrs = reinterpret_cast<StageHdr*>(smem + kGatherBarBytes + kGatherRing * sizeof(TileMasks));
  double* warp_acc = reinterpret_cast<double*>(smem + kGatherBarBytes + kGatherRing * sizeof(TileMasks) + kGatherMaxStages * sizeof(StageHdr));
  unsigned char* wring = reinterpret_cast<unsigned char*>(warp_acc + kAccRows * kMaxW);
  const uint32_t rd_buf = G.rd_cap * 512u;                 // RD: bytes of one scratch buffer
  unsigned char* rscratch = wring + kWireRing * kRowR;     // RD: kRdBuffers buffers per warp that reads stale copies
  unsigned char* stage0 = rscratch + (RD ? (uint32_t)(kND ? kND : kNR) * GatherShape<CW, RD>::kRdBuffers * rd_buf : 0u);
  const uint32_t S = G.stages;
  const uint32_t off_th = G.grad_slots * kRowG;
  const uint32_t off_m = off_th + kTile * 4, off_v = off_m + kTile * 4;

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t W = P.W;
  const uint32_t lgP = 31u - (uint32_t)__clz((int)P.P);                 // packets are powers of two here
  auto full_bar = [&](uint32_t s) { return smem_u32(&bars[s]); };
  auto done_bar = [&](uint32_t s) { return smem_u32(&bars[kGatherMaxStages + s]); };
  auto empty_bar = [&](uint32_t s) { return smem_u32(&bars[2 * kGatherMaxStages + s]); };
  auto mfull_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kGatherMaxStages + q]); };
  auto mempty_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kGatherMaxStages + kGatherRing + q]); };
  auto wfull_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kGatherMaxStages + 2 * kGatherRing + q]); };
  auto wempty_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kGatherMaxStages + 2 * kGatherRing + kWireRing + q]); };

  for (uint32_t q = threadIdx.x; q < (uint32_t)kAccRows * kMaxW; q += blockDim.x) warp_acc[q] = 0.0;
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 32u * kNP + 1u);        // every gather lane's copies, and the header's writer
      mbar_init(done_bar(s), CW);
      mbar_init(empty_bar(s), 1);
    }
    for (uint32_t q = 0; q < kGatherRing; ++q) {
      mbar_init(mfull_bar(q), 1);
      mbar_init(mempty_bar(q), kNR + kND);           // the replica (and drift) warps are the last readers of a tile's masks
    }
    for (uint32_t q = 0; q < kWireRing; ++q) {
      mbar_init(wfull_bar(q), CW);
      mbar_init(wempty_bar(q), kNR + kND);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();

  constexpr int kChunks = kRowR / 512u;                     // a replica's row of a tile in 512-byte chunks
  constexpr uint32_t kElemsPerChunk = 512u / kRB;
  // Wide RD builds. A replica's row of a tile is cut into 2^lgf parts (the host balances the W * 2^lgf parts over
  // the drift warps); a warp takes parts first, first + stride, ... PASS 0 requests the old copies of their stale
  // (replica, sub-packet) pairs into `buffer`, chunk after chunk in the order (part, chunk); pass 1 takes their
  // squared differences against the wire tile: fp32 per lane within a part's chunks, one warp reduction per part
  // and tile, fp64 from there on (each (replica, part) has one accumulator, touched by one warp alone, in tile
  // order; the CTA's exit adds a replica's parts in ascending order).
  // One warp runs this alone, so its instructions are fetched for it alone: the walk visits the stale chunks only
  // and is kept short (one loop body for both passes, nothing unrolled), and each role calls it from one place.
  constexpr uint32_t kLgEpc = kElemsPerChunk == 256u ? 8u : 7u;
  auto drift_pass = [&](const TileMasks& tm, uint32_t first, uint32_t stride, unsigned char* buffer, int pass, const unsigned char* wt) {
    const uint32_t lgf = G.rd_lgsplit, part = G.packets_per_tile >> lgf;   // a replica's row in 2^lgf parts of `part` sub-packets
    const uint64_t stale_l = tm.stale[lane & (kMaxSub - 1)];
    const uint32_t j_l = tm.j[lane & (kMaxSub - 1)];
    const uint32_t live_tile = (1u << tm.npk) - 1u;       // entries behind a short last tile are marked stale everywhere
    const uint64_t e0 = tm.e0;
    const bool whole = lgP >= kLgEpc;                      // a sub-packet is one or more whole chunks (else a chunk holds several)
    const uint32_t sh = whole ? lgP - kLgEpc : kLgEpc - lgP;
    uint32_t n = 0;                                        // stale chunks met so far (warp-uniform)
#pragma unroll 1
    for (uint32_t u = first; u < (W << lgf); u += stride) {
      const uint32_t i = u >> lgf, h = u & ((1u << lgf) - 1u);
      const uint32_t live = __ballot_sync(0xFFFFFFFFu, (stale_l >> i) & 1ull) & live_tile & (((1u << part) - 1u) << (h * part));
      if (live == 0u) continue;
      const unsigned char* base = reinterpret_cast<const unsigned char*>(P.replicas[i]);
      float2 sq2 = make_float2(0.0f, 0.0f);                // two running sums (packed fp32 pairs of sm_100)
      uint32_t rem = live;
#pragma unroll 1
      while (rem) {
        const uint32_t sp0 = (uint32_t)__ffs((int)rem) - 1u;
        uint32_t c, c_end;
        if (whole) { c = sp0 << sh; c_end = c + (1u << sh); rem &= rem - 1u; }
        else { c = sp0 >> sh; c_end = c + 1u; rem &= ~(((1u << (1u << sh)) - 1u) << (c << sh)); }
#pragma unroll 1
        for (; c < c_end; ++c) {
          const uint32_t q = n++;
          const uint32_t off = c * 512u + (uint32_t)lane * 16u;
          const uint32_t el = off / kRB, sp = el >> lgP;
          const uint32_t j_sp = __shfl_sync(0xFFFFFFFFu, j_l, (int)sp);
          if (!((live >> sp) & 1u)) continue;              // this lane's 16 bytes are not stale ones
          unsigned char* sc = buffer + q * 512u + (uint32_t)lane * 16u;
          const unsigned char* old = base + rep_index(P, i, j_sp, e0 + el) * kRB;
          if (pass == 0) {
            if (q < G.rd_cap) cp_async16(smem_u32(sc), old);
          } else {
            // each lane reads back what it copied itself; a chunk the scratch had no room for comes from memory now
            const uint4 ov = q < G.rd_cap ? *reinterpret_cast<const uint4*>(sc) : __ldcs(reinterpret_cast<const uint4*>(old));
            const uint4 wv = *reinterpret_cast<const uint4*>(wt + off);
            const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
            if constexpr (RT::kVecs == 2) {                // fp32 replicas: one element per word
#pragma unroll
              for (int h = 0; h < 4; h += 2) {
                const float2 d = __fadd2_rn(make_float2(__uint_as_float(ow[h]), __uint_as_float(ow[h + 1])),
                                            make_float2(-__uint_as_float(ww[h]), -__uint_as_float(ww[h + 1])));
                sq2 = __fadd2_rn(sq2, __fmul2_rn(d, d));
              }
            } else {                                        // bf16 replicas: two elements per word
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const float2 d = __fadd2_rn(make_float2(__uint_as_float(ow[h] << 16), __uint_as_float(ow[h] & 0xFFFF0000u)),
                                            make_float2(-__uint_as_float(ww[h] << 16), -__uint_as_float(ww[h] & 0xFFFF0000u)));
                sq2 = __fadd2_rn(sq2, __fmul2_rn(d, d));
              }
            }
          }
        }
      }
      if (pass == 1) {
        const float tot = warp_sum(__fadd_rn(sq2.x, sq2.y));
        if (lane == 0) warp_acc[h * kMaxW + i] += (double)tot;   // one accumulator per replica and part, touched by one warp alone
      }
    }
  };
  if (warp == CW) {
    // ================================= mask warp =================================
    uint32_t slot = 0, par = 0;
    uint32_t Wp = 32;
    const bool batched = W <= 32 && !P.ghat_prev;          // Algorithm 1 draws once per packet
    if (batched) { Wp = 1; while (Wp < W) Wp <<= 1; }
    const uint32_t lgWp = 31u - (uint32_t)__clz((int)Wp);
    const uint32_t Bp = 32u >> lgWp;                        // sub-packets per pass of draws
    const uint32_t wmask = Wp == 32 ? 0xFFFFFFFFu : ((1u << Wp) - 1u);
    // the old copy of a (replica, sub-packet) pair that misses the broadcast is read several tiles later for the
    // drift term (by a compute warp, or by a replica warp in the RD builds): start it toward L2 now (one bulk
    // prefetch per pair)
    // (G.hints bit 2: the host asks for it where few pairs per tile are stale — it gains about 5 % there and
    // loses as much where they are many: the prefetches then crowd the bulk-copy unit that moves theta, m, v)
    const bool prefetch_on = kWarpDrift && (G.hints & 4u);
    auto prefetch_stale = [&](uint32_t i, uint32_t j, uint32_t k) {
      bulk_prefetch_l2(reinterpret_cast<const typename RT::raw*>(P.replicas[i]) + rep_index(P, i, j, (uint64_t)k * P.P), P.P * kRB);
    };
    for (uint32_t tile = blockIdx.x; tile < G.num_tiles; tile += gridDim.x) {
      if (!mbar_wait(mempty_bar(slot), par ^ 1u, abort_flag)) break;
      const uint32_t kfirst = tile * G.packets_per_tile;
      const uint32_t npk = min(G.packets_per_tile, G.full_packets - kfirst);
      if constexpr (kDevCheck) {   // debug build: every sub-packet's range, in the slab and in every replica
        bool fine = true;
        for (uint32_t sp = 0; sp < npk; ++sp)
          fine = tile_ok(P, kfirst + sp, (P.k0 + kfirst + sp) / P.pps, (uint64_t)(kfirst + sp) * P.P, P.P, kSiteGather, lane) && fine;
        if (!fine) { *abort_flag = 1u; break; }
      }
      TileMasks& tm = ring[slot];
      auto report = [&](uint32_t sp, uint32_t j, uint64_t r, uint64_t st, uint64_t gbad, uint64_t pbad) {   // one lane
        const uint32_t k = kfirst + sp;
        tm.recv[sp] = r;
        tm.stale[sp] = st;
        tm.j[sp] = j;
        if (P.count) P.count[k] = (uint8_t)__popcll(r);
        if (P.recv_bits) P.recv_bits[k] = r;
        if (P.stale_bits) P.stale_bits[k] = st;
        if (P.burst_out) {
          P.burst_out[k] = gbad;
          P.burst_out[(size_t)P.K + k] = pbad;
        }
      };
      if (batched) {
        for (uint32_t q0 = 0; q0 < npk; q0 += Bp) {
          const uint32_t sp_l = q0 + ((uint32_t)lane >> lgWp), i_l = (uint32_t)lane & (Wp - 1u);
          const uint32_t k_l = kfirst + (sp_l < npk ? sp_l : 0u);
          const uint32_t j_l = (P.k0 + k_l) / P.pps;
          const BatchDraws d = batch_draws<AGG | BCAST>(P, k_l, j_l, i_l, sp_l < npk && i_l < W);
          uint64_t st_l = 0;                                 // the stale set of this lane's own sub-packet
          for (uint32_t x = 0; x < Bp && q0 + x < npk; ++x) {
            uint64_t r, st, gbad, pbad;
            batch_masks<AGG | BCAST>(P, d, kfirst + q0 + x, (int)(x * Wp), wmask, r, st, gbad, pbad);
            const uint32_t j_x = __shfl_sync(0xFFFFFFFFu, j_l, (int)(x * Wp));
            if (x == ((uint32_t)lane >> lgWp)) st_l = st;
            if ((uint32_t)lane == x) report(q0 + x, j_x, r, st, gbad, pbad);
          }
          if (prefetch_on && sp_l < npk && i_l < W && ((st_l >> i_l) & 1ull)) prefetch_stale(i_l, j_l, k_l);
        }
      } else {
        for (uint32_t sp = 0; sp < npk; ++sp) {
          uint64_t r, st, gbad, pbad;
          const uint32_t j_sp = (P.k0 + kfirst + sp) / P.pps;
          packet_masks<AGG | BCAST>(P, kfirst + sp, j_sp, lane, r, st, gbad, pbad);
          if (lane == 0) report(sp, j_sp, r, st, gbad, pbad);
          if (prefetch_on) {
            for (uint32_t i = lane; i < W; i += 32)
              if ((st >> i) & 1ull) prefetch_stale(i, j_sp, kfirst + sp);
          }
        }
      }
      if ((uint32_t)lane >= npk && lane < kMaxSub) {      // entries behind a short last tile: nothing delivered, nothing to do
        tm.recv[lane] = 0;
        tm.stale[lane] = ~0ull;
        tm.j[lane] = 0;
      }
      if (lane == 0) {
        tm.e0 = (uint64_t)kfirst * P.P;
        tm.npk = npk;
        tm.len = npk * P.P;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(mfull_bar(slot));
      if (++slot == kGatherRing) { slot = 0; par ^= 1u; }
    }
  } else if (warp > CW && warp <= CW + kNP) {
    // ================================ gather warps ================================
    const uint32_t pw = (uint32_t)(warp - CW - 1);          // which gather warp
    uint32_t s = 0, par = 0, slot = 0, mpar = 0;
    bool ok = true;
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      if (!mbar_wait(mfull_bar(slot), mpar, abort_flag)) { ok = false; break; }
      const TileMasks& tm = ring[slot];
      const uint64_t e0 = tm.e0;
      const uint32_t len = tm.len;
      // lane l holds sub-packet (l & 7)'s receive mask; a ballot per worker turns that column into the worker's
      // row of delivered sub-packets
      const uint64_t recv_l = tm.recv[lane & (kMaxSub - 1)];
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag)) { ok = false; break; }
        const bool last = g + 1 == G.groups;
        const uint32_t in_group = min((uint32_t)kGroup, W - g * kGroup);
        const uint32_t st = smem_u32(stage0 + (size_t)s * G.stage_bytes);
        if (pw == 0) {
          // the header, and theta / m / v as three bulk copies on the same barrier
          if (lane == 0) {
            StageHdr& h = hdrs[s];
            h.recv = 0; h.stale = 0; h.e0 = e0; h.k = slot; h.len = len; h.cnt = 0; h.last = last ? 1u : 0u; h.own = 0; h.j = 0;
            if (last) mbar_arrive_expect_tx(full_bar(s), (OPT == 1 ? 3u : 1u) * len * 4u);   // publishes the header
            else mbar_arrive(full_bar(s));
          }
          __syncwarp();
          if (last) {
            if (lane == 8) bulk_g2s(st + off_th, P.master + e0, len * 4u, full_bar(s), false, 0);
            if constexpr (OPT == 1) {
              if (lane == 9) bulk_g2s(st + off_m, P.m + e0, len * 4u, full_bar(s), false, 0);
              if (lane == 10) bulk_g2s(st + off_v, P.v + e0, len * 4u, full_bar(s), false, 0);
            }
          }
        }
        // Delivered pieces of this group's workers: a row is copied in chunks of 512 bytes (one warp
        // instruction, 16 bytes per lane), each lane testing the sub-packet its 16 bytes lie in.
        auto copy_row = [&](uint32_t u, uint32_t c_first, uint32_t c_step) {
          const uint32_t rowmask = __ballot_sync(0xFFFFFFFFu, (recv_l >> (g * kGroup + u)) & 1ull) & 0xFFu;
          if (rowmask == 0u) return;
          const unsigned char* src = reinterpret_cast<const unsigned char*>(P.grads[g * kGroup + u]) + e0 * kGB;
          const uint32_t dst = st + u * kRowG;
#pragma unroll
          for (uint32_t c = c_first; c < kRowG / 512u; c += c_step) {
            const uint32_t off = c * 512u + (uint32_t)lane * 16u;   // byte within the row
            if ((rowmask >> ((off / kGB) >> lgP)) & 1u) cp_async16(dst + off, src + off);
          }
        };
        // Two gather warps deal out either the group's workers (a row of several chunks per warp and turn: half the
        // ballots) or every row's chunks (both warps in the same row); the host picks (G.hints bit 3 = chunks).
        // (One gather warp keeps the loop it had: the same copies written as the two-warp form ran 6-14 % slower in
        // the twin geometry.)
        if (kNP > 1 && !(G.hints & 8u)) {
          for (uint32_t u = pw; u < in_group; u += kNP) copy_row(u, 0u, 1u);
        } else {
          for (uint32_t u = 0; u < in_group; ++u) copy_row(u, pw, kNP);
        }
        cp_async_arrive(full_bar(s));
      }
      if (++slot == kGatherRing) { slot = 0; mpar ^= 1u; }
    }
    // copies in flight at an abort: wait for this warp's own before the CTA exits
    if (!ok || *abort_flag) asm volatile("cp.async.wait_all;" ::: "memory");
  } else if (warp == CW + kNP + 1) {
    // ================================ store warp =================================
    uint32_t s = 0, par = 0;
    bool ok = true;
    const bool sh_hint = G.hints & 2u;
    const uint64_t pol = policy_evict_first();
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(done_bar(s), par, abort_flag)) { ok = false; break; }
        if (g + 1 == G.groups) {
          const uint64_t e0 = hdrs[s].e0;
          const uint32_t len = hdrs[s].len;
          unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
          if (lane == 0) bulk_s2g(P.master + e0, smem_u32(st + off_th), len * 4u, sh_hint, pol);
          if constexpr (OPT == 1) {
            if (lane == 1) bulk_s2g(P.m + e0, smem_u32(st + off_m), len * 4u, sh_hint, pol);
            if (lane == 2) bulk_s2g(P.v + e0, smem_u32(st + off_v), len * 4u, sh_hint, pol);
          }
          bulk_commit();
          bulk_wait_read0();          // shared memory of this stage may be overwritten after this
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(s));
      }
    }
    bulk_wait0();
  } else if (kND > 0 && warp > CW + kNP + 1 + kNR) {
    // ================================ drift warps ================================
    // (wide RD builds) warp d takes replicas d, d + kND, ...: requests a tile's stale copies when its masks are
    // published, uses them when its wire tile is, and releases both
    const uint32_t dw = (uint32_t)(warp - CW - kNP - 2 - kNR);
    unsigned char* scratch = rscratch + (size_t)dw * rd_buf;
    uint32_t slot = 0, mpar = 0, wslot = 0, wpar = 0;
    bool ok = true;
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      if (!mbar_wait(mfull_bar(slot), mpar, abort_flag)) break;
      const TileMasks& tm = ring[slot];
#pragma unroll 1
      for (int pass = 0; pass < 2; ++pass) {
        if (pass == 1) {
          if (!mbar_wait(wfull_bar(wslot), wpar, abort_flag)) { ok = false; break; }
          asm volatile("cp.async.wait_all;" ::: "memory");
        }
        drift_pass(tm, dw, kND, scratch, pass, wring + (size_t)wslot * kRowR);
      }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(wempty_bar(wslot));
        mbar_arrive(mempty_bar(slot));
      }
      if (++slot == kGatherRing) { slot = 0; mpar ^= 1u; }
      if (++wslot == kWireRing) { wslot = 0; wpar ^= 1u; }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else if (warp > CW + kNP + 1) {
    // =============================== replica warps ===============================
    const uint32_t rw = (uint32_t)(warp - CW - kNP - 2);    // this warp owns replicas rw, rw + kNR, ...
    constexpr bool kReadsStale = RD && kND == 0;            // twin RD: these warps also take the drift terms
    unsigned char* scratch = rscratch + (size_t)rw * 2u * rd_buf;
    uint32_t slot = 0, wslot = 0, wpar = 0, mpar = 0, buf = 0;
    // twin RD: the walk of this warp's replicas' rows, unrolled over a row's few chunks (measured faster here than the
    // drift warps' loop over the stale chunks). PASS 0 requests the old copies of a tile's stale (replica, sub-packet)
    // pairs into scratch buffer `b`
    // (chunk after chunk in the order (replica, chunk)); pass 1 takes their squared differences against the wire
    // tile: fp32 per lane within a replica's chunks, one warp reduction per replica and tile, fp64 from there on
    // (each replica has one accumulator, touched by this warp alone, in tile order).
    auto row_pass = [&](const TileMasks& tm, uint32_t b, int pass, const unsigned char* wt) {
      const uint64_t stale_l = tm.stale[lane & (kMaxSub - 1)];
      const uint32_t j_l = tm.j[lane & (kMaxSub - 1)];
      const uint32_t live_tile = (1u << tm.npk) - 1u;       // entries behind a short last tile are marked stale everywhere
      const uint64_t e0 = tm.e0;
      uint32_t n = 0;                                       // chunks with a stale sub-packet met so far (warp-uniform)
      for (uint32_t i = rw; i < W; i += kNR) {
        const uint32_t live = __ballot_sync(0xFFFFFFFFu, (stale_l >> i) & 1ull) & 0xFFu & live_tile;
        if (live == 0u) continue;
        const unsigned char* base = reinterpret_cast<const unsigned char*>(P.replicas[i]);
        float2 sq2 = make_float2(0.0f, 0.0f);                                 // two running sums (packed fp32 pairs of sm_100)
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          const uint32_t el0 = (uint32_t)c * kElemsPerChunk;                    // the chunk's sub-packets, as bits
          const uint32_t in_chunk = ((2u << ((el0 + kElemsPerChunk - 1u) >> lgP)) - 1u) & ~((1u << (el0 >> lgP)) - 1u);
          if ((live & in_chunk) == 0u) continue;
          const uint32_t q = n++;
          const uint32_t off = (uint32_t)c * 512u + (uint32_t)lane * 16u;
          const uint32_t el = off / kRB, sp = el >> lgP;
          const uint32_t j_sp = __shfl_sync(0xFFFFFFFFu, j_l, (int)sp);
          const bool mine = (live >> sp) & 1u;                                  // this lane's 16 bytes are stale ones
          unsigned char* sc = scratch + (size_t)b * rd_buf + q * 512u + (uint32_t)lane * 16u;
          if (pass == 0) {
            if (mine) cp_async16(smem_u32(sc), base + rep_index(P, i, j_sp, e0 + el) * kRB);
          } else if (mine) {
            const uint4 ov = *reinterpret_cast<const uint4*>(sc);               // each lane reads back what it copied itself
            const uint4 wv = *reinterpret_cast<const uint4*>(wt + off);
            const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w}, ww[4] = {wv.x, wv.y, wv.z, wv.w};
            if constexpr (RT::kVecs == 2) {                // fp32 replicas: one element per word
#pragma unroll
              for (int h = 0; h < 4; h += 2) {
                const float2 d = __fadd2_rn(make_float2(__uint_as_float(ow[h]), __uint_as_float(ow[h + 1])),
                                            make_float2(-__uint_as_float(ww[h]), -__uint_as_float(ww[h + 1])));
                sq2 = __fadd2_rn(sq2, __fmul2_rn(d, d));
              }
            } else {                                        // bf16 replicas: two elements per word
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const float2 d = __fadd2_rn(make_float2(__uint_as_float(ow[h] << 16), __uint_as_float(ow[h] & 0xFFFF0000u)),
                                            make_float2(-__uint_as_float(ww[h] << 16), -__uint_as_float(ww[h] & 0xFFFF0000u)));
                sq2 = __fadd2_rn(sq2, __fmul2_rn(d, d));
              }
            }
          }
        }
        if (pass == 1) {
          const float tot = warp_sum(__fadd_rn(sq2.x, sq2.y));
          if (lane == 0) warp_acc[i] += (double)tot;        // row 0 of the sums: one accumulator per replica
        }
      }
    };
    if constexpr (kReadsStale) {
      if (blockIdx.x < G.num_tiles) {
        if (mbar_wait(mfull_bar(0), 0u, abort_flag)) row_pass(ring[0], 0u, 0, nullptr);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (uint32_t tile = blockIdx.x; tile < G.num_tiles; tile += gridDim.x) {
      if constexpr (kReadsStale) {
        // the next tile's old copies first: they have this tile's duration to arrive
        if (tile + gridDim.x < G.num_tiles) {
          const uint32_t nslot = slot + 1u == kGatherRing ? 0u : slot + 1u;
          if (!mbar_wait(mfull_bar(nslot), nslot == 0u ? mpar ^ 1u : mpar, abort_flag)) break;
          row_pass(ring[nslot], buf ^ 1u, 0, nullptr);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
      // the wire tile is complete: every compute warp has arrived, and each had waited for the tile's masks first
      if (!mbar_wait(wfull_bar(wslot), wpar, abort_flag)) break;
      const TileMasks& tm = ring[slot];
      const uint64_t e0 = tm.e0;
      const unsigned char* wt = wring + (size_t)wslot * kRowR;
      // lane l holds sub-packet (l & 7)'s masks; a ballot per replica turns that column into the replica's row
      const uint32_t j_l = tm.j[lane & (kMaxSub - 1)];
      const uint64_t keep_l = tm.stale[lane & (kMaxSub - 1)] | own_bit(P, j_l);   // not written: missed the broadcast, or does not exist
      uint32_t jc[kChunks];                                 // owner of the sub-packet this lane's bytes of chunk c lie in
#pragma unroll
      for (int c = 0; c < kChunks; ++c)
        jc[c] = __shfl_sync(0xFFFFFFFFu, j_l, (int)((((uint32_t)c * 512u + (uint32_t)lane * 16u) / kRB) >> lgP));
      for (uint32_t i = rw; i < W; i += kNR) {
        const uint32_t fresh = __ballot_sync(0xFFFFFFFFu, !((keep_l >> i) & 1ull)) & 0xFFu;   // bit sp: replica i takes it
        if (fresh == 0u) continue;
        unsigned char* base = reinterpret_cast<unsigned char*>(P.replicas[i]);
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          const uint32_t off = (uint32_t)c * 512u + (uint32_t)lane * 16u;
          const uint32_t el = off / kRB;
          if ((fresh >> (el >> lgP)) & 1u)
            __stcs(reinterpret_cast<uint4*>(base + rep_index(P, i, jc[c], e0 + el) * kRB),
                   *reinterpret_cast<const uint4*>(wt + off));
        }
      }
      if constexpr (kReadsStale) {
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // everything but the next tile's requests has landed
        row_pass(tm, buf, 1, wt);
        buf ^= 1u;
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(wempty_bar(wslot));
        mbar_arrive(mempty_bar(slot));
      }
      if (++slot == kGatherRing) { slot = 0; mpar ^= 1u; }
      if (++wslot == kWireRing) { wslot = 0; wpar ^= 1u; }
    }
    if constexpr (kReadsStale) asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // =============================== compute warps ===============================
    const uint32_t idx = threadIdx.x * kEpl;               // first element of this lane within the tile
    const uint32_t my_sp = ((uint32_t)(threadIdx.x & ~31) * kEpl) >> lgP;   // this warp's sub-packet, always the same
    uint32_t s = 0, par = 0, slot = 0, mpar = 0, wslot = 0, wpar = 0;
    bool ok = true;
    float acc[kEpl];
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    constexpr int kWords = LaneWords<RT>::value;
    // Stale copies requested before the tile's arithmetic. Four: with eight (16 more registers per lane for bf16)
    // every point measured slower (W = 8, P = 256, p = 0.3: 0.83 -> 0.71), although a copy requested only
    // afterwards exposes its latency.
    constexpr int kPre = 4;
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      if (!mbar_wait(mfull_bar(slot), mpar, abort_flag)) { ok = false; break; }
      const TileMasks& tm = ring[slot];
      const uint32_t len = tm.len;
      const uint64_t e0 = tm.e0;
      const bool active = idx < len;
      const uint64_t my_recv = tm.recv[my_sp];             // zero behind a short last tile
      // The old copies this warp compares against for the drift term (in L2 by now: the mask warp asked for them
      // tiles ago) are requested first, so that their latency hides behind the wait for the tile and its arithmetic.
      [[maybe_unused]] uint32_t pre_raw[kPre][4];
      [[maybe_unused]] uint64_t early = 0;                 // the replicas whose copies were requested early
      [[maybe_unused]] uint32_t my_j = 0;
      uint64_t stale_rest = 0;
      if constexpr (kWarpDrift) {
        if (active) {
          stale_rest = tm.stale[my_sp];
          my_j = tm.j[my_sp];
        }
#pragma unroll
        for (int b = 0; b < kPre; ++b) {
          if (stale_rest) {
            const int id = __ffsll((long long)stale_rest) - 1;
            stale_rest &= stale_rest - 1;
            early |= 1ull << id;
            load_words_stream<kWords>(reinterpret_cast<const typename RT::raw*>(P.replicas[id]) +
                                          rep_index(P, (uint32_t)id, my_j, e0 + idx), pre_raw[b]);
          }
        }
      }
#pragma unroll
      for (int x = 0; x < kEpl; ++x) acc[x] = 0.0f;
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
        unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
        const uint32_t bits = (uint32_t)(my_recv >> (g * kGroup)) & 0xFFu;
#pragma unroll
        for (int u = 0; u < kGroup; ++u)
          if ((bits >> u) & 1u) {
            float f[kEpl];
            lds_lane<GT>(st + (size_t)u * kRowG, idx, f);
#pragma unroll
            for (int x = 0; x < kEpl; ++x) acc[x] = __fadd_rn(acc[x], f[x]);
          }
        if (g + 1 == G.groups) {
          // the wire tile goes into the ring the replica warps drain
          if (!mbar_wait(wempty_bar(wslot), wpar ^ 1u, abort_flag)) { ok = false; break; }
          float wire[kEpl];
#pragma unroll
          for (int x = 0; x < kEpl; ++x) wire[x] = 0.0f;
          if (active)
            finish_tile_lane<RT, OPT>(P, acc, (uint32_t)__popcll(my_recv), st, off_th, off_m, off_v,
                                      wring + (size_t)wslot * kRowR, idx, e0 + idx, wire);
          fence_proxy_async();          // make theta / m / v visible to the bulk stores
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(wfull_bar(wslot));
            mbar_arrive(done_bar(s));
          }
          if (++wslot == kWireRing) { wslot = 0; wpar ^= 1u; }
          if constexpr (kWarpDrift) {
            // squared differences of up to four copies at a time, their warp totals in one multi-value reduction;
            // the first lane of segment b adds copy b's total to this warp's fp64 sum of that replica
            auto reduce4 = [&](float (&sq)[4], const int (&ids)[4]) {
              const float tot = warp_sum_multi<4>(sq, lane);
              const int b = lane >> 3;
              int id = ids[0];
#pragma unroll
              for (int x = 1; x < 4; ++x) id = b == x ? ids[x] : id;
              if ((lane & 7) == 0 && id >= 0) warp_acc[warp * kMaxW + id] += (double)tot;
            };
            if (early) {              // warp-uniform: the warp's elements lie in one sub-packet
              float sq[4];
#pragma unroll
              for (int b0 = 0; b0 < kPre; b0 += 4) {
                if (b0 > 0 && early == 0) break;
                int ids[4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                  sq[b] = 0.0f;
                  ids[b] = -1;
                  if (early) {
                    ids[b] = __ffsll((long long)early) - 1;
                    early &= early - 1;
                    float old[kEpl];
                    unpack_lane<RT>(pre_raw[b0 + b], old);
#pragma unroll
                    for (int x = 0; x < kEpl; ++x) {
                      const float d = __fsub_rn(old[x], wire[x]);
                      sq[b] = __fadd_rn(sq[b], __fmul_rn(d, d));
                    }
                  }
                }
                reduce4(sq, ids);
              }
              while (stale_rest) {     // more stale copies than were requested early
                int ids[4];
                uint32_t raw[4][4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                  ids[b] = -1;
                  if (stale_rest) {
                    ids[b] = __ffsll((long long)stale_rest) - 1;
                    stale_rest &= stale_rest - 1;
                    load_words_stream<kWords>(reinterpret_cast<const typename RT::raw*>(P.replicas[ids[b]]) +
                                                  rep_index(P, (uint32_t)ids[b], my_j, e0 + idx), raw[b]);
                  }
                }
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                  sq[b] = 0.0f;
                  if (ids[b] >= 0) {
                    float old[kEpl];
                    unpack_lane<RT>(raw[b], old);
#pragma unroll
                    for (int x = 0; x < kEpl; ++x) {
                      const float d = __fsub_rn(old[x], wire[x]);
                      sq[b] = __fadd_rn(sq[b], __fmul_rn(d, d));
                    }
                  }
                }
                reduce4(sq, ids);
              }
            }
          }
        } else {
          __syncwarp();
          if (lane == 0) mbar_arrive(done_bar(s));
        }
      }
      if (++slot == kGatherRing) { slot = 0; mpar ^= 1u; }
    }
  }

  // ---- common exit: per-CTA drift partials in fixed order, status word ---------------
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) atomicExch(G.status, 1u);
  if constexpr (DRIFTK) {
    if (threadIdx.x < kMaxW) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < kAccRows; ++w) t += warp_acc[w * kMaxW + threadIdx.x];
      P.partials[(size_t)blockIdx.x * kMaxW + threadIdx.x] = t;
    }
    if (P.ticket) drift_last_block(P, warp, lane, GatherShape<CW, RD>::kThreads / 32);
  }
}

}  // namespace lossy
