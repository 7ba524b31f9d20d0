// The four single-phase calls (aggregate, optimizer step, broadcast, drift norms) as bulk-copy (TMA)
// pipelines for sm_100a: the same CTA shape, barriers and bounded waits as the fused kernel, one phase
// per build.
//
// A tile is at most kTile contiguous elements inside one packet. Per tile the producer warp arms an
// mbarrier and issues 1-D bulk copies global -> shared memory, the compute warps work in shared
// memory, and the store warp writes results with bulk copies shared -> global memory:
//   AGG   : groups of up to GS delivered gradient pieces in, summed in ascending worker order, divided
//           by the received count; the fp32 estimate goes out as one tile (dropped packets are not read)
//   STEP  : ghat, theta (and m, v) in, updated in place, theta (and m, v) out
//   BCAST : theta in, rounded to the wire type once, one bulk store per replica that receives it
//   DRIFT : theta and groups of up to GS replica pieces in, squared differences accumulated, nothing out
// Packets shorter than a tile and a ragged last packet stay on the register kernel. Algorithm 1's aggregate
// (P.ghat_prev set) runs here too: one draw per packet, the saved aggregate read or written by the compute warps.
#pragma once
#include "lossy_tma.cuh"

namespace lossy {

constexpr int kPhaseMaxStages = 8;     // as many as fit, up to eight (the host caps the optimizer step at three)
static_assert(3 * kPhaseMaxStages * 8 + 4 <= (int)kTmaBarBytes, "barrier area too small");

// bytes of one pipeline stage; `slots` = arrays of the streamed group (AGG, DRIFT), `eb` = their element size
template <int PH>
__host__ __device__ constexpr uint32_t phase_stage_bytes(uint32_t tile, uint32_t slots, uint32_t eb, bool adam) {
  return PH == AGG     ? slots * tile * eb + tile * 4u
         : PH == STEP  ? (adam ? 4u : 2u) * tile * 4u
         : PH == BCAST ? tile * 4u + (eb == 4u ? 0u : tile * eb)
                       : slots * tile * eb + tile * 4u;
}

// T = element type of the streamed arrays: gradients (AGG) or replicas (BCAST, DRIFT); F32 for STEP.
template <int PH, class T, int OPT, int CW, int GS>
__global__ void __launch_bounds__(TmaShape<CW>::kThreads, TmaShape<CW>::kCtasPerSm)
    lossy_phase_tma_kernel(const __grid_constant__ Params P, const __grid_constant__ TmaGeom G) {
  static_assert(PH == AGG || PH == STEP || PH == BCAST || PH == DRIFT, "one phase per build");
  static_assert(kEpl == 4, "the drift arithmetic pairs four elements per lane");
  constexpr int kConsumerWarps = CW;
  constexpr int kTile = TmaShape<CW>::kTile;
  constexpr uint32_t kEB = sizeof(typename T::raw);
  constexpr bool kGrouped = PH == AGG || PH == DRIFT;   // W arrays streamed in groups of GS
  extern __shared__ __align__(128) unsigned char smem[];
  // layout: [full, done, empty barriers | abort flag] (kTmaBarBytes) | headers (kPhaseMaxStages x 64 B) | stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kTmaBarBytes - 4);
  StageHdr* hdrs = reinterpret_cast<StageHdr*>(smem + kTmaBarBytes);
  unsigned char* stage0 = smem + kTmaBarBytes + kPhaseMaxStages * sizeof(StageHdr);
  const uint32_t S = G.stages;
  // offsets inside a stage
  const uint32_t off_tail = G.grad_slots * kTile * kEB;          // AGG: estimate tile, DRIFT: theta tile
  constexpr uint32_t off_th = PH == STEP ? kTile * 4u : 0u;       // STEP: ghat | theta | m | v; BCAST: theta | wire
  constexpr uint32_t off_m = 2u * kTile * 4u, off_v = 3u * kTile * 4u;
  constexpr uint32_t off_wire = kEB == 4u ? 0u : kTile * 4u;      // fp32 replicas are stored from the theta tile

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t W = P.W;
  auto full_bar = [&](uint32_t s) { return smem_u32(&bars[s]); };
  auto done_bar = [&](uint32_t s) { return smem_u32(&bars[kPhaseMaxStages + s]); };
  auto empty_bar = [&](uint32_t s) { return smem_u32(&bars[2 * kPhaseMaxStages + s]); };

  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(done_bar(s), kConsumerWarps);
      mbar_init(empty_bar(s), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();

  double dacc0 = 0.0, dacc1 = 0.0;   // DRIFT, compute warps: lane l holds replicas l and l + 32

  if (warp == kConsumerWarps) {
    // =============================== producer warp ===============================
    // One warp's chain of dependent instructions per tile bounds the whole CTA when a tile carries few
    // bytes, so the delivery draws (the hash is most of that chain) are taken for a batch of tiles at
    // once: with W <= 32 the warp's lanes cover 32 / Wp tiles (Wp = W rounded up to a power of two), one
    // link per lane, and one ballot returns the masks of all of them.
    uint32_t s = 0, par = 0, armed_mask = 0, armed_par = 0;
    bool ok = true;
    const bool lh = G.hints & 1u;
    const uint64_t pol = policy_evict_first();
    constexpr bool kMasked = PH == AGG || PH == BCAST;
    uint32_t Wp = 32;
    const bool batched = kMasked && W <= 32 && !(PH == AGG && P.ghat_prev);   // Algorithm 1 draws once per packet
    if (batched && W <= 16) { Wp = 1; while (Wp < W) Wp <<= 1; }
    const uint32_t lgWp = 31u - (uint32_t)__clz((int)Wp);
    const uint32_t B = 32u >> lgWp;                                // tiles per batch
    const uint32_t wmask = Wp == 32 ? 0xFFFFFFFFu : ((1u << Wp) - 1u);
    const uint64_t all = W == 64 ? ~0ull : ((1ull << W) - 1ull);
    for (uint32_t tile0 = blockIdx.x; ok && tile0 < G.num_tiles; tile0 += B * gridDim.x) {
      // this lane's tile of the batch and its worker there
      const uint32_t b_l = (uint32_t)lane >> lgWp, i_l = (uint32_t)lane & (Wp - 1u);
      const uint32_t tile_l = tile0 + b_l * gridDim.x;
      const bool tv = tile_l < G.num_tiles;
      const uint32_t k_l = tv ? tile_l / G.tiles_per_packet : 0u;
      const uint32_t c_l = tv ? tile_l - k_l * G.tiles_per_packet : 0u;
      const uint32_t j_l = (P.k0 + k_l) / P.pps;
      BatchDraws draws = {0u, 0u, 0u};         // W <= 32: one bit per (tile of the batch, worker)
      if constexpr (kMasked) {
        if (batched) draws = batch_draws<PH>(P, k_l, j_l, i_l, tv && i_l < W);
      }
      for (uint32_t b = 0; ok && b < B; ++b) {
        const uint32_t tile = tile0 + b * gridDim.x;
        if (tile >= G.num_tiles) break;
        const int src = (int)(b * Wp);
        const uint32_t k = __shfl_sync(0xFFFFFFFFu, k_l, src);
        const uint32_t c = __shfl_sync(0xFFFFFFFFu, c_l, src);
        const uint32_t j = __shfl_sync(0xFFFFFFFFu, j_l, src);
        const uint64_t e0 = (uint64_t)k * P.P + (uint64_t)c * kTile;
        const uint32_t len = min((uint32_t)kTile, P.P - c * kTile);
        if (!tile_ok(P, k, j, e0, len, kSitePhase, lane)) { *abort_flag = 1u; ok = false; break; }   // debug build only
        uint64_t recv = 0, stale = 0, gbad = 0, pbad = 0;
        uint32_t cnt = 1;
        if constexpr (kMasked) {
          if (batched) {
            batch_masks<PH>(P, draws, k, src, wmask, recv, stale, gbad, pbad);
          } else {
            packet_masks<PH>(P, k, j, lane, recv, stale, gbad, pbad);
          }
        }
        if constexpr (PH == AGG) {
          cnt = __popcll(recv);
          if (c == 0 && lane == 0) {
            if (P.count) P.count[k] = (uint8_t)cnt;
            if (P.recv_bits) P.recv_bits[k] = recv;
            if (P.burst_out) P.burst_out[k] = gbad;
          }
        } else if constexpr (PH == BCAST) {
          if (c == 0 && lane == 0) {
            if (P.stale_bits) P.stale_bits[k] = stale;
            if (P.burst_out) P.burst_out[(size_t)P.K + k] = pbad;
          }
        } else if constexpr (PH == STEP) {
          if (P.flags & 2u) cnt = P.count_in[k];
        } else {
          recv = all & ~own_bit(P, j);   // standalone drift: every copy that exists is compared
        }
        for (uint32_t g = 0; g < G.groups; ++g) {
          if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag)) { ok = false; break; }
          const bool last = g + 1 == G.groups;
          const uint32_t bits = kGrouped ? (uint32_t)(recv >> (g * GS)) & ((1u << GS) - 1u) : 0u;
          unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
          if (lane == 0) {
            StageHdr& h = hdrs[s];
            h.recv = recv; h.stale = stale; h.e0 = e0; h.k = k; h.len = len; h.cnt = cnt; h.last = last ? 1u : 0u;
            h.own = own_bit(P, j); h.j = j;
            uint32_t bytes = __popc(bits) * len * kEB;
            if constexpr (PH == STEP) bytes = (OPT == 1 ? 4u : 2u) * len * 4u;
            if constexpr (PH == BCAST) bytes = len * 4u;
            if constexpr (PH == DRIFT) bytes += g == 0 ? len * 4u : 0u;
            mbar_arrive_expect_tx(full_bar(s), bytes);
          }
          __syncwarp();
          if constexpr (kGrouped) {
            if (lane < GS && ((bits >> lane) & 1u)) {
              const void* src_p = PH == AGG ? P.grads[g * GS + lane] : P.replicas[g * GS + lane];
              const uint64_t at = PH == AGG ? e0 : rep_index(P, g * GS + (uint32_t)lane, j, e0);
              bulk_g2s(smem_u32(st + (size_t)lane * kTile * kEB), reinterpret_cast<const typename T::raw*>(src_p) + at,
                       len * kEB, full_bar(s), lh, pol);
            }
            if constexpr (PH == DRIFT) {
              if (g == 0 && lane == 8) bulk_g2s(smem_u32(st + off_tail), P.master + e0, len * 4u, full_bar(s), lh, pol);
            }
          } else if constexpr (PH == STEP) {
            if (lane == 0) bulk_g2s(smem_u32(st), P.ghat + e0, len * 4u, full_bar(s), lh, pol);
            if (lane == 1) bulk_g2s(smem_u32(st + off_th), P.master + e0, len * 4u, full_bar(s), lh, pol);
            if constexpr (OPT == 1) {
              if (lane == 2) bulk_g2s(smem_u32(st + off_m), P.m + e0, len * 4u, full_bar(s), lh, pol);
              if (lane == 3) bulk_g2s(smem_u32(st + off_v), P.v + e0, len * 4u, full_bar(s), lh, pol);
            }
          } else {
            if (lane == 0) bulk_g2s(smem_u32(st + off_th), P.master + e0, len * 4u, full_bar(s), lh, pol);
          }
          armed_mask |= 1u << s;
          armed_par = (armed_par & ~(1u << s)) | (par << s);
          if (++s == S) { s = 0; par ^= 1u; }
        }
      }
    }
    if (!ok || *abort_flag) {
      // give this CTA's copies in flight a bounded time to land before the CTA exits
      for (uint32_t q = 0; q < S; ++q)
        if ((armed_mask >> q) & 1u)
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(full_bar(q), (armed_par >> q) & 1u)) break;
    }
  } else if (warp == kConsumerWarps + 1) {
    // ================================ store warp =================================
    uint32_t s = 0, par = 0;
    bool ok = true;
    const bool sh_hint = G.hints & 2u;
    const uint64_t pol = policy_evict_first();
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(done_bar(s), par, abort_flag)) { ok = false; break; }
        if (PH == DRIFT || g + 1 < G.groups) {   // nothing to store from this stage
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_bar(s));
          continue;
        }
        const StageHdr& h = hdrs[s];
        const uint64_t e0 = h.e0;
        const uint32_t len = h.len;
        unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
        if constexpr (PH == AGG) {
          if (lane == 0) bulk_s2g(P.ghat + e0, smem_u32(st + off_tail), len * 4u, sh_hint, pol);
        } else if constexpr (PH == STEP) {
          if (!((P.flags & 2u) && h.cnt == 0)) {   // a packet nobody reported on keeps its state untouched
            if (lane == 0) bulk_s2g(P.master + e0, smem_u32(st + off_th), len * 4u, sh_hint, pol);
            if constexpr (OPT == 1) {
              if (lane == 1) bulk_s2g(P.m + e0, smem_u32(st + off_m), len * 4u, sh_hint, pol);
              if (lane == 2) bulk_s2g(P.v + e0, smem_u32(st + off_v), len * 4u, sh_hint, pol);
            }
          }
        } else if constexpr (PH == BCAST) {
          const uint64_t keep = h.stale | h.own;   // replicas that are not written: they missed the broadcast, or do not exist
          for (uint32_t i = lane; i < W; i += 32)
            if (!((keep >> i) & 1ull))
              bulk_s2g(reinterpret_cast<typename T::raw*>(P.replicas[i]) + rep_index(P, i, h.j, e0), smem_u32(st + off_wire), len * kEB,
                       sh_hint, pol);
        }
        bulk_commit();
        bulk_wait_read0();            // shared memory of this stage may be overwritten after this
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(s));
      }
    }
    bulk_wait0();
  } else {
    // =============================== compute warps ===============================
    const uint32_t idx = threadIdx.x * kEpl;   // first element of this lane within the tile
    uint32_t s = 0, par = 0;
    bool ok = true;
    float acc[kEpl];                            // AGG: running sum; DRIFT: the wire value of the tile
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
        const StageHdr& h = hdrs[s];
        const uint32_t len = h.len;
        const bool active = idx < len;
        unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
        if constexpr (PH == AGG) {
          if (g == 0) {
#pragma unroll
            for (int x = 0; x < kEpl; ++x) acc[x] = 0.0f;
          }
          const uint32_t bits = (uint32_t)(h.recv >> (g * GS)) & ((1u << GS) - 1u);
          if (active) {
#pragma unroll
            for (int u = 0; u < GS; ++u)
              if ((bits >> u) & 1u) {
                float f[kEpl];
                lds_lane<T>(st + (size_t)u * kTile * kEB, idx, f);
#pragma unroll
                for (int x = 0; x < kEpl; ++x) acc[x] = __fadd_rn(acc[x], f[x]);
              }
            if (g + 1 == G.groups) {
              divide_by_count<kEpl>(acc, h.cnt);
              if (P.ghat_prev) {
                // Algorithm 1: a dropped packet falls back to the saved aggregate, a surviving one is saved
                uint32_t pw[4];
                if (h.cnt == 0) {
                  load_words_stream<kEpl>(P.ghat_prev + h.e0 + idx, pw);
                  unpack_lane<F32>(pw, acc);
                } else {
#pragma unroll
                  for (int x = 0; x < kEpl; ++x) pw[x] = __float_as_uint(acc[x]);
                  __stcs(reinterpret_cast<uint4*>(P.ghat_prev + h.e0 + idx), make_uint4(pw[0], pw[1], pw[2], pw[3]));
                }
              }
              sts_lane_f32(st + off_tail, idx, acc);
            }
          }
        } else if constexpr (PH == STEP) {
          if (active && !((P.flags & 2u) && h.cnt == 0)) {
            float gh[kEpl], th[kEpl], m[kEpl], v[kEpl];
            lds_lane<F32>(st, idx, gh);
            lds_lane<F32>(st + off_th, idx, th);
            if constexpr (OPT == 1) {
              lds_lane<F32>(st + off_m, idx, m);
              lds_lane<F32>(st + off_v, idx, v);
            }
            optimizer_n<OPT, kEpl>(P, gh, th, m, v);
            sts_lane_f32(st + off_th, idx, th);
            if constexpr (OPT == 1) {
              sts_lane_f32(st + off_m, idx, m);
              sts_lane_f32(st + off_v, idx, v);
            }
          }
        } else if constexpr (PH == BCAST) {
          if constexpr (kEB == 2u) {
            if (active) {
              float th[kEpl];
              uint32_t ww[4];
              lds_lane<F32>(st + off_th, idx, th);
              pack_bf16_lane(th, ww);
              store_words<kEpl / 2>(st + off_wire + (size_t)idx * 2, ww);
            }
          }
        } else {
          if (g == 0) {
            // the value every copy is compared with: theta rounded to the replicas' type
            if (active) {
              lds_lane<F32>(st + off_tail, idx, acc);
              if constexpr (kEB == 2u) {
                uint32_t ww[4];
                pack_bf16_lane(acc, ww);
                unpack_lane<BF16>(ww, acc);
              }
            } else {
#pragma unroll
              for (int x = 0; x < kEpl; ++x) acc[x] = 0.0f;
            }
          }
          // squared differences of this lane's elements against each copy of the group ...
          const uint32_t in_group = min((uint32_t)GS, W - g * GS);
          const uint32_t have = (uint32_t)(h.recv >> (g * GS)) & ((1u << GS) - 1u);   // the copies that were fetched
          float sq[GS];
#pragma unroll
          for (int u = 0; u < GS; ++u) {
            sq[u] = 0.0f;
            if (active && ((have >> u) & 1u)) {
              // two elements per instruction (packed fp32 pairs of sm_100)
              float old[kEpl];
              lds_lane<T>(st + (size_t)u * kTile * kEB, idx, old);
              const float2 d0 = __fadd2_rn(make_float2(old[0], old[1]), make_float2(-acc[0], -acc[1]));
              const float2 d1 = __fadd2_rn(make_float2(old[2], old[3]), make_float2(-acc[2], -acc[3]));
              const float2 q = __ffma2_rn(d1, d1, __fmul2_rn(d0, d0));
              sq[u] = __fadd_rn(q.x, q.y);
            }
          }
          // ... summed over the warp for all GS copies at once; the lane that owns a copy's fp64
          // accumulator (lane l: replicas l and l + 32) then fetches that copy's total
          const float tot = warp_sum_multi<GS>(sq, lane);
          const uint32_t u = ((uint32_t)lane - g * GS) & 31u;      // copy of this group that this lane owns
          const float mine = __shfl_sync(0xFFFFFFFFu, tot, (int)((u * (32u / GS)) & 31u));
          if (u < in_group) {
            if (g * GS < 32u) dacc0 += (double)mine; else dacc1 += (double)mine;
          }
        }
        if constexpr (PH != DRIFT) fence_proxy_async();   // results must be visible to the bulk stores
        __syncwarp();
        if (lane == 0) mbar_arrive(done_bar(s));
      }
    }
  }

  // ---- common exit: status word; per-CTA drift partials in fixed order ----------------
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) atomicExch(G.status, 1u);
  if constexpr (PH == DRIFT) {
    double* sh = reinterpret_cast<double*>(stage0);   // stages are idle now
    if (warp < kConsumerWarps) {
      sh[warp * kMaxW + lane] = dacc0;
      sh[warp * kMaxW + lane + 32] = dacc1;
    }
    __syncthreads();
    if (threadIdx.x < kMaxW) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) t += sh[w * kMaxW + threadIdx.x];
      P.partials[((size_t)P.partials_row0 + blockIdx.x) * kMaxW + threadIdx.x] = t;
    }
    if (P.ticket) drift_last_block(P, warp, lane, kConsumerWarps + 2);
  }
}

}  // namespace lossy
