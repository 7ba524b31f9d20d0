// Fused lossy step as a bulk-copy (TMA) pipeline for sm_100a.
//
// One CTA = CW compute warps + 1 producer warp + 1 store warp (see TmaShape for the two builds).
// The bucket's full packets are cut into tiles of at most kTile contiguous elements inside one
// packet (kTile = 128 * CW), so one set of delivery masks covers a tile. Per tile and per group of
// up to GS (4 or 8) workers the producer arms an mbarrier and issues 1-D bulk copies global ->
// shared memory for the DELIVERED workers' pieces only (dropped packets are never read) and, with
// the last group, for theta / m / v. Compute warps sum the pieces in ascending worker order from shared memory,
// divide by the received count, run the optimizer in place in shared memory and write the wire
// value (fp32 or RNE bf16) once; the store warp then fans that single shared-memory tile out with
// one bulk copy per replica that receives the broadcast, plus theta / m / v. Replicas that miss
// the broadcast are not written; their old packet is read (L2-prefetched by the producer) only to
// accumulate the drift term. No cluster launch and no multicast: the path has no cross-CTA reuse.
//
// Template variants, picked per context by the host's launch policy: CW (compute warps: 16 = one CTA per
// SM with 2048-element tiles, 8 = two CTAs per SM with 1024-element tiles), GS (workers per pipeline stage, 4
// or 8), PRE (how the old copies of stale replicas are read: 0 = by the compute warps in the drift phase, 16 =
// the first ones requested before the tile's arithmetic into 16 registers per lane, 1 = as extra pipeline
// stages), PACKED (packets shorter than a tile: several whole packets per tile, masks evaluated by the
// compute warps a tile ahead) and SPLIT (theta / m / v and the wire tile in two state slots of their own, stages of
// gradient slots only).
// Drift norms are finalised by the last CTA to finish (fence + ticket counter; nothing waits on another CTA).
//
// Every wait on an mbarrier is bounded: after kMaxPolls unsuccessful polls the CTA raises a
// shared abort flag, records a code in the context's device status word and every role leaves
// its loop; the producer then gives its own copies in flight a bounded time to land.
#pragma once
#include "lossy_kernels.cuh"

namespace lossy {

constexpr int kEpl = 4;                                   // elements per compute lane
// Two geometries are built: "wide" = 16 compute warps, one CTA per SM, tiles of 2048 elements
// (best for W <= 16); "twin" = 8 compute warps, two CTAs per SM, tiles of 1024 elements (best when
// a tile takes many worker groups). Each comes with pipeline stages of 4 or of 8 workers (GS).
template <int CW> struct TmaShape {
  static constexpr int kConsumerWarps = CW;
  static constexpr int kTile = CW * 32 * kEpl;
  static constexpr int kThreads = (CW + 2) * 32;          // + producer warp + store warp
  static constexpr int kCtasPerSm = CW >= 16 ? 1 : 2;
};
constexpr int kStaleBatch = 4;                            // stale replica packets in flight per compute lane (8 measured slower)
constexpr int kMaxStages = 4;                             // deeper pipelines measured no faster
// PACKED builds: a tile's masks are evaluated one tile ahead and shared through a ring of kMaskBufs buffers.
// Per warp and iteration n the order is write(n+1), arrive(n+1), wait(n), read(n). A warp that has passed
// wait(n-1) knows that every warp has arrived for tile n-1, i.e. has entered iteration n-2 and so has finished
// read(n-3): tile n+1 may therefore reuse the buffer of tile n-3, and no earlier one. Hence four buffers (with
// two, a warp that is ahead overwrites masks a slower warp has yet to read).
constexpr uint32_t kMaskBufs = 4;
constexpr uint32_t kTmaBarBytes = 256;                   // barriers (3 per stage, 4 of the state slots, kMaskBufs of the PACKED masks; 8 B each) and the abort flag
static_assert((3 * kMaxStages + 4 + kMaskBufs) * 8 + 4 <= kTmaBarBytes, "barrier area too small");
constexpr uint32_t kMaxPolls = 1u << 22;

struct TmaGeom {
  uint32_t num_tiles;         // full packets * tiles_per_packet
  uint32_t tiles_per_packet;
  uint32_t stages;
  uint32_t stage_bytes;       // per stage, 128-byte multiple
  uint32_t state_bytes;       // SPLIT builds: one state slot (theta, m, v, wire tile), 128-byte multiple
  uint32_t groups;            // ceil(W / GS)
  uint32_t grad_slots;        // min(W, GS)
  uint32_t hints;             // bit 0: evict-first on bulk loads, bit 1: on bulk stores, bit 2 (gather pipeline): L2 prefetch of stale copies, bit 3 (gather pipeline): the gather warps split a row's chunks, not the workers
  uint32_t packets_per_tile;  // PACKED build: whole small packets per tile (2, 4 or 8), else 1
  uint32_t full_packets;      // PACKED build: complete packets of the bucket
  uint32_t rd_cap;            // gather pipeline, RD builds: 512-byte chunks per scratch buffer
  uint32_t rd_lgsplit;        // gather pipeline, wide RD builds: log2 of the parts a replica's row of a tile is cut into
  uint32_t* status;           // device status word (0 = fine)
};

// PACKED build, for packets shorter than a tile: a tile holds up to kMaxSub whole packets. The producer
// fetches every worker's piece of the tile in ONE bulk copy each (bulk copies under ~2 KB run far below the
// memory rate, and a single warp cannot evaluate eight packets' masks per tile fast enough); the masks are
// evaluated by the compute warps instead, which split a tile's sub-packets among themselves one tile ahead and
// share the result in shared memory, so dropped sub-packets are fetched but never used. A compute warp's 128
// elements lie in one sub-packet, whose masks it reads from there. The store warp writes each replica the
// runs of consecutive sub-packets whose broadcast it received.
constexpr int kMaxSub = 8;
struct __align__(16) PackedStale { uint64_t stale[kMaxSub]; uint32_t j[kMaxSub]; };   // per sub-packet: replicas not written, owner
struct __align__(16) PackedMasks { uint64_t recv[kMaxSub], stale[kMaxSub]; uint32_t j[kMaxSub]; };   // a tile's masks and owners, shared by its compute warps

struct __align__(16) StageHdr {
  uint64_t recv, stale, e0;
  uint32_t k, len, cnt, last;
  uint64_t own;          // owner-elided replicas: the bit of the replica that does not exist for this packet
  uint32_t j;            // owner of the packet
  uint32_t pad[3];
};
static_assert(sizeof(StageHdr) == 64, "header is one 64-byte slot");

// ---- PTX wrappers ---------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// `hint` = mark the lines evict-first in L2 (they are touched once per step)
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, bool hint,
                                         uint64_t pol) {
  if (hint)
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar), "l"(pol)
                 : "memory");
  else
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes, bool hint, uint64_t pol) {
  if (hint)
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(dst), "r"(src),
                 "r"(bytes), "l"(pol)
                 : "memory");
  else
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Bounded wait; false = gave up (or another role already aborted).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t max_polls = kMaxPolls) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1u;
  return false;
}

// Self-test of the failure report: one small CTA initialises a barrier that nothing ever arms or arrives on,
// waits on it with the pipelines' own bounded wait (a short poll limit, no copy in flight), and leaves through
// the pipelines' exit path: abort flag -> the context's status word.
static __global__ void wait_expiry_kernel(uint32_t max_polls, uint32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_word;
  volatile uint32_t* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  mbar_wait(smem_u32(&bar), 0u, abort_flag, max_polls);   // phase 0 never completes
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) atomicExch(status, 1u);
}

// kEpl consecutive elements of one lane, to and from shared or global memory
template <class T>
__device__ __forceinline__ void unpack_lane(const uint32_t (&w)[4], float (&f)[kEpl]) {
  if constexpr (T::kVecs == 2) {
#pragma unroll
    for (int x = 0; x < kEpl; ++x) f[x] = __uint_as_float(w[x]);
  } else {
#pragma unroll
    for (int x = 0; x < kEpl / 2; ++x) {
      f[2 * x] = __uint_as_float(w[x] << 16);
      f[2 * x + 1] = __uint_as_float(w[x] & 0xFFFF0000u);
    }
  }
}
// words of kEpl elements: fp32 -> kEpl words, bf16 -> kEpl/2 words
template <class T> struct LaneWords { static constexpr int value = T::kVecs == 2 ? kEpl : kEpl / 2; };

template <int WORDS>
__device__ __forceinline__ void load_words(const void* p, uint32_t (&w)[4]) {
  if constexpr (WORDS == 4) {
    const uint4 r = *reinterpret_cast<const uint4*>(p); w[0] = r.x; w[1] = r.y; w[2] = r.z; w[3] = r.w;
  } else if constexpr (WORDS == 2) {
    const uint2 r = *reinterpret_cast<const uint2*>(p); w[0] = r.x; w[1] = r.y;
  } else {
    w[0] = *reinterpret_cast<const uint32_t*>(p);
  }
}
template <int WORDS>
__device__ __forceinline__ void load_words_stream(const void* p, uint32_t (&w)[4]) {
  if constexpr (WORDS == 4) {
    const uint4 r = __ldcs(reinterpret_cast<const uint4*>(p)); w[0] = r.x; w[1] = r.y; w[2] = r.z; w[3] = r.w;
  } else if constexpr (WORDS == 2) {
    const uint2 r = __ldcs(reinterpret_cast<const uint2*>(p)); w[0] = r.x; w[1] = r.y;
  } else {
    w[0] = __ldcs(reinterpret_cast<const uint32_t*>(p));
  }
}
template <int WORDS>
__device__ __forceinline__ void store_words(void* p, const uint32_t (&w)[4]) {
  if constexpr (WORDS == 4) *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  else if constexpr (WORDS == 2) *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
  else *reinterpret_cast<uint32_t*>(p) = w[0];
}
template <class T>
__device__ __forceinline__ void lds_lane(const unsigned char* base, uint32_t idx, float (&f)[kEpl]) {
  uint32_t w[4];
  load_words<LaneWords<T>::value>(base + (size_t)idx * sizeof(typename T::raw), w);
  unpack_lane<T>(w, f);
}
__device__ __forceinline__ void sts_lane_f32(unsigned char* base, uint32_t idx, const float (&f)[kEpl]) {
  uint32_t w[4];
#pragma unroll
  for (int x = 0; x < kEpl; ++x) w[x] = __float_as_uint(f[x]);
  store_words<kEpl>(base + (size_t)idx * 4, w);
}
__device__ __forceinline__ void pack_bf16_lane(const float (&f)[kEpl], uint32_t (&w)[4]) {
#pragma unroll
  for (int x = 0; x < kEpl / 2; ++x) {
    __nv_bfloat162 a = __floats2bfloat162_rn(f[2 * x], f[2 * x + 1]);
    w[x] = *reinterpret_cast<uint32_t*>(&a);
  }
}

// PRE = 32-bit registers per lane that hold stale replica data requested EARLY (before the tile's
// arithmetic) so that its latency is hidden; 0 = every stale copy is fetched in the drift phase. The early
// variant gains 8-10 % when a tile has several stale replicas (W >= 16 at p = 0.3) and costs 1-6 % when
// it has about one or none, so both are built and the launch policy picks.
// PRE = 1 selects another way altogether: the old copies of the replicas that miss a tile's broadcast come
// through the pipeline as extra stages after the tile's last gradient group (up to GS copies per stage, in
// the gradient slots), so the compute warps never wait on a global load. It needs replica elements no
// larger than gradient elements and wins when a tile has many stale replicas.
// SPLIT: theta / m / v and the wire tile live in a ring of two state slots with barriers of their own
// instead of in every stage, so that a stage is gradient slots only and more of them fit (a tile of W > 8
// workers takes several stages, of which only the last needs the state).
template <class GT, class RT, int OPT, bool DRIFTK, int CW, int GS, int PRE, bool PACKED = false, bool SPLIT = false>
__global__ void __launch_bounds__(TmaShape<CW>::kThreads, TmaShape<CW>::kCtasPerSm)
    lossy_fused_tma_kernel(const __grid_constant__ Params P, const __grid_constant__ TmaGeom G) {
  constexpr int kConsumerWarps = CW;
  constexpr int kGroup = GS;                // workers whose pieces share one pipeline stage
  constexpr int kTile = TmaShape<CW>::kTile;
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr uint32_t kGB = sizeof(typename GT::raw), kRB = sizeof(typename RT::raw);
  constexpr bool kStaleStages = DRIFTK && PRE == 1 && !PACKED;   // stale copies arrive as pipeline stages
  static_assert(!(SPLIT && PACKED), "the PACKED builds keep the state in the stage");
  static_assert(!kStaleStages || (sizeof(typename RT::raw) <= sizeof(typename GT::raw) && GS == 8), "stale stages reuse the gradient slots");
  // layout: [full, done, empty barriers | abort flag] (kTmaBarBytes) | headers (kMaxStages x 64 B) |
  //         stale masks and owners per sub-packet of the PACKED build (one per stage) | the ring of tile masks of
  //         the PACKED build (kMaskBufs) | stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kTmaBarBytes - 4);
  StageHdr* hdrs = reinterpret_cast<StageHdr*>(smem + kTmaBarBytes);
  PackedStale* pks = reinterpret_cast<PackedStale*>(smem + kTmaBarBytes + kMaxStages * sizeof(StageHdr));
  PackedMasks* tmasks = reinterpret_cast<PackedMasks*>(smem + kTmaBarBytes + kMaxStages * (sizeof(StageHdr) + sizeof(PackedStale)));   // [kMaskBufs]
  unsigned char* stage0 = smem + kTmaBarBytes + kMaxStages * (sizeof(StageHdr) + sizeof(PackedStale)) + kMaskBufs * sizeof(PackedMasks);
  const uint32_t S = G.stages;
  // SPLIT builds: two state slots behind the stages
  unsigned char* state0 = stage0 + (size_t)S * G.stage_bytes;
  // stale-stage builds: fp64 drift sums per compute warp and replica, behind everything else
  double* warp_acc = reinterpret_cast<double*>(state0 + (SPLIT ? 2u * G.state_bytes : 0u));
  const uint32_t off_th = SPLIT ? 0u : G.grad_slots * kTile * kGB;   // within the stage, or within the state slot
  const uint32_t off_m = off_th + kTile * 4, off_v = off_m + kTile * 4, off_wire = off_v + kTile * 4;

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t W = P.W;
  auto full_bar = [&](uint32_t s) { return smem_u32(&bars[s]); };
  auto done_bar = [&](uint32_t s) { return smem_u32(&bars[kMaxStages + s]); };
  auto empty_bar = [&](uint32_t s) { return smem_u32(&bars[2 * kMaxStages + s]); };
  auto sfull_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kMaxStages + q]); };        // SPLIT: state slot loaded
  auto sempty_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kMaxStages + 2 + q]); };   // SPLIT: state slot stored
  auto mask_bar = [&](uint32_t q) { return smem_u32(&bars[3 * kMaxStages + 4 + q]); };     // PACKED: a tile's masks are written

  if constexpr (kStaleStages) {
    for (uint32_t q = threadIdx.x; q < (uint32_t)kConsumerWarps * kMaxW; q += blockDim.x) warp_acc[q] = 0.0;
  }
  if (threadIdx.x == 0) {
    *abort_flag = 0u;
    for (uint32_t s = 0; s < S; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(done_bar(s), kConsumerWarps);
      mbar_init(empty_bar(s), 1);
    }
    if constexpr (SPLIT) {
      for (uint32_t q = 0; q < 2; ++q) {
        mbar_init(sfull_bar(q), 1);
        mbar_init(sempty_bar(q), 1);
      }
    }
    if constexpr (PACKED) {
      for (uint32_t q = 0; q < kMaskBufs; ++q) mbar_init(mask_bar(q), kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();

  double dacc0 = 0.0, dacc1 = 0.0;   // compute warps: lane l holds replicas l and l + 32

  if (warp == kConsumerWarps) {
    // =============================== producer warp ===============================
    uint32_t s = 0, par = 0, armed_mask = 0, armed_par = 0;
    uint32_t sq = 0, spar = 0, sarmed_mask = 0, sarmed_par = 0;   // SPLIT: state slot ring
    bool ok = true;
    const bool lh = G.hints & 1u;
    const uint64_t pol = policy_evict_first();
    if constexpr (PACKED) {
      // no masks here: every worker's piece of the tile is fetched, the compute warps decide what counts
      for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
        const uint32_t kfirst = tile * G.packets_per_tile;
        const uint32_t npk = min(G.packets_per_tile, G.full_packets - kfirst);
        const uint64_t e0 = (uint64_t)kfirst * P.P;
        const uint32_t len = npk * P.P;
        if constexpr (kDevCheck) {   // debug build: every sub-packet's range, in the slab and in every replica
          bool fine = true;
          for (uint32_t sp = 0; sp < npk; ++sp)
            fine = tile_ok(P, kfirst + sp, (P.k0 + kfirst + sp) / P.pps, e0 + (uint64_t)sp * P.P, P.P, kSiteFusedPacked, lane) && fine;
          if (!fine) { *abort_flag = 1u; ok = false; break; }
        }
        for (uint32_t g = 0; g < G.groups; ++g) {
          if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag)) { ok = false; break; }
          const bool last = g + 1 == G.groups;
          const uint32_t in_group = min((uint32_t)kGroup, W - g * kGroup);
          unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
          if (lane == 0) {
            StageHdr& h = hdrs[s];
            h.recv = 0; h.stale = 0; h.e0 = e0; h.k = npk; h.len = len; h.cnt = 0; h.last = last ? 1u : 0u; h.own = 0; h.j = 0;
            uint32_t bytes = in_group * len * kGB;
            if (last) bytes += (OPT == 1 ? 3u : 1u) * len * 4u;
            mbar_arrive_expect_tx(full_bar(s), bytes);
          }
          __syncwarp();
          if ((uint32_t)lane < in_group)
            bulk_g2s(smem_u32(st + (size_t)lane * kTile * kGB),
                     reinterpret_cast<const typename GT::raw*>(P.grads[g * kGroup + lane]) + e0, len * kGB, full_bar(s), lh, pol);
          if (last) {
            if (lane == 8) bulk_g2s(smem_u32(st + off_th), P.master + e0, len * 4u, full_bar(s), lh, pol);
            if constexpr (OPT == 1) {
              if (lane == 9) bulk_g2s(smem_u32(st + off_m), P.m + e0, len * 4u, full_bar(s), lh, pol);
              if (lane == 10) bulk_g2s(smem_u32(st + off_v), P.v + e0, len * 4u, full_bar(s), lh, pol);
            }
          }
          armed_mask |= 1u << s;
          armed_par = (armed_par & ~(1u << s)) | (par << s);
          if (++s == S) { s = 0; par ^= 1u; }
        }
      }
    } else {
      // The delivery draws are taken for a batch of tiles per ballot where the lanes allow it (W <= 16, not
      // Algorithm 1): one warp hashing one packet at a time is a chain of dependent instructions that would
      // bound the CTA when a tile carries few bytes.
      uint32_t Wp = 32;
      if (W <= 16 && !P.ghat_prev) { Wp = 1; while (Wp < W) Wp <<= 1; }
      const uint32_t lgWp = 31u - (uint32_t)__clz((int)Wp);
      const uint32_t B = 32u >> lgWp;                                // tiles per batch
      const uint32_t wmask = Wp == 32 ? 0xFFFFFFFFu : ((1u << Wp) - 1u);
      for (uint32_t tile0 = blockIdx.x; ok && tile0 < G.num_tiles; tile0 += B * gridDim.x) {
        const uint32_t b_l = (uint32_t)lane >> lgWp, i_l = (uint32_t)lane & (Wp - 1u);
        const uint32_t tile_l = tile0 + b_l * gridDim.x;
        const bool tv = tile_l < G.num_tiles;
        const uint32_t k_l = tv ? tile_l / G.tiles_per_packet : 0u;
        const uint32_t c_l = tv ? tile_l - k_l * G.tiles_per_packet : 0u;
        const uint32_t j_l = (P.k0 + k_l) / P.pps;
        BatchDraws draws = {0u, 0u, 0u};
        if (B > 1) draws = batch_draws<AGG | BCAST>(P, k_l, j_l, i_l, tv && i_l < W);
        for (uint32_t b = 0; ok && b < B; ++b) {
          const uint32_t tile = tile0 + b * gridDim.x;
          if (tile >= G.num_tiles) break;
          const int src = (int)(b * Wp);
          const uint32_t k = __shfl_sync(0xFFFFFFFFu, k_l, src);
          const uint32_t c = __shfl_sync(0xFFFFFFFFu, c_l, src);
          const uint32_t j = __shfl_sync(0xFFFFFFFFu, j_l, src);
          const uint64_t e0 = (uint64_t)k * P.P + (uint64_t)c * kTile;
          const uint32_t len = min((uint32_t)kTile, P.P - c * kTile);
          if (!tile_ok(P, k, j, e0, len, kSiteFused, lane)) { *abort_flag = 1u; ok = false; break; }   // debug build only
          uint64_t recv = 0, stale = 0, gbad = 0, pbad = 0;
          if (B > 1) batch_masks<AGG | BCAST>(P, draws, k, src, wmask, recv, stale, gbad, pbad);
          else packet_masks<AGG | BCAST>(P, k, j, lane, recv, stale, gbad, pbad);
          const uint32_t cnt = __popcll(recv);
          if (c == 0 && lane == 0) {
            if (P.count) P.count[k] = (uint8_t)cnt;
            if (P.recv_bits) P.recv_bits[k] = recv;
            if (P.stale_bits) P.stale_bits[k] = stale;
            if (P.burst_out) {   // bursty loss: the packet's first tile stores its links' new states
              P.burst_out[k] = gbad;
              P.burst_out[(size_t)P.K + k] = pbad;
            }
          }
          if constexpr (DRIFTK && !kStaleStages) {
            for (uint32_t i = lane; i < W; i += 32)
              if ((stale >> i) & 1ull)
                bulk_prefetch_l2(reinterpret_cast<const typename RT::raw*>(P.replicas[i]) + rep_index(P, i, j, e0), len * kRB);
          }
          if (P.ghat_prev && cnt == 0 && lane == 0) bulk_prefetch_l2(P.ghat_prev + e0, len * 4u);   // Algorithm 1 fallback
          if constexpr (SPLIT) {
            // the tile's theta / m / v go to state slot sq, ahead of its gradient groups
            if (!mbar_wait(sempty_bar(sq), spar ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sb = state0 + (size_t)sq * G.state_bytes;
            if (lane == 0) mbar_arrive_expect_tx(sfull_bar(sq), (OPT == 1 ? 3u : 1u) * len * 4u);
            __syncwarp();
            if (lane == 8) bulk_g2s(smem_u32(sb + off_th), P.master + e0, len * 4u, sfull_bar(sq), lh, pol);
            if constexpr (OPT == 1) {
              if (lane == 9) bulk_g2s(smem_u32(sb + off_m), P.m + e0, len * 4u, sfull_bar(sq), lh, pol);
              if (lane == 10) bulk_g2s(smem_u32(sb + off_v), P.v + e0, len * 4u, sfull_bar(sq), lh, pol);
            }
            sarmed_mask |= 1u << sq;
            sarmed_par = (sarmed_par & ~(1u << sq)) | (spar << sq);
            if (++sq == 2u) { sq = 0; spar ^= 1u; }
          }
          for (uint32_t g = 0; g < G.groups; ++g) {
            if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag)) { ok = false; break; }
            const bool last = !SPLIT && g + 1 == G.groups;   // the stage that also carries the state
            const uint32_t bits = (uint32_t)(recv >> (g * kGroup)) & ((1u << kGroup) - 1u);
            unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
            if (lane == 0) {
              StageHdr& h = hdrs[s];
              h.recv = recv; h.stale = stale; h.e0 = e0; h.k = k; h.len = len; h.cnt = cnt; h.last = g + 1 == G.groups ? 1u : 0u;
              h.own = own_bit(P, j); h.j = j;
              uint32_t bytes = __popc(bits) * len * kGB;
              if (last) bytes += (OPT == 1 ? 3u : 1u) * len * 4u;
              mbar_arrive_expect_tx(full_bar(s), bytes);
            }
            __syncwarp();
            if (lane < kGroup && ((bits >> lane) & 1u))
              bulk_g2s(smem_u32(st + (size_t)lane * kTile * kGB),
                       reinterpret_cast<const typename GT::raw*>(P.grads[g * kGroup + lane]) + e0, len * kGB, full_bar(s), lh, pol);
            if (last) {
              if (lane == 8) bulk_g2s(smem_u32(st + off_th), P.master + e0, len * 4u, full_bar(s), lh, pol);
              if constexpr (OPT == 1) {
                if (lane == 9) bulk_g2s(smem_u32(st + off_m), P.m + e0, len * 4u, full_bar(s), lh, pol);
                if (lane == 10) bulk_g2s(smem_u32(st + off_v), P.v + e0, len * 4u, full_bar(s), lh, pol);
              }
            }
            armed_mask |= 1u << s;
            armed_par = (armed_par & ~(1u << s)) | (par << s);
            if (++s == S) { s = 0; par ^= 1u; }
          }
          if constexpr (kStaleStages) {
            // the old copies of the replicas that miss this broadcast, up to kGroup per extra stage; lane u
            // fetches the u-th of them into gradient slot u
            uint64_t sm = stale;
            while (ok && sm) {
              if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag)) { ok = false; break; }
              uint64_t ids = 0;
              int mine = -1;
#pragma unroll
              for (int u = 0; u < kGroup; ++u)
                if (sm) {
                  const int i = __ffsll((long long)sm) - 1;
                  sm &= sm - 1;
                  ids |= 1ull << i;
                  if (lane == u) mine = i;
                }
              unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
              if (lane == 0) {
                StageHdr& h = hdrs[s];
                h.recv = ids; h.stale = 0; h.e0 = e0; h.k = k; h.len = len; h.cnt = (uint32_t)__popcll(ids); h.last = 2u; h.own = 0; h.j = j;
                mbar_arrive_expect_tx(full_bar(s), (uint32_t)__popcll(ids) * len * kRB);
              }
              __syncwarp();
              if (mine >= 0)
                bulk_g2s(smem_u32(st + (size_t)lane * kTile * kGB),
                         reinterpret_cast<const typename RT::raw*>(P.replicas[mine]) + rep_index(P, (uint32_t)mine, j, e0), len * kRB,
                         full_bar(s), lh, pol);
              armed_mask |= 1u << s;
              armed_par = (armed_par & ~(1u << s)) | (par << s);
              if (++s == S) { s = 0; par ^= 1u; }
            }
          }
        }
      }
    }
    if (!ok || *abort_flag) {
      // give this CTA's copies in flight a bounded time to land before the CTA exits
      for (uint32_t q = 0; q < S; ++q)
        if ((armed_mask >> q) & 1u)
          for (uint32_t i = 0; i < (1u << 16); ++i)
            if (mbar_try_wait(full_bar(q), (armed_par >> q) & 1u)) break;
      if constexpr (SPLIT) {
        for (uint32_t q = 0; q < 2; ++q)
          if ((sarmed_mask >> q) & 1u)
            for (uint32_t i = 0; i < (1u << 16); ++i)
              if (mbar_try_wait(sfull_bar(q), (sarmed_par >> q) & 1u)) break;
      }
    }
  } else if (warp == kConsumerWarps + 1) {
    // ================================ store warp =================================
    uint32_t s = 0, par = 0, sq = 0;
    bool ok = true;
    const bool sh_hint = G.hints & 2u;
    const uint64_t pol = policy_evict_first();
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(done_bar(s), par, abort_flag)) { ok = false; break; }
        if (g + 1 == G.groups) {
          const StageHdr& h = hdrs[s];
          const uint64_t e0 = h.e0, stale = h.stale;
          const uint64_t keep = stale | h.own;     // replicas that are not written: they missed the broadcast, or do not exist
          const uint32_t len = h.len;
          unsigned char* st = SPLIT ? state0 + (size_t)sq * G.state_bytes : stage0 + (size_t)s * G.stage_bytes;
          if (lane == 0) bulk_s2g(P.master + e0, smem_u32(st + off_th), len * 4u, sh_hint, pol);
          if constexpr (OPT == 1) {
            if (lane == 1) bulk_s2g(P.m + e0, smem_u32(st + off_m), len * 4u, sh_hint, pol);
            if (lane == 2) bulk_s2g(P.v + e0, smem_u32(st + off_v), len * 4u, sh_hint, pol);
          }
          if constexpr (PACKED) {
            // replica i takes every run of consecutive sub-packets whose broadcast it received
            const uint32_t npk = h.k;
            for (uint32_t i = lane; i < W; i += 32) {
              int run = -1;
              for (uint32_t sp = 0; sp <= npk; ++sp) {
                const bool fresh = sp < npk && !((pks[s].stale[sp < npk ? sp : 0] >> i) & 1ull);
                if (fresh && run < 0) run = (int)sp;
                if (!fresh && run >= 0) {
                  // (with owner-elided replicas a run never holds a packet of worker i's own shard, so one
                  // index shift serves the whole run)
                  bulk_s2g(reinterpret_cast<typename RT::raw*>(P.replicas[i]) +
                               rep_index(P, i, pks[s].j[run], e0 + (uint64_t)run * P.P),
                           smem_u32(st + off_wire + (size_t)run * P.P * kRB), (sp - (uint32_t)run) * P.P * kRB, sh_hint, pol);
                  run = -1;
                }
              }
            }
          } else {
            for (uint32_t i = lane; i < W; i += 32)
              if (!((keep >> i) & 1ull))
                bulk_s2g(reinterpret_cast<typename RT::raw*>(P.replicas[i]) + rep_index(P, i, h.j, e0), smem_u32(st + off_wire), len * kRB,
                         sh_hint, pol);
          }
          bulk_commit();
          bulk_wait_read0();          // shared memory of this stage may be overwritten after this
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_bar(s));
          if constexpr (SPLIT) {
            if (lane == 0) mbar_arrive(sempty_bar(sq));
            sq ^= 1u;
          }
          if constexpr (kStaleStages) {
            // the tile's stale stages carry nothing to store: hand each back once the compute warps are done
            for (uint32_t n = ((uint32_t)__popcll(stale) + kGroup - 1) / kGroup; ok && n > 0; --n) {
              next_stage();
              if (!mbar_wait(done_bar(s), par, abort_flag)) { ok = false; break; }
              __syncwarp();
              if (lane == 0) mbar_arrive(empty_bar(s));
            }
          }
          continue;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar(s));
      }
    }
    bulk_wait0();
  } else {
    // =============================== compute warps ===============================
    const uint32_t idx = threadIdx.x * kEpl;   // first element of this lane within the tile
    uint32_t s = 0, par = 0, sq = 0, spar = 0;
    bool ok = true;
    float acc[kEpl];
    auto next_stage = [&]() { if (++s == S) { s = 0; par ^= 1u; } };
    // PACKED: this warp's 128 elements lie in one sub-packet of the tile, always the same one
    const uint32_t my_sp = PACKED ? min((uint32_t)(threadIdx.x & ~31) * kEpl / P.P, (uint32_t)kMaxSub - 1u) : 0u;
    uint32_t mbuf = 0, mpar = 0;                 // PACKED: buffer and phase of the shared tile masks
    uint32_t pk_Wp = 32;
    const bool pk_batched = PACKED && W <= 32 && !P.ghat_prev;
    if (pk_batched) { pk_Wp = 1; while (pk_Wp < W) pk_Wp <<= 1; }
    const uint32_t pk_lgWp = 31u - (uint32_t)__clz((int)pk_Wp);
    // sub-packets per pass of draws: at most two, so that the work spreads over several warps instead of
    // lengthening one warp's tile (with W <= 4 a single pass could cover all eight, and did so at a loss)
    const uint32_t pk_Bp = min(32u >> pk_lgWp, 2u);
    const uint32_t pk_wmask = pk_Wp == 32 ? 0xFFFFFFFFu : ((1u << pk_Wp) - 1u);
    // PACKED: a tile's masks are evaluated once, one tile ahead, and shared through the ring of kMaskBufs
    // buffers (see there for why a warp that is ahead never overwrites masks still to be read): with W <= 32
    // (not Algorithm 1) warp w
    // takes the w-th batch of 32 / Wp sub-packets in one pass of draws; otherwise the first warp of each
    // sub-packet takes its own. Every compute warp arrives on the buffer's barrier once per tile.
    auto eval_masks = [&](uint32_t tile, uint32_t buf) {
      const uint32_t kfirst = tile * G.packets_per_tile;
      const uint32_t npk = min(G.packets_per_tile, G.full_packets - kfirst);
      const uint32_t widx = (uint32_t)(threadIdx.x & ~31) * kEpl;
      PackedMasks& tm = tmasks[buf];
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
      if (pk_batched) {
        const uint32_t q0 = (uint32_t)warp * pk_Bp;
        if (q0 < npk) {
          const uint32_t sp_l = q0 + ((uint32_t)lane >> pk_lgWp), i_l = (uint32_t)lane & (pk_Wp - 1u);
          const uint32_t k_l = kfirst + (sp_l < npk ? sp_l : 0u);
          const uint32_t j_l = (P.k0 + k_l) / P.pps;
          const BatchDraws d = batch_draws<AGG | BCAST>(P, k_l, j_l, i_l, sp_l < npk && i_l < W);
          for (uint32_t x = 0; x < pk_Bp && q0 + x < npk; ++x) {
            uint64_t r, st, gbad, pbad;
            batch_masks<AGG | BCAST>(P, d, kfirst + q0 + x, (int)(x * pk_Wp), pk_wmask, r, st, gbad, pbad);
            const uint32_t j_x = __shfl_sync(0xFFFFFFFFu, j_l, (int)(x * pk_Wp));   // the owner of sub-packet q0 + x
            if ((uint32_t)lane == x) report(q0 + x, j_x, r, st, gbad, pbad);
          }
        }
      } else if (widx < npk * P.P && widx == my_sp * P.P) {
        uint64_t r, st, gbad, pbad;
        const uint32_t j_sp = (P.k0 + kfirst + my_sp) / P.pps;
        packet_masks<AGG | BCAST>(P, kfirst + my_sp, j_sp, lane, r, st, gbad, pbad);
        if (lane == 0) report(my_sp, j_sp, r, st, gbad, pbad);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(mask_bar(buf));
    };
    if constexpr (PACKED) {
      if (blockIdx.x < G.num_tiles) eval_masks(blockIdx.x, 0u);
    }
    for (uint32_t tile = blockIdx.x; ok && tile < G.num_tiles; tile += gridDim.x) {
      uint64_t my_recv = 0, my_stale = 0;
      uint32_t my_j = 0;                 // PACKED: the owner of the packet this warp's elements lie in
      bool my_first = false;
      if constexpr (PACKED) {
        const uint32_t kfirst = tile * G.packets_per_tile;
        const uint32_t npk = min(G.packets_per_tile, G.full_packets - kfirst);
        const uint32_t widx = (uint32_t)(threadIdx.x & ~31) * kEpl;
        // the next tile's masks first (their latency hides behind the wait for this tile's), into the buffer
        // three behind this tile's
        if (tile + gridDim.x < G.num_tiles) eval_masks(tile + gridDim.x, (mbuf + 1u) & (kMaskBufs - 1u));
        if (!mbar_wait(mask_bar(mbuf), mpar, abort_flag)) { ok = false; break; }
        if (widx < npk * P.P) {
          my_first = widx == my_sp * P.P;
          my_recv = tmasks[mbuf].recv[my_sp];
          my_stale = tmasks[mbuf].stale[my_sp];
          my_j = tmasks[mbuf].j[my_sp];
          if constexpr (DRIFTK) {   // the old copies this warp will compare against: start them toward L2 right away
            uint64_t sm = my_stale;
            while (sm) {
              const int i = __ffsll((long long)sm) - 1;
              sm &= sm - 1;
              prefetch_l2(reinterpret_cast<const typename RT::raw*>(P.replicas[i]) +
                          rep_index(P, (uint32_t)i, my_j, (uint64_t)kfirst * P.P + idx));
            }
          }
        }
        if (++mbuf == kMaskBufs) { mbuf = 0; mpar ^= 1u; }
      }
      for (uint32_t g = 0; g < G.groups; ++g, next_stage()) {
        if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
        const StageHdr& h = hdrs[s];
        const uint64_t recv = PACKED ? my_recv : h.recv;
        const uint32_t len = h.len;
        const bool active = idx < len;
        unsigned char* st = stage0 + (size_t)s * G.stage_bytes;
        if (g == 0) {
#pragma unroll
          for (int x = 0; x < kEpl; ++x) acc[x] = 0.0f;
        }
        const uint32_t bits = (uint32_t)(recv >> (g * kGroup)) & ((1u << kGroup) - 1u);
        if (active) {
#pragma unroll
          for (int u = 0; u < kGroup; ++u)
            if ((bits >> u) & 1u) {
              float f[kEpl];
              lds_lane<GT>(st + (size_t)u * kTile * kGB, idx, f);
#pragma unroll
              for (int x = 0; x < kEpl; ++x) acc[x] = __fadd_rn(acc[x], f[x]);
            }
        }
        if (g + 1 < G.groups) {
          __syncwarp();
          if (lane == 0) mbar_arrive(done_bar(s));
          continue;
        }
        // ---- last group of the tile: estimate, update, wire value -----------------
        unsigned char* sb = st;       // where theta / m / v and the wire tile live
        if constexpr (SPLIT) {
          if (!mbar_wait(sfull_bar(sq), spar, abort_flag)) { ok = false; break; }
          sb = state0 + (size_t)sq * G.state_bytes;
          if (++sq == 2u) { sq = 0; spar ^= 1u; }
        }
        const uint32_t cnt = PACKED ? (uint32_t)__popcll(my_recv) : h.cnt;
        const uint64_t stale = PACKED ? my_stale : h.stale, e0 = h.e0;
        const uint32_t jj = PACKED ? my_j : h.j;      // the owner of the packet of this lane's elements
        if constexpr (PACKED) {
          // for the store warp, before this warp's arrive: the replicas that do not take this sub-packet
          if (my_first && lane == 0) {
            pks[s].stale[my_sp] = my_stale | own_bit(P, my_j);
            pks[s].j[my_sp] = my_j;
          }
        }
        float wire[kEpl];
        // The first stale copies are requested now, so that their (L2) latency hides behind the arithmetic
        // below; they are used in the drift phase after this warp has handed the stage to the store warp.
        constexpr int kPre = kStaleStages ? 0 : PRE / LaneWords<RT>::value;   // PRE = 16: 8 bf16 or 4 fp32 copies
        uint32_t pre_raw[kPre > 0 ? kPre : 1][4];
        int pre_id[kPre > 0 ? kPre : 1];
        uint64_t stale_rest = stale;
        if constexpr (DRIFTK) {
#pragma unroll
          for (int b = 0; b < kPre; ++b) {
            pre_id[b] = -1;
            if (stale_rest) {
              pre_id[b] = __ffsll((long long)stale_rest) - 1;
              stale_rest &= stale_rest - 1;
              if (active)
                load_words_stream<LaneWords<RT>::value>(
                    reinterpret_cast<const typename RT::raw*>(P.replicas[pre_id[b]]) + rep_index(P, (uint32_t)pre_id[b], jj, e0 + idx),
                    pre_raw[b]);
            }
          }
        }
        if (active) {
          divide_by_count<kEpl>(acc, cnt);
          if (P.ghat_prev) {
            // Algorithm 1: a dropped packet falls back to the saved aggregate, a surviving one is saved
            uint32_t pw[4];
            if (cnt == 0) {
              load_words_stream<kEpl>(P.ghat_prev + e0 + idx, pw);
              unpack_lane<F32>(pw, acc);
            } else {
#pragma unroll
              for (int x = 0; x < kEpl; ++x) pw[x] = __float_as_uint(acc[x]);
              __stcs(reinterpret_cast<uint4*>(P.ghat_prev + e0 + idx), make_uint4(pw[0], pw[1], pw[2], pw[3]));
            }
          }
          if (P.ghat) {
            uint32_t gw[4];
#pragma unroll
            for (int x = 0; x < kEpl; ++x) gw[x] = __float_as_uint(acc[x]);
            store_words<kEpl>(P.ghat + e0 + idx, gw);
          }
          float th[kEpl], m[kEpl], v[kEpl];
          lds_lane<F32>(sb + off_th, idx, th);
          if (!((P.flags & 2u) && cnt == 0)) {
            if constexpr (OPT == 1) {
              lds_lane<F32>(sb + off_m, idx, m);
              lds_lane<F32>(sb + off_v, idx, v);
            }
#pragma unroll
            for (int x = 0; x < kEpl; ++x) {
              if constexpr (OPT == 0) {
                th[x] = __fsub_rn(th[x], __fmul_rn(P.lr, acc[x]));
              } else {
                const float mn = __fadd_rn(__fmul_rn(P.b1, m[x]), __fmul_rn(P.omb1, acc[x]));
                const float vn = __fadd_rn(__fmul_rn(P.b2, v[x]), __fmul_rn(__fmul_rn(P.omb2, acc[x]), acc[x]));
                const float mh = __fmul_rn(mn, P.ibc1);
                const float vh = __fmul_rn(vn, P.ibc2);
                const float den = __fadd_rn(__fsqrt_rn(vh), P.eps);
                th[x] = __fsub_rn(th[x], __fdiv_rn(__fmul_rn(P.lr, mh), den));
                m[x] = mn;
                v[x] = vn;
              }
            }
            sts_lane_f32(sb + off_th, idx, th);
            if constexpr (OPT == 1) {
              sts_lane_f32(sb + off_m, idx, m);
              sts_lane_f32(sb + off_v, idx, v);
            }
          }
          if constexpr (RT::kVecs == 2) {
            sts_lane_f32(sb + off_wire, idx, th);
#pragma unroll
            for (int x = 0; x < kEpl; ++x) wire[x] = th[x];
          } else {
            uint32_t ww[4];
            pack_bf16_lane(th, ww);
            store_words<kEpl / 2>(sb + off_wire + (size_t)idx * 2, ww);
            unpack_lane<BF16>(ww, wire);
          }
        } else {
#pragma unroll
          for (int x = 0; x < kEpl; ++x) wire[x] = 0.0f;
        }
        fence_proxy_async();          // make the shared-memory results visible to the bulk stores
        __syncwarp();
        if (lane == 0) mbar_arrive(done_bar(s));

        // ---- drift of the replicas that missed this broadcast ---------------------
        if constexpr (kStaleStages) {
          // their old copies follow as stages of up to kGroup copies in the gradient slots
          uint64_t sm = stale;
          while (sm) {
            next_stage();
            if (!mbar_wait(full_bar(s), par, abort_flag)) { ok = false; break; }
            const uint64_t ids = hdrs[s].recv;
            const unsigned char* sst = stage0 + (size_t)s * G.stage_bytes;
            const uint32_t n_in = (uint32_t)__popcll(ids);
            float sq[kGroup];
#pragma unroll
            for (int u = 0; u < kGroup; ++u) {
              sq[u] = 0.0f;
              if (active && (uint32_t)u < n_in) {
                float old[kEpl];
                lds_lane<RT>(sst + (size_t)u * kTile * kGB, idx, old);
#pragma unroll
                for (int x = 0; x < kEpl; ++x) {
                  const float d = __fsub_rn(old[x], wire[x]);
                  sq[u] = __fadd_rn(sq[u], __fmul_rn(d, d));
                }
              }
            }
            // all copies' warp totals at once; the first lane of segment u adds copy u's total to this warp's
            // fp64 sum of that replica
            const float tot = warp_sum_multi<kGroup>(sq, lane);
            const uint32_t u = (uint32_t)lane / (32u / kGroup);
            if ((lane & (32 / kGroup - 1)) == 0 && u < n_in) {
              uint64_t t = ids;
              for (uint32_t q = 0; q < u; ++q) t &= t - 1;
              warp_acc[warp * kMaxW + (__ffsll((long long)t) - 1)] += (double)tot;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(done_bar(s));
            sm &= ~ids;
          }
          if (!ok) break;
        } else if constexpr (DRIFTK) {
#pragma unroll
          for (int b = 0; b < kPre; ++b) {
            if (pre_id[b] >= 0) {
              float old[kEpl];
              if (active) {
                unpack_lane<RT>(pre_raw[b], old);
              } else {
#pragma unroll
                for (int x = 0; x < kEpl; ++x) old[x] = 0.0f;
              }
              float sq = 0.0f;
#pragma unroll
              for (int x = 0; x < kEpl; ++x) {
                const float d = __fsub_rn(old[x], wire[x]);
                sq = __fadd_rn(sq, __fmul_rn(d, d));
              }
              const float tot = warp_sum(sq);
              if ((pre_id[b] & 31) == lane) {
                if (pre_id[b] < 32) dacc0 += (double)tot; else dacc1 += (double)tot;
              }
            }
          }
          uint64_t sm = stale_rest;   // more stale copies than were requested early
          while (sm) {
            // up to kStaleBatch stale copies are fetched before the first is used
            int ids[kStaleBatch];
            float old[kStaleBatch][kEpl];
            int nb = 0;
#pragma unroll
            for (int b = 0; b < kStaleBatch; ++b) {
              ids[b] = -1;
              if (sm) {
                ids[b] = __ffsll((long long)sm) - 1;
                sm &= sm - 1;
                nb = b + 1;
                if (active) {
                  const typename RT::raw* rp =
                      reinterpret_cast<const typename RT::raw*>(P.replicas[ids[b]]) + rep_index(P, (uint32_t)ids[b], jj, e0 + idx);
                  uint32_t ow[4];
                  load_words_stream<LaneWords<RT>::value>(rp, ow);
                  unpack_lane<RT>(ow, old[b]);
                } else {
#pragma unroll
                  for (int x = 0; x < kEpl; ++x) old[b][x] = 0.0f;
                }
              }
            }
#pragma unroll
            for (int b = 0; b < kStaleBatch; ++b) {
              if (b < nb) {
                float sq = 0.0f;
#pragma unroll
                for (int x = 0; x < kEpl; ++x) {
                  const float d = __fsub_rn(old[b][x], wire[x]);
                  sq = __fadd_rn(sq, __fmul_rn(d, d));
                }
                const float tot = warp_sum(sq);
                if ((ids[b] & 31) == lane) {
                  if (ids[b] < 32) dacc0 += (double)tot; else dacc1 += (double)tot;
                }
              }
            }
          }
        }
      }
    }
  }

  // ---- common exit: per-CTA drift partials in fixed order, status word ---------------
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) atomicExch(G.status, 1u);
  if constexpr (DRIFTK) {
    double* sh = kStaleStages ? warp_acc : reinterpret_cast<double*>(stage0);   // stages are idle now
    if constexpr (!kStaleStages) {
      if (warp < kConsumerWarps) {
        sh[warp * kMaxW + lane] = dacc0;
        sh[warp * kMaxW + lane + 32] = dacc1;
      }
      __syncthreads();
    }
    if (threadIdx.x < kMaxW) {
      double t = 0.0;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) t += sh[w * kMaxW + threadIdx.x];
      P.partials[(size_t)blockIdx.x * kMaxW + threadIdx.x] = t;
    }
    if (P.ticket) drift_last_block(P, warp, lane, kConsumerWarps + 2);
  }
}

}  // namespace lossy
