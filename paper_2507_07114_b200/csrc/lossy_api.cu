// C ABI of the lossy data-parallel step (see include/lossy.h for the contract).
// Host side: argument validation, threshold and hash-key derivation, launches.
#include "../../include/lossy.h"

#include <math.h>
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <new>

#include "lossy_gather.cuh"
#include "lossy_phase_tma.cuh"

using namespace lossy;

struct lossy_ctx {
  lossy_config cfg;
  uint64_t K;
  uint32_t chunks_per_packet;
  uint32_t num_chunks;
  uint32_t pps;
  uint32_t Tg, Tp;
  int device;
  int num_sms;
  uint32_t max_blocks;   // capacity of `partials`
  double* partials;      // device, [max_blocks][kMaxW], followed by the status word
  uint32_t* status;      // device status words: [0] 0 = fine, 1 = a bounded wait in a kernel gave up; [1..4] debug build: a failed index check
  uint64_t check_shrink; // debug build self-test: the index checks hold ranges against n - check_shrink
  uint32_t* ticket;      // device counter of finished blocks (last-block drift finalisation), zero between calls
  bool plan_only;        // launch helpers only report their grid size
  const uint64_t* reliable;  // caller-owned device array [2][K] of reliable-link bits, or NULL
  uint64_t* burst_state; // bursty loss: caller-owned device array [2 buffers][2 rows][K], or NULL
  uint32_t Tenter, Tstay;
  int smem_optin;        // largest dynamic shared memory a block may opt in to
  uint64_t launches;
  char* plan;            // lossy_describe_plan: where try_tma notes the build it would launch (else NULL)
  size_t plan_size;
  char err[256];
};

namespace {

constexpr int kBlocksPerSmCap = 8;

int fail(lossy_ctx* ctx, int code, const char* msg) {
  if (ctx) snprintf(ctx->err, sizeof ctx->err, "%s", msg);
  return code;
}
int fail_cuda(lossy_ctx* ctx, const char* what, cudaError_t e) {
  if (ctx) snprintf(ctx->err, sizeof ctx->err, "%s: %s", what, cudaGetErrorString(e));
  return LOSSY_ECUDA;
}
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

uint32_t threshold_of(double p) { return (uint32_t)floor(p * 4294967296.0); }

int check_table(lossy_ctx* ctx, const void* const* tab, const char* name) {
  if (!tab) return fail(ctx, LOSSY_EINVAL, name);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i)
    if (!tab[i] || !aligned16(tab[i])) return fail(ctx, LOSSY_EINVAL, name);
  return LOSSY_OK;
}

// elements of worker i's shard inside this context's packet range (what an owner-elided replica leaves out)
uint64_t own_elems(const lossy_ctx* ctx, uint32_t i) {
  const lossy_config& c = ctx->cfg;
  const uint64_t s0 = (uint64_t)i * ctx->pps, s1 = s0 + ctx->pps;
  const uint64_t c0 = c.shard_packet0, c1 = c.shard_packet0 + ctx->K;
  const uint64_t lo = s0 > c0 ? s0 : c0, hi = s1 < c1 ? s1 : c1;
  if (lo >= hi) return 0;
  const uint64_t e0 = (lo - c0) * c.packet_elems, e1 = (hi - c0) * c.packet_elems;
  return (e1 < c.n ? e1 : c.n) - (e0 < c.n ? e0 : c.n);
}

// The replica table: W aligned device pointers; an owner-elided replica that holds nothing may be NULL.
int check_replicas(lossy_ctx* ctx, const void* const* tab) {
  const char* name = "replicas: NULL or misaligned pointer";
  if (!tab) return fail(ctx, LOSSY_EINVAL, name);
  const bool elide = ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER;
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) {
    if (elide && own_elems(ctx, i) == ctx->cfg.n) continue;
    if (!tab[i] || !aligned16(tab[i])) return fail(ctx, LOSSY_EINVAL, name);
  }
  return LOSSY_OK;
}

void fill_common(const lossy_ctx* ctx, uint64_t step, Params& P) {
  memset(&P, 0, sizeof P);
  const lossy_config& c = ctx->cfg;
  P.n = c.n;
  P.packet_base = c.packet_base + c.shard_packet0;   // the hash sees the global id of every packet
  P.k0 = (uint32_t)c.shard_packet0;
  P.step_key = step_key_of(c.seed, step);
  P.num_chunks = ctx->num_chunks;
  P.chunks_per_packet = ctx->chunks_per_packet;
  P.pps = ctx->pps;
  P.P = c.packet_elems;
  P.W = c.W;
  P.Tg = ctx->Tg;
  P.Tp = ctx->Tp;
  P.flags = c.flags;
  P.lr = c.lr;
  P.b1 = c.beta1;
  P.b2 = c.beta2;
  P.omb1 = 1.0f - c.beta1;   // (1 - beta) in fp32
  P.omb2 = 1.0f - c.beta2;
  P.ibc1 = (float)(1.0 / (1.0 - pow((double)c.beta1, (double)step)));
  P.ibc2 = (float)(1.0 / (1.0 - pow((double)c.beta2, (double)step)));
  P.eps = c.eps;
  P.partials = ctx->partials;
  P.K = (uint32_t)ctx->K;
  P.reliable = ctx->reliable;
  P.check = ctx->status + 1;
  P.check_n = c.n - (ctx->check_shrink < c.n ? ctx->check_shrink : c.n);
  fill_rep_skip(P, (c.flags & LOSSY_REPLICA_SKIP_OWNER) != 0);
  if (ctx->burst_state) {
    // the states after step t-1 live in buffer (t-1)&1, those after step t go to buffer t&1
    const size_t buf = 2 * (size_t)ctx->K;
    P.burst_in = ctx->burst_state + ((step - 1) & 1u) * buf;
    P.burst_out = ctx->burst_state + (step & 1u) * buf;
    P.Tenter = ctx->Tenter;
    P.Tstay = ctx->Tstay;
  }
}

// ---- bulk-copy pipeline (fused step only) --------------------------------------------------
constexpr uint32_t kTmaSmemFixed = kTmaBarBytes + kMaxStages * (sizeof(StageHdr) + sizeof(PackedStale)) + kMaskBufs * sizeof(PackedMasks);

// Launch policy of the bulk-copy pipeline, from sweeps on B200 over W = 2..64, p = 0.05..0.3
// (CUDA-event timings of bench.py with each build forced): which of the four builds runs and whether its bulk copies carry an
// L2 evict-first hint (bit 0 loads, bit 1 stores).
struct TmaPolicy {
  bool wide;      // 16 compute warps, one CTA per SM, 2048-element tiles (else 8 warps, two CTAs, 1024)
  int group;      // workers per pipeline stage: 4 or 8
  int early_stale;   // stale copies: 0 = fetched in the drift phase, 16 = first ones requested before the tile's arithmetic, 1 = extra pipeline stages (stages of 8 only)
  uint32_t hints;
  bool split;     // state slots apart from the stages (twin build, stages of 8, high loss)
  uint32_t split_stages;
};
TmaPolicy tma_policy(const lossy_config& c) {
  const double pm = c.p_grad > c.p_param ? c.p_grad : c.p_param;
  TmaPolicy t;
  // wide tiles win whenever a tile takes at most two 8-worker groups and the packet is a multiple of the tile
  t.wide = c.W <= 16 && c.packet_elems % TmaShape<16>::kTile == 0;
  // stages of 4 workers (finer-grained pipeline) win for few workers at low loss: +5 % at W = 8, p = 0.1,
  // but -9 % at W = 8, p = 0.3; the crossover at W = 8 sits near p = 0.17
  t.group = c.W <= 4 ? 4 : (c.W <= 8 && pm < 0.175 ? 4 : 8);
  // hints: +2-4 % on the twin build at high loss, or at W = 64 from moderate loss (p = 0.1: 0.957 against
  // 0.934); neutral to -2 % elsewhere (W = 64, p = 0.01: 0.944 against 0.961)
  t.hints = t.wide ? (pm >= 0.28 ? 3u : 0u) : ((pm >= 0.2 || (c.W > 32 && pm >= 0.05)) ? 3u : 0u);
  // early stale requests pay from about two stale replicas per tile at high loss: +8-10 % at W >= 16,
  // p = 0.3; at p = 0.1 they lose 1-2 % even with six stale replicas per tile (W = 64)
  t.early_stale = t.group == 8 && (c.W - 1) * c.p_param >= 2.0 && c.p_param >= 0.15 ? 16 : 0;
  // State slots apart from the stages (one more gradient stage fits): the twin build at p >= 0.2, where the
  // compute warps spend long on stale replicas and the extra stage keeps the loads going meanwhile: W = 32,
  // p = 0.3: 0.89 -> 0.96; W = 48, p = 0.2: 0.91 -> 0.97; W = 64, p = 0.3: 0.90 -> 0.95. The fourth stage pays
  // from about 6.5 stale replicas per tile; below that three (W = 24, p = 0.2: 0.93 -> 0.95), and at lower
  // loss the plain build is as fast or faster (W = 64, p = 0.1: 0.96 against 0.94 with four stages).
  t.split = !t.wide && t.group == 8 && c.W > 16 && c.p_param >= 0.2;
  t.split_stages = (c.W - 1) * c.p_param >= 6.5 ? 4u : 3u;
  // With the fourth stage the stale replicas' old copies come through the pipeline as extra stages instead
  // of being read by the compute warps (W = 64, p = 0.3: 0.88 -> 0.95; W = 48, p = 0.3: 0.91 -> 0.97; W = 17,
  // p = 0.5: 0.71 -> 0.79); with fewer stale replicas per tile the early requests stay ahead (W = 24, p = 0.2:
  // 0.95 against 0.92).
  if (t.split && t.split_stages == 4u) t.early_stale = 1;
  return t;
}

constexpr int kMaxDevices = 64;
// The launch helpers below remember, per kernel instantiation and device, what they set up once (the raised
// shared-memory limit, the occupancy). Those tables are process-wide, so host threads that drive different
// contexts take this lock around the look-up; it is never held across a launch.
std::mutex g_setup_mu;

// Dynamic shared memory one CTA of the bulk-copy kernel may use: the CTAs of one SM share 227 KB.
template <int CW>
uint32_t tma_smem_budget(const lossy_ctx* ctx) {
  uint32_t budget = (227u * 1024u) / TmaShape<CW>::kCtasPerSm - 1024u;
  if ((uint32_t)ctx->smem_optin < budget) budget = (uint32_t)ctx->smem_optin;
  return budget;
}

template <int CW, int GS, bool PACKED, bool SPLIT>
bool tma_geometry(const lossy_ctx* ctx, TmaGeom& G) {
  constexpr uint32_t kGroup = GS;
  constexpr uint32_t kTile = TmaShape<CW>::kTile;
  const lossy_config& c = ctx->cfg;
  const uint64_t kfull = c.n / c.packet_elems;               // packets that are complete
  if (kfull == 0 || kfull >= (1ull << 31)) return false;
  G.packets_per_tile = 1;
  G.full_packets = (uint32_t)kfull;
  if (PACKED) {
    // small packets: a tile packs 2, 4 or 8 whole packets; a compute warp's 128 elements stay inside one
    if (c.packet_elems >= kTile || kTile % c.packet_elems != 0 || c.packet_elems % 128 != 0 ||
        kTile / c.packet_elems > (uint32_t)kMaxSub)
      return false;
    G.packets_per_tile = kTile / c.packet_elems;
  } else if (c.packet_elems < kTile) {
    return false;
  }
  const uint32_t gb = c.grad_dtype == LOSSY_BF16 ? 2 : 4, rb = c.replica_dtype == LOSSY_BF16 ? 2 : 4;
  G.grad_slots = c.W < (uint32_t)kGroup ? c.W : (uint32_t)kGroup;
  G.groups = (c.W + kGroup - 1) / kGroup;
  const uint32_t state = 3 * kTile * 4 + kTile * rb;           // theta, m, v and the wire tile
  const uint32_t sb = G.grad_slots * kTile * gb + (SPLIT ? 0u : state);
  G.stage_bytes = (sb + 127u) & ~127u;
  G.state_bytes = SPLIT ? (state + 127u) & ~127u : 0u;
  // behind the stages: the two state slots of the SPLIT builds, and fp64 drift sums per compute warp and
  // replica (used by the stale-stage builds)
  const uint32_t budget = tma_smem_budget<CW>(ctx) - CW * kMaxW * (uint32_t)sizeof(double) - 2u * G.state_bytes;
  if (budget < kTmaSmemFixed + 2 * G.stage_bytes) return false;
  G.stages = (budget - kTmaSmemFixed) / G.stage_bytes;
  const uint32_t cap = SPLIT ? tma_policy(c).split_stages : 4u;   // with the state in the stage a fifth measured no faster
  if (G.stages > cap) G.stages = cap;
  // One tile per stage (a single worker group): with a fourth stage the loads run too far ahead of the
  // stores (W = 4, p = 0.1: 0.98 of the copy rate with three stages, 0.92 with four; W = 2: 0.96 / 0.95);
  // a single worker still gains from the fourth (0.97 / 0.91).
  if (G.groups == 1 && c.W >= 2 && G.stages > 3u) G.stages = 3u;
  G.tiles_per_packet = PACKED ? 1u : (c.packet_elems + kTile - 1) / kTile;
  const uint64_t tiles = PACKED ? (kfull + G.packets_per_tile - 1) / G.packets_per_tile : kfull * G.tiles_per_packet;
  if (tiles >= (1ull << 31)) return false;
  G.num_tiles = (uint32_t)tiles;
  G.status = ctx->status;
  G.hints = tma_policy(c).hints;
  return true;
}

template <class GT, class RT, int OPT, bool DRIFTK, int CW, int GS, int PRE, bool PACKED, bool SPLIT>
int launch_tma(lossy_ctx* ctx, const Params& P, const TmaGeom& G, cudaStream_t s, uint32_t* blocks_out) {
  auto kern = lossy_fused_tma_kernel<GT, RT, OPT, DRIFTK, CW, GS, PRE, PACKED, SPLIT>;
  constexpr int kThreadsTma = TmaShape<CW>::kThreads;
  const uint32_t smem = kTmaSmemFixed + G.stages * G.stage_bytes + 2u * G.state_bytes + CW * kMaxW * (uint32_t)sizeof(double);
  // launch bounds and the shared-memory budget guarantee kCtasPerSm resident CTAs per SM
  uint32_t blocks = (uint32_t)(ctx->num_sms * TmaShape<CW>::kCtasPerSm);
  if (blocks > G.num_tiles) blocks = G.num_tiles;
  *blocks_out = blocks;
  if (ctx->plan_only) return LOSSY_OK;
  static bool opted_in[kMaxDevices];   // per kernel instantiation and device: raise the dynamic shared memory limit once
  cudaError_t e;
  {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (ctx->device >= kMaxDevices || !opted_in[ctx->device]) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tma_smem_budget<CW>(ctx));
      if (e != cudaSuccess) return fail_cuda(ctx, "shared memory opt-in", e);
      if (ctx->device < kMaxDevices) opted_in[ctx->device] = true;
    }
  }
  kern<<<blocks, kThreadsTma, smem, s>>>(P, G);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "bulk-copy kernel launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

template <bool DRIFTK, int CW, int GS, int PRE, bool PACKED, bool SPLIT>
int dispatch_tma(lossy_ctx* ctx, const Params& P, const TmaGeom& G, cudaStream_t s, uint32_t* blocks) {
  const bool gb = ctx->cfg.grad_dtype == LOSSY_BF16;
  const bool rb = ctx->cfg.replica_dtype == LOSSY_BF16;
  const bool adam = ctx->cfg.optimizer == LOSSY_ADAM;
  if (gb && rb) return adam ? launch_tma<BF16, BF16, 1, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks) : launch_tma<BF16, BF16, 0, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks);
  // stale copies as pipeline stages (PRE = 1) reuse the gradient slots: fp32 replicas with bf16 gradients do not fit
  constexpr int PRE_WIDER = PRE == 1 ? 16 : PRE;
  if (gb && !rb) return adam ? launch_tma<BF16, F32, 1, DRIFTK, CW, GS, PRE_WIDER, PACKED, SPLIT>(ctx, P, G, s, blocks) : launch_tma<BF16, F32, 0, DRIFTK, CW, GS, PRE_WIDER, PACKED, SPLIT>(ctx, P, G, s, blocks);
  if (!gb && rb) return adam ? launch_tma<F32, BF16, 1, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks) : launch_tma<F32, BF16, 0, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks);
  return adam ? launch_tma<F32, F32, 1, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks) : launch_tma<F32, F32, 0, DRIFTK, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks);
}

template <int CW, int GS, int PRE = 0, bool PACKED = false, bool SPLIT = false>
int try_tma(lossy_ctx* ctx, const Params& P, bool drift, cudaStream_t s, uint32_t* blocks, bool* used) {
  TmaGeom G = {};
  if (!tma_geometry<CW, GS, PACKED, SPLIT>(ctx, G)) return LOSSY_OK;
  *used = true;
  if (ctx->plan) {
    // dispatch_tma runs the early-request build where staged copies do not fit the gradient slots
    const bool fits = !(ctx->cfg.grad_dtype == LOSSY_BF16 && ctx->cfg.replica_dtype == LOSSY_F32);
    snprintf(ctx->plan, ctx->plan_size, "bulk-copy %s group=%d stale=%s%s%s stages=%u", CW == 16 ? "wide" : "twin", GS,
             !drift || PRE == 0 ? "late" : PRE == 1 && fits ? "staged" : "early", PACKED ? " packed" : "",
             SPLIT ? " split" : "", G.stages);
  }
  // without drift norms nothing reads the stale copies: the plain build serves
  return drift ? dispatch_tma<true, CW, GS, PRE, PACKED, SPLIT>(ctx, P, G, s, blocks)
               : dispatch_tma<false, CW, GS, 0, PACKED, SPLIT>(ctx, P, G, s, blocks);
}

// ---- gather pipeline (packets shorter than a tile) ------------------------------------------
// barriers, the ring of tile masks, stage headers; the drift sums per compute warp, the wire ring and the stages follow
constexpr uint32_t kGatherSmemFixed = kGatherBarBytes + kGatherRing * sizeof(TileMasks) + kGatherMaxStages * sizeof(StageHdr);

// rd: the stale copies are read outside the compute warps (twin geometry: by the replica warps, one replica each;
// wide geometry: by drift warps of their own)
template <int CW>
bool gather_geometry(const lossy_ctx* ctx, bool rd, TmaGeom& G) {
  constexpr uint32_t kTile = GatherShape<CW>::kTile;
  const lossy_config& c = ctx->cfg;
  const uint64_t kfull = c.n / c.packet_elems;               // packets that are complete
  if (kfull == 0 || kfull >= (1ull << 31)) return false;
  // whole packets per tile: powers of two from 128 elements that divide the tile, at most kMaxSub of them
  const uint32_t P = c.packet_elems;
  if (P >= kTile || (P & (P - 1u)) != 0 || P < 128u || kTile / P > (uint32_t)kMaxSub) return false;
  memset(&G, 0, sizeof G);
  G.packets_per_tile = kTile / P;
  G.full_packets = (uint32_t)kfull;
  const uint32_t gb = c.grad_dtype == LOSSY_BF16 ? 2 : 4, rb = c.replica_dtype == LOSSY_BF16 ? 2 : 4;
  G.grad_slots = c.W < 8u ? c.W : 8u;
  G.groups = (c.W + 7u) / 8u;
  // a stage holds the group's gradient rows and theta, m, v
  G.stage_bytes = (G.grad_slots * kTile * gb + 3 * kTile * 4 + 127u) & ~127u;
  // fp64 drift sums per adding warp and replica, the wire ring, and (rd) the scratch for the stale copies
  G.state_bytes = (uint32_t)(rd ? GatherShape<CW, true>::kAccRows : CW) * kMaxW * (uint32_t)sizeof(double) + kWireRing * kTile * rb;
  const uint32_t row_chunks = kTile * rb / 512u;             // 512-byte chunks of one replica's row of a tile
  uint32_t scratch_unit = 0;                                  // bytes of scratch per chunk of capacity
  if (rd) {
    using Shape = GatherShape<CW, true>;
    scratch_unit = (uint32_t)(Shape::kDriftWarps ? Shape::kDriftWarps : Shape::kReplicaWarps) * Shape::kRdBuffers * 512u;
    // twin: a replica warp owns one replica, its whole row fits; wide: at least four chunks per drift warp, more below
    G.rd_cap = Shape::kDriftWarps ? 4u : row_chunks;
    G.state_bytes += G.rd_cap * scratch_unit;
  }
  const uint32_t budget = (227u * 1024u) / GatherShape<CW>::kCtasPerSm - 1024u;
  const uint32_t avail = (uint32_t)ctx->smem_optin < budget ? (uint32_t)ctx->smem_optin : budget;
  if (avail < kGatherSmemFixed + G.state_bytes + 2 * G.stage_bytes) return false;
  G.stages = (avail - kGatherSmemFixed - G.state_bytes) / G.stage_bytes;
  if (G.stages > 4u) G.stages = 4u;                           // more measured no faster (W = 2..32)
  if (rd && GatherShape<CW, true>::kDriftWarps) {
    // wide: what the stages leave goes to the scratch, up to every chunk of a drift warp's replicas
    const uint32_t left = avail - kGatherSmemFixed - G.state_bytes - G.stages * G.stage_bytes;
    // a replica's row in 2^lgsplit parts, W * 2^lgsplit parts dealt round robin: the fewest parts that balance the drift warps
    const uint32_t nd = GatherShape<CW, true>::kDriftWarps;
    // (a warp's cost: its share of a row, plus about a sixteenth of a row per part whatever the part holds: W = 17 in 8
    // parts per row, 17 parts per warp, ran at 0.56 where W = 16 in whole rows, 2 per warp, ran at 0.85; W = 12 in
    // halves 0.79 against 0.74 in whole rows; W = 5, P = 512 in quarters 0.86 against 0.83)
    uint32_t best = ~0u, share = 8u;
    for (uint32_t lg = 0; (1u << lg) <= G.packets_per_tile && lg <= 2u; ++lg) {
      const uint32_t parts = ((c.W << lg) + nd - 1u) / nd;                   // a warp's parts ...
      const uint32_t eighths = parts * (8u >> lg);                            // ... and its share in eighths of a row
      const uint32_t cost = 2u * eighths + parts;
      if (cost < best) { best = cost; share = eighths; G.rd_lgsplit = lg; }
    }
    const uint32_t most = (share * row_chunks + 7u) / 8u;
    uint32_t more = left / scratch_unit;
    if (G.rd_cap + more > most) more = most > G.rd_cap ? most - G.rd_cap : 0u;
    G.rd_cap += more;
    G.state_bytes += more * scratch_unit;
    // A drift warp's stale chunks of a tile should mostly fit its scratch: what does not fit is loaded directly at
    // its full latency. Where not even their mean count fits (fp32 replicas, whose wire ring takes the room: a
    // scratch of 4 chunks for a mean of 9) the compute warps' reads serve better; the caller falls back to them,
    // unless it was told to use this build (LOSSY_GATHER_PATH: comparison and tests). (W = 16, P = 256, p = 0.3,
    // bf16: 8 chunks for a mean of 4.5; W = 24: 8 for 6.9.)
    const double mean = share / 8.0 * row_chunks * c.p_param * (c.W - 1.0) / c.W;
    if (!(c.flags & LOSSY_GATHER_PATH) && G.rd_cap < mean) return false;
  }
  G.tiles_per_packet = 1;
  const uint64_t tiles = (kfull + G.packets_per_tile - 1) / G.packets_per_tile;
  if (tiles >= (1ull << 31)) return false;
  G.num_tiles = (uint32_t)tiles;
  G.status = ctx->status;
  // bit 2: the mask warp sends the stale pairs' old copies toward L2 tiles ahead (W = 16, p = 0.1: 0.94 -> 0.99;
  // with more than about two stale replicas per sub-packet it loses: W = 12, p = 0.2: 0.86 -> 0.78)
  G.hints = (c.W - 1) * c.p_param < 1.8 ? 4u : 0u;
  // bit 3: how the wide geometry's two gather warps share a group. Dealing out the workers halves each warp's
  // ballots and is ahead wherever rows have holes (W = 16, P = 256: +1 / +7 / +1 % at p = 0.1 / 0.2 / 0.3; P = 512,
  // p = 0.3: +4 %) and with 9-12 or more than 16 workers at any loss (W = 24: +4 % at p = 0, +6 % at 0.1; W = 64,
  // P = 512: +9 %); where most rows are whole, up to 8 or with 13-16 workers, both warps in one row do better
  // (W = 16: 0.98-0.99 against 0.91-0.94 up to p = 0.05; W = 8: +1 %). Same-process A/B pairs, repeatable to 0.002.
  const double whole_rows = pow(1.0 - c.p_grad, (double)G.packets_per_tile);
  if (whole_rows >= 0.6 && (c.W <= 8u || (c.W >= 13u && c.W <= 16u))) G.hints |= 8u;
  return true;
}

template <class GT, class RT, int OPT, bool DRIFTK, int CW, bool RD>
int launch_gather(lossy_ctx* ctx, const Params& P, const TmaGeom& G, cudaStream_t s, uint32_t* blocks_out) {
  auto kern = lossy_fused_gather_kernel<GT, RT, OPT, DRIFTK, CW, RD>;
  const uint32_t smem = kGatherSmemFixed + G.state_bytes + G.stages * G.stage_bytes;
  uint32_t blocks = (uint32_t)(ctx->num_sms * GatherShape<CW>::kCtasPerSm);
  if (blocks > G.num_tiles) blocks = G.num_tiles;
  *blocks_out = blocks;
  if (ctx->plan_only) return LOSSY_OK;
  static bool opted_in[kMaxDevices];   // per kernel instantiation and device: raise the dynamic shared memory limit once
  cudaError_t e;
  {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (ctx->device >= kMaxDevices || !opted_in[ctx->device]) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tma_smem_budget<CW>(ctx));
      if (e != cudaSuccess) return fail_cuda(ctx, "shared memory opt-in", e);
      if (ctx->device < kMaxDevices) opted_in[ctx->device] = true;
    }
  }
  kern<<<blocks, GatherShape<CW, RD>::kThreads, smem, s>>>(P, G);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "gather kernel launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

template <bool DRIFTK, int CW, bool RD>
int dispatch_gather(lossy_ctx* ctx, const Params& P, const TmaGeom& G, cudaStream_t s, uint32_t* blocks) {
  const bool gb = ctx->cfg.grad_dtype == LOSSY_BF16;
  const bool rb = ctx->cfg.replica_dtype == LOSSY_BF16;
  const bool adam = ctx->cfg.optimizer == LOSSY_ADAM;
  if (gb && rb) return adam ? launch_gather<BF16, BF16, 1, DRIFTK, CW, RD>(ctx, P, G, s, blocks) : launch_gather<BF16, BF16, 0, DRIFTK, CW, RD>(ctx, P, G, s, blocks);
  if (gb && !rb) return adam ? launch_gather<BF16, F32, 1, DRIFTK, CW, RD>(ctx, P, G, s, blocks) : launch_gather<BF16, F32, 0, DRIFTK, CW, RD>(ctx, P, G, s, blocks);
  if (!gb && rb) return adam ? launch_gather<F32, BF16, 1, DRIFTK, CW, RD>(ctx, P, G, s, blocks) : launch_gather<F32, BF16, 0, DRIFTK, CW, RD>(ctx, P, G, s, blocks);
  return adam ? launch_gather<F32, F32, 1, DRIFTK, CW, RD>(ctx, P, G, s, blocks) : launch_gather<F32, F32, 0, DRIFTK, CW, RD>(ctx, P, G, s, blocks);
}

template <int CW>
int try_gather(lossy_ctx* ctx, const Params& P, bool drift, bool rd, cudaStream_t s, uint32_t* blocks, bool* used) {
  TmaGeom G = {};
  if (!gather_geometry<CW>(ctx, drift && rd, G)) return LOSSY_OK;
  *used = true;
  if (ctx->plan)
    snprintf(ctx->plan, ctx->plan_size, "gather %s packets/tile=%u stages=%u%s", CW == 16 ? "wide" : "twin", G.packets_per_tile, G.stages,
             drift && rd && CW == 16 ? " drift-warps" : "");
  if (drift && rd) return dispatch_gather<true, CW, true>(ctx, P, G, s, blocks);
  return drift ? dispatch_gather<true, CW, false>(ctx, P, G, s, blocks) : dispatch_gather<false, CW, false>(ctx, P, G, s, blocks);
}

// Run the build the policy picks; *used stays false when no bulk-copy launch fits (packets shorter
// than a tile, or no complete packet): the register path then takes everything.
int run_tma(lossy_ctx* ctx, const Params& P, bool drift, cudaStream_t s, uint32_t* blocks, bool* used) {
  *used = false;
  if (ctx->cfg.flags & LOSSY_REGISTER_PATH) return LOSSY_OK;
  const TmaPolicy t = tma_policy(ctx->cfg);
  if (!(ctx->cfg.flags & LOSSY_PACKED_BULK) && ctx->cfg.packet_elems < (uint32_t)TmaShape<8>::kTile) {
    // Packets shorter than a tile (128, 256 or 512 elements): the gather pipeline, where it beats the register
    // kernel. Fractions of the copy rate, 20 steps of a 202 M element bucket, P = 256, taken back to back in one
    // process (power-capped clocks; a point measured alone runs 3-6 % higher), S = (W - 1) p_param = stale replicas
    // per sub-packet:
    //  * the wide geometry with drift warps of its own for 4..24 workers, packets of 256 or 512 elements and
    //    0.2 (W - 8) <= S < 7.5 (W = 8: 0.97 / 0.97 / 0.94 / 0.85 at p = 0.05 / 0.1 / 0.2 / 0.3, where the compute
    //    warps' reads gave 0.89 / 0.84 / 0.82 / 0.77 and the register kernel 0.77 and 0.67 at p = 0.1 and 0.3; W = 16:
    //    0.92 / 0.88 / 0.84 at p = 0.1 / 0.2 / 0.3 against 0.90 / 0.81 / 0.69, register kernel 0.82 / 0.79 / 0.76;
    //    W = 24: 0.83 and 0.78 at p = 0.2 and 0.3 against 0.81 and 0.72; W = 4: 0.77-0.83 against 0.75-0.84 for the
    //    twin geometry);
    //  * below that band (many workers, few stale copies) the compute warps' reads stay ahead (W = 16, p = 0.05: 0.98
    //    against 0.91; W = 24, p = 0.1: 0.88 against 0.85; W = 32, p = 0.05: 0.96 against 0.91);
    //  * above it the drift warps fall behind (W = 17, p = 0.5: 0.43): many workers at high loss stay with the
    //    register kernel (p = 0.2, W = 32: 0.85 against 0.79-0.84; W = 17, p = 0.5: 0.56);
    //  * two or three workers, and packets of 128 elements: the twin geometry (W = 2: 0.78-0.81 against 0.69-0.74
    //    for the wide one), whose replica warps also read the stale copies up to four workers.
    const lossy_config& c = ctx->cfg;
    const double pm = c.p_grad > c.p_param ? c.p_grad : c.p_param;
    const bool wide_fits = c.packet_elems * (uint32_t)kMaxSub >= (uint32_t)GatherShape<16>::kTile;
    const double stale = (c.W - 1u) * c.p_param;
    // (bf16 replicas: with fp32 ones a row has twice the chunks and the wire ring leaves the drift warps little
    // scratch; the compute warps' reads gave 0.71-0.73 where drift warps gave 0.48-0.59; LOSSY_GATHER_PATH asks
    // for the drift warps all the same, for tests)
    const bool drift_warps = wide_fits && c.W >= 4u && c.W <= 24u && stale < 7.5 && stale >= 0.2 * ((double)c.W - 8.0) &&
                             (c.replica_dtype == LOSSY_BF16 || (c.flags & LOSSY_GATHER_PATH));
    // (the register kernel's lead at high loss was measured with bf16 replicas; with fp32 ones the compute warps'
    // reads are ahead at W = 12-16, p = 0.3: 0.71-0.73 against 0.57-0.62)
    const bool reg_ahead = !(c.flags & LOSSY_GATHER_PATH) && !drift_warps &&
                           (c.replica_dtype == LOSSY_BF16 ? (c.W >= 12 && pm >= 0.25) || (c.W >= 24 && pm >= 0.15) : c.W >= 24 && pm >= 0.25);
    if (!reg_ahead) {
      int rc = LOSSY_OK;
      if (c.W >= 4u) rc = try_gather<16>(ctx, P, drift, drift_warps, s, blocks, used);
      if (rc || *used) return rc;
      if (c.W > kRdTwinMaxWorkers && drift && drift_warps) rc = try_gather<16>(ctx, P, drift, false, s, blocks, used);   // scratch too small
      if (rc || *used) return rc;
      rc = try_gather<8>(ctx, P, drift, c.W <= kRdTwinMaxWorkers, s, blocks, used);
      if (rc || *used) return rc;
    }
  }
  {
    // Packets of exactly half a wide tile with 13..16 workers at low loss: the PACKED wide build (two packets
    // per tile, one CTA per SM) beats the twin build, whose pieces are 2 KB (W = 16: 0.96-0.98 against 0.93 up
    // to p = 0.1; W = 13-14: 0.97-1.0 against 0.94 up to p = 0.05); beyond that its fetches of dropped packets
    // cost more than the wider tile gains, and from 12 workers down the twin build is ahead at every p.
    const lossy_config& c = ctx->cfg;
    const double pm = c.p_grad > c.p_param ? c.p_grad : c.p_param;
    if (c.packet_elems * 2u == (uint32_t)TmaShape<16>::kTile && c.W >= 13 && c.W <= 16 && pm <= (c.W == 16 ? 0.1 : 0.05)) {
      int rc = try_tma<16, 8, 0, true>(ctx, P, drift, s, blocks, used);
      if (rc || *used) return rc;
    }
  }
  if (ctx->cfg.packet_elems < (uint32_t)TmaShape<8>::kTile) {
    // Packets shorter than a tile: the PACKED builds, where they beat the register kernel. They fetch the
    // dropped sub-packets too, so they win at low loss (+8..17 % at W = 8-16, P = 256-512, p <= 0.1; +3..5 % at
    // p = 0.2) and lose at p = 0.3 from W = 16 and at p >= 0.1 from W = 32; with 2..8 workers they win at every loss rate
    // (+1..13 %); below 256 elements the register kernel's 256-element chunks are mostly idle lanes and the
    // PACKED build always wins.
    const lossy_config& c = ctx->cfg;
    const double pm = c.p_grad > c.p_param ? c.p_grad : c.p_param;
    if (c.packet_elems < 256 || (c.W >= 2 && c.W <= 8) || (pm <= 0.2 && c.W <= 24) || (pm <= 0.075 && c.W <= 32)) {
      if (c.W <= 16) {
        int rc = try_tma<16, 8, 0, true>(ctx, P, drift, s, blocks, used);
        if (rc || *used) return rc;
      }
      int rc = try_tma<8, 8, 0, true>(ctx, P, drift, s, blocks, used);
      if (rc || *used) return rc;
    }
  }
  if (t.split) {
    // the state lives in its own two-slot ring (SPLIT builds, twin geometry only)
    return t.early_stale == 1 ? try_tma<8, 8, 1, false, true>(ctx, P, drift, s, blocks, used)
           : t.early_stale ? try_tma<8, 8, 16, false, true>(ctx, P, drift, s, blocks, used)
                           : try_tma<8, 8, 0, false, true>(ctx, P, drift, s, blocks, used);
  }
  if (t.wide) {
    int rc = t.group == 4 ? try_tma<16, 4>(ctx, P, drift, s, blocks, used)
             : t.early_stale ? try_tma<16, 8, 16>(ctx, P, drift, s, blocks, used)
                             : try_tma<16, 8>(ctx, P, drift, s, blocks, used);
    if (rc || *used) return rc;
  }
  return t.group == 4 ? try_tma<8, 4>(ctx, P, drift, s, blocks, used)
         : t.early_stale ? try_tma<8, 8, 16>(ctx, P, drift, s, blocks, used)
                         : try_tma<8, 8>(ctx, P, drift, s, blocks, used);
}

template <int PH, class GT, class RT, int OPT, bool ELIDE = false>
int launch(lossy_ctx* ctx, const Params& P, cudaStream_t s, uint32_t* blocks_out) {
  auto kern = lossy_kernel<PH, GT, RT, OPT, ELIDE>;
  static int occupancy[kMaxDevices];   // per kernel instantiation and device: resident blocks per SM
  int per_sm = 0;
  cudaError_t e;
  {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    per_sm = ctx->device < kMaxDevices ? occupancy[ctx->device] : 0;
    if (per_sm == 0) {
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, 0);
      if (e != cudaSuccess) return fail_cuda(ctx, "occupancy query", e);
      if (per_sm < 1) per_sm = 1;
      if (per_sm > kBlocksPerSmCap) per_sm = kBlocksPerSmCap;
      if (ctx->device < kMaxDevices) occupancy[ctx->device] = per_sm;
    }
  }
  uint32_t blocks = (uint32_t)(ctx->num_sms * per_sm);
  const uint32_t need = (P.num_chunks - P.chunk_begin + kWarps - 1) / kWarps;
  if (blocks > need) blocks = need;
  if (blocks > ctx->max_blocks - P.partials_row0) blocks = ctx->max_blocks - P.partials_row0;
  if (blocks == 0) blocks = 1;
  if (blocks_out) *blocks_out = blocks;
  if (ctx->plan_only) return LOSSY_OK;
  kern<<<blocks, kThreads, 0, s>>>(P);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "kernel launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

// dispatch on the runtime element types / optimizer
template <int PH>
int dispatch(lossy_ctx* ctx, const Params& P, cudaStream_t s, uint32_t* blocks) {
  const bool gb = ctx->cfg.grad_dtype == LOSSY_BF16;
  const bool rb = ctx->cfg.replica_dtype == LOSSY_BF16;
  const bool adam = ctx->cfg.optimizer == LOSSY_ADAM;
  if constexpr (PH == AGG) {
    return gb ? launch<PH, BF16, F32, 0>(ctx, P, s, blocks) : launch<PH, F32, F32, 0>(ctx, P, s, blocks);
  } else if constexpr (PH == STEP) {
    return adam ? launch<PH, F32, F32, 1>(ctx, P, s, blocks) : launch<PH, F32, F32, 0>(ctx, P, s, blocks);
  } else if constexpr (PH == BCAST || PH == DRIFT) {
    if (ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER)   // owner-elided replicas: builds of their own
      return rb ? launch<PH, F32, BF16, 0, true>(ctx, P, s, blocks) : launch<PH, F32, F32, 0, true>(ctx, P, s, blocks);
    return rb ? launch<PH, F32, BF16, 0>(ctx, P, s, blocks) : launch<PH, F32, F32, 0>(ctx, P, s, blocks);
  } else {
    if (ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER) {
      if (gb && rb) return adam ? launch<PH, BF16, BF16, 1, true>(ctx, P, s, blocks) : launch<PH, BF16, BF16, 0, true>(ctx, P, s, blocks);
      if (gb && !rb) return adam ? launch<PH, BF16, F32, 1, true>(ctx, P, s, blocks) : launch<PH, BF16, F32, 0, true>(ctx, P, s, blocks);
      if (!gb && rb) return adam ? launch<PH, F32, BF16, 1, true>(ctx, P, s, blocks) : launch<PH, F32, BF16, 0, true>(ctx, P, s, blocks);
      return adam ? launch<PH, F32, F32, 1, true>(ctx, P, s, blocks) : launch<PH, F32, F32, 0, true>(ctx, P, s, blocks);
    }
    if (gb && rb) return adam ? launch<PH, BF16, BF16, 1>(ctx, P, s, blocks) : launch<PH, BF16, BF16, 0>(ctx, P, s, blocks);
    if (gb && !rb) return adam ? launch<PH, BF16, F32, 1>(ctx, P, s, blocks) : launch<PH, BF16, F32, 0>(ctx, P, s, blocks);
    if (!gb && rb) return adam ? launch<PH, F32, BF16, 1>(ctx, P, s, blocks) : launch<PH, F32, BF16, 0>(ctx, P, s, blocks);
    return adam ? launch<PH, F32, F32, 1>(ctx, P, s, blocks) : launch<PH, F32, F32, 0>(ctx, P, s, blocks);
  }
}


// ---- the single-phase calls through the bulk-copy pipeline ---------------------------------
constexpr uint32_t kPhaseSmemFixed = kTmaBarBytes + kPhaseMaxStages * sizeof(StageHdr);

template <int PH, int CW, int GS>
bool phase_geometry(const lossy_ctx* ctx, TmaGeom& G) {
  constexpr uint32_t kTile = TmaShape<CW>::kTile;
  constexpr bool kGrouped = PH == AGG || PH == DRIFT;
  const lossy_config& c = ctx->cfg;
  const uint64_t kfull = c.n / c.packet_elems;               // packets that are complete
  if (kfull == 0 || kfull >= (1ull << 31) || c.packet_elems < kTile) return false;
  memset(&G, 0, sizeof G);
  G.packets_per_tile = 1;
  G.full_packets = (uint32_t)kfull;
  const uint32_t gb = c.grad_dtype == LOSSY_BF16 ? 2 : 4, rb = c.replica_dtype == LOSSY_BF16 ? 2 : 4;
  const uint32_t eb = PH == AGG ? gb : PH == STEP ? 4u : rb;
  G.grad_slots = kGrouped ? (c.W < (uint32_t)GS ? c.W : (uint32_t)GS) : 0u;
  G.groups = kGrouped ? (c.W + GS - 1) / GS : 1u;
  G.stage_bytes = (phase_stage_bytes<PH>(kTile, G.grad_slots, eb, c.optimizer == LOSSY_ADAM) + 127u) & ~127u;
  const uint32_t budget = tma_smem_budget<CW>(ctx);
  if (budget < kPhaseSmemFixed + 2 * G.stage_bytes) return false;
  G.stages = (budget - kPhaseSmemFixed) / G.stage_bytes;
  if (G.stages > (uint32_t)kPhaseMaxStages) G.stages = kPhaseMaxStages;
  // the optimizer step reads and writes equal amounts: deeper than three stages its loads run too far ahead
  // of its stores (measured 1.01 of the copy rate with three stages, 0.90 with seven)
  if (PH == STEP && G.stages > 3u) G.stages = 3u;
  G.tiles_per_packet = (c.packet_elems + kTile - 1) / kTile;
  const uint64_t tiles = kfull * G.tiles_per_packet;
  if (tiles >= (1ull << 31)) return false;
  G.num_tiles = (uint32_t)tiles;
  G.status = ctx->status;
  G.hints = 0;
  return true;
}

template <int PH, class T, int OPT, int CW, int GS>
int launch_phase_tma(lossy_ctx* ctx, const Params& P, const TmaGeom& G, cudaStream_t s, uint32_t* blocks_out) {
  auto kern = lossy_phase_tma_kernel<PH, T, OPT, CW, GS>;
  const uint32_t smem = kPhaseSmemFixed + G.stages * G.stage_bytes;
  uint32_t blocks = (uint32_t)(ctx->num_sms * TmaShape<CW>::kCtasPerSm);
  if (blocks > G.num_tiles) blocks = G.num_tiles;
  *blocks_out = blocks;
  if (ctx->plan_only) return LOSSY_OK;
  static bool opted_in[kMaxDevices];   // per kernel instantiation and device: raise the dynamic shared memory limit once
  cudaError_t e;
  {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (ctx->device >= kMaxDevices || !opted_in[ctx->device]) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tma_smem_budget<CW>(ctx));
      if (e != cudaSuccess) return fail_cuda(ctx, "shared memory opt-in", e);
      if (ctx->device < kMaxDevices) opted_in[ctx->device] = true;
    }
  }
  kern<<<blocks, TmaShape<CW>::kThreads, smem, s>>>(P, G);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "bulk-copy kernel launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

template <int PH, int CW, int GS>
int try_phase_tma(lossy_ctx* ctx, const Params& P, cudaStream_t s, uint32_t* blocks, bool* used) {
  TmaGeom G;
  if (!phase_geometry<PH, CW, GS>(ctx, G)) return LOSSY_OK;
  *used = true;
  const bool adam = ctx->cfg.optimizer == LOSSY_ADAM;
  if constexpr (PH == AGG) {
    return ctx->cfg.grad_dtype == LOSSY_BF16 ? launch_phase_tma<PH, BF16, 0, CW, GS>(ctx, P, G, s, blocks)
                                             : launch_phase_tma<PH, F32, 0, CW, GS>(ctx, P, G, s, blocks);
  } else if constexpr (PH == STEP) {
    return adam ? launch_phase_tma<PH, F32, 1, CW, GS>(ctx, P, G, s, blocks)
                : launch_phase_tma<PH, F32, 0, CW, GS>(ctx, P, G, s, blocks);
  } else {
    return ctx->cfg.replica_dtype == LOSSY_BF16 ? launch_phase_tma<PH, BF16, 0, CW, GS>(ctx, P, G, s, blocks)
                                                : launch_phase_tma<PH, F32, 0, CW, GS>(ctx, P, G, s, blocks);
  }
}

// One single-phase call: complete packets through the bulk-copy pipeline where a build fits (packets of at
// least one tile), a ragged last packet or everything else through the register kernel. With drift norms, pass 0 only sizes the grids: the blocks of both launches draw tickets from one
// counter and the last of them finalises the norms.
template <int PH>
int run_phase(lossy_ctx* ctx, const Params& P, float* norms, double* sumsq, cudaStream_t s) {
  const lossy_config& c = ctx->cfg;
  const bool bulk = !(c.flags & LOSSY_REGISTER_PATH);
  // wide tiles (one CTA per SM) when they divide the packet and the streamed arrays fit two groups
  const bool wide = c.packet_elems % TmaShape<16>::kTile == 0 && c.W <= 16;
  uint32_t tma_blocks = 0, tail_blocks = 0;
  for (int pass = PH == DRIFT ? 0 : 1; pass < 2; ++pass) {
    ctx->plan_only = pass == 0;
    Params Q = P;
    if (PH == DRIFT && pass == 1) {
      Q.ticket = ctx->ticket;
      Q.total_rows = tma_blocks + tail_blocks;
      Q.norms = norms;
      Q.sumsq = sumsq;
    }
    bool used = false;
    int rc = LOSSY_OK;
    if (bulk) {
      if (wide) rc = try_phase_tma<PH, 16, 8>(ctx, Q, s, &tma_blocks, &used);
      if (!rc && !used) rc = try_phase_tma<PH, 8, 8>(ctx, Q, s, &tma_blocks, &used);
    }
    if (!rc) {
      if (used) {
        Q.chunk_begin = (uint32_t)((c.n / c.packet_elems) * ctx->chunks_per_packet);
        Q.partials_row0 = tma_blocks;
      } else {
        tma_blocks = 0;
      }
      if (Q.chunk_begin < Q.num_chunks) rc = dispatch<PH>(ctx, Q, s, &tail_blocks);
      else tail_blocks = 0;
    }
    ctx->plan_only = false;
    if (rc) {
      // a ticketed launch may already be queued: the counter must be zero again before the next call
      if (Q.ticket) cudaMemsetAsync(ctx->ticket, 0, sizeof(uint32_t), s);
      return rc;
    }
  }
  return LOSSY_OK;
}

}  // namespace

extern "C" {

int lossy_init(const lossy_config* cfg, lossy_ctx** out) {
  if (!cfg || !out) return LOSSY_EINVAL;
  *out = nullptr;
  if (cfg->W == 0 || cfg->W > LOSSY_MAX_WORKERS) return LOSSY_EINVAL;
  if (cfg->packet_elems == 0 || cfg->packet_elems % 8 != 0) return LOSSY_EINVAL;
  if (!(cfg->p_grad >= 0.0 && cfg->p_grad < 1.0) || !(cfg->p_param >= 0.0 && cfg->p_param < 1.0)) return LOSSY_EINVAL;
  if (cfg->grad_dtype > LOSSY_BF16 || cfg->replica_dtype > LOSSY_BF16 || cfg->optimizer > LOSSY_ADAM) return LOSSY_EINVAL;
  if (cfg->flags & ~(uint32_t)(LOSSY_SELF_LOSSLESS | LOSSY_ZERO_SKIP | LOSSY_REGISTER_PATH | LOSSY_REPLICA_SKIP_OWNER | LOSSY_PACKED_BULK | LOSSY_GATHER_PATH))
    return LOSSY_EINVAL;
  const uint64_t K = (cfg->n + cfg->packet_elems - 1) / cfg->packet_elems;
  const uint64_t cpp = (cfg->packet_elems + kChunk - 1) / kChunk;
  if (K * cpp >= (1ull << 31)) return LOSSY_EINVAL;  // stream larger models bucket by bucket
  if (cfg->bucket_packets) {
    // a packet range of a larger bucket: inside it, and ragged only where the bucket ends
    if (cfg->bucket_packets >= (1ull << 31) || cfg->shard_packet0 + K > cfg->bucket_packets) return LOSSY_EINVAL;
    if (cfg->n % cfg->packet_elems != 0 && cfg->shard_packet0 + K != cfg->bucket_packets) return LOSSY_EINVAL;
  } else if (cfg->shard_packet0) {
    return LOSSY_EINVAL;
  }

  lossy_ctx* ctx = new (std::nothrow) lossy_ctx;
  if (!ctx) return LOSSY_ENOMEM;
  memset(ctx, 0, sizeof *ctx);
  ctx->cfg = *cfg;
  ctx->K = K;
  ctx->chunks_per_packet = (uint32_t)cpp;
  ctx->num_chunks = (uint32_t)(K * cpp);
  // shard map of the WHOLE bucket: this context may cover only the packet range starting at shard_packet0
  const uint64_t Kb = cfg->bucket_packets ? cfg->bucket_packets : K;
  const uint64_t pps = (Kb + cfg->W - 1) / cfg->W;
  ctx->pps = pps ? (uint32_t)pps : 1u;
  ctx->Tg = threshold_of(cfg->p_grad);
  ctx->Tp = threshold_of(cfg->p_param);
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e != cudaSuccess) { delete ctx; return LOSSY_ECUDA; }
  ctx->max_blocks = (uint32_t)(ctx->num_sms * kBlocksPerSmCap);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device);
  if (e != cudaSuccess) { delete ctx; return LOSSY_ECUDA; }
  const size_t pbytes = (size_t)ctx->max_blocks * kMaxW * sizeof(double);
  e = cudaMalloc(&ctx->partials, pbytes + 256);
  if (e != cudaSuccess) { delete ctx; return e == cudaErrorMemoryAllocation ? LOSSY_ENOMEM : LOSSY_ECUDA; }
  ctx->status = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(ctx->partials) + pbytes);
  ctx->ticket = ctx->status + 16;
  e = cudaMemset(ctx->status, 0, 256);
  if (e != cudaSuccess) { cudaFree(ctx->partials); delete ctx; return LOSSY_ECUDA; }
  *out = ctx;
  return LOSSY_OK;
}

void lossy_destroy(lossy_ctx* ctx) {
  if (!ctx) return;
  if (ctx->partials) cudaFree(ctx->partials);
  delete ctx;
}

int lossy_set_bursty(lossy_ctx* ctx, double p_enter_bad, double p_leave_bad, uint64_t* state) {
  if (!ctx) return LOSSY_EINVAL;
  if (!state) {
    ctx->burst_state = nullptr;
    return LOSSY_OK;
  }
  if (!(p_enter_bad >= 0.0 && p_enter_bad < 1.0) || !(p_leave_bad > 0.0 && p_leave_bad <= 1.0))
    return fail(ctx, LOSSY_EINVAL, "bursty loss: need 0 <= P(good->bad) < 1 and 0 < P(bad->good) <= 1");
  if (ctx->K >= (1ull << 32)) return fail(ctx, LOSSY_EINVAL, "too many packets for bursty loss");
  if (reinterpret_cast<uintptr_t>(state) & 7u) return fail(ctx, LOSSY_EINVAL, "state: misaligned");
  ctx->burst_state = state;
  ctx->Tenter = threshold_of(p_enter_bad);
  ctx->Tstay = p_leave_bad >= 1.0 ? 0u : threshold_of(1.0 - p_leave_bad);
  return LOSSY_OK;
}

int lossy_set_reliable(lossy_ctx* ctx, const uint64_t* reliable) {
  if (!ctx) return LOSSY_EINVAL;
  if (reinterpret_cast<uintptr_t>(reliable) & 7u) return fail(ctx, LOSSY_EINVAL, "reliable: misaligned");
  if (ctx->K >= (1ull << 32)) return fail(ctx, LOSSY_EINVAL, "too many packets");
  ctx->reliable = reliable;
  return LOSSY_OK;
}

int lossy_packet_sqnorms(lossy_ctx* ctx, const void* const* grads, float* out, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (!out) return fail(ctx, LOSSY_EINVAL, "out: NULL");
  if (int rc = check_table(ctx, grads, "grads: NULL or misaligned pointer")) return rc;
  if (ctx->cfg.n == 0) return LOSSY_OK;
  SqnormArgs A;
  memset(&A, 0, sizeof A);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) A.grads[i] = grads[i];
  A.out = out;
  A.n = ctx->cfg.n;
  A.W = ctx->cfg.W;
  A.P = ctx->cfg.packet_elems;
  A.K = (uint32_t)ctx->K;
  uint64_t blocks = ((uint64_t)A.W * A.K + 7) / 8;
  const uint64_t cap = (uint64_t)ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  cudaStream_t s = (cudaStream_t)stream;
  if (ctx->cfg.grad_dtype == LOSSY_BF16) packet_sqnorms_kernel<BF16><<<(uint32_t)blocks, 256, 0, s>>>(A);
  else packet_sqnorms_kernel<F32><<<(uint32_t)blocks, 256, 0, s>>>(A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "packet norm launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

int lossy_set_lr(lossy_ctx* ctx, float lr) {
  if (!ctx) return LOSSY_EINVAL;
  ctx->cfg.lr = lr;
  return LOSSY_OK;
}

static int aggregate_impl(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev, float* ghat,
                          uint8_t* count, uint64_t* recv_bits, void* stream) {
  if (ctx->cfg.n == 0) return LOSSY_OK;
  if (step == 0) return fail(ctx, LOSSY_EINVAL, "step is 1-based");
  if (int rc = check_table(ctx, grads, "grads: NULL or misaligned pointer")) return rc;
  if (!ghat || !aligned16(ghat)) return fail(ctx, LOSSY_EINVAL, "ghat: NULL or misaligned");
  Params P;
  fill_common(ctx, step, P);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) P.grads[i] = grads[i];
  P.ghat = ghat;
  P.ghat_prev = ghat_prev;
  P.count = count;
  P.recv_bits = recv_bits;
  return run_phase<AGG>(ctx, P, nullptr, nullptr, (cudaStream_t)stream);
}

int lossy_aggregate(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat, uint8_t* count,
                    uint64_t* recv_bits, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  return aggregate_impl(ctx, step, grads, nullptr, ghat, count, recv_bits, stream);
}

static int check_alg1(lossy_ctx* ctx, const float* ghat_prev) {
  if (ctx->cfg.flags & LOSSY_SELF_LOSSLESS)
    return fail(ctx, LOSSY_EINVAL, "LOSSY_SELF_LOSSLESS has no meaning in Algorithm 1 mode");
  if (ctx->cfg.n && (!ghat_prev || !aligned16(ghat_prev))) return fail(ctx, LOSSY_EINVAL, "ghat_prev: NULL or misaligned");
  return LOSSY_OK;
}

int lossy_aggregate_alg1(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev, float* ghat,
                         uint8_t* count, uint64_t* recv_bits, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (int rc = check_alg1(ctx, ghat_prev)) return rc;
  return aggregate_impl(ctx, step, grads, ghat_prev, ghat, count, recv_bits, stream);
}

int lossy_step(lossy_ctx* ctx, uint64_t step, const float* ghat, const uint8_t* count, float* master, float* m,
               float* v, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (ctx->cfg.n == 0) return LOSSY_OK;
  if (step == 0) return fail(ctx, LOSSY_EINVAL, "step is 1-based");
  if (!ghat || !aligned16(ghat) || !master || !aligned16(master)) return fail(ctx, LOSSY_EINVAL, "ghat/master: NULL or misaligned");
  if (ctx->cfg.optimizer == LOSSY_ADAM && (!m || !v || !aligned16(m) || !aligned16(v)))
    return fail(ctx, LOSSY_EINVAL, "Adam needs m and v");
  if ((ctx->cfg.flags & LOSSY_ZERO_SKIP) && !count) return fail(ctx, LOSSY_EINVAL, "LOSSY_ZERO_SKIP needs count");
  Params P;
  fill_common(ctx, step, P);
  P.ghat = const_cast<float*>(ghat);
  P.count_in = count;
  P.master = master;
  P.m = m;
  P.v = v;
  return run_phase<STEP>(ctx, P, nullptr, nullptr, (cudaStream_t)stream);
}

int lossy_broadcast(lossy_ctx* ctx, uint64_t step, const float* master, void* const* replicas, uint64_t* stale_bits,
                    void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (ctx->cfg.n == 0) return LOSSY_OK;
  if (step == 0) return fail(ctx, LOSSY_EINVAL, "step is 1-based");
  if (int rc = check_replicas(ctx, replicas)) return rc;
  if (!master || !aligned16(master)) return fail(ctx, LOSSY_EINVAL, "master: NULL or misaligned");
  Params P;
  fill_common(ctx, step, P);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) P.replicas[i] = replicas[i];
  P.master = const_cast<float*>(master);
  P.stale_bits = stale_bits;
  return run_phase<BCAST>(ctx, P, nullptr, nullptr, (cudaStream_t)stream);
}

int drift_norms(lossy_ctx* ctx, const float* master, const void* const* replicas, float* norms, double* sumsq,
                void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (int rc = check_replicas(ctx, replicas)) return rc;
  if (ctx->cfg.n == 0) {
    if (norms) {
      cudaError_t e = cudaMemsetAsync(norms, 0, ctx->cfg.W * sizeof(float), (cudaStream_t)stream);
      if (e != cudaSuccess) return fail_cuda(ctx, "memset", e);
    }
    return LOSSY_OK;
  }
  if (!master || !aligned16(master)) return fail(ctx, LOSSY_EINVAL, "master: NULL or misaligned");
  Params P;
  fill_common(ctx, 1, P);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) P.replicas[i] = const_cast<void*>(replicas[i]);
  P.master = const_cast<float*>(master);
  return run_phase<DRIFT>(ctx, P, norms, sumsq, (cudaStream_t)stream);
}

static int fused_impl(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev, float* master,
                      float* m, float* v, void* const* replicas, float* ghat, uint8_t* count, uint64_t* recv_bits,
                      uint64_t* stale_bits, float* norms, double* sumsq, void* stream) {
  if (step == 0) return fail(ctx, LOSSY_EINVAL, "step is 1-based");
  if (int rc = check_table(ctx, grads, "grads: NULL or misaligned pointer")) return rc;
  if (int rc = check_replicas(ctx, replicas)) return rc;
  if (ctx->cfg.n == 0) {
    if (norms) {
      cudaError_t e = cudaMemsetAsync(norms, 0, ctx->cfg.W * sizeof(float), (cudaStream_t)stream);
      if (e != cudaSuccess) return fail_cuda(ctx, "memset", e);
    }
    return LOSSY_OK;
  }
  if (!master || !aligned16(master)) return fail(ctx, LOSSY_EINVAL, "master: NULL or misaligned");
  if (ctx->cfg.optimizer == LOSSY_ADAM && (!m || !v || !aligned16(m) || !aligned16(v)))
    return fail(ctx, LOSSY_EINVAL, "Adam needs m and v");
  if (ghat && !aligned16(ghat)) return fail(ctx, LOSSY_EINVAL, "ghat: misaligned");
  Params P;
  fill_common(ctx, step, P);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) {
    P.grads[i] = grads[i];
    P.replicas[i] = replicas[i];
  }
  P.master = master;
  P.m = m;
  P.v = v;
  P.ghat = ghat;
  P.ghat_prev = ghat_prev;
  P.count = count;
  P.recv_bits = recv_bits;
  P.stale_bits = stale_bits;
  // register kernel, all phases fused: prefetching the warp's next chunk pays for W <= 8 (+3..13 %);
  // it costs 20 % on the single-phase kernels, which never set it
  P.prefetch_next = ctx->cfg.W <= 8u ? 1u : 0u;
  cudaStream_t s = (cudaStream_t)stream;
  const bool drift = norms || sumsq;
  // Complete packets go through the bulk-copy pipeline, a short last packet (or everything, when no
  // bulk-copy build fits) through the register kernel. Pass 0 only sizes the grids: the blocks of both
  // launches draw tickets from one counter and the last of them finalises the drift norms.
  uint32_t tma_blocks = 0, tail_blocks = 0;
  for (int pass = 0; pass < 2; ++pass) {
    ctx->plan_only = pass == 0;
    Params Q = P;
    if (pass == 1 && drift) {
      Q.ticket = ctx->ticket;
      Q.total_rows = tma_blocks + tail_blocks;
      Q.norms = norms;
      Q.sumsq = sumsq;
    }
    bool used_tma = false;
    int rc = run_tma(ctx, Q, drift, s, &tma_blocks, &used_tma);
    if (!rc) {
      if (used_tma) {
        Q.chunk_begin = (uint32_t)((ctx->cfg.n / ctx->cfg.packet_elems) * ctx->chunks_per_packet);
        Q.partials_row0 = tma_blocks;
      } else {
        tma_blocks = 0;
      }
      if (Q.chunk_begin < Q.num_chunks)
        rc = drift ? dispatch<AGG | STEP | BCAST | DRIFT>(ctx, Q, s, &tail_blocks) : dispatch<AGG | STEP | BCAST>(ctx, Q, s, &tail_blocks);
      else
        tail_blocks = 0;
    }
    ctx->plan_only = false;
    if (rc) {
      // a ticketed launch may already be queued: the counter must be zero again before the next call
      if (Q.ticket) cudaMemsetAsync(ctx->ticket, 0, sizeof(uint32_t), s);
      return rc;
    }
  }
  return LOSSY_OK;
}

int lossy_fused_step(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* master, float* m, float* v,
                     void* const* replicas, float* ghat, uint8_t* count, uint64_t* recv_bits, uint64_t* stale_bits,
                     float* norms, double* sumsq, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  return fused_impl(ctx, step, grads, nullptr, master, m, v, replicas, ghat, count, recv_bits, stale_bits, norms, sumsq,
                    stream);
}

int lossy_fused_step_alg1(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev, float* master,
                          float* m, float* v, void* const* replicas, float* ghat, uint8_t* count,
                          uint64_t* recv_bits, uint64_t* stale_bits, float* norms, double* sumsq, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (int rc = check_alg1(ctx, ghat_prev)) return rc;
  return fused_impl(ctx, step, grads, ghat_prev, master, m, v, replicas, ghat, count, recv_bits, stale_bits, norms,
                    sumsq, stream);
}

int drift_pairwise(lossy_ctx* ctx, const void* const* replicas, double* d2, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (!d2) return fail(ctx, LOSSY_EINVAL, "d2: NULL");
  if (int rc = check_replicas(ctx, replicas)) return rc;
  if (ctx->cfg.n == 0) return LOSSY_OK;
  PairwiseArgs A;
  memset(&A, 0, sizeof A);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) A.replicas[i] = replicas[i];
  A.d2 = d2;
  A.n = ctx->cfg.n;
  A.W = ctx->cfg.W;
  A.nblk = (ctx->cfg.W + 3) / 4;
  if (ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER) {
    A.elide = 1u;
    A.P = ctx->cfg.packet_elems;
    A.pps = ctx->pps;
    A.k0 = (uint32_t)ctx->cfg.shard_packet0;
    for (uint32_t i = 0; i < ctx->cfg.W; ++i) A.rep_skip[i] = own_elems(ctx, i);
  }
  const uint32_t pairs = A.nblk * (A.nblk + 1) / 2;
  const uint64_t nvec = (A.n + 7) / 8;
  uint64_t bx = (nvec + 255) / 256;
  const uint64_t cap = (uint64_t)ctx->num_sms * 4;
  if (bx > cap) bx = cap;
  const dim3 grid((uint32_t)bx, pairs);
  cudaStream_t s = (cudaStream_t)stream;
  if (ctx->cfg.replica_dtype == LOSSY_BF16) drift_pairwise_kernel<BF16><<<grid, 256, 0, s>>>(A);
  else drift_pairwise_kernel<F32><<<grid, 256, 0, s>>>(A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "pairwise drift launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

int lossy_closed_loop_grads(lossy_ctx* ctx, const float* curv, const float* target, const void* const* noise,
                            const void* const* replicas, void* const* grads_out, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (ctx->cfg.n == 0) return LOSSY_OK;
  if (ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER)
    return fail(ctx, LOSSY_EINVAL, "closed-loop gradients need every worker's full copy (no LOSSY_REPLICA_SKIP_OWNER)");
  if (!curv || !target || !aligned16(curv) || !aligned16(target)) return fail(ctx, LOSSY_EINVAL, "curv/target: NULL or misaligned");
  if (int rc = check_table(ctx, noise, "noise: NULL or misaligned pointer")) return rc;
  if (int rc = check_replicas(ctx, replicas)) return rc;
  if (int rc = check_table(ctx, grads_out, "grads_out: NULL or misaligned pointer")) return rc;
  ClosedLoopArgs A;
  memset(&A, 0, sizeof A);
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) {
    A.noise[i] = noise[i];
    A.replicas[i] = replicas[i];
    A.grads[i] = grads_out[i];
  }
  A.curv = curv;
  A.target = target;
  A.n = ctx->cfg.n;
  A.W = ctx->cfg.W;
  const uint64_t nvec = (A.n + 7) / 8;
  uint64_t blocks = (nvec + 255) / 256;
  const uint64_t cap = (uint64_t)ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  const bool gb = ctx->cfg.grad_dtype == LOSSY_BF16, rb = ctx->cfg.replica_dtype == LOSSY_BF16;
  cudaStream_t s = (cudaStream_t)stream;
  if (gb && rb) closed_loop_grads_kernel<BF16, BF16><<<(uint32_t)blocks, 256, 0, s>>>(A);
  else if (gb) closed_loop_grads_kernel<BF16, F32><<<(uint32_t)blocks, 256, 0, s>>>(A);
  else if (rb) closed_loop_grads_kernel<F32, BF16><<<(uint32_t)blocks, 256, 0, s>>>(A);
  else closed_loop_grads_kernel<F32, F32><<<(uint32_t)blocks, 256, 0, s>>>(A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "closed-loop gradient launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

int lossy_device_status(lossy_ctx* ctx, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  uint32_t word[5] = {0, 0, 0, 0, 0};
  cudaError_t e = cudaMemcpyAsync(word, ctx->status, sizeof word, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(ctx, "status read", e);
  if (word[1] != 0) {   // debug build only; a pipeline that skipped a tile also left through its wait exit (word[0])
    static const char* const kSites[] = {"?", "register kernel", "fused bulk-copy pipeline (packed)", "fused bulk-copy pipeline",
                                         "single-phase bulk-copy pipeline", "gather pipeline"};
    const uint32_t site = word[1] & 15u;
    snprintf(ctx->err, sizeof ctx->err, "device index check failed in the %s: %s elements [%llu, +%u) lie outside the array; not touched, the results of that call are invalid",
             site < 6 ? kSites[site] : kSites[0], (word[1] & kSiteReplica) ? "replica" : "slab",
             (unsigned long long)(((uint64_t)word[3] << 32) | word[2]), word[4]);
    return LOSSY_EDEVCHECK;
  }
  if (word[0] != 0) return fail(ctx, LOSSY_EDEVICE, "a bounded wait inside a kernel gave up; results of that call are invalid");
  return LOSSY_OK;
}

int lossy_has_device_checks(void) { return kDevCheck ? 1 : 0; }

int lossy_selftest_shrink_checks(lossy_ctx* ctx, uint64_t elems) {
  if (!ctx) return LOSSY_EINVAL;
  if (!kDevCheck) return fail(ctx, LOSSY_EINVAL, "this library was built without device index checks");
  ctx->check_shrink = elems;
  return LOSSY_OK;
}

int lossy_reset_status(lossy_ctx* ctx, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  cudaError_t e = cudaMemsetAsync(ctx->status, 0, 5 * sizeof(uint32_t), (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ticket, 0, sizeof(uint32_t), (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(ctx, "status reset", e);
  ctx->err[0] = 0;
  return LOSSY_OK;
}

int lossy_selftest_wait_expiry(lossy_ctx* ctx, uint32_t max_polls, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (max_polls == 0 || max_polls > (1u << 20)) return fail(ctx, LOSSY_EINVAL, "max_polls: 1 .. 2^20");
  wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(max_polls, ctx->status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "self-test launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

int lossy_fused_step_host(lossy_ctx* ctx, uint64_t step, const void* const* host_grads, void* const* dev_grads,
                          float* master, float* m, float* v, void* const* replicas, float* dev_norms,
                          float* host_norms, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (!host_grads || !dev_norms || !host_norms) return fail(ctx, LOSSY_EINVAL, "NULL argument");
  cudaStream_t s = (cudaStream_t)stream;
  const size_t gbytes = (size_t)ctx->cfg.n * (ctx->cfg.grad_dtype == LOSSY_BF16 ? 2 : 4);
  // Zero-copy: when every host buffer is pinned and mapped into the device's address space, the kernel
  // reads the gradients over PCIe itself, so packets that the network dropped are never transferred at all
  // and no staging copy is made. Otherwise (pageable memory) each buffer is staged with cudaMemcpyAsync.
  const void* mapped[LOSSY_MAX_WORKERS];
  bool zero_copy = true;
  for (uint32_t i = 0; i < ctx->cfg.W; ++i) {
    if (!host_grads[i]) return fail(ctx, LOSSY_EINVAL, "NULL gradient pointer");
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_grads[i]) != cudaSuccess) { cudaGetLastError(); zero_copy = false; continue; }
    if (attr.type != cudaMemoryTypeHost || !attr.devicePointer || !aligned16(attr.devicePointer)) zero_copy = false;
    mapped[i] = attr.devicePointer;
  }
  const void* const* step_grads = mapped;
  if (!zero_copy) {
    for (uint32_t i = 0; i < ctx->cfg.W; ++i) {
      if (!dev_grads || !dev_grads[i]) return fail(ctx, LOSSY_EINVAL, "pageable host gradients need staging buffers");
      if (gbytes) {
        cudaError_t e = cudaMemcpyAsync(dev_grads[i], host_grads[i], gbytes, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return fail_cuda(ctx, "gradient upload", e);
      }
    }
    step_grads = dev_grads;
  }
  if (int rc = lossy_fused_step(ctx, step, step_grads, master, m, v, replicas, nullptr, nullptr, nullptr, nullptr,
                                dev_norms, nullptr, stream))
    return rc;
  cudaError_t e = cudaMemcpyAsync(host_norms, dev_norms, ctx->cfg.W * sizeof(float), cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return fail_cuda(ctx, "norm download", e);
  return lossy_device_status(ctx, stream);   // synchronises the stream
}

uint32_t lossy_hash_u32(uint64_t seed, uint64_t step, uint32_t src, uint32_t dst, uint64_t packet) {
  return pair_hash(packet_key_of(step_key_of(seed, step), packet), src, dst);
}

int lossy_mask(const lossy_ctx* ctx, uint64_t step, uint32_t src, uint32_t dst, uint64_t packet, int is_param) {
  if (!ctx) return -1;
  const uint32_t T = is_param ? ctx->Tp : ctx->Tg;
  return lossy_hash_u32(ctx->cfg.seed, step, src, dst, packet) >= T ? 1 : 0;
}

int lossy_mask_grid(lossy_ctx* ctx, uint64_t step, const uint32_t* src, const uint32_t* dst, const uint64_t* packet,
                    uint64_t count, int is_param, uint8_t* out, void* stream) {
  if (!ctx) return LOSSY_EINVAL;
  if (count == 0) return LOSSY_OK;
  if (!src || !dst || !packet || !out) return fail(ctx, LOSSY_EINVAL, "NULL argument");
  const uint64_t blocks = (count + 255) / 256;
  if (blocks > 0x7FFFFFFFull) return fail(ctx, LOSSY_EINVAL, "grid too large");
  mask_grid_kernel<<<(uint32_t)blocks, 256, 0, (cudaStream_t)stream>>>(ctx->cfg.seed, step, src, dst, packet, count,
                                                                      is_param ? ctx->Tp : ctx->Tg, out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail_cuda(ctx, "mask grid launch", e);
  ctx->launches++;
  return LOSSY_OK;
}

const char* lossy_last_error(const lossy_ctx* ctx) { return ctx ? ctx->err : "NULL context"; }
uint64_t lossy_num_packets(const lossy_ctx* ctx) { return ctx ? ctx->K : 0; }
uint64_t lossy_replica_elems(const lossy_ctx* ctx, uint32_t worker) {
  if (!ctx || worker >= ctx->cfg.W) return 0;
  return (ctx->cfg.flags & LOSSY_REPLICA_SKIP_OWNER) ? ctx->cfg.n - own_elems(ctx, worker) : ctx->cfg.n;
}
uint64_t lossy_kernel_launches(const lossy_ctx* ctx) { return ctx ? ctx->launches : 0; }

int lossy_describe_plan(lossy_ctx* ctx, int with_drift, char* buf, size_t size) {
  if (!ctx || !buf || size == 0) return LOSSY_EINVAL;
  snprintf(buf, size, "register kernel");
  if (ctx->cfg.n == 0) return LOSSY_OK;
  Params P;
  fill_common(ctx, 1, P);
  uint32_t blocks = 0;
  bool used = false;
  ctx->plan = buf;
  ctx->plan_size = size;
  ctx->plan_only = true;             // sizes grids, launches nothing
  const int rc = run_tma(ctx, P, with_drift != 0, nullptr, &blocks, &used);
  ctx->plan_only = false;
  ctx->plan = nullptr;
  return rc;
}

}  // extern "C"
