/*
 * lossy_oracle.c — TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-threaded CPU statement of one iteration of the paper's
 * packet-loss-tolerant data-parallel step (Section 3 "Model Formulation", steps
 * (2) gradient communication, (3) local update, (4) parameter broadcast, and the
 * drift quantity of "Quantifying Model Drift"). Scalar loops in the paper's
 * order: packet -> masks -> element -> worker. No blocking, no fusion tricks.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 * It shares no code with the CUDA library and includes none of its headers.
 *
 * The file compiles twice:
 *   default            REAL = float : the contract precision (fp32 accumulation in
 *                      ascending worker order, every operation rounded separately;
 *                      build with -ffp-contract=off). Symbols: oracle_*.
 *   -DORACLE_F64       REAL = double: the same steps in fp64, used by the CPU
 *                      tests to show that the fp32 contract path stays within
 *                      tolerance of the mathematical definition. Symbols: oracle64_*.
 *
 * Pins (tests/test_oracle_*.py): p = 0 equals the plain mean; exhaustive
 * enumeration of all delivery patterns for tiny W, K; unbiasedness over seeds;
 * the four-case drift rule of the Bounded Model Drift proof; exact stationary
 * drift for i.i.d. increments; optimizer trajectories against closed forms; hash
 * statistics; slab by slab equals the whole bucket. The paper prints no worked
 * numeric example, so values at scale rest on the enumeration of tiny cases plus
 * that packet independence; no function here is without a pin.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef ORACLE_F64
typedef double REAL;
#define NAME(x) oracle64_##x
#else
typedef float REAL;
#define NAME(x) oracle_##x
#endif

enum { DT_F32 = 0, DT_BF16 = 1 };
enum { OPT_SGD = 0, OPT_ADAM = 1 };
enum { FLAG_SELF_LOSSLESS = 1u, FLAG_ZERO_SKIP = 2u,
       /* Section 3 step (4) sends a shard's update "to all OTHER workers": worker i never needs a replica of
        * its own shard (what it owns IS the master). With this flag replicas[i] holds only the packets that
        * worker i does not own, in bucket order, back to back. */
       FLAG_REPLICA_SKIP_OWNER = 8u };

typedef struct {
  uint32_t W;            /* workers = shards = replicas (paper's N)                    */
  uint32_t packet_elems; /* P                                                         */
  uint64_t n;            /* elements of the WHOLE bucket (fixes K and the shard map)   */
  uint64_t packet_base;  /* global id of the bucket's packet 0                         */
  double p_grad, p_param;
  uint64_t seed;
  uint32_t grad_dtype, replica_dtype, optimizer, flags;
  float lr, beta1, beta2, eps;
} oracle_config;

/* ------------------------------------------------------------------------- */
/* Delivery indicators: Section 3 draws s ~ Bernoulli(1-p) per (src,dst)      */
/* transmission; Algorithm 1 tests Uniform(0,1) < p. Here the uniform is a    */
/* counter-based hash of (seed, step, src, dst, packet): two keyed rounds of  */
/* the splitmix64 output mix, then one round over the (src,dst) pair.         */
/* ------------------------------------------------------------------------- */
/* exported so a test can pin it to the published splitmix64 test vector */
uint64_t NAME(mix64)(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
  z ^= z >> 27; z *= 0x94D049BB133111EBULL;
  z ^= z >> 31;
  return z;
}

uint32_t NAME(hash_u32)(uint64_t seed, uint64_t step, uint32_t src, uint32_t dst, uint64_t packet) {
  uint64_t seed_key = NAME(mix64)(seed ^ 0x6A09E667F3BCC908ULL);
  uint64_t step_key = NAME(mix64)(seed_key + step * 0x9E3779B97F4A7C15ULL);
  uint64_t pkt_key = NAME(mix64)(step_key ^ (packet * 0xD6E8FEB86659FD93ULL));
  uint64_t pair = ((uint64_t)src << 32) | (uint64_t)dst;
  return (uint32_t)(NAME(mix64)(pkt_key + pair * 0xC2B2AE3D27D4EB4FULL) >> 32);
}

/* Drop iff u < T with T = floor(p * 2^32): p = 0 never drops. */
uint32_t NAME(threshold)(double p) { return (uint32_t)floor(p * 4294967296.0); }

int NAME(delivered)(uint64_t seed, uint64_t step, uint32_t src, uint32_t dst, uint64_t packet, double p) {
  return NAME(hash_u32)(seed, step, src, dst, packet) >= NAME(threshold)(p);
}

/* ------------------------------------------------------------------------- */
/* bf16 <-> fp32. Widening is exact; narrowing is IEEE round-to-nearest-even. */
/* ------------------------------------------------------------------------- */
static float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return f;
}
uint16_t NAME(f32_to_bf16)(float f) {
  uint32_t u; memcpy(&u, &f, 4);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;                       /* ties go to the even 16-bit pattern */
  return (uint16_t)(u >> 16);
}

static REAL load_grad(const void* g, uint32_t dt, uint64_t e) {
  return dt == DT_BF16 ? (REAL)bf16_to_f32(((const uint16_t*)g)[e]) : (REAL)((const float*)g)[e];
}

/* Shard map: K = ceil(n/P) packets, contiguous shards of pps = ceil(K/W) packets. */
uint64_t NAME(num_packets)(const oracle_config* c) {
  return (c->n + c->packet_elems - 1) / c->packet_elems;
}
uint32_t NAME(owner)(const oracle_config* c, uint64_t k) {
  uint64_t K = NAME(num_packets)(c);
  uint64_t pps = (K + c->W - 1) / c->W;
  return (uint32_t)(k / pps);
}

/*
 * One iteration over a slab of the bucket.
 *
 * The slab starts at packet k0 of the bucket and holds n_slab elements (it ends
 * on a packet boundary or at the end of the bucket). Every array argument is
 * indexed from the slab's first element / first packet; packets evolve
 * independently, so a bucket may be checked slab by slab.
 *
 *   grads[i]        worker i's gradient slab (cfg.grad_dtype), read only
 *   master, m, v    REAL [n_slab], updated in place (m, v ignored for SGD)
 *   replicas[i]     worker i's copy of the slab (cfg.replica_dtype), updated in place; with
 *                   FLAG_REPLICA_SKIP_OWNER the slab's packets that worker i does not own, back to back
 *   ghat_prev       NULL: Section 3's per-link loss (the default). Non-NULL (REAL [n_slab], in/out):
 *                   Algorithm 1's gradient half — the reduce over all W workers is reliable,
 *                   then ONE draw per packet decides whether the owner keeps the fresh aggregate
 *                   (and saves it as "prev") or falls back to the saved previous aggregate
 *   burst           NULL: independent Bernoulli drops (the paper's model). Non-NULL: double[2] =
 *                   {P(good->bad), P(bad->good)} of a two-state (Gilbert-Elliott) chain per link
 *                   and packet, the bursty loss the paper's Limitations leave open: with u the same
 *                   hash value, bad_t = bad_{t-1} ? (u >= T_leave) : (u < T_enter), T = floor(p 2^32);
 *                   a transmission is lost iff its link is bad at step t. p_grad / p_param are unused.
 *   burst_in/out    [2][packets] uint64 (row 0 gradient links, row 1 broadcast links; bit i = link of
 *                   worker i is bad): state after step t-1 (read) and after step t (written)
 *   reliable        optional [2][packets] uint64 (row 0 gradient links, row 1 broadcast links): bit i set =
 *                   that transmission travels on a reliable channel and is never lost (the hybrid
 *                   reliable/unreliable transport of the paper's Future Directions)
 *   recv_force      optional [packets] uint64: use these delivery bits (bit i = s_i)
 *                   instead of the hash — the hook the exhaustive-pattern test uses
 *                   (Algorithm 1 mode: bit 0 = the packet's aggregate survives)
 *   stale_force     optional [packets] uint64: bit i = replica i misses the broadcast
 *   ghat            optional REAL [n_slab] out
 *   count           optional uint8 [packets] out; recv_bits / stale_bits optional uint64 [packets] out
 *   age[i]          optional uint32 [packets] in/out: steps since replica i last took packet k
 *   sumsq           optional double [W]: sum_e (replica_i[e] - cast(theta[e]))^2 is ADDED per replica
 * Returns 0, or 1 for a bad argument.
 */
int NAME(step)(const oracle_config* c, uint64_t step, uint64_t k0, uint64_t n_slab,
               const void* const* grads, REAL* master, REAL* m, REAL* v, void* const* replicas,
               REAL* ghat_prev, const double* burst, const uint64_t* burst_in, uint64_t* burst_out,
               const uint64_t* reliable, const uint64_t* recv_force, const uint64_t* stale_force,
               REAL* ghat, uint8_t* count, uint64_t* recv_bits, uint64_t* stale_bits,
               uint32_t* const* age, double* sumsq) {
  if (!c || c->W == 0 || c->W > 64 || c->packet_elems == 0) return 1;
  if (!(c->p_grad >= 0.0 && c->p_grad < 1.0) || !(c->p_param >= 0.0 && c->p_param < 1.0)) return 1;
  const uint32_t W = c->W;
  const uint64_t P = c->packet_elems;
  const uint32_t Tg = NAME(threshold)(c->p_grad), Tp = NAME(threshold)(c->p_param);
  const uint64_t slab_start = k0 * P;
  if (slab_start + n_slab > c->n) return 1;
  const uint64_t packets = (n_slab + P - 1) / P;
  uint32_t Tenter = 0, Tleave = 0;
  if (burst) {
    if (!burst_in || !burst_out) return 1;
    if (!(burst[0] >= 0.0 && burst[0] < 1.0) || !(burst[1] > 0.0 && burst[1] <= 1.0)) return 1;
    Tenter = NAME(threshold)(burst[0]);
    /* P(bad->good) = 1 means "always leave": the compare u >= T can then never fail */
    Tleave = burst[1] >= 1.0 ? 0u : NAME(threshold)(1.0 - burst[1]);
  }

  /* Adam's scalars: (1-beta) in fp32, bias corrections in double then rounded once. */
  const REAL lr = (REAL)c->lr, b1 = (REAL)c->beta1, b2 = (REAL)c->beta2, eps = (REAL)c->eps;
  const REAL omb1 = (REAL)1 - b1, omb2 = (REAL)1 - b2;
  const REAL ibc1 = (REAL)(1.0 / (1.0 - pow((double)c->beta1, (double)step)));
  const REAL ibc2 = (REAL)(1.0 / (1.0 - pow((double)c->beta2, (double)step)));

  /* owner-elided replicas: where the current packet starts inside replicas[i] */
  const int elide = (c->flags & FLAG_REPLICA_SKIP_OWNER) != 0;
  uint64_t cursor[64];
  for (uint32_t i = 0; i < 64; ++i) cursor[i] = 0;

  for (uint64_t kl = 0; kl < packets; ++kl) {
    const uint64_t k = k0 + kl;                 /* packet within the bucket */
    const uint64_t kg = c->packet_base + k;     /* global packet id (hash only) */
    const uint32_t j = NAME(owner)(c, k);       /* owner W_j of this packet */
    const uint64_t e0 = kl * P;
    const uint64_t e1 = (e0 + P < n_slab) ? e0 + P : n_slab;

    /* (2) which workers' pieces reached the owner: s^(i,j) */
    uint64_t recv = 0;
    uint64_t gbad = 0, pbad = 0;   /* link states after this step (bursty mode) */
    if (ghat_prev) {
      /* Algorithm 1: "reduce-scatter" is lossless, then Uniform(0,1) < p_grad drops the whole packet */
      int keep;
      if (recv_force) keep = (int)(recv_force[kl] & 1ULL);
      else if (burst) {
        uint32_t u = NAME(hash_u32)(c->seed, step, j, j, kg);
        int was_bad = (int)(burst_in[kl] & 1ULL);
        int bad = was_bad ? (u < Tleave) : (u < Tenter);
        gbad = (uint64_t)bad;
        keep = !bad;
      } else keep = NAME(hash_u32)(c->seed, step, j, j, kg) >= Tg;
      if (keep) recv = W == 64 ? ~0ULL : ((1ULL << W) - 1ULL);
    } else if (recv_force) recv = recv_force[kl];
    else
      for (uint32_t i = 0; i < W; ++i) {
        uint32_t u = NAME(hash_u32)(c->seed, step, i, j, kg);
        int s;
        if (burst) {
          int was_bad = (int)((burst_in[kl] >> i) & 1ULL);
          int bad = was_bad ? (u < Tleave) : (u < Tenter);   /* stays bad unless u >= T_leave */
          if ((c->flags & FLAG_SELF_LOSSLESS) && i == j) bad = 0;
          if (bad) gbad |= 1ULL << i;
          s = !bad;
        } else {
          s = u >= Tg;
          if ((c->flags & FLAG_SELF_LOSSLESS) && i == j) s = 1;
        }
        if (s) recv |= 1ULL << i;
      }
    if (reliable && !recv_force) {
      const uint64_t all = W == 64 ? ~0ULL : ((1ULL << W) - 1ULL);
      /* Algorithm 1 mode has one transmission per packet: bit 0 makes it reliable */
      if (ghat_prev) { if (reliable[kl] & 1ULL) recv = all; }
      else recv |= reliable[kl] & all;
    }
    uint32_t cnt = 0;
    for (uint32_t i = 0; i < W; ++i) cnt += (uint32_t)((recv >> i) & 1ULL);
    if (count) count[kl] = (uint8_t)cnt;
    if (recv_bits) recv_bits[kl] = recv;

    /* (4) which replicas take the broadcast of this packet: r^(j,i); the owner always has it */
    uint64_t stale = 0;
    if (stale_force) stale = stale_force[kl] & ~(1ULL << j);
    else if (burst) {
      for (uint32_t i = 0; i < W; ++i) {
        if (i == j) continue;
        uint32_t u = NAME(hash_u32)(c->seed, step, j, i, kg);
        int was_bad = (int)((burst_in[packets + kl] >> i) & 1ULL);
        int bad = was_bad ? (u < Tleave) : (u < Tenter);
        if (bad) { pbad |= 1ULL << i; stale |= 1ULL << i; }
      }
    } else
      for (uint32_t i = 0; i < W; ++i)
        if (i != j && NAME(hash_u32)(c->seed, step, j, i, kg) < Tp) stale |= 1ULL << i;
    if (burst) { burst_out[kl] = gbad; burst_out[packets + kl] = pbad; }
    if (reliable && !stale_force) stale &= ~reliable[packets + kl];
    if (stale_bits) stale_bits[kl] = stale;

    for (uint64_t e = e0; e < e1; ++e) {
      /* unbiased estimate: masked sum in ascending worker order over the received count */
      REAL acc = 0;
      for (uint32_t i = 0; i < W; ++i)
        if ((recv >> i) & 1ULL) acc = acc + load_grad(grads[i], c->grad_dtype, e);
      REAL gh = cnt > 0 ? acc / (REAL)cnt : (REAL)0;
      if (ghat_prev) {
        /* Algorithm 1: dropped => g <- g_prev ; else g_prev <- g */
        if (cnt == 0) gh = ghat_prev[e];
        else ghat_prev[e] = gh;
      }
      if (ghat) ghat[e] = gh;

      /* (3) the owner's update of its shard */
      if (!(cnt == 0 && (c->flags & FLAG_ZERO_SKIP))) {
        if (c->optimizer == OPT_SGD) {
          REAL t1 = lr * gh;
          master[e] = master[e] - t1;
        } else {
          REAL t1 = b1 * m[e], t2 = omb1 * gh;
          REAL mn = t1 + t2;
          REAL t3 = b2 * v[e], t4 = omb2 * gh;
          REAL t5 = t4 * gh;
          REAL vn = t3 + t5;
          REAL mh = mn * ibc1, vh = vn * ibc2;
          REAL num = lr * mh;
#ifdef ORACLE_F64
          REAL den = sqrt(vh) + eps;
#else
          REAL den = sqrtf(vh) + eps;
#endif
          REAL upd = num / den;
          m[e] = mn; v[e] = vn;
          master[e] = master[e] - upd;
        }
      }

      /* (4) broadcast the value that goes on the wire; a miss keeps the old copy */
      const float wire_f = (float)master[e];
      const uint16_t wire_h = NAME(f32_to_bf16)(wire_f);
      const double x = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(wire_h) : (double)wire_f;
      for (uint32_t i = 0; i < W; ++i) {
        if (elide && i == j) continue;           /* the owner keeps no replica of its own shard: drift term 0 */
        const uint64_t at = elide ? cursor[i] + (e - e0) : e;
        if (!((stale >> i) & 1ULL)) {
          if (c->replica_dtype == DT_BF16) ((uint16_t*)replicas[i])[at] = wire_h;
          else ((float*)replicas[i])[at] = wire_f;
        } else if (sumsq) {
          double r = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(((const uint16_t*)replicas[i])[at])
                                                 : (double)((const float*)replicas[i])[at];
          double d = r - x;
          sumsq[i] += d * d;
        }
      }
    }
    for (uint32_t i = 0; i < W; ++i)
      if (i != j) cursor[i] += e1 - e0;
    if (age)
      for (uint32_t i = 0; i < W; ++i) age[i][kl] = ((stale >> i) & 1ULL) ? age[i][kl] + 1u : 0u;
  }
  return 0;
}

/*
 * Drift of every replica from the owners' current values, on its own (no
 * broadcast): sumsq[i] += sum_e (replica_i[e] - cast(master[e]))^2 in double.
 * The slab starts at bucket packet k0 (only the owner-elided layout needs it: there
 * worker i has no copy of its own packets, which add nothing to its sum).
 */
int NAME(drift_sumsq)(const oracle_config* c, uint64_t k0, uint64_t n_slab, const REAL* master,
                      const void* const* replicas, double* sumsq) {
  if (!c || !sumsq) return 1;
  const int elide = (c->flags & FLAG_REPLICA_SKIP_OWNER) != 0;
  uint64_t at[64];                               /* next element of replicas[i] */
  for (uint32_t i = 0; i < 64; ++i) at[i] = 0;
  for (uint64_t e = 0; e < n_slab; ++e) {
    const uint32_t j = NAME(owner)(c, k0 + e / c->packet_elems);
    const float wire_f = (float)master[e];
    const double x = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(NAME(f32_to_bf16)(wire_f)) : (double)wire_f;
    for (uint32_t i = 0; i < c->W; ++i) {
      if (elide && i == j) continue;
      const uint64_t q = at[i]++;
      double r = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(((const uint16_t*)replicas[i])[q])
                                             : (double)((const float*)replicas[i])[q];
      double d = r - x;
      sumsq[i] += d * d;
    }
  }
  return 0;
}

/*
 * Closed-loop stand-in for "(1) Local gradient computation" of Section 3: worker i evaluates the
 * gradient of a diagonal quadratic, L(theta) = 1/2 sum_e a[e] (theta[e] - x*[e])^2, at ITS OWN
 * (possibly stale) replica and adds its mini-batch noise:
 *     g_i[e] = cast( a[e] * (replica_i[e] - x*[e]) + noise_i[e] )
 * sub, mul, add each rounded on its own; cast = identity (fp32 gradients) or RNE to bf16.
 */
int NAME(closed_loop_grads)(const oracle_config* c, uint64_t n_slab, const float* curv, const float* target,
                            const void* const* noise, const void* const* replicas, void* const* grads_out) {
  if (!c || !curv || !target || !noise || !replicas || !grads_out) return 1;
  if (c->flags & FLAG_REPLICA_SKIP_OWNER) return 1;   /* needs every worker's full copy */
  for (uint32_t i = 0; i < c->W; ++i)
    for (uint64_t e = 0; e < n_slab; ++e) {
      REAL rep = c->replica_dtype == DT_BF16 ? (REAL)bf16_to_f32(((const uint16_t*)replicas[i])[e])
                                             : (REAL)((const float*)replicas[i])[e];
      REAL d = rep - (REAL)target[e];
      REAL q = (REAL)curv[e] * d;
      REAL r = q + load_grad(noise[i], c->grad_dtype, e);
      if (c->grad_dtype == DT_BF16) ((uint16_t*)grads_out[i])[e] = NAME(f32_to_bf16)((float)r);
      else ((float*)grads_out[i])[e] = (float)r;
    }
  return 0;
}

/*
 * The theorem's own quantity ("Quantifying Model Drift": D = theta^(i,j) - theta^(k,j) between two
 * workers' copies): d2[i*W + k] += sum_e (replica_i[e] - replica_k[e])^2 for every pair, in double.
 */
int NAME(pairwise_sumsq)(const oracle_config* c, uint64_t k0, uint64_t n_slab, const void* const* replicas, double* d2) {
  if (!c || !replicas || !d2) return 1;
  const uint32_t W = c->W;
  /* Owner-elided layout: the owner of an element holds no replica of it, so on that element the sums run
   * over the pairs of the other workers only (the theorem's D is between two receivers of shard j). */
  const int elide = (c->flags & FLAG_REPLICA_SKIP_OWNER) != 0;
  uint64_t at[64];
  for (uint32_t i = 0; i < 64; ++i) at[i] = 0;
  for (uint64_t e = 0; e < n_slab; ++e) {
    const uint32_t j = NAME(owner)(c, k0 + e / c->packet_elems);
    for (uint32_t i = 0; i < W; ++i) {
      if (elide && i == j) continue;
      double ri = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(((const uint16_t*)replicas[i])[at[i]])
                                              : (double)((const float*)replicas[i])[at[i]];
      for (uint32_t k = 0; k < W; ++k) {
        if (elide && k == j) continue;
        double rk = c->replica_dtype == DT_BF16 ? (double)bf16_to_f32(((const uint16_t*)replicas[k])[at[k]])
                                                : (double)((const float*)replicas[k])[at[k]];
        double d = ri - rk;
        d2[(size_t)i * W + k] += d * d;
      }
    }
    for (uint32_t i = 0; i < W; ++i)
      if (!(elide && i == j)) at[i]++;
  }
  return 0;
}

/*
 * Per (worker, packet) squared norm of the gradient pieces, the input of an importance rule
 * (Future Directions: gradients of large norm are the traffic to send reliably): out[i * packets + k], double.
 */
int NAME(packet_sqnorms)(const oracle_config* c, uint64_t n_slab, const void* const* grads, double* out) {
  if (!c || !grads || !out) return 1;
  const uint64_t P = c->packet_elems, packets = (n_slab + P - 1) / P;
  for (uint32_t i = 0; i < c->W; ++i)
    for (uint64_t k = 0; k < packets; ++k) {
      double s = 0.0;
      const uint64_t e1 = (k + 1) * P < n_slab ? (k + 1) * P : n_slab;
      for (uint64_t e = k * P; e < e1; ++e) {
        double g = (double)load_grad(grads[i], c->grad_dtype, e);
        s += g * g;
      }
      out[(size_t)i * packets + k] = s;
    }
  return 0;
}

/*
 * Delivery indicators alone (Section 3's s and r for independent loss), for `packets` packets starting at
 * bucket packet k0: recv bit i = worker i's piece reached the owner, stale bit i = replica i missed the
 * broadcast, count = received pieces. Lets a test compare EVERY packet of a full-size bucket.
 */
int NAME(masks)(const oracle_config* c, uint64_t step, uint64_t k0, uint64_t packets, uint64_t* recv_bits,
                uint64_t* stale_bits, uint8_t* count) {
  if (!c || !recv_bits || !stale_bits || !count) return 1;
  const uint32_t Tg = NAME(threshold)(c->p_grad), Tp = NAME(threshold)(c->p_param);
  for (uint64_t kl = 0; kl < packets; ++kl) {
    const uint64_t k = k0 + kl, kg = c->packet_base + k;
    const uint32_t j = NAME(owner)(c, k);
    uint64_t recv = 0, stale = 0;
    uint32_t cnt = 0;
    for (uint32_t i = 0; i < c->W; ++i) {
      int s = NAME(hash_u32)(c->seed, step, i, j, kg) >= Tg;
      if ((c->flags & FLAG_SELF_LOSSLESS) && i == j) s = 1;
      if (s) { recv |= 1ULL << i; ++cnt; }
      if (i != j && NAME(hash_u32)(c->seed, step, j, i, kg) < Tp) stale |= 1ULL << i;
    }
    recv_bits[kl] = recv; stale_bits[kl] = stale; count[kl] = (uint8_t)cnt;
  }
  return 0;
}
