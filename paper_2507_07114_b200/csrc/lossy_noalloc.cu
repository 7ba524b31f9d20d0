// drift_norms_static: the drift norms for callers that must not allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits. Examples are a training loop
// whose memory is handed out once by a framework's caching allocator and then frozen, a
// process that has given every free byte of HBM to its parameter buffers, and a service that
// forbids allocation calls after start-up because an allocation synchronises the device. Such
// a caller cannot use lossy_init (it allocates the per-block partial sums), so this entry point
// takes the configuration directly and keeps its partial sums in the array below, which is part
// of the library image: every GPU that loads the library holds these 512 KB until the process
// exits.
#include "../../include/lossy.h"

#include <mutex>

#include "lossy_kernels.cuh"

using namespace lossy;

namespace {

constexpr uint32_t kStaticRows = 1024;   // per-block partial rows: at most 1024 blocks per call
// Scratch shared by every call in the process (per device): [kStaticRows][kMaxW] doubles = 512 KB.
static __device__ __align__(256) double g_static_partials[kStaticRows * kMaxW];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
double* g_ptr[kMaxDevices];     // device address of g_static_partials, per device
int g_sms[kMaxDevices];

// Set-up, once per device, with that device current: the array's name is only a host-side
// handle here, so ask the runtime for its device address before giving it to a kernel.
// This first call on a device is also the one that may load the library's device code (CUDA loads
// modules lazily), which reserves memory for the kernels and for the array itself: it belongs at
// start-up, before the caller commits or freezes its memory and before any stream capture. The
// cached address is valid until the device is reset (cudaDeviceReset); a process that resets a
// device must not call this entry point on it afterwards.
int static_scratch(double** out, int* sms) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return LOSSY_ECUDA;
  if (dev < 0 || dev >= kMaxDevices) return LOSSY_ELIMIT;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_ptr[dev]) {
    double* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials);
    if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return LOSSY_ENOMEM; }   // no room left to load the library image
    if (e != cudaSuccess || !p) return LOSSY_ECUDA;
    int n = 0;
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || n < 1) return LOSSY_ECUDA;
    g_sms[dev] = n;
    g_ptr[dev] = p;
  }
  *out = g_ptr[dev];
  *sms = g_sms[dev];
  return LOSSY_OK;
}

template <class RT, bool ELIDE>
int launch_static(const Params& P, int sms, cudaStream_t s, uint32_t* blocks_out) {
  auto kern = lossy_kernel<DRIFT, F32, RT, 0, ELIDE>;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, 0) != cudaSuccess) return LOSSY_ECUDA;
  if (per_sm < 1) per_sm = 1;
  uint64_t blocks = (uint64_t)sms * (uint64_t)per_sm;
  const uint64_t need = ((uint64_t)P.num_chunks + kWarps - 1) / kWarps;
  if (blocks > need) blocks = need;
  if (blocks > kStaticRows) blocks = kStaticRows;   // the grid never outgrows the static rows
  kern<<<(uint32_t)blocks, kThreads, 0, s>>>(P);
  if (cudaGetLastError() != cudaSuccess) return LOSSY_ECUDA;
  *blocks_out = (uint32_t)blocks;
  return LOSSY_OK;
}

}  // namespace

extern "C" int drift_norms_static(const lossy_config* cfg, const float* master, const void* const* replicas,
                                  float* norms, double* sumsq, void* stream) {
  if (!cfg || !replicas || (!norms && !sumsq)) return LOSSY_EINVAL;
  if (cfg->W == 0 || cfg->packet_elems == 0 || cfg->packet_elems % 8 != 0) return LOSSY_EINVAL;
  if (cfg->replica_dtype > LOSSY_BF16) return LOSSY_EINVAL;
  // sizes beyond what the static scratch and the 32-bit chunk index cover
  if (cfg->W > LOSSY_MAX_WORKERS) return LOSSY_ELIMIT;
  const uint64_t K = (cfg->n + cfg->packet_elems - 1) / cfg->packet_elems;
  const uint64_t cpp = (cfg->packet_elems + kChunk - 1) / kChunk;
  if (K * cpp > LOSSY_STATIC_MAX_CHUNKS) return LOSSY_ELIMIT;
  // the shard map (only the owner-elided replica layout depends on it): a packet range of a larger bucket, or the whole bucket
  const bool elide = (cfg->flags & LOSSY_REPLICA_SKIP_OWNER) != 0;
  if (cfg->bucket_packets ? (cfg->bucket_packets >= (1ull << 31) || cfg->shard_packet0 + K > cfg->bucket_packets)
                          : cfg->shard_packet0 != 0)
    return LOSSY_EINVAL;
  const uint64_t Kb = cfg->bucket_packets ? cfg->bucket_packets : K;
  const uint64_t pps = (Kb + cfg->W - 1) / cfg->W;

  cudaStream_t s = (cudaStream_t)stream;
  if (cfg->n == 0) {
    if (norms && cudaMemsetAsync(norms, 0, cfg->W * sizeof(float), s) != cudaSuccess) return LOSSY_ECUDA;
    return LOSSY_OK;
  }
  if (!master || (reinterpret_cast<uintptr_t>(master) & 15u)) return LOSSY_EINVAL;

  double* scratch = nullptr;
  int sms = 0;
  if (int rc = static_scratch(&scratch, &sms)) return rc;

  Params P;
  memset(&P, 0, sizeof P);
  P.n = cfg->n;
  P.num_chunks = (uint32_t)(K * cpp);
  P.chunks_per_packet = (uint32_t)cpp;
  P.pps = pps ? (uint32_t)pps : 1u;
  P.k0 = (uint32_t)cfg->shard_packet0;
  P.K = (uint32_t)K;
  P.P = cfg->packet_elems;
  P.W = cfg->W;
  P.flags = elide ? kSkipOwner : 0u;
  fill_rep_skip(P, elide);
  for (uint32_t i = 0; i < cfg->W; ++i) {
    if (elide && P.rep_skip[i] == cfg->n) continue;           // this worker owns everything here: its replica holds nothing
    if (!replicas[i] || (reinterpret_cast<uintptr_t>(replicas[i]) & 15u)) return LOSSY_EINVAL;
  }
  P.master = const_cast<float*>(master);
  for (uint32_t i = 0; i < cfg->W; ++i) P.replicas[i] = const_cast<void*>(replicas[i]);
  // Every row that the finalize kernel reads is written in full by this call's own blocks
  // first, so nothing in the shared array has to start at zero.
  P.partials = scratch;
  uint32_t blocks = 0;
  int rc;
  if (elide) rc = cfg->replica_dtype == LOSSY_BF16 ? launch_static<BF16, true>(P, sms, s, &blocks) : launch_static<F32, true>(P, sms, s, &blocks);
  else rc = cfg->replica_dtype == LOSSY_BF16 ? launch_static<BF16, false>(P, sms, s, &blocks) : launch_static<F32, false>(P, sms, s, &blocks);
  if (rc) return rc;
  drift_finalize_kernel<<<cfg->W, 32, 0, s>>>(scratch, blocks, cfg->W, norms, sumsq);
  return cudaGetLastError() == cudaSuccess ? LOSSY_OK : LOSSY_ECUDA;
}
