// Tensor-core (tcgen05) path, host side: tensor maps, workspace carving, slice-width choice, launches.
//
// Both kernels go on the caller's stream; the chain kernel is launched as a programmatic dependent of the
// prep kernel, so it may start once every prep CTA is running.  Two modes:
//   sequential: the chain kernel sets itself up under the prep kernel's tail and then waits for that whole grid;
//   concurrent: when the chain CTAs need at most half of the SMs and the cost model below expects a gain, the
//     prep kernel is sized to the other SMs
//     (one CTA per SM) and the chain kernel consumes each chunk as soon as the prep work group of that chunk
//     has published it (release/acquire flag per chunk in the workspace, stamped with a per-call epoch so that
//     nothing has to be cleared).  The flags' producer is running (or done) before a consumer starts, whatever
//     else the GPU is doing, so the consumer's bounded waits cannot starve.
// HA_LA_TC_OVERLAP=0 forces the sequential mode, =2 the concurrent one wherever it is legal.
#include <cuda.h>
#include <stdlib.h>

#include <atomic>
#include <random>

#include "tc_common.cuh"

namespace ha_la {

cudaError_t launch_tc_prep(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                           const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, int64_t epoch,
                           int reserved_sms, cudaStream_t stream);
cudaError_t launch_tc_chain(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                            const CUtensorMap& mk, const CUtensorMap& mo, int nv, int64_t epoch, bool dependent,
                            uint32_t spin_limit, const SegBuffers& sg, cudaStream_t stream);
cudaError_t launch_tc_seg_fix(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const SegBuffers& sg,
                              cudaStream_t stream);

cudaError_t configure_tc_prep(const Problem& p);
cudaError_t configure_tc_chain(const Problem& p, int nv);

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime, so the library does not link libcuda.
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// [T][H][128] bf16 token-major tensor; box = 64 features x 1 head x 64 tokens, 128-byte swizzle.
// The innermost coordinate of every load is 0 or 64 elements (a multiple of 16 bytes).
bool make_map(CUtensorMap* m, const void* base, int T, int H) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)H, (cuuint64_t)(T > 0 ? T : 1)};
  const cuuint64_t strides[2] = {128 * 2, (cuuint64_t)H * 128 * 2};
  const cuuint32_t box[3] = {64, 1, 64};
  const cuuint32_t es[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The output o as the chain kernel stores it: box = one slice block (nv <= 64 channels) x 1 head x 64 tokens,
// swizzled like the kernel's staging tile.  Store coordinates are multiples of 32 channels (64 bytes).
bool make_map_o(CUtensorMap* m, const void* base, int T, int H, int nv) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)H, (cuuint64_t)(T > 0 ? T : 1)};
  const cuuint64_t strides[2] = {128 * 2, (cuuint64_t)H * 128 * 2};
  const cuuint32_t box[3] = {(cuuint32_t)(nv < 64 ? nv : 64), 1, 64};
  const cuuint32_t es[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, nv < 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int n = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    return v;
  }();
  return n;
}

constexpr int kMaxDevices = 64;
constexpr uint32_t kDefaultSpinLimit = 4u << 20;      // polls before a device-side bounded wait gives up
std::atomic<uint32_t> g_calls{0};

// Epoch of a concurrent-mode call: (random per-process tag, never 0) << 40 | call counter << 8; the low byte is zero
// (the chain kernel's slices count in it).
int64_t next_epoch() {
  static const uint32_t tag = [] {
    std::random_device rd;
    uint32_t t = rd();
    return (t & 0x7fffffu) ? t : 0x9e3779b9u;
  }();
  return (int64_t)(((uint64_t)(tag & 0x7fffffu) << 40) | ((uint64_t)(uint32_t)g_calls.fetch_add(1) << 8));
}

// Slice width (value channels per chain CTA) and launch mode, from a cost model measured on B200.
// Chain kernel: bound by the latency of its two MMA round trips per chunk, which grows with the slice width (about
// 0.9 / 1.23 / 1.5 us per chunk at 32 / 64 / 128 channels; the last is a kernel of its own that keeps the whole head's
// state in tensor memory) and does not depend on the number of CTAs.  Each CTA
// needs an SM of its own, so the kernel's time is about  max(longest sequence, all sequences / SMs)  in chunk-times
// when the lengths differ (more CTAs than SMs are started longest sequence first and pack well), and whole rounds
// when they do not: with few chains the narrow slice wins, with many a wider one may.
// Prep kernel: throughput-bound, about 3.45 (GDN) / 9.8 (KDA) SM-microseconds per (chunk, head), and never
// faster than its rounds of one item per work group (3 per SM for GDN, 1 for KDA) at 9 / 10.5 us per item.
// Back to back the two times add.  Concurrently (allowed while the chain's CTAs leave at least half of the SMs to
// the prep kernel) the call takes the longer of the chain and of the prep kernel on the remaining SMs (plus some
// interference), plus the wait for the first chunks; with several sequences the prep kernel works through them
// one after the other, so the last sequence's chain starts only when most of the prep work is done.
// Only bounds are known on the host: max_len for the longest sequence, max_chunks for the total.
struct TcPlan { int nv; bool concurrent; int nseg; };

TcPlan plan_tc(const Problem& p) {
  const int sms = sm_count();
  const long long chains = (long long)p.N * p.HV;
  const double longest = (double)((p.max_len + kChunk - 1) / kChunk);
  const double items = (double)p.max_chunks * p.HV;
  const int widths[3] = {32, 64, 128};
  const double per_chunk_us[3] = {0.90, 1.23, 1.50};
  const bool kda = p.variant == HA_LA_KDA;
  auto prep_time = [&](int on_sms) {                     // the prep kernel on `on_sms` SMs
    const double thru = items * (kda ? 9.8 : 3.45) / on_sms;
    const double groups = (double)on_sms * (kda ? 1 : 3);
    const double rounds = (double)(long long)((items + groups - 1) / groups) * (kda ? 10.5 : 9.0);
    return thru > rounds ? thru : rounds;
  };
  const double prep_us = prep_time(sms);
  // sequences of about the same length (batch rows, or a packed batch whose longest is close to its average)
  // cannot be packed any better than in rounds of one CTA per SM
  const double avg_len = p.N > 0 ? (double)p.T_total / p.N : 0.0;
  const bool even = avg_len <= 0.0 || p.max_len < 1.5 * avg_len;
  bool may_overlap = p.max_chunks > 1;
  bool force_overlap = false;                            // "2": side by side whenever that is legal (tests)
  if (const char* e = getenv("HA_LA_TC_OVERLAP")) {
    may_overlap = may_overlap && e[0] != '0';
    force_overlap = may_overlap && e[0] == '2';
  }
  int forced_nv = 0;
  if (const char* e = getenv("HA_LA_TC_NV")) {
    const int v = atoi(e);
    if (v == 32 || v == 64 || v == 128) forced_nv = v;
  }
  TcPlan plan{32, false, 1};
  double best = 1e30;
  for (int w = 0; w < 3; ++w) {
    if (forced_nv && widths[w] != forced_nv) continue;
    const long long ctas = chains * (128 / widths[w]);
    const double serial = longest * per_chunk_us[w];
    double chain_us = serial;
    if (ctas > sms) {
      const double spread = 1.15 * items * (128 / widths[w]) * per_chunk_us[w] / sms;
      chain_us = even ? serial * (double)((ctas + sms - 1) / sms) : (serial > spread ? serial : spread);
    }
    const double back_to_back = prep_us + chain_us + (force_overlap ? 1e9 : 0.0);
    if (back_to_back < best) { best = back_to_back; plan = TcPlan{widths[w], false, 1}; }
    if (may_overlap && ctas * 2 <= sms) {
      const double prep_beside = 1.1 * prep_time(sms - (int)ctas);
      double overlapped = (chain_us > prep_beside ? chain_us : prep_beside) + 12.0;
      if (p.N > 1) {
        const double last = prep_beside * (1.0 - 1.0 / p.N) + chain_us + 12.0;
        if (last > overlapped) overlapped = last;
      }
      if (overlapped < best) { best = overlapped; plan = TcPlan{widths[w], true, 1}; }
    }
  }
  // Segment-parallel state passing (equal-length rows, sliced kernels, back to back with the prep kernel): a
  // sequence's chain is cut into nseg segments that run at once; a later segment costs three times the columns of
  // the first (its own from a zero state plus 128 transition columns), so it only pays while all those CTAs have an
  // SM each, i.e. for few heads and long sequences.  Costs measured on B200: the chain's per-chunk times above,
  // 7 us + 3.1 us per further segment for the start states (S - 1 products of 128^3 in turn) and 9 us + 15 ns per
  // corrected chunk-head for the outputs.
  int forced_seg = 0;
  if (const char* e = getenv("HA_LA_TC_SEGMENTS")) {
    const int v = atoi(e);
    if (v == 1 || v == 2 || v == 4 || v == 8) forced_seg = v;
  }
  if ((!p.varlen || forced_seg > 1) && forced_seg != 1 && longest >= 2) {
    for (int w = 0; w < 2; ++w) {                          // 32- and 64-channel slices
      if (forced_nv && widths[w] != forced_nv) continue;
      for (int nseg = 2; nseg <= 8; nseg *= 2) {
        if (forced_seg && nseg != forced_seg) continue;
        if (nseg > longest) continue;
        const long long ctas = chains * (128 / widths[w]) * (2 * nseg - 1);
        if (ctas > sms && !forced_seg) continue;
        const double cpseg = (double)(long long)((longest + nseg - 1) / nseg);
        const double waves = (double)((ctas + sms - 1) / sms);
        const double later = items * (1.0 - 1.0 / nseg);
        const double t = prep_us + waves * cpseg * per_chunk_us[w] + (7.0 + 3.1 * (nseg - 1)) + (9.0 + 0.015 * later);
        if (t < best || (forced_seg && plan.nseg != forced_seg)) { best = t; plan = TcPlan{widths[w], false, nseg}; }
      }
    }
  }
  return plan;
}

}  // namespace

bool tc_supported(const Problem& p) {
  return p.dtype == HA_LA_BF16 && p.dk == 128 && p.dv == 128;
}

// Images plus, when the planner cuts the sequences into segments, the segment scratch for that many.  (The call
// checks the caller's size against this same function, so an environment switch that is changed between sizing and
// calling ends in HA_LA_ERR_WORKSPACE, not in an overrun.)
size_t tc_workspace_bytes(const Problem& p) {
  const size_t img = tc_ws_bytes_for((size_t)p.max_chunks * p.HV, p.variant == HA_LA_KDA);
  return img + tc_seg_bytes((size_t)p.N * p.HV, plan_tc(p).nseg, (size_t)p.T_total, p.HV);
}

int tc_num_launches(const Problem& p) { return plan_tc(p).nseg > 1 ? 4 : 2; }

int tc_num_segments(const Problem& p) { return plan_tc(p).nseg; }

void tc_launch_plan(const Problem& p, int* slice_width, int* concurrent) {
  const TcPlan tp = plan_tc(p);
  *slice_width = tp.nv;
  *concurrent = tp.concurrent ? 1 : 0;
}

cudaError_t launch_tc(const Problem& p, const ha_la_prefill_args& a, PlanView plan, void* tc_ws, cudaStream_t stream) {
  const TcPlan tp = plan_tc(p);
  const int nv = tp.nv;
  CUtensorMap mq, mk, mv, mo;
  if (!make_map(&mq, a.q, p.T_total, p.HK) || !make_map(&mk, a.k, p.T_total, p.HK) ||
      !make_map(&mv, a.v, p.T_total, p.HV) || !make_map_o(&mo, a.o, p.T_total, p.HV, nv))
    return cudaErrorInvalidValue;
  const size_t ncj = (size_t)p.max_chunks * p.HV;
  const TcWorkspace ws = tc_ws_view(tc_ws, ncj, p.variant == HA_LA_KDA);
  const SegBuffers sg = tc_seg_view(reinterpret_cast<uint8_t*>(tc_ws) + tc_ws_bytes_for(ncj, p.variant == HA_LA_KDA),
                                    (size_t)p.N * p.HV, tp.nseg, (size_t)p.T_total, p.HV);
  const bool concurrent = tp.concurrent && !g_timer;     // (per-kernel timing wants one kernel at a time)
  // Configure (and load) both kernels before anything is enqueued: loading a kernel for the first time can
  // wait for the device, and in the concurrent mode the chain kernel would be spinning meanwhile.
  // (Once per device and kernel instance: the attributes stick, and the calls are not free on the host.)
  static std::atomic<uint32_t> configured[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
  const uint32_t bit = 1u << ((p.variant == HA_LA_KDA ? 3 : 0) + (nv == 32 ? 0 : (nv == 64 ? 1 : 2)));
  if (dev < 0 || dev >= kMaxDevices || !(configured[dev].load() & bit)) {
    cudaError_t ce = configure_tc_prep(p);
    if (ce != cudaSuccess) return ce;
    ce = configure_tc_chain(p, nv);
    if (ce != cudaSuccess) return ce;
    if (dev >= 0 && dev < kMaxDevices) configured[dev].fetch_or(bit);
  }
  int64_t epoch = 0;                                     // 0 means "sequential"
  int reserved_sms = 0;
  if (concurrent) {
    epoch = next_epoch();
    reserved_sms = p.N * p.HV * (128 / nv);              // a chain CTA fills its SM
  }
  if (concurrent) {
    // A call captured into a CUDA graph is replayed with the epoch it was captured with, and the flags its last
    // replay left behind carry exactly that epoch: the chain kernel would run ahead of the prep kernel on stale
    // images.  Under capture the flags are therefore cleared first (a memset node, replayed with the rest).
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) {
      (void)cudaGetLastError();
      cs = cudaStreamCaptureStatusNone;
    }
    if (cs == cudaStreamCaptureStatusActive) {
      const cudaError_t me = cudaMemsetAsync(ws.flags, 0, ncj * sizeof(int64_t), stream);
      if (me != cudaSuccess) return me;
    }
  }
  cudaError_t e = launch_tc_prep(p, a, plan, ws, mq, mk, mv, epoch, reserved_sms, stream);
  if (e != cudaSuccess) return e;
  e = launch_tc_chain(p, a, plan, ws, mk, mo, nv, epoch, /*dependent=*/g_timer == nullptr, kDefaultSpinLimit, sg, stream);
  if (e != cudaSuccess) return e;
  return launch_tc_seg_fix(p, a, plan, sg, stream);
}

// Test hook behind ha_la_debug_wait_timeout: the sequential kernel alone, in the concurrent mode, with an epoch that
// nothing will ever publish and a small poll limit.  Its first flag wait runs out, it records the time-out, and then
// walks the chunks on whatever the workspace holds (valid memory, meaningless numbers) to a normal exit.
cudaError_t launch_tc_chain_unpublished(const Problem& p, const ha_la_prefill_args& a, void* tc_ws, uint32_t spin_limit,
                                        cudaStream_t stream) {
  const int nv = 32;
  CUtensorMap mk, mo;
  if (!make_map(&mk, a.k, p.T_total, p.HK) || !make_map_o(&mo, a.o, p.T_total, p.HV, nv)) return cudaErrorInvalidValue;
  const TcWorkspace ws = tc_ws_view(tc_ws, (size_t)p.max_chunks * p.HV, p.variant == HA_LA_KDA);
  cudaError_t ce = configure_tc_chain(p, nv);
  if (ce != cudaSuccess) return ce;
  return launch_tc_chain(p, a, PlanView{}, ws, mk, mo, nv, next_epoch(), /*dependent=*/false, spin_limit,
                         SegBuffers{1, nullptr, nullptr, nullptr, nullptr}, stream);
}

}  // namespace ha_la
