// ha_la_prefill_noalloc: the prefill for callers that cannot provide scratch memory.
//
// Some callers have no way to hand this library a workspace: code running inside a framework's
// allocator-free region (a custom-op hook that must not touch the caching allocator), a runtime
// that froze its memory pool at start-up, or a plug-in that only ever sees the tensors of the
// operator it implements.  For them the chunk table that ha_la_prefill keeps in the caller's
// workspace lives here instead, in a fixed array that is part of the library image.  Every GPU
// that loads the library holds that array (kScratchBytes) until the process exits.
//
// The array's name is only a host-side handle: it is not a device address and must never be
// passed to a kernel from host code.  The device address is looked up once per device with
// cudaGetSymbolAddress, with that device current, on the entry point's first call on that device.
#include "common.cuh"

#include <atomic>

namespace ha_la {
namespace {

constexpr int kMaxSeqs = 1024;        // sequences (batch rows or packed sequences)
constexpr int kMaxChunks = 16384;     // chunk slots: about one million tokens
constexpr size_t kScratchInts = 8 + 3 * (size_t)kMaxSeqs + (kMaxSeqs + 1) + 3 * (size_t)kMaxChunks;
// rounded like plan_bytes() (to 1 KiB), so that a problem at exactly both limits fits: 209 KiB
constexpr size_t kScratchBytes = (kScratchInts * sizeof(int32_t) + 1023) / 1024 * 1024;

static __device__ __align__(256) unsigned char g_plan_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
// Device address of g_plan_scratch on each device, once known.  Host threads may race on a slot: every writer
// stores the same value (the address is a property of the device's primary context), so the race is between
// equal stores; the slots are atomics only to make that well defined.  A cached address belongs to the
// device's primary context and does not survive cudaDeviceReset.
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Looks the array's device address up (first call on this device) or returns the cached one.
int scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HA_LA_ERR_CUDA;
  void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_plan_scratch) != cudaSuccess || !p) return HA_LA_ERR_CUDA;
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return HA_LA_OK;
}

}  // namespace
}  // namespace ha_la

using namespace ha_la;

extern "C" int ha_la_prefill_noalloc(const ha_la_prefill_args* a, void* cuda_stream) {
  if (!a) return HA_LA_ERR_INVALID_ARG;
  // Shape validation is the same as ha_la_prefill's: ask the workspace query (host only, no CUDA call).
  size_t unused = 0;
  const int rc = ha_la_prefill_workspace_bytes(a, &unused);
  if (rc != HA_LA_OK) return rc;
  const bool packed = a->num_seqs > 0 || a->cu_seqlens;

  Problem p;
  p.variant = a->variant; p.dtype = a->dtype;
  p.N = packed ? a->num_seqs : a->batch;
  p.T_total = a->batch * a->seqlen;
  p.T_row = a->seqlen;
  p.HK = a->num_qk_heads; p.HV = a->num_v_heads; p.dk = a->d_k; p.dv = a->d_v;
  p.scale = a->scale;
  p.varlen = packed ? 1 : 0;
  if (packed) {
    p.max_len = (a->max_seqlen > 0 && a->max_seqlen < a->seqlen) ? a->max_seqlen : a->seqlen;
    p.max_chunks = (int)(((long long)p.T_total + 63LL * p.N) / kChunk);
  } else {
    p.max_len = a->seqlen;
    p.max_chunks = a->batch * ((a->seqlen + kChunk - 1) / kChunk);
  }
  p.max_seq_chunks = (p.max_len + kChunk - 1) / kChunk;
  if (!simt_supported(p)) return HA_LA_ERR_UNSUPPORTED;
  // sizes first (shapes alone decide them), then the pointers
  if (p.N > kMaxSeqs || p.max_chunks > kMaxChunks || plan_bytes(p) > kScratchBytes) return HA_LA_ERR_TOO_LARGE;
  if (!a->q || !a->k || !a->v || !a->g || !a->beta || !a->o) return HA_LA_ERR_INVALID_ARG;
  if (packed && !a->cu_seqlens) return HA_LA_ERR_INVALID_ARG;
  const uintptr_t al16 = (uintptr_t)a->q | (uintptr_t)a->k | (uintptr_t)a->v | (uintptr_t)a->o |
                         (uintptr_t)a->h0 | (uintptr_t)a->hT;
  if (al16 & 15) return HA_LA_ERR_INVALID_ARG;
  if (((uintptr_t)a->g | (uintptr_t)a->beta | (uintptr_t)a->cu_seqlens | (uintptr_t)a->status_word) & 3)
    return HA_LA_ERR_INVALID_ARG;

  void* scratch = nullptr;
  const int src = scratch_address(&scratch);
  if (src != HA_LA_OK) return src;

  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  // The plan kernel writes every entry the compute kernel reads (header, per-sequence rows, and all
  // max_chunks slots of this problem), so nothing left in the array by an earlier call is ever read.
  PlanView plan = plan_view(scratch, p);
  if (launch_plan(p, a->cu_seqlens, plan, a->status_word, stream) != cudaSuccess) return HA_LA_ERR_CUDA;
  if (p.T_total == 0 && !a->hT) return HA_LA_OK;
  return launch_simt(p, *a, plan, stream) == cudaSuccess ? HA_LA_OK : HA_LA_ERR_CUDA;
}

extern "C" size_t ha_la_prefill_noalloc_scratch_bytes(void) { return kScratchBytes; }
