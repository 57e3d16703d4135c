// C ABI of the ha_la library: argument validation, workspace carving and kernel dispatch.
// See include/ha_la.h for the contract of every entry point.
#include "common.cuh"

#include <stdlib.h>

using namespace ha_la;

namespace ha_la { thread_local KernelTimer* g_timer = nullptr; }


namespace {

bool dim_ok(int d) { return d == 64 || d == 128; }

// Shape-only validation (no pointer checks).  Fills `p` on success.
int make_problem(const ha_la_prefill_args* a, Problem* p) {
  if (!a) return HA_LA_ERR_INVALID_ARG;
  if (a->variant != HA_LA_GDN && a->variant != HA_LA_KDA) return HA_LA_ERR_INVALID_ARG;
  if (a->dtype != HA_LA_BF16 && a->dtype != HA_LA_FP32) return HA_LA_ERR_INVALID_ARG;
  if (a->batch < 1 || a->seqlen < 0) return HA_LA_ERR_INVALID_ARG;
  if (a->num_qk_heads < 1 || a->num_v_heads < 1 || a->num_v_heads % a->num_qk_heads != 0)
    return HA_LA_ERR_INVALID_ARG;
  if (a->d_k < 1 || a->d_v < 1) return HA_LA_ERR_INVALID_ARG;
  if (!dim_ok(a->d_k) || !dim_ok(a->d_v)) return HA_LA_ERR_UNSUPPORTED;
  if (a->chunk != kChunk) return HA_LA_ERR_UNSUPPORTED;
  if (!(a->scale == a->scale)) return HA_LA_ERR_INVALID_ARG;   // NaN
  const bool varlen = a->cu_seqlens != nullptr || a->num_seqs > 0;
  if (varlen) {
    if (a->batch != 1 || a->num_seqs < 1) return HA_LA_ERR_INVALID_ARG;
    if (a->max_seqlen < 0) return HA_LA_ERR_INVALID_ARG;
  }
  const long long rows = (long long)a->batch * a->seqlen;
  if (rows > 0x7fffffffLL - 64) return HA_LA_ERR_UNSUPPORTED;   // token rows are indexed in int32

  p->variant = a->variant;
  p->dtype = a->dtype;
  p->N = varlen ? a->num_seqs : a->batch;
  p->T_total = (int)rows;
  p->T_row = a->seqlen;
  p->HK = a->num_qk_heads;
  p->HV = a->num_v_heads;
  p->dk = a->d_k;
  p->dv = a->d_v;
  p->scale = a->scale;
  p->varlen = varlen ? 1 : 0;
  if (varlen) {
    p->max_len = (a->max_seqlen > 0 && a->max_seqlen < a->seqlen) ? a->max_seqlen : a->seqlen;
    p->max_chunks = (int)(((long long)p->T_total + 63LL * p->N) / kChunk);
  } else {
    p->max_len = a->seqlen;
    p->max_chunks = a->batch * ((a->seqlen + kChunk - 1) / kChunk);
  }
  p->max_seq_chunks = (p->max_len + kChunk - 1) / kChunk;
  if (!tc_supported(*p) && !simt_supported(*p)) return HA_LA_ERR_UNSUPPORTED;
  return HA_LA_OK;
}

bool use_tc(const Problem& p) {
  static const bool forced_off = [] {
    const char* e = getenv("HA_LA_FORCE_SIMT");
    return e && e[0] == '1';
  }();
  return !forced_off && tc_supported(p);
}

}  // namespace

extern "C" {

int ha_la_prefill_workspace_bytes(const ha_la_prefill_args* args, size_t* out_bytes) {
  if (!out_bytes) return HA_LA_ERR_INVALID_ARG;
  Problem p;
  const int rc = make_problem(args, &p);
  if (rc != HA_LA_OK) return rc;
  size_t bytes = plan_bytes(p);
  if (tc_supported(p)) bytes += tc_workspace_bytes(p);
  *out_bytes = align_up(bytes, 256);
  return HA_LA_OK;
}

const char* ha_la_prefill_path(const ha_la_prefill_args* args) {
  Problem p;
  if (make_problem(args, &p) != HA_LA_OK) return nullptr;
  return use_tc(p) ? "tc" : "simt";
}

// The chunk table is only needed for packed batches and by the CUDA-core kernel; the tensor-core
// kernels index equal-length rows arithmetically.
static bool needs_plan(const ha_la_prefill_args* a, const Problem& p) {
  return a->num_seqs > 0 || a->cu_seqlens != nullptr || !use_tc(p);
}

int ha_la_prefill_num_launches(const ha_la_prefill_args* args) {
  Problem p;
  if (make_problem(args, &p) != HA_LA_OK) return 0;
  return (needs_plan(args, p) ? 1 : 0) + (use_tc(p) ? tc_num_launches(p) : 1);
}

int ha_la_prefill_num_segments(const ha_la_prefill_args* args) {
  Problem p;
  if (make_problem(args, &p) != HA_LA_OK) return 0;
  return use_tc(p) ? tc_num_segments(p) : 1;
}

int ha_la_prefill_launch_plan(const ha_la_prefill_args* args, int* slice_width, int* concurrent) {
  Problem p;
  const int rc = make_problem(args, &p);
  if (rc != HA_LA_OK) return rc;
  if (!slice_width || !concurrent) return HA_LA_ERR_INVALID_ARG;
  *slice_width = 0;
  *concurrent = 0;
  if (use_tc(p)) tc_launch_plan(p, slice_width, concurrent);
  return HA_LA_OK;
}

int ha_la_prefill(const ha_la_prefill_args* a, void* cuda_stream) {
  Problem p;
  int rc = make_problem(a, &p);
  if (rc != HA_LA_OK) return rc;
  if (!a->q || !a->k || !a->v || !a->g || !a->beta || !a->o) return HA_LA_ERR_INVALID_ARG;
  const bool varlen = a->num_seqs > 0 || a->cu_seqlens;
  if (varlen && !a->cu_seqlens) return HA_LA_ERR_INVALID_ARG;
  const uintptr_t al16 = (uintptr_t)a->q | (uintptr_t)a->k | (uintptr_t)a->v | (uintptr_t)a->o |
                         (uintptr_t)a->h0 | (uintptr_t)a->hT;
  if (al16 & 15) return HA_LA_ERR_INVALID_ARG;
  if (((uintptr_t)a->g | (uintptr_t)a->beta | (uintptr_t)a->cu_seqlens | (uintptr_t)a->status_word) & 3)
    return HA_LA_ERR_INVALID_ARG;
  if (a->variant == HA_LA_KDA && ((uintptr_t)a->g & 15)) return HA_LA_ERR_INVALID_ARG;   // fetched by bulk copies

  size_t need = 0;
  rc = ha_la_prefill_workspace_bytes(a, &need);
  if (rc != HA_LA_OK) return rc;
  if (!a->workspace || ((uintptr_t)a->workspace & 255) || a->workspace_bytes < need) return HA_LA_ERR_WORKSPACE;

  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  PlanView plan = plan_view(a->workspace, p);
  if (needs_plan(a, p)) {
    if (launch_plan(p, a->cu_seqlens, plan, a->status_word, stream) != cudaSuccess) return HA_LA_ERR_CUDA;
  } else {
    plan = PlanView{};                                   // null table: equal-length rows, indexed arithmetically
  }
  if (p.T_total == 0 && !a->hT) return HA_LA_OK;

  cudaError_t e;
  if (use_tc(p)) {
    void* tc_ws = reinterpret_cast<char*>(a->workspace) + plan_bytes(p);
    e = launch_tc(p, *a, plan, tc_ws, stream);
  } else {
    e = launch_simt(p, *a, plan, stream);
  }
  return e == cudaSuccess ? HA_LA_OK : HA_LA_ERR_CUDA;
}

int ha_la_prefill_timed(const ha_la_prefill_args* a, void* cuda_stream, int max_kernels, float* ms_out,
                        const char** names_out, int* num_kernels_out) {
  if (!ms_out || !num_kernels_out || max_kernels < 1) return HA_LA_ERR_INVALID_ARG;
  *num_kernels_out = 0;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  KernelTimer t;
  for (int i = 0; i <= KernelTimer::kMax; ++i)
    if (cudaEventCreate(&t.ev[i]) != cudaSuccess) return HA_LA_ERR_CUDA;
  g_timer = &t;
  int rc = ha_la_prefill(a, cuda_stream);
  g_timer = nullptr;
  if (rc == HA_LA_OK) {
    cudaEventRecord(t.ev[t.n], stream);
    if (cudaStreamSynchronize(stream) != cudaSuccess) rc = HA_LA_ERR_CUDA;
  }
  if (rc == HA_LA_OK) {
    const int n = t.n < max_kernels ? t.n : max_kernels;
    for (int i = 0; i < n; ++i) {
      float ms = 0.f;
      cudaEventElapsedTime(&ms, t.ev[i], t.ev[i + 1]);
      ms_out[i] = ms;
      if (names_out) names_out[i] = t.name[i];
    }
    *num_kernels_out = n;
  }
  for (int i = 0; i <= KernelTimer::kMax; ++i) cudaEventDestroy(t.ev[i]);
  return rc;
}

int ha_la_debug_wait_timeout(const ha_la_prefill_args* a, void* cuda_stream, unsigned int spin_limit) {
  Problem p;
  int rc = make_problem(a, &p);
  if (rc != HA_LA_OK) return rc;
  if (!tc_supported(p) || a->cu_seqlens || a->num_seqs > 0) return HA_LA_ERR_UNSUPPORTED;
  if (!a->q || !a->k || !a->v || !a->g || !a->beta || !a->o || !a->status_word) return HA_LA_ERR_INVALID_ARG;
  if (spin_limit < 1 || spin_limit > (1u << 20)) return HA_LA_ERR_INVALID_ARG;
  size_t need = 0;
  rc = ha_la_prefill_workspace_bytes(a, &need);
  if (rc != HA_LA_OK) return rc;
  if (!a->workspace || ((uintptr_t)a->workspace & 255) || a->workspace_bytes < need) return HA_LA_ERR_WORKSPACE;
  void* tc_ws = reinterpret_cast<char*>(a->workspace) + plan_bytes(p);
  return launch_tc_chain_unpublished(p, *a, tc_ws, spin_limit, reinterpret_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? HA_LA_OK : HA_LA_ERR_CUDA;
}

const char* ha_la_status_string(int status) {
  switch (status) {
    case HA_LA_OK: return "ok";
    case HA_LA_ERR_INVALID_ARG: return "invalid argument";
    case HA_LA_ERR_UNSUPPORTED: return "unsupported shape or option";
    case HA_LA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case HA_LA_ERR_CUDA: return "CUDA call or kernel launch failed";
    case HA_LA_ERR_TIMEOUT: return "device-side wait ran out";
    case HA_LA_ERR_DEVICE_CHECK: return "device-side check failed";
    case HA_LA_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of ha_la_prefill_noalloc";
    default: return "unknown status";
  }
}

int ha_la_version(void) { return 1; }

}  // extern "C"
