// Tensor-core (tcgen05) path, host side: tensor maps, workspace carving, slice-width choice, launches.
#include <cuda.h>
#include <stdlib.h>

#include "tc_common.cuh"

namespace ha_la {

cudaError_t launch_tc_prep(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                           const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, int nv,
                           cudaStream_t stream);
cudaError_t launch_tc_chain(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                            const CUtensorMap& mk, int nv, cudaStream_t stream);

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

int sm_count() {
  static int n = [] {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    return v;
  }();
  return n;
}

// Value channels per chain CTA: the narrowest slice that still gives every CTA its own SM.
int pick_nv(const Problem& p) {
  if (const char* e = getenv("HA_LA_TC_NV")) {
    const int v = atoi(e);
    if (v == 32 || v == 64 || v == 128) return v;
  }
  const long long chains = (long long)p.N * p.HV;
  const int sms = sm_count();
  if (chains * 4 <= sms) return 32;
  if (chains * 2 <= sms) return 64;
  return 128;
}

}  // namespace

bool tc_supported(const Problem& p) {
  return p.dtype == HA_LA_BF16 && p.dk == 128 && p.dv == 128;
}

size_t tc_workspace_bytes(const Problem& p) {
  return tc_ws_bytes_for((size_t)p.max_chunks * p.HV, p.variant == HA_LA_KDA);
}

int tc_num_launches(const Problem&) { return 2; }

cudaError_t launch_tc(const Problem& p, const ha_la_prefill_args& a, PlanView plan, void* tc_ws, cudaStream_t stream) {
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, a.q, p.T_total, p.HK) || !make_map(&mk, a.k, p.T_total, p.HK) ||
      !make_map(&mv, a.v, p.T_total, p.HV))
    return cudaErrorInvalidValue;
  const TcWorkspace ws = tc_ws_view(tc_ws, (size_t)p.max_chunks * p.HV, p.variant == HA_LA_KDA);
  const int nv = pick_nv(p);
  cudaError_t e = launch_tc_prep(p, a, plan, ws, mq, mk, mv, nv, stream);
  if (e != cudaSuccess) return e;
  return launch_tc_chain(p, a, plan, ws, mk, nv, stream);
}

}  // namespace ha_la
