// One decoding step of the delta-rule layer (one new token per sequence): see ha_la_decode in ha_la.h.
//
// The step reads and rewrites the whole fp32 state (d_k x d_v per sequence and V-head, 64 KiB at d = 128) for
// about 6 d_k d_v flops, so it is bound by HBM traffic: 2 x 4 d_k d_v bytes per (sequence, V-head).  One CTA
// per (sequence, V-head), one thread per value channel: a thread keeps its column of the state in registers
// (d_k values), so the state crosses the memory system exactly once in each direction, with every load and
// store of a warp covering 128 contiguous bytes and all d_k loads of a thread independent (in flight together).
#include "common.cuh"

#include <cuda_bf16.h>

namespace ha_la {

namespace {

struct DecodeParams {
  const void* q; const void* k; const void* v;
  const float* g; const float* beta; const float* h_in;
  float* h_out; void* o;
  int HK, HV;
  float scale;
};

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <typename In, int D, bool KDA>
__global__ void __launch_bounds__(D) decode_kernel(DecodeParams p) {
  __shared__ __align__(16) float sk[D];                  // k, then q, then the per-row decay
  __shared__ __align__(16) float sq[D];
  __shared__ __align__(16) float sdec[D];
  const int tid = threadIdx.x;
  const size_t nj = blockIdx.x;                          // (sequence, V-head)
  const int j = (int)(nj % p.HV);
  const size_t n = nj / p.HV;
  const int jq = j / (p.HV / p.HK);
  const size_t qk_off = (n * p.HK + jq) * D + tid;
  sk[tid] = to_f32(reinterpret_cast<const In*>(p.k)[qk_off]);
  sq[tid] = to_f32(reinterpret_cast<const In*>(p.q)[qk_off]);
  sdec[tid] = __expf(KDA ? p.g[nj * D + tid] : p.g[nj]);
  const float vv = to_f32(reinterpret_cast<const In*>(p.v)[nj * D + tid]);
  const float beta = p.beta[nj];

  // column `tid` of the state, all d_k rows; the loads do not depend on anything above
  float h[D];
  const float* hin = p.h_in ? p.h_in + nj * D * D + tid : nullptr;
#pragma unroll
  for (int c = 0; c < D; ++c) h[c] = hin ? __ldcs(hin + (size_t)c * D) : 0.f;   // streaming: read once
  __syncthreads();

  float r = 0.f;                                         // (decayed h)^T k
#pragma unroll
  for (int c = 0; c < D; ++c) {
    h[c] *= sdec[c];
    r = fmaf(h[c], sk[c], r);
  }
  const float u = beta * (vv - r);
  float acc = 0.f;
  float* hout = p.h_out + nj * D * D + tid;
#pragma unroll
  for (int c = 0; c < D; ++c) {
    h[c] = fmaf(sk[c], u, h[c]);
    acc = fmaf(h[c], sq[c], acc);
    __stcs(hout + (size_t)c * D, h[c]);
  }
  reinterpret_cast<In*>(p.o)[nj * D + tid] = from_f32<In>(p.scale * acc);
}

template <typename In, int D, bool KDA>
cudaError_t launch(const DecodeParams& dp, size_t grid, cudaStream_t stream) {
  decode_kernel<In, D, KDA><<<(unsigned)grid, D, 0, stream>>>(dp);
  return cudaGetLastError();
}

}  // namespace

}  // namespace ha_la

using namespace ha_la;

extern "C" int ha_la_decode(const ha_la_decode_args* a, void* cuda_stream) {
  if (!a) return HA_LA_ERR_INVALID_ARG;
  if (a->variant != HA_LA_GDN && a->variant != HA_LA_KDA) return HA_LA_ERR_INVALID_ARG;
  if (a->dtype != HA_LA_BF16 && a->dtype != HA_LA_FP32) return HA_LA_ERR_INVALID_ARG;
  if (a->num_seqs < 0 || a->num_qk_heads < 1 || a->num_v_heads < 1 || a->num_v_heads % a->num_qk_heads != 0)
    return HA_LA_ERR_INVALID_ARG;
  if (a->d_k < 1 || a->d_v < 1) return HA_LA_ERR_INVALID_ARG;
  if (a->d_k != a->d_v || (a->d_k != 64 && a->d_k != 128)) return HA_LA_ERR_UNSUPPORTED;
  if (!(a->scale == a->scale)) return HA_LA_ERR_INVALID_ARG;
  const unsigned long long grid = (unsigned long long)a->num_seqs * a->num_v_heads;
  if (grid > 0x7fffffffULL) return HA_LA_ERR_UNSUPPORTED;
  if (grid == 0) return HA_LA_OK;
  if (!a->q || !a->k || !a->v || !a->g || !a->beta || !a->h_out || !a->o) return HA_LA_ERR_INVALID_ARG;
  const uintptr_t al16 = (uintptr_t)a->q | (uintptr_t)a->k | (uintptr_t)a->v | (uintptr_t)a->o |
                         (uintptr_t)a->h_in | (uintptr_t)a->h_out;
  if (al16 & 15) return HA_LA_ERR_INVALID_ARG;
  if (((uintptr_t)a->g | (uintptr_t)a->beta) & 3) return HA_LA_ERR_INVALID_ARG;

  DecodeParams dp{a->q, a->k, a->v, a->g, a->beta, a->h_in, a->h_out, a->o, a->num_qk_heads, a->num_v_heads, a->scale};
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const bool kda = a->variant == HA_LA_KDA, bf = a->dtype == HA_LA_BF16, big = a->d_k == 128;
  cudaError_t e;
  if (bf) {
    if (big) e = kda ? launch<__nv_bfloat16, 128, true>(dp, grid, stream) : launch<__nv_bfloat16, 128, false>(dp, grid, stream);
    else e = kda ? launch<__nv_bfloat16, 64, true>(dp, grid, stream) : launch<__nv_bfloat16, 64, false>(dp, grid, stream);
  } else {
    if (big) e = kda ? launch<float, 128, true>(dp, grid, stream) : launch<float, 128, false>(dp, grid, stream);
    else e = kda ? launch<float, 64, true>(dp, grid, stream) : launch<float, 64, false>(dp, grid, stream);
  }
  return e == cudaSuccess ? HA_LA_OK : HA_LA_ERR_CUDA;
}
