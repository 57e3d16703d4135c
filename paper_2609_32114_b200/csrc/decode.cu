// One decoding step of the delta-rule layer (one new token per sequence): see ha_la_decode in ha_la.h.
//
// The step reads and rewrites the whole fp32 state (d_k x d_v per sequence and V-head, 64 KiB at d = 128) for
// about 6 d_k d_v flops, so it is bound by HBM traffic: 2 x 4 d_k d_v bytes per (sequence, V-head).  One CTA
// per (sequence, V-head), one or two threads per value channel: a thread keeps (half of) its column of the state
// in registers, so the state crosses the memory system exactly once in each direction, with every load and
// store of a warp covering 128 contiguous bytes and all loads of a thread independent (in flight together);
// the state is read and written with streaming hints (it is used once per step and exceeds L2).
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

// R threads share a column of the state (R = 2 at d = 128: 64 rows and 64 registers each, which lets four
// CTAs instead of two be resident per SM; the two partial dot products meet in shared memory).
template <typename In, int D, bool KDA, int R>
__global__ void __launch_bounds__(D * R) decode_kernel(DecodeParams p) {
  constexpr int ROWS = D / R;
  __shared__ __align__(16) float sk[D];
  __shared__ __align__(16) float sq[D];
  __shared__ __align__(16) float sdec[D];
  __shared__ float spart[R][D];
  const int tid = threadIdx.x;
  const int col = tid % D, part = tid / D;               // value channel, which block of rows
  const size_t nj = blockIdx.x;                          // (sequence, V-head)
  const int j = (int)(nj % p.HV);
  const size_t n = nj / p.HV;
  const int jq = j / (p.HV / p.HK);
  if (part == 0) {
    const size_t qk_off = (n * p.HK + jq) * D + col;
    sk[col] = to_f32(reinterpret_cast<const In*>(p.k)[qk_off]);
    sq[col] = to_f32(reinterpret_cast<const In*>(p.q)[qk_off]);
    sdec[col] = __expf(KDA ? p.g[nj * D + col] : p.g[nj]);
  }
  const float vv = to_f32(reinterpret_cast<const In*>(p.v)[nj * D + col]);
  const float beta = p.beta[nj];

  // rows part*ROWS .. of column `col`; the loads do not depend on anything above and are read exactly once
  float h[ROWS];
  const size_t base = nj * D * D + (size_t)part * ROWS * D + col;
  const float* hin = p.h_in ? p.h_in + base : nullptr;
#pragma unroll
  for (int c = 0; c < ROWS; ++c) h[c] = hin ? __ldcs(hin + (size_t)c * D) : 0.f;
  __syncthreads();

  const float* k_ = sk + part * ROWS;
  const float* q_ = sq + part * ROWS;
  const float* dec_ = sdec + part * ROWS;
  float r = 0.f;                                         // (decayed h)^T k, this thread's rows
#pragma unroll
  for (int c = 0; c < ROWS; ++c) {
    h[c] *= dec_[c];
    r = fmaf(h[c], k_[c], r);
  }
  if (R > 1) {
    spart[part][col] = r;
    __syncthreads();
    r = 0.f;
#pragma unroll
    for (int pp = 0; pp < R; ++pp) r += spart[pp][col];
    __syncthreads();
  }
  const float u = beta * (vv - r);
  float acc = 0.f;
  float* hout = p.h_out + base;
#pragma unroll
  for (int c = 0; c < ROWS; ++c) {
    h[c] = fmaf(k_[c], u, h[c]);
    acc = fmaf(h[c], q_[c], acc);
    __stcs(hout + (size_t)c * D, h[c]);
  }
  if (R > 1) {
    spart[part][col] = acc;
    __syncthreads();
    acc = 0.f;
#pragma unroll
    for (int pp = 0; pp < R; ++pp) acc += spart[pp][col];
  }
  if (part == 0) reinterpret_cast<In*>(p.o)[nj * D + col] = from_f32<In>(p.scale * acc);
}

template <typename In, int D, bool KDA>
cudaError_t launch(const DecodeParams& dp, size_t grid, cudaStream_t stream) {
  constexpr int R = D == 128 ? 2 : 1;
  decode_kernel<In, D, KDA, R><<<(unsigned)grid, D * R, 0, stream>>>(dp);
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
