// Segment-parallel state passing, second half (paper Section "Head-Level Mapping with Cross-Operator Fusion": the
// Chunk-Seg-Seg mapping of its FlashQLA baseline cuts a head's sequential Reduce into segments that run concurrently
// after an extra pre-computation; Section "Peak Device Memory" warns that materialising cumulative gates for it costs
// memory -- nothing of that kind is stored here, the chunk images already carry their decays).
//
// The chain kernel has walked every segment s >= 1 of a sequence twice over at the same time as segment 0: from a zero
// state (provisional outputs in o, end state b_s) and, with U = O_loc = 0, from the identity (end state Phi_s; its
// output rows R = scale Q~ Phi_c).  The state recurrence is affine in its start state, so with the true start h_s
//     h_{s+1} = Phi_s h_s + b_s          (h_1 is segment 0's end state: it started from the real h0)
//     o_t    += R_t h_s                  for every token t of segment s
// Two small kernels do that:
//   seg_fix_kernel   per (sequence, V-head) and tile of 16 state columns: the S - 1 products in turn, fp32 on the
//                    CUDA cores (128 x 128 x 16 each); writes hT and a bf16 copy of every h_s;
//   seg_out_kernel   per (chunk of a later segment, V-head): o += R h_s on the legacy tensor path (wmma bf16,
//                    fp32 accumulation), 64 x 128 x 128; chunk-parallel, no dependency between CTAs.
#include <mma.h>

#include "tc_common.cuh"

namespace ha_la {

namespace {

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr int kFixCols = 16;             // state columns per CTA of the fix-up kernel
constexpr int kPhiLd = 129;              // padded row stride (floats) of the transition in shared memory
constexpr size_t kFixSmem = (size_t)128 * kPhiLd * 4 + 128 * kFixCols * 4;

__global__ void __launch_bounds__(256) seg_fix_kernel(SegBuffers sg, float* hT) {
  extern __shared__ __align__(16) float fsm[];
  float* sPhi = fsm;                     // [128][kPhiLd]: Phi_s, whole (every thread walks one row of it)
  float* sh = fsm + 128 * kPhiLd;        // [128][kFixCols]: h_s, this CTA's columns
  const int nj = blockIdx.x;
  const int x0 = blockIdx.y * kFixCols;
  const int i = threadIdx.x & 127;       // state row
  const int xh = (threadIdx.x >> 7) * 8; // which 8 of the 16 columns
  const size_t seg_stride = 128 * 128;
  const float* b = sg.seg_b + (size_t)nj * sg.nseg * seg_stride;
  const float* phi = sg.seg_phi + (size_t)nj * sg.nseg * seg_stride;
  __nv_bfloat16* hs = sg.hs + (size_t)nj * sg.nseg * seg_stride;
  float h[8];
  {
    const float4 a0 = *reinterpret_cast<const float4*>(b + (size_t)i * 128 + x0 + xh);
    const float4 a1 = *reinterpret_cast<const float4*>(b + (size_t)i * 128 + x0 + xh + 4);
    h[0] = a0.x; h[1] = a0.y; h[2] = a0.z; h[3] = a0.w; h[4] = a1.x; h[5] = a1.y; h[6] = a1.z; h[7] = a1.w;   // h_1
  }
  for (int s = 1; s < sg.nseg; ++s) {
    // the whole transition of this segment: coalesced 16-byte loads, all in flight together
    const float4* g4 = reinterpret_cast<const float4*>(phi + (size_t)s * seg_stride);
    float4 t[16];
#pragma unroll
    for (int q = 0; q < 16; ++q) t[q] = g4[q * 256 + threadIdx.x];
    float acc[8];
    {
      const float* bs = b + (size_t)s * seg_stride + (size_t)i * 128 + x0 + xh;
      const float4 a0 = *reinterpret_cast<const float4*>(bs), a1 = *reinterpret_cast<const float4*>(bs + 4);
      acc[0] = a0.x; acc[1] = a0.y; acc[2] = a0.z; acc[3] = a0.w; acc[4] = a1.x; acc[5] = a1.y; acc[6] = a1.z; acc[7] = a1.w;
    }
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const int e = (q * 256 + threadIdx.x) * 4, r = e >> 7, c = e & 127;
      float* d = sPhi + r * kPhiLd + c;
      d[0] = t[q].x; d[1] = t[q].y; d[2] = t[q].z; d[3] = t[q].w;
    }
    const uint4 w = make_uint4(pack2(h[0], h[1]), pack2(h[2], h[3]), pack2(h[4], h[5]), pack2(h[6], h[7]));
    *reinterpret_cast<uint4*>(hs + (size_t)s * seg_stride + (size_t)i * 128 + x0 + xh) = w;   // h_s for the output kernel
#pragma unroll
    for (int q = 0; q < 8; ++q) sh[i * kFixCols + xh + q] = h[q];
    __syncthreads();
    const float* prow = sPhi + i * kPhiLd;
#pragma unroll 8
    for (int v = 0; v < 128; ++v) {
      const float f = prow[v];
      const float4 s0 = *reinterpret_cast<const float4*>(sh + v * kFixCols + xh);
      const float4 s1 = *reinterpret_cast<const float4*>(sh + v * kFixCols + xh + 4);
      acc[0] = fmaf(f, s0.x, acc[0]); acc[1] = fmaf(f, s0.y, acc[1]); acc[2] = fmaf(f, s0.z, acc[2]); acc[3] = fmaf(f, s0.w, acc[3]);
      acc[4] = fmaf(f, s1.x, acc[4]); acc[5] = fmaf(f, s1.y, acc[5]); acc[6] = fmaf(f, s1.z, acc[6]); acc[7] = fmaf(f, s1.w, acc[7]);
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 8; ++q) h[q] = acc[q];
  }
  if (hT) {
    float* d = hT + (size_t)nj * seg_stride + (size_t)i * 128 + x0 + xh;
    *reinterpret_cast<float4*>(d) = make_float4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<float4*>(d + 4) = make_float4(h[4], h[5], h[6], h[7]);
  }
}

// o[t][:] += R[t][:] h_s  for the 64 tokens of one chunk of one V-head.  Four warps, 16 token rows each; R, h_s and
// the result go through shared memory (operand loads straight from global memory were latency-bound: 64 small tile
// loads per warp).
constexpr int kLdR = 128 + 8, kLdC = 64 + 4;
constexpr size_t kOutSmem = (size_t)(64 + 128) * kLdR * 2 + (size_t)4 * 16 * kLdC * 4;

__global__ void __launch_bounds__(128) seg_out_kernel(SegBuffers sg, __nv_bfloat16* o, int T_row, int cps, int HV) {
  using namespace nvcuda;
  extern __shared__ __align__(32) uint8_t osm[];
  __nv_bfloat16* sR = reinterpret_cast<__nv_bfloat16*>(osm);                  // [64][kLdR]
  __nv_bfloat16* sB = sR + 64 * kLdR;                                          // [128][kLdR]: h_s
  float* sC = reinterpret_cast<float*>(sB + 128 * kLdR);                       // [4][16][kLdC]
  const int slot = blockIdx.x;                           // chunk slot: chunk cc of batch row n
  const int j = blockIdx.y;
  const int n = slot / cps, cc = slot % cps;
  const int nch = (T_row + kChunk - 1) / kChunk;
  const int cpseg = (nch + sg.nseg - 1) / sg.nseg;
  const int seg = cc / cpseg;
  if (cc >= nch || seg == 0) return;                     // segment 0 ran from the real start state
  const int L = min(kChunk, T_row - cc * kChunk);
  const size_t row0 = (size_t)n * T_row + (size_t)cc * kChunk;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const __nv_bfloat16* hs = sg.hs + (((size_t)n * HV + j) * sg.nseg + seg) * 128 * 128;
  // R tile (rows past the end of the sequence as zeros) and h_s -> shared memory
#pragma unroll 4
  for (int idx = tid; idx < 64 * 16; idx += 128) {
    const int t = idx >> 4, p8 = idx & 15;
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if (t < L) w = *reinterpret_cast<const uint4*>(sg.r + ((row0 + t) * HV + j) * 128 + p8 * 8);
    *reinterpret_cast<uint4*>(sR + t * kLdR + p8 * 8) = w;
  }
#pragma unroll 4
  for (int idx = tid; idx < 128 * 16; idx += 128) {
    const int v = idx >> 4, p8 = idx & 15;
    *reinterpret_cast<uint4*>(sB + v * kLdR + p8 * 8) = *reinterpret_cast<const uint4*>(hs + (size_t)v * 128 + p8 * 8);
  }
  __syncthreads();
  wmma::fragment<wmma::accumulator, 16, 16, 16, float> acc[8];
#pragma unroll
  for (int x = 0; x < 8; ++x) wmma::fill_fragment(acc[x], 0.f);
#pragma unroll 2
  for (int k = 0; k < 8; ++k) {
    wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> fa;
    wmma::load_matrix_sync(fa, sR + (warp * 16) * kLdR + k * 16, kLdR);
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> fb;
      wmma::load_matrix_sync(fb, sB + (k * 16) * kLdR + x * 16, kLdR);
      wmma::mma_sync(acc[x], fa, fb, acc[x]);
    }
  }
  float* myC = sC + warp * 16 * kLdC;
  for (int half = 0; half < 2; ++half) {                 // 64 output columns at a time through shared memory
#pragma unroll
    for (int x = 0; x < 4; ++x) wmma::store_matrix_sync(myC + x * 16, acc[4 * half + x], kLdC, wmma::mem_row_major);
    __syncwarp();
    // each lane adds two columns of every row: all loads first (interleaved with the stores they would run one
    // after the other, a memory latency each)
    __nv_bfloat162* op = reinterpret_cast<__nv_bfloat162*>(o + ((row0 + warp * 16) * HV + j) * 128 + half * 64 + lane * 2);
    const size_t rstride = (size_t)HV * 64;              // one token row further, in bf16 pairs
    const int rows = min(16, L - warp * 16);
    __nv_bfloat162 ov[16];
#pragma unroll
    for (int r = 0; r < 16; ++r)
      if (r < rows) ov[r] = op[r * rstride];
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      if (r < rows) {
        const float2 c = *reinterpret_cast<const float2*>(myC + r * kLdC + lane * 2);
        const float2 f = __bfloat1622float2(ov[r]);
        op[r * rstride] = __floats2bfloat162_rn(f.x + c.x, f.y + c.y);
      }
    }
    __syncwarp();
  }
}

}  // namespace

// Both kernels, behind the chain kernel on the same stream.
cudaError_t launch_tc_seg_fix(const Problem& p, const ha_la_prefill_args& a, const SegBuffers& sg, cudaStream_t stream) {
  if (sg.nseg <= 1 || p.N * p.HV == 0) return cudaSuccess;
  // (per device and idempotent; a few microseconds on the host, on a path that is already several launches long)
  cudaError_t ce = cudaFuncSetAttribute(seg_fix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFixSmem);
  if (ce == cudaSuccess) ce = cudaFuncSetAttribute(seg_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kOutSmem);
  if (ce != cudaSuccess) return ce;
  timer_mark(stream, "tc_seg_fix");
  seg_fix_kernel<<<dim3((unsigned)(p.N * p.HV), 128 / kFixCols), 256, kFixSmem, stream>>>(sg, a.hT);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  timer_mark(stream, "tc_seg_out");
  const int cps = p.max_seq_chunks > 0 ? p.max_seq_chunks : 1;
  seg_out_kernel<<<dim3((unsigned)(p.N * cps), (unsigned)p.HV), 128, kOutSmem, stream>>>(
      sg, reinterpret_cast<__nv_bfloat16*>(a.o), p.T_row, cps, p.HV);
  return cudaGetLastError();
}

}  // namespace ha_la
