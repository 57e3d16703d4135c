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
//   seg_fix_kernel   per (sequence, V-head) and tile of 16 state columns: the S - 1 products in turn, TF32 on the
//                    legacy tensor path (128 x 128 x 16 each); writes hT and a bf16 copy of every h_s;
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

// Warp-level bf16 products on the legacy tensor path (mma.sync m16n8k16, fp32 accumulation), operands fetched by
// ldmatrix from row-major bf16 matrices in shared memory (the wmma interface spends ten times the instructions on
// fragment loads, and the correction kernel is bound by its instruction count).
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const __nv_bfloat16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const __nv_bfloat16* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// h_{s+1} = Phi_s h_s + b_s, s = 1 .. S-1 in turn, for 16 of the 128 state columns per CTA (columns are
// independent; narrow tiles, because a step is a chain of dependent instructions whose length, not the GPU's
// throughput, sets the time: eight CTAs per (sequence, V-head)).  Eight warps, 16 state rows each; the product runs
// on the legacy tensor path in TF32 (wmma m16n16k8, fp32 accumulation starting from b_s): Phi_s and h_s round to
// 11 significant bits, finer than the bf16 operands of every other product of the path.  The transition of a
// segment (64 KiB) goes through shared memory: coalesced 16-byte loads, all of a thread's in flight together, the
// next segment's -- and the next b_s tile -- fetched under this one's product.
constexpr int kFixCols = 16;             // state columns per CTA
constexpr int kPhiLd = 128 + 4;          // row strides (floats) in shared memory
constexpr int kHLd = kFixCols + 4;
constexpr size_t kFixSmem = (size_t)128 * kPhiLd * 4 + (size_t)128 * kHLd * 4;

__global__ void __launch_bounds__(256) seg_fix_kernel(SegBuffers sg, float* hT, int T_row, int HV, const int32_t* seq_len) {
  using namespace nvcuda;
  extern __shared__ __align__(32) float fsm[];
  float* sPhi = fsm;                     // [128][kPhiLd]: Phi_s
  float* sh = fsm + 128 * kPhiLd;        // [128][kHLd]: h_s, this CTA's columns
  const int nj = blockIdx.x;
  const int x0 = blockIdx.y * kFixCols;
  const int tid = threadIdx.x, warp = tid >> 5;
  const size_t seg_stride = 128 * 128;
  const float* b = sg.seg_b + (size_t)nj * sg.nseg * seg_stride;
  const float* phi = sg.seg_phi + (size_t)nj * sg.nseg * seg_stride;
  __nv_bfloat16* hs = sg.hs + (size_t)nj * sg.nseg * seg_stride;
  const int hr = tid >> 1, hc = (tid & 1) * 8;           // this thread's 8 values of the 128 x 16 tile (copies)
  // segments past the end of a short sequence are empty: their transition is the identity and the state passes
  // through untouched (bit for bit, which the TF32 product would not do)
  const int len = seq_len ? seq_len[nj / HV] : T_row;
  const int nch = (len + kChunk - 1) / kChunk;
  const int cpseg = (nch + sg.nseg - 1) / sg.nseg;
  asm volatile("griddepcontrol.wait;" ::: "memory");     // (launched as a programmatic dependent of the chain kernel)
  float4 t[16];
  wmma::fragment<wmma::accumulator, 16, 16, 8, float> acc;
  auto fetch = [&](int s) {                              // Phi_s into registers, b_s's tile into the accumulator
    const float4* g4 = reinterpret_cast<const float4*>(phi + (size_t)s * seg_stride);
#pragma unroll
    for (int q = 0; q < 16; ++q) t[q] = g4[q * 256 + tid];
    wmma::load_matrix_sync(acc, b + (size_t)s * seg_stride + (size_t)(warp * 16) * 128 + x0, 128, wmma::mem_row_major);
  };
  if (sg.nseg > 1) fetch(1);
  // h_1 = end state of segment 0 (which started from the real initial state)
#pragma unroll
  for (int q = 0; q < 2; ++q)
    *reinterpret_cast<float4*>(sh + hr * kHLd + hc + 4 * q) = *reinterpret_cast<const float4*>(b + (size_t)hr * 128 + x0 + hc + 4 * q);
  for (int s = 1; s < sg.nseg; ++s) {
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const int e = (q * 256 + tid) * 4;
      *reinterpret_cast<float4*>(sPhi + (e >> 7) * kPhiLd + (e & 127)) = t[q];
    }
    __syncthreads();                                     // Phi_s and h_s are in shared memory
    {                                                    // h_s as bf16, for the output kernel
      const float4 lo = *reinterpret_cast<const float4*>(sh + hr * kHLd + hc);
      const float4 hi = *reinterpret_cast<const float4*>(sh + hr * kHLd + hc + 4);
      *reinterpret_cast<uint4*>(hs + (size_t)s * seg_stride + (size_t)hr * 128 + x0 + hc) =
          make_uint4(pack2(lo.x, lo.y), pack2(lo.z, lo.w), pack2(hi.x, hi.y), pack2(hi.z, hi.w));
    }
    const bool empty = s * cpseg >= nch;                 // (the same for every thread of the CTA)
    if (!empty) {
#pragma unroll 4
      for (int k = 0; k < 16; ++k) {
        wmma::fragment<wmma::matrix_a, 16, 16, 8, wmma::precision::tf32, wmma::row_major> fa;
        wmma::fragment<wmma::matrix_b, 16, 16, 8, wmma::precision::tf32, wmma::row_major> fb;
        wmma::load_matrix_sync(fa, sPhi + (warp * 16) * kPhiLd + k * 8, kPhiLd);
        wmma::load_matrix_sync(fb, sh + (k * 8) * kHLd, kHLd);
#pragma unroll
        for (int e = 0; e < fa.num_elements; ++e) fa.x[e] = wmma::__float_to_tf32(fa.x[e]);
#pragma unroll
        for (int e = 0; e < fb.num_elements; ++e) fb.x[e] = wmma::__float_to_tf32(fb.x[e]);
        wmma::mma_sync(acc, fa, fb, acc);
      }
    }
    __syncthreads();                                     // every warp has read h_s and Phi_s
    if (!empty) wmma::store_matrix_sync(sh + (warp * 16) * kHLd, acc, kHLd, wmma::mem_row_major);
    if (s + 1 < sg.nseg) fetch(s + 1);                   // (in flight across the barrier and the next staging)
    __syncthreads();                                     // h_{s+1} is complete
  }
  if (hT) {
#pragma unroll
    for (int q = 0; q < 2; ++q)
      *reinterpret_cast<float4*>(hT + (size_t)nj * seg_stride + (size_t)hr * 128 + x0 + hc + 4 * q) =
          *reinterpret_cast<const float4*>(sh + hr * kHLd + hc + 4 * q);
  }
}

// o[t][:] += R[t][:] h_s  for one chunk (64 tokens) of one later segment of one V-head.  Eight warps: warp w takes
// 16 token rows (w & 3) and 64 of the 128 value channels (w >> 2).  h_s, R and the result go through shared memory
// (operand loads straight from global memory were latency-bound: 64 small tile loads per warp); the o values to be
// corrected are fetched at the very start, with the operands, so that their latency is paid once.
constexpr int kLdR = 128 + 8, kLdC = 64 + 4;
constexpr size_t kOutSmem = (size_t)(64 + 128) * kLdR * 2 + (size_t)8 * 16 * kLdC * 4;

__global__ void __launch_bounds__(256) seg_out_kernel(SegBuffers sg, __nv_bfloat16* o, int T_row, int HV, int cps,
                                                      const int32_t* seq_tok0, const int32_t* seq_len) {
  using namespace nvcuda;
  extern __shared__ __align__(32) uint8_t osm[];
  __nv_bfloat16* sR = reinterpret_cast<__nv_bfloat16*>(osm);                  // [64][kLdR]: the chunk's rows of R
  __nv_bfloat16* sB = sR + 64 * kLdR;                                          // [128][kLdR]: h_s
  float* sC = reinterpret_cast<float*>(sB + 128 * kLdR);                       // [8][16][kLdC]
  // `cps` = chunks per segment of the longest sequence the grid was sized for; shorter sequences leave CTAs idle
  const int j = blockIdx.y;
  const int cin = blockIdx.x % cps;
  const int seg = 1 + (blockIdx.x / cps) % (sg.nseg - 1);
  const int n = blockIdx.x / (cps * (sg.nseg - 1));
  const int len = seq_len ? seq_len[n] : T_row;          // (packed batches: the plan kernel's per-sequence table)
  const int tok0 = seq_tok0 ? seq_tok0[n] : n * T_row;
  const int nch = (len + kChunk - 1) / kChunk;
  const int cpseg = (nch + sg.nseg - 1) / sg.nseg;
  const int cc = seg * cpseg + cin;                      // this CTA's chunk of the sequence
  const int cend = min((seg + 1) * cpseg, nch);          // end of the segment
  asm volatile("griddepcontrol.wait;" ::: "memory");     // (programmatic dependent of the fix-up kernel)
  if (cin >= cpseg || cc >= cend) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t row0 = (size_t)tok0 + (size_t)cc * kChunk;
  const int rows_here = min(kChunk, len - cc * kChunk);  // valid token rows of the chunk
  const int rt = warp & 3, half = warp >> 2;
  const int rows = min(16, rows_here - rt * 16);         // this warp's valid rows
  const __nv_bfloat16* hs = sg.hs + (((size_t)n * HV + j) * sg.nseg + seg) * 128 * 128;
  __nv_bfloat162* op = reinterpret_cast<__nv_bfloat162*>(o + ((row0 + rt * 16) * HV + j) * 128 + half * 64 + lane * 2);
  const size_t rstride = (size_t)HV * 64;                // one token row further, in bf16 pairs
  __nv_bfloat162 ov[16];
  {
    uint4 w[8], r[4];                                    // all loads of a thread in flight together
#pragma unroll
    for (int q = 0; q < 8; ++q) w[q] = *reinterpret_cast<const uint4*>(hs + (size_t)(q * 256 + tid) * 8);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = q * 256 + tid, t = idx >> 4, p8 = idx & 15;
      r[q] = make_uint4(0u, 0u, 0u, 0u);                 // rows past the chunk's end as zeros
      if (t < rows_here) r[q] = *reinterpret_cast<const uint4*>(sg.r + ((row0 + t) * HV + j) * 128 + p8 * 8);
    }
#pragma unroll
    for (int rr = 0; rr < 16; ++rr)
      if (rr < rows) ov[rr] = op[rr * rstride];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int idx = q * 256 + tid;
      *reinterpret_cast<uint4*>(sB + (idx >> 4) * kLdR + (idx & 15) * 8) = w[q];
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int idx = q * 256 + tid;
      *reinterpret_cast<uint4*>(sR + (idx >> 4) * kLdR + (idx & 15) * 8) = r[q];
    }
  }
  __syncthreads();
  if (rows <= 0) return;
  float acc[8][4];                                       // eight tiles of 8 columns; mma.sync's accumulator layout
#pragma unroll
  for (int x = 0; x < 8; ++x) acc[x][0] = acc[x][1] = acc[x][2] = acc[x][3] = 0.f;
  // ldmatrix addresses: A, lane l -> row l % 16, columns 8 (l / 16)..; B (transposed on the way in), lane l ->
  // row (k) l % 16, columns 8 (l / 16)..: two 8-column tiles per instruction
  const __nv_bfloat16* pa = sR + (rt * 16 + (lane & 15)) * kLdR + (lane >> 4) * 8;
  const __nv_bfloat16* pb = sB + (lane & 15) * kLdR + half * 64 + (lane >> 4) * 8;
#pragma unroll 2
  for (int k = 0; k < 8; ++k) {
    uint32_t a[4];
    ldsm_x4(a, pa + k * 16);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      uint32_t b[4];
      ldsm_x4_trans(b, pb + (k * 16) * kLdR + x * 16);
      mma_bf16(acc[2 * x], a, b[0], b[1]);
      mma_bf16(acc[2 * x + 1], a, b[2], b[3]);
    }
  }
  float* myC = sC + warp * 16 * kLdC;
  {
    const int g = lane >> 2, t2 = (lane & 3) * 2;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      *reinterpret_cast<float2*>(myC + g * kLdC + x * 8 + t2) = make_float2(acc[x][0], acc[x][1]);
      *reinterpret_cast<float2*>(myC + (g + 8) * kLdC + x * 8 + t2) = make_float2(acc[x][2], acc[x][3]);
    }
  }
  __syncwarp();
#pragma unroll
  for (int rr = 0; rr < 16; ++rr) {                      // each lane adds two columns of every row
    if (rr < rows) {
      const float2 c = *reinterpret_cast<const float2*>(myC + rr * kLdC + lane * 2);
      const float2 f = __bfloat1622float2(ov[rr]);
      op[rr * rstride] = __floats2bfloat162_rn(f.x + c.x, f.y + c.y);
    }
  }
}

}  // namespace

// Both kernels, behind the chain kernel on the same stream.
cudaError_t launch_tc_seg_fix(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const SegBuffers& sg,
                              cudaStream_t stream) {
  if (sg.nseg <= 1 || p.N * p.HV == 0) return cudaSuccess;
  // (per device and idempotent; a few microseconds on the host, on a path that is already several launches long)
  cudaError_t ce = cudaFuncSetAttribute(seg_fix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFixSmem);
  if (ce == cudaSuccess) ce = cudaFuncSetAttribute(seg_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kOutSmem);
  if (ce != cudaSuccess) return ce;
  // Both kernels are launched as programmatic dependents of the kernel before them (each waits for it on the
  // device before its first read), which hides their launch latency under that kernel's tail.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = g_timer ? 0 : 1;                        // (per-kernel timing wants one kernel at a time)
  timer_mark(stream, "tc_seg_fix");
  cfg.gridDim = dim3((unsigned)(p.N * p.HV), 128 / kFixCols);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = kFixSmem;
  ce = cudaLaunchKernelEx(&cfg, seg_fix_kernel, sg, a.hT, p.T_row, p.HV, (const int32_t*)plan.seq_len);
  if (ce != cudaSuccess) return ce;
  const int nch = p.max_seq_chunks;                      // longest sequence (a bound, for packed batches)
  const int cpseg = (nch + sg.nseg - 1) / sg.nseg;
  if (nch <= cpseg) return cudaSuccess;                  // (everything is in segment 0)
  timer_mark(stream, "tc_seg_out");
  cfg.gridDim = dim3((unsigned)(p.N * (sg.nseg - 1) * cpseg), (unsigned)p.HV);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = kOutSmem;
  return cudaLaunchKernelEx(&cfg, seg_out_kernel, sg, reinterpret_cast<__nv_bfloat16*>(a.o), p.T_row, p.HV, cpseg,
                            (const int32_t*)plan.seq_tok0, (const int32_t*)plan.seq_len);
}

}  // namespace ha_la
