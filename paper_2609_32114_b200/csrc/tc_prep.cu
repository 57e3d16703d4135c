// Chunk-local operators of the delta-rule prefill on tcgen05 tensor cores (GDN).
//
// One CTA per (chunk slot, V-head).  Implements, for its chunk (paper Section 2.1, "Chunkwise
// Map-Reduce-Map Execution"):
//   #1 Gate   G = chunk-local cumulative log-gate (warp scan)
//   #2 KKT    S = [K; Q] K^T on the tensor cores (one M=128 MMA covers K K^T and Q K^T), then
//             A_ij = beta_i e^{G_i-G_j} S_kk[i,j] (j<i)  and  P_ij = e^{G_i-G_j} S_qk[i,j] (j<=i) in fp32
//   #3 Solve  T = (I + A)^-1 in fp32: two 32x32 diagonal blocks by forward substitution, the
//             off-diagonal block as -T_11 (A_10 T_00)
//   #4 W/U    W^T = K^T (T diag(beta e^G))^T,  U^T = V^T (T diag(beta))^T   (M = feature dim = 128)
// and the chunk-local halves of operator #6, so that the sequential kernel needs one stacked MMA:
//             Q~ = Q e^G - P W      O_loc = P U        (o = scale [Q~ h + O_loc])
// Operands arrive by TMA (bf16, 128-byte swizzle), accumulators live in tensor memory, results go
// to the workspace as ready-to-use operand images (tc_common.cuh).
//
// Tokens past the end of a sequence are made no-ops by beta = 0 and g = 0; whatever the TMA box
// read for them (the next sequence's rows, or zero fill past the end of the tensor) is multiplied
// by exact zeros.  This relies on the inputs being finite.
#include <cuda.h>

#include "tc_common.cuh"
#include "tc_ptx.cuh"

namespace ha_la {

using namespace ptx;

namespace {

constexpr int kPrepThreads = 128;
constexpr int LDF = 68;                  // row stride (floats) of the fp32 64x64 matrices
constexpr int LDX = 36;                  // row stride of the 32x32 scratch

// shared-memory map (bytes from the 1024-aligned base)
constexpr uint32_t OFF_KQ = 0;           // [kb][K 8K | Q 8K], kb = 0,1 (feature halves)
constexpr uint32_t OFF_V = 32768;        // [kb][V 8K]
constexpr uint32_t OFF_R1 = 49152;       // solve scratch, later the W^T / U^T operand tiles
constexpr uint32_t OFF_A = OFF_R1;                       // fp32 [64][LDF]; later T^W, T^U tiles
constexpr uint32_t OFF_T = OFF_R1 + 64 * LDF * 4;        // fp32 [64][LDF]
constexpr uint32_t OFF_X = OFF_T + 64 * LDF * 4;         // fp32 [32][LDX]
constexpr uint32_t OFF_TW = OFF_R1;                      // bf16 [64][64] K-major, swizzled (8 KiB)
constexpr uint32_t OFF_TU = OFF_R1 + 8192;
constexpr uint32_t OFF_WT = OFF_R1;                      // bf16 [128][64] K-major, swizzled (16 KiB)
constexpr uint32_t OFF_UT = OFF_R1 + 16384;
constexpr uint32_t OFF_P = OFF_R1 + 40960;               // bf16 [64][64] K-major, swizzled
constexpr uint32_t OFF_MISC = OFF_P + 8192;              // floats: G[64], beta[64], e^G[64], beta e^G[64]
constexpr uint32_t OFF_BAR = OFF_MISC + 4 * 64 * 4;
constexpr uint32_t kPrepSmem = OFF_BAR + 64;
static_assert(OFF_X + 32 * LDX * 4 <= OFF_P, "solve scratch overlaps P");
static_assert(OFF_UT + 16384 <= OFF_P, "operand tiles overlap P");

struct PrepParams {
  const float* g;
  const float* beta;
  const int32_t* chunk_tok0;
  const int32_t* chunk_len;
  TcWorkspace ws;
  int HK, HV;
  int32_t* status;
};

__device__ __forceinline__ void ld64(uint32_t taddr, float (&v)[64]) {
  uint32_t r0[32], r1[32];
  tmem_ld32(taddr, r0);
  tmem_ld32(taddr + 32, r1);
  tmem_ld_wait();
#pragma unroll
  for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(r0[i]); v[32 + i] = __uint_as_float(r1[i]); }
}

// 64 fp32 values of one feature row -> eight 16-byte pieces of bf16, swizzled, to shared and/or global
__device__ __forceinline__ void store_row_image(const float (&v)[64], int row, uint8_t* smem_tile, uint8_t* gmem_img) {
#pragma unroll
  for (int ch = 0; ch < 8; ++ch) {
    uint4 w;
    w.x = pack_bf16(v[ch * 8 + 0], v[ch * 8 + 1]);
    w.y = pack_bf16(v[ch * 8 + 2], v[ch * 8 + 3]);
    w.z = pack_bf16(v[ch * 8 + 4], v[ch * 8 + 5]);
    w.w = pack_bf16(v[ch * 8 + 6], v[ch * 8 + 7]);
    const uint32_t off = sw128_offset(row, ch);
    if (smem_tile) *reinterpret_cast<uint4*>(smem_tile + off) = w;
    if (gmem_img) *reinterpret_cast<uint4*>(gmem_img + off) = w;
  }
}

__global__ void __launch_bounds__(kPrepThreads, 2)
tc_prep_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, PrepParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* sA = reinterpret_cast<float*>(sm + OFF_A);
  float* sT = reinterpret_cast<float*>(sm + OFF_T);
  float* sX = reinterpret_cast<float*>(sm + OFF_X);
  float* sG = reinterpret_cast<float*>(sm + OFF_MISC);
  float* sBeta = sG + 64;
  float* sEG = sG + 128;
  float* sBE = sG + 192;
  uint64_t* bar_load = reinterpret_cast<uint64_t*>(sm + OFF_BAR);
  uint64_t* bar_mma = bar_load + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_load + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sTmp = reinterpret_cast<float*>(tmem_slot + 2);

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int cj = blockIdx.x;
  const int s = cj / p.HV, j = cj % p.HV;
  const int jq = j / (p.HV / p.HK);
  const int L = p.chunk_len[s];
  if (L <= 0) return;                                    // unused chunk slot (uniform for the CTA)
  const int tok0 = p.chunk_tok0[s];

  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
  }
  if (warp == 0) tmem_alloc(tmem_slot, 256);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t TM_S = tmem, TM_W = tmem + 64, TM_U = tmem + 128, TM_Q = tmem, TM_O = tmem + 192;
  const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;

  if (tid == 0) {
    mbar_expect_tx(bar_load, 6 * 8192);
    for (int kb = 0; kb < 2; ++kb) {
      tma_load_3d(sm + OFF_KQ + kb * 16384, &map_k, bar_load, kb * 64, jq, tok0);
      tma_load_3d(sm + OFF_KQ + kb * 16384 + 8192, &map_q, bar_load, kb * 64, jq, tok0);
      tma_load_3d(sm + OFF_V + kb * 8192, &map_v, bar_load, kb * 64, j, tok0);
    }
  }

  // ---- op #1 Gate: inclusive scan of the log-gate over the chunk (threads 0..63)
  if (tid < 64) {
    const bool valid = tid < L;
    float x = valid ? p.g[(size_t)(tok0 + tid) * p.HV + j] : 0.f;
    const float b = valid ? p.beta[(size_t)(tok0 + tid) * p.HV + j] : 0.f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (tid == 31) *sTmp = x;
    sBeta[tid] = b;
    sG[tid] = x;                                         // warp 1 adds warp 0's total below
  }
  __syncthreads();
  if (tid >= 32 && tid < 64) sG[tid] += *sTmp;
  __syncthreads();
  if (tid < 64) {
    const float e = __expf(sG[tid]);
    sEG[tid] = e;
    sBE[tid] = e * sBeta[tid];
  }

  // ---- op #2 KKT (+ Q K^T): S[0:64] = K K^T, S[64:128] = Q K^T
  if (tid == 0) {
    mbar_wait(bar_load, 0, abort_flag);
    tc_fence_after_sync();
    const uint32_t id = idesc_bf16(128, 64, false, false);
    const uint32_t base = smem_u32(sm + OFF_KQ);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint32_t a = base + (ks >> 2) * 16384 + (ks & 3) * 32;
      umma_ss(TM_S, smem_desc(a, 16, 1024, kSwizzle128B), smem_desc(a, 16, 1024, kSwizzle128B), id, ks > 0);
    }
    umma_commit(bar_mma);
  }
  __syncthreads();                                       // sEG / sBE visible to everyone
  mbar_wait(bar_mma, 0, abort_flag);
  tc_fence_after_sync();
  {
    float v[64];
    ld64(TM_S + lane_base, v);
    if (tid < 64) {                                      // row i of A (strictly lower, beta-scaled), fp32
      const int i = tid;
      const float gi = sG[i], bi = sBeta[i];
#pragma unroll
      for (int jj = 0; jj < 64; ++jj) {
        const float e = __expf(fminf(gi - sG[jj], 0.f));
        sA[i * LDF + jj] = jj < i ? bi * e * v[jj] : 0.f;
      }
    } else {                                             // row i of P (lower incl. diagonal), bf16 operand tile
      const int i = tid - 64;
      const float gi = sG[i];
#pragma unroll
      for (int jj = 0; jj < 64; ++jj) {
        const float e = __expf(fminf(gi - sG[jj], 0.f));
        v[jj] = jj <= i ? e * v[jj] : 0.f;
      }
      store_row_image(v, i, sm + OFF_P, nullptr);
    }
  }
  __syncthreads();

  // ---- op #3 Solve: T = (I + A)^-1, fp32
  if (warp < 2) {
    // diagonal 32x32 block `warp`: thread = column, forward substitution down the rows
    const int o = 32 * warp, c = lane;
    float x[32];
#pragma unroll
    for (int r = 0; r < 32; ++r) {
      float acc = r == c ? 1.f : 0.f;
      const float* arow = sA + (o + r) * LDF + o;
#pragma unroll
      for (int jj = 0; jj < r; ++jj) acc = fmaf(-arow[jj], x[jj], acc);
      x[r] = acc;
      sT[(o + r) * LDF + o + c] = acc;
    }
  } else {
    // upper-right 32x32 block of T is zero
    const int t2 = tid - 64;
    for (int idx = t2; idx < 32 * 32; idx += 64) sT[(idx >> 5) * LDF + 32 + (idx & 31)] = 0.f;
  }
  __syncthreads();
  {
    // X = A_10 T_00 ; thread -> row r, 8 columns
    const int r = tid >> 2, c0 = (tid & 3) * 8;
    float acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = 0.f;
#pragma unroll 8
    for (int m = 0; m < 32; ++m) {
      const float a = sA[(32 + r) * LDF + m];
      const float4 t0 = *reinterpret_cast<const float4*>(sT + m * LDF + c0);
      const float4 t1 = *reinterpret_cast<const float4*>(sT + m * LDF + c0 + 4);
      acc[0] = fmaf(a, t0.x, acc[0]); acc[1] = fmaf(a, t0.y, acc[1]);
      acc[2] = fmaf(a, t0.z, acc[2]); acc[3] = fmaf(a, t0.w, acc[3]);
      acc[4] = fmaf(a, t1.x, acc[4]); acc[5] = fmaf(a, t1.y, acc[5]);
      acc[6] = fmaf(a, t1.z, acc[6]); acc[7] = fmaf(a, t1.w, acc[7]);
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) sX[r * LDX + c0 + q] = acc[q];
  }
  __syncthreads();
  {
    // T_10 = -T_11 X
    const int r = tid >> 2, c0 = (tid & 3) * 8;
    float acc[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) acc[q] = 0.f;
#pragma unroll 8
    for (int m = 0; m < 32; ++m) {
      const float a = -sT[(32 + r) * LDF + 32 + m];      // zero for m > r
      const float4 x0 = *reinterpret_cast<const float4*>(sX + m * LDX + c0);
      const float4 x1 = *reinterpret_cast<const float4*>(sX + m * LDX + c0 + 4);
      acc[0] = fmaf(a, x0.x, acc[0]); acc[1] = fmaf(a, x0.y, acc[1]);
      acc[2] = fmaf(a, x0.z, acc[2]); acc[3] = fmaf(a, x0.w, acc[3]);
      acc[4] = fmaf(a, x1.x, acc[4]); acc[5] = fmaf(a, x1.y, acc[5]);
      acc[6] = fmaf(a, x1.z, acc[6]); acc[7] = fmaf(a, x1.w, acc[7]);
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) sT[(32 + r) * LDF + c0 + q] = acc[q];
  }
  __syncthreads();

  // ---- column-scaled copies of T as bf16 operand tiles: T^W = T diag(beta e^G), T^U = T diag(beta)
  {
    const int i = tid >> 1, hf = tid & 1;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int ch = hf * 4 + q;
      float tw[8], tu[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int jj = ch * 8 + e;
        const float t = sT[i * LDF + jj];
        tw[e] = t * sBE[jj];
        tu[e] = t * sBeta[jj];
      }
      uint4 w, u;
      w.x = pack_bf16(tw[0], tw[1]); w.y = pack_bf16(tw[2], tw[3]); w.z = pack_bf16(tw[4], tw[5]); w.w = pack_bf16(tw[6], tw[7]);
      u.x = pack_bf16(tu[0], tu[1]); u.y = pack_bf16(tu[2], tu[3]); u.z = pack_bf16(tu[4], tu[5]); u.w = pack_bf16(tu[6], tu[7]);
      const uint32_t off = sw128_offset(i, ch);
      *reinterpret_cast<uint4*>(sm + OFF_TW + off) = w;   // overwrites sA, which is dead by now
      *reinterpret_cast<uint4*>(sm + OFF_TU + off) = u;
    }
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();

  // ---- op #4 W/U: W^T = K^T (T^W)^T, U^T = V^T (T^U)^T  (A operands feature-major straight from the TMA tiles)
  if (tid == 0) {
    tc_fence_after_sync();
    const uint32_t id = idesc_bf16(128, 64, true, false);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(TM_W, smem_desc(smem_u32(sm + OFF_KQ) + ks * 2048, 16384, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_TW) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(TM_U, smem_desc(smem_u32(sm + OFF_V) + ks * 2048, 8192, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_TU) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
    umma_commit(bar_mma);
  }
  mbar_wait(bar_mma, 1, abort_flag);
  tc_fence_after_sync();
  {
    float v[64];
    ld64(TM_W + lane_base, v);                           // row = key channel tid, columns = tokens
    store_row_image(v, tid, sm + OFF_WT, p.ws.wq + (size_t)cj * 2 * kImgBytes);
    ld64(TM_U + lane_base, v);
    store_row_image(v, tid, sm + OFF_UT, p.ws.u + (size_t)cj * kImgBytes);
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();

  // ---- chunk-local halves of op #6: (P W)^T = W^T P^T, O_loc^T = U^T P^T
  if (tid == 0) {
    tc_fence_after_sync();
    const uint32_t id = idesc_bf16(128, 64, false, false);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(TM_Q, smem_desc(smem_u32(sm + OFF_WT) + ks * 32, 16, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_P) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(TM_O, smem_desc(smem_u32(sm + OFF_UT) + ks * 32, 16, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_P) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
    umma_commit(bar_mma);
  }
  mbar_wait(bar_mma, 0, abort_flag);
  tc_fence_after_sync();
  {
    float v[64];
    ld64(TM_Q + lane_base, v);
    // Q~^T[c][i] = Q[i][c] e^{G_i} - (P W)[i][c], c = tid
    const uint8_t* qtile = sm + OFF_KQ + (tid >> 6) * 16384 + 8192;
    const int cc = tid & 63;
#pragma unroll
    for (int i = 0; i < 64; ++i) {
      const __nv_bfloat16 qv = *reinterpret_cast<const __nv_bfloat16*>(qtile + sw128_offset(i, cc >> 3) + (cc & 7) * 2);
      v[i] = fmaf(__bfloat162float(qv), sEG[i], -v[i]);
    }
    store_row_image(v, tid, nullptr, p.ws.wq + (size_t)cj * 2 * kImgBytes + kImgBytes);
    ld64(TM_O + lane_base, v);
    store_row_image(v, tid, nullptr, p.ws.ol + (size_t)cj * kImgBytes);
  }
  {
    float* sc = p.ws.sc + (size_t)cj * kScFloats;
    const float gl = sG[63];
    if (tid < 64) sc[tid] = __expf(gl - sG[tid]);
    sc[64 + tid] = __expf(gl);
  }
  if (*abort_flag && tid == 0) report_status(p.status, HA_LA_ERR_TIMEOUT);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

cudaError_t launch_tc_prep(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                           const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t stream) {
  PrepParams pp;
  pp.g = a.g; pp.beta = a.beta;
  pp.chunk_tok0 = plan.chunk_tok0; pp.chunk_len = plan.chunk_len;
  pp.ws = ws; pp.HK = p.HK; pp.HV = p.HV; pp.status = a.status_word;
  const int smem = kPrepSmem + 1024;
  cudaError_t e = cudaFuncSetAttribute(tc_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  const long long grid = (long long)p.max_chunks * p.HV;
  if (grid == 0) return cudaSuccess;
  timer_mark(stream, "tc_prep");
  tc_prep_kernel<<<(unsigned)grid, kPrepThreads, smem, stream>>>(mq, mk, mv, pp);
  return cudaGetLastError();
}

}  // namespace ha_la
