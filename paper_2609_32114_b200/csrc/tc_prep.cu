// Chunk-local operators of the delta-rule prefill on tcgen05 tensor cores (GDN and KDA).
//
// A persistent kernel, one CTA per SM, whose work items are (chunk slot, V-head) pairs in chunk-major order.
// GDN: a CTA holds three independent work groups of 8 warps (own shared memory, named barrier and quarter of
// tensor memory), i.e. three items are in flight per SM.  KDA: one group of 16 warps per CTA; warps 8..15 only
// run the gate-dependent element-wise passes, stage the next item's gate rows and prefetch later ones into L2.
// A group implements, for its chunk (paper Section 2.1, "Chunkwise Map-Reduce-Map Execution"):
//   #1 Gate   G = chunk-local cumulative log-gate (GDN: one scalar per token; KDA: one per key channel)
//   #2 KKT    GDN: S = [K; Q] K^T on the tensor cores (one M=128 MMA covers K K^T and Q K^T), then
//             A_ij = beta_i e^{G_i-G_j} S_kk[i,j] (j<i)  and  P_ij = e^{G_i-G_j} S_qk[i,j] (j<=i) in fp32.
//             KDA: the decay sits inside the contraction; see the comment at that pass.
//   #3 Solve  T = (I + A)^-1 by blocked forward substitution: four 16x16 diagonal blocks in fp32 registers,
//             then the off-diagonal blocks level by level as T_lo = -T_hi (A_lo T_lo') on mma.sync (fp16
//             operands, fp32 accumulation).  A and T are held in shared memory as fp16 (T is rounded to bf16
//             for the next operator anyway); this assumes the delta rule's usual normalisation
//             (beta |k|^2 of order one), far inside the fp16 range.
//   #4 W/U    W^T = K^T (T diag(beta e^G))^T,  U^T = V^T (T diag(beta))^T   (M = feature dim = 128)
// and the chunk-local halves of operator #6, so that the sequential kernel needs one stacked MMA:
//             Q~ = Q e^G - P W      O_loc = P U        (o = scale [Q~ h + O_loc])
// (Q e^G enters the Q~ accumulator as one more MMA, Q^T diag(e^G), and P W with the negate-A flag.)
// Operands arrive by TMA (bf16, 128-byte swizzle), accumulators live in tensor memory, results are
// assembled in shared memory as ready-to-use operand images (tc_common.cuh) and leave by bulk copy.  The next
// item's tiles, gates and position are fetched while the current one finishes.  When the chain kernel runs
// concurrently, each item is published with a release flag once its bulk stores have completed.
//
// Warp w (of the first 8) reads tensor-memory lanes 32*(w%4)..+31 (accumulator rows) and columns 32*(w/4)..+31.
//
// Tokens past the end of a sequence are made no-ops by beta = 0 and g = 0; whatever the TMA box
// read for them (the next sequence's rows, or zero fill past the end of the tensor) is multiplied
// by exact zeros.  This relies on the inputs being finite.
#include <cuda.h>
#include <cuda_fp16.h>

#include "tc_common.cuh"
#include "tc_ptx.cuh"
#include "prof.cuh"

namespace ha_la {

using namespace ptx;

HA_PROF_DECL(prep)

namespace {

constexpr int kPrepThreads = 256;        // threads of one work group that run every phase (a CTA holds kGroups groups)
constexpr int kKdaThreads = 512;         // KDA: the group has 8 more warps, which only run the gate-dependent passes
constexpr int LDH = 72;                  // row stride (halfs) of the fp16 64x64 matrix A / T

// shared-memory map (bytes from the 1024-aligned base); 73.3 KiB, so that three CTAs fit one SM
constexpr uint32_t OFF_KQ = 0;           // [kb][K 8K | Q 8K], kb = 0,1 (feature halves)
constexpr uint32_t OFF_E = OFF_KQ;       // bf16 [64][64] diag(e^G) tile over the first K piece, once K is dead
constexpr uint32_t OFF_V = 32768;        // [kb][V 8K]; later the U image, then the O_loc image
constexpr uint32_t OFF_UT = OFF_V;
constexpr uint32_t OFF_R1 = 49152;       // 16 KiB: A / T (fp16), then T^W | T^U, then the W image, then the Q~ image
constexpr uint32_t OFF_A = OFF_R1;                       // fp16 [64][LDH]: A, overwritten in place by T
constexpr uint32_t OFF_D = OFF_R1 + 64 * LDH * 2;        // fp16 4 x [16][16]: inverses of the diagonal blocks
constexpr uint32_t OFF_TW = OFF_R1;                      // bf16 [64][64] K-major, swizzled (8 KiB)
constexpr uint32_t OFF_TU = OFF_R1 + 8192;
constexpr uint32_t OFF_WT = OFF_R1;                      // bf16 [128][64] K-major, swizzled (16 KiB)
constexpr uint32_t OFF_P = OFF_R1 + 16384;               // bf16 [64][64] K-major, swizzled
constexpr uint32_t OFF_MISC = OFF_P + 8192;              // floats: G[64], beta[64], e^G[64], beta e^G[64], G log2e[64]
constexpr uint32_t OFF_RAW = OFF_MISC + 5 * 64 * 4;      // floats: log-gate[64], beta[64] of the NEXT item (cp.async)
constexpr uint32_t OFF_BAR = OFF_RAW + 2 * 64 * 4;
constexpr uint32_t kPrepSmem = OFF_BAR + 64;
static_assert(OFF_D + 4 * 256 * 2 <= OFF_P, "solve scratch overlaps P");
// GDN: one CTA per SM holds three independent work groups (256 threads and one copy of this map each, their own
// named barrier and quarter of tensor memory), which is the occupancy of three small CTAs but leaves whole SMs
// to a concurrently running chain kernel.  KDA (larger map): one group.
constexpr uint32_t kGroupSmem = (kPrepSmem + 1023) / 1024 * 1024;
template <bool KDA> constexpr int kGroups = KDA ? 1 : 3;
static_assert(3 * kGroupSmem <= 227 * 1024, "three work groups per CTA");
// KDA only: per-channel cumulative log-gate (fp32, times log2 e) and the K e^{G_L - G} operand image
constexpr int LDG = 132;                                  // row stride (floats) of the 64 x 128 gate matrix
constexpr uint32_t OFF_G = (kPrepSmem + 1023) / 1024 * 1024;
constexpr uint32_t OFF_KD = (OFF_G + 64 * LDG * 4 + 1023) / 1024 * 1024;   // [kb][64 tok][64 feat], like the K tile
// K+ / Q+ rows (block b: 16 K+ rows then 16 Q+ rows): one M = 128 operand
constexpr uint32_t OFF_KQP = OFF_KD + 16384;              // [kb][128 rows][128 B], K-major, swizzled
constexpr uint32_t KQP_KB = 128 * 128;
// K- rows for block-rows I = 0..3 (16, 32, 48, 64 rows, starting at rows 0, 16, 48, 96)
constexpr uint32_t OFF_KM = OFF_KQP + 2 * KQP_KB;         // [kb][160 rows][128 B], K-major, swizzled
constexpr uint32_t KM_KB = 160 * 128;
constexpr uint32_t OFF_FALL = OFF_KM + 2 * KM_KB;         // int[4]: diagonal block needs the element-wise evaluation
constexpr uint32_t OFF_QT = OFF_FALL + 16;                // float[4][128]: per-channel totals of the scan's four quarters
constexpr uint32_t kPrepSmemKda = OFF_QT + 4 * 128 * 4;
constexpr float kMaxUpExp = 100.f;                        // largest exponent (base 2) allowed in a K- factor
static_assert(kPrepSmemKda <= 227 * 1024, "KDA shared memory budget");

struct PrepParams {
  const float* g;
  const float* beta;
  const int32_t* chunk_tok0;   // chunk table of the plan kernel, or NULL for equal-length rows:
  const int32_t* chunk_len;    //   then slot s is chunk s % cps of row s / cps, T_row tokens per row
  int T_row, cps;
  TcWorkspace ws;
  int HK, HV;
  long long total;        // work items = chunk slots x V-heads
  int64_t epoch;          // published to ws.flags[cj] when this CTA's results are in memory (0: do not publish)
  int32_t* status;
};

__device__ __forceinline__ void ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  tmem_ld32(taddr, r);
  tmem_ld_wait();
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void cp_async4(void* sdst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(sdst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {          // 2^x, flushes to zero for very negative x
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8]) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = __uint_as_float(u[e] << 16);
    f[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}

__device__ __forceinline__ void unpack8h(const uint4& w, float (&f)[8]) {          // 8 fp16 -> fp32
  const __half2* h = reinterpret_cast<const __half2*>(&w);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 t = __half22float2(h[e]);
    f[2 * e] = t.x;
    f[2 * e + 1] = t.y;
  }
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Warp-level fp16 matrix products on the legacy tensor path (mma.sync m16n8k16, fp32 accumulation) with
// operands fetched by ldmatrix from row-major fp16 matrices in shared memory.
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const __half* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)) : "memory");
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], const __half* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];"
               : "=r"(r[0]), "=r"(r[1]) : "r"(smem_u32(p)) : "memory");
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One level of the blocked solve for BS x BS blocks (BS = 16 or 32):  T10 = -T11 (A10 T00), evaluated
// transposed so that the first product's accumulators are the second product's A fragments:
//   X^T = T00^T A10^T  (all BS/8 column tiles, needed as the contraction index of the second product),
//   R^T = X^T T11^T    (NT2 tiles of 8 rows of T10, starting at tile nt2_0),
// for the 16 columns mt*16.. of T10.  Results stay in registers (c2); store_merge() writes them over A10.
template <int BS, int NT2>
__device__ __forceinline__ void merge_compute(float (&c2)[NT2][4], const __half* T00, int ld00, const __half* A10,
                                              int ldA, const __half* T11, int ld11, int mt, int nt2_0, int lane) {
  constexpr int KS = BS / 16, NT = BS / 8;
  float c1[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) c1[nt][0] = c1[nt][1] = c1[nt][2] = c1[nt][3] = 0.f;
  const int j = lane >> 3, r = lane & 7;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    uint32_t a[4];
    ldsm_x4_t(a, T00 + (ks * 16 + (j >> 1) * 8 + r) * ld00 + mt * 16 + (j & 1) * 8);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      uint32_t b[2];
      ldsm_x2(b, A10 + (nt * 8 + r) * ldA + ks * 16 + (j & 1) * 8);
      mma_f16(c1[nt], a, b);
    }
  }
#pragma unroll
  for (int n2 = 0; n2 < NT2; ++n2) c2[n2][0] = c2[n2][1] = c2[n2][2] = c2[n2][3] = 0.f;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const uint32_t a[4] = {pack_f16(c1[2 * ks][0], c1[2 * ks][1]), pack_f16(c1[2 * ks][2], c1[2 * ks][3]),
                           pack_f16(c1[2 * ks + 1][0], c1[2 * ks + 1][1]), pack_f16(c1[2 * ks + 1][2], c1[2 * ks + 1][3])};
#pragma unroll
    for (int n2 = 0; n2 < NT2; ++n2) {
      uint32_t b[2];
      ldsm_x2(b, T11 + ((nt2_0 + n2) * 8 + r) * ld11 + ks * 16 + (j & 1) * 8);
      mma_f16(c2[n2], a, b);
    }
  }
}
template <int NT2>
__device__ __forceinline__ void merge_store(const float (&c2)[NT2][4], __half* T10, int ld, int mt, int nt2_0, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int n2 = 0; n2 < NT2; ++n2) {
    __half* d = T10 + ((nt2_0 + n2) * 8 + 2 * t) * ld + mt * 16 + g;
    d[0] = __float2half_rn(-c2[n2][0]);
    d[ld] = __float2half_rn(-c2[n2][1]);
    d[8] = __float2half_rn(-c2[n2][2]);
    d[ld + 8] = __float2half_rn(-c2[n2][3]);
  }
}

// 32 fp32 values (columns 32*hf .. +31 of one 64-column row) -> four 16-byte pieces of bf16, swizzled
__device__ __forceinline__ void store_half_row(const float (&v)[32], int row, int hf, uint8_t* tile) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 w;
    w.x = pack_bf16(v[q * 8 + 0], v[q * 8 + 1]);
    w.y = pack_bf16(v[q * 8 + 2], v[q * 8 + 3]);
    w.z = pack_bf16(v[q * 8 + 4], v[q * 8 + 5]);
    w.w = pack_bf16(v[q * 8 + 6], v[q * 8 + 7]);
    *reinterpret_cast<uint4*>(tile + sw128_offset(row, hf * 4 + q)) = w;
  }
}

template <bool KDA>
__global__ void __launch_bounds__(KDA ? kKdaThreads : kPrepThreads * kGroups<KDA>, 1)
tc_prep_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, PrepParams p) {
  constexpr int G = kGroups<KDA>;
  extern __shared__ __align__(1024) uint8_t smem_raw[];  // no static shared memory in this kernel: 1024-aligned
  constexpr int NT = KDA ? kKdaThreads : kPrepThreads;   // threads of a work group
  // Where the Q~ and O_loc images are staged for their bulk stores.  GDN: over the W and U images (which must
  // have left by then).  KDA: over the gate-scaled operand copies, dead once the first product is complete, so
  // that the group does not wait for the W / U / K e^{G_L-G} images to be read (48 KiB, some 1.5 k cycles).
  constexpr uint32_t OFF_QI = KDA ? OFF_KQP : OFF_WT;
  constexpr uint32_t OFF_OI = KDA ? OFF_KQP + 16384 : OFF_UT;
  const int grp = threadIdx.x / NT;                      // work group of this thread
  uint8_t* sm = smem_raw + grp * kGroupSmem;
  auto gsync = [&]() {                                   // barrier of the 8 warps of a group that run every phase
    asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "r"(kPrepThreads) : "memory");
  };
  auto bsync = [&]() {                                   // KDA: barrier of all 16 warps of the group
    asm volatile("bar.sync 8, %0;" ::"r"(kKdaThreads) : "memory");
  };
  __half* sAh = reinterpret_cast<__half*>(sm + OFF_A);  // A, then T in place
  __half* sD = reinterpret_cast<__half*>(sm + OFF_D);
  float* sG = reinterpret_cast<float*>(sm + OFF_MISC);
  float* sBeta = sG + 64;
  float* sEG = sG + 128;
  float* sBE = sG + 192;
  float* sRaw = reinterpret_cast<float*>(sm + OFF_RAW);
  uint64_t* bar_load = reinterpret_cast<uint64_t*>(sm + OFF_BAR);
  uint64_t* bar_mma = bar_load + 1;
  uint64_t* bar_v = bar_load + 2;                        // the V tiles arrive on their own barrier
  uint64_t* bar_g = bar_load + 7;                        // KDA: the log-gate rows of the next item
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_load + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* sNext = reinterpret_cast<int*>(tmem_slot + 2);    // next item: have, j, jq, L, tok0 (written by thread 0)

  const int tid = threadIdx.x % NT;
  const int warp = tid >> 5, lane = tid & 31;
  const bool is_main = !KDA || tid < kPrepThreads;       // KDA: warps 8..15 only help with the gate-dependent passes
  if (smem_u32(smem_raw) & 1023u) {                            // the swizzled layouts need it; never seen to fail
    if (threadIdx.x == 0) report_status(p.status, HA_LA_ERR_DEVICE_CHECK);
    return;
  }
  HA_PROF(prep, 0);
  if (blockIdx.x == 0 && threadIdx.x == 0) HA_PROF_GT(prep, 900);
#define PP(slot) HA_PROF(prep, 16 + 16 * (int)(cjl / vstride) + (slot))

  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_g, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
  }
  // the CTA's first warp allocates tensor memory for all groups (a power of two: everything, for three groups)
  if (threadIdx.x < 32) tmem_alloc(reinterpret_cast<uint32_t*>(smem_raw + OFF_BAR + 24), G == 1 ? 256 : 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // This kernel is launched as a programmatic dependent of whatever precedes it in the stream; when that is the
  // previous call's chain kernel, which lets its dependents go a few chunks before its end, everything above ran
  // under that kernel's tail.  Nothing of this call has been read or written so far: wait for the stream's earlier
  // work to complete here.  (A no-op after a kernel that triggers nothing early, or without the launch attribute.)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Every CTA of this grid is running now: a dependent launch (the chain kernel) may be scheduled.  It either
  // waits for this grid to finish or consumes chunks as they are published.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t tmem_cta = *reinterpret_cast<const uint32_t*>(smem_raw + OFF_BAR + 24);
  const uint32_t tmem = tmem_cta + grp * 128;
  const int rowq = (warp & 3) * 32 + lane;               // accumulator row owned by this thread
  const int hf = warp >> 2;                              // which 32 of the 64 columns
  const uint32_t my_tmem = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16) + hf * 32;
  HA_PROF(prep, 1);

  // Persistent groups: work items (chunk slot, V-head) g, g + #groups, ... for group g of the grid, so
  // that early chunks are finished first (the chain kernel may be consuming them concurrently).
  uint32_t mph = 0;                                      // parity of the next MMA-completion wait
  uint32_t lph = 0;                                      // parity of the next tile-load wait
  long long prev_cj = -1;                                // item whose bulk stores are still in flight (thread 0)
  auto item_geom = [&](long long c, int& j_, int& jq_, int& L_, int& tok0_) {   // (the item count fits 31 bits)
    const int s_ = (int)((unsigned)c / (unsigned)p.HV);
    j_ = (int)((unsigned)c - (unsigned)s_ * (unsigned)p.HV);
    jq_ = j_ / (p.HV / p.HK);
    if (p.chunk_len) {
      L_ = p.chunk_len[s_];
      tok0_ = p.chunk_tok0[s_];
    } else {
      const int cc_ = s_ % p.cps;
      tok0_ = (s_ / p.cps) * p.T_row + cc_ * kChunk;
      L_ = min(kChunk, p.T_row - cc_ * kChunk);
    }
  };
  auto issue_tiles_kb = [&](int jq_, int tok0_, int kb) { // feature half kb of the K and Q tiles of one item
    tma_load_3d(sm + OFF_KQ + kb * 16384, &map_k, bar_load, kb * 64, jq_, tok0_);
    tma_load_3d(sm + OFF_KQ + kb * 16384 + 8192, &map_q, bar_load, kb * 64, jq_, tok0_);
  };
  auto issue_tiles = [&](int jq_, int tok0_) {           // one thread: K and Q tiles of one item
    mbar_expect_tx(bar_load, 4 * 8192);
    issue_tiles_kb(jq_, tok0_, 0);
    issue_tiles_kb(jq_, tok0_, 1);
  };
  auto issue_v = [&](int j_, int tok0_) {                // thread 0: V tiles (their room is free later than K's)
    mbar_expect_tx(bar_v, 2 * 8192);
    for (int kb = 0; kb < 2; ++kb) tma_load_3d(sm + OFF_V + kb * 8192, &map_v, bar_v, kb * 64, j_, tok0_);
  };
  auto publish_prev = [&]() {                            // thread 0, concurrent mode: hand the previous item over
    if (p.epoch != 0 && prev_cj >= 0) {
      bulk_wait_all();
      fence_proxy_async_all();
      __threadfence();
      st_release_gpu(p.ws.flags + prev_cj, p.epoch);
      if (prev_cj % p.HV == 0) HA_PROF_GT(prep, 512 + (int)(prev_cj / p.HV));
    }
  };
  // The groups of a CTA start a third of an item apart, so that they are in different phases (tensor core /
  // CUDA cores / waiting for memory) at any time instead of in lock step.
  if (G > 1 && grp > 0) __nanosleep(2000u * grp);
  const long long vstride = (long long)gridDim.x * G;    // work groups in the grid
  long long cjl = (long long)grp * gridDim.x + blockIdx.x;   // group-major: a last partial round spreads over the SMs
  int j = 0, jq = 0, L = 0, tok0 = 0;
  bool have = cjl < p.total;
  if (have) { item_geom(cjl, j, jq, L, tok0); have = L > 0; }   // unused chunk slots come last
  // Warp 1 stages the per-token scalars of an item one item ahead: GDN, log-gate and beta with cp.async (two
  // tokens per lane), scanned at the top of that item; KDA, beta likewise and the 64 x 128 log-gate rows by
  // bulk copies straight into the gate matrix (512 contiguous bytes per token).
  auto stage_gates = [&](int j_, int L_, int tok0_, bool rows) {
    if (warp == 1) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int t = lane + 32 * h;
        if (t < L_) {
          if (!KDA) cp_async4(sRaw + t, p.g + (size_t)(tok0_ + t) * p.HV + j_);
          cp_async4(sRaw + 64 + t, p.beta + (size_t)(tok0_ + t) * p.HV + j_);
        } else {
          sRaw[t] = 0.f;
          sRaw[64 + t] = 0.f;
        }
      }
    }
    if (KDA && rows && warp == 8) {                      // a helper warp: off the other warps' critical path
      if (lane == 0) mbar_expect_tx(bar_g, (uint32_t)L_ * 512u);
      __syncwarp();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int t = lane + 32 * h;
        if (t < L_) {
          bulk_load(sm + OFF_G + t * LDG * 4, p.g + ((size_t)(tok0_ + t) * p.HV + j_) * 128, 512, bar_g);
        } else {
          float4* row = reinterpret_cast<float4*>(sm + OFF_G + t * LDG * 4);
          for (int c = 0; c < 32; ++c) row[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
    }
  };
  // KDA, helper warps (8..15): where the next item is (one thread), its gate rows (warp 8), and the gate rows of
  // the item after it into L2 (warp 9; 32 KiB from HBM take a while).
  auto helper_geom = [&]() {
    if (tid == kPrepThreads) {
      int jn = 0, jqn = 0, Ln = 0, tok0n = 0;
      bool hn = cjl + vstride < p.total;
      if (hn) { item_geom(cjl + vstride, jn, jqn, Ln, tok0n); hn = Ln > 0; }
      sNext[0] = hn ? 1 : 0; sNext[1] = jn; sNext[2] = jqn; sNext[3] = Ln; sNext[4] = tok0n;
    }
  };
  auto helper_fetch = [&]() {                            // (after helper_geom and a barrier or __syncwarp)
    if (warp == 8 && sNext[0]) stage_gates(sNext[1], sNext[3], sNext[4], true);
    if (warp == 9) {
      int j2 = 0, jq2 = 0, L2 = 0, t2 = 0;
      if (lane == 0 && cjl + 2 * vstride < p.total) item_geom(cjl + 2 * vstride, j2, jq2, L2, t2);
      j2 = __shfl_sync(0xffffffffu, j2, 0);
      L2 = __shfl_sync(0xffffffffu, L2, 0);
      t2 = __shfl_sync(0xffffffffu, t2, 0);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int t = lane + 32 * h;
        if (t < L2) bulk_prefetch_l2(p.g + ((size_t)(t2 + t) * p.HV + j2) * 128, 512);
      }
    }
  };
  if (have) {
    if (tid == 0) issue_tiles(jq, tok0);
    stage_gates(j, L, tok0, true);
  }
  while (have) {
  const size_t cj = (size_t)cjl;
  if constexpr (KDA) {
    // The previous item's W / U / K e^{G_L-G} images (its first group of bulk stores, issued long ago) have left
    // shared memory: V lands on one, the rescaling pass rewrites another.  Its Q~ / O_loc images (second group)
    // sit where the gate-scaled operand copies go, and are waited for just before those are written.
    if (tid == 0) {
      if (prev_cj >= 0) bulk_wait_read_1();
      issue_v(j, tok0);
      publish_prev();
    }
    bsync();
    // ---- op #1 Gate, per key channel: G[i][c] = cumulative log-gate, kept times log2(e) for ex2
    float* sGc = reinterpret_cast<float*>(sm + OFF_G);
    float* sQt = reinterpret_cast<float*>(sm + OFF_QT);    // totals of the four 16-row quarters of the scan
    int* sFall = reinterpret_cast<int*>(sm + OFF_FALL);
    PP(2);
    {
      if (warp == 1) {
        cp_async_wait_all();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float b = sRaw[64 + lane + 32 * h];
          sBeta[lane + 32 * h] = b;
          sBE[lane + 32 * h] = b;                        // the gate factor lives in the K operand, not in T^W
          sEG[lane + 32 * h] = 1.f;                      // and Q is rescaled in place: E = identity
        }
      }
      if (tid < 4) sFall[tid] = 0;
    }
    if (warp == 0) mbar_wait(bar_g, lph, abort_flag);    // the raw log-gate rows (staged during the previous item)
    bsync();
    PP(3);
    const int sc_c = tid & 127, sc_q = tid >> 7;         // scan: four threads per channel, 16 rows each
    {
      float acc = 0.f;
      for (int i = 0; i < 16; ++i) {
        acc = fmaf(sGc[(16 * sc_q + i) * LDG + sc_c], 1.4426950408889634f, acc);
        sGc[(16 * sc_q + i) * LDG + sc_c] = acc;
      }
      sQt[sc_q * 128 + sc_c] = acc;
    }
    bsync();
    if (sc_q > 0) {
      float add = sQt[sc_c];
      if (sc_q > 1) add += sQt[128 + sc_c];
      if (sc_q > 2) add += sQt[256 + sc_c];
      for (int i = 0; i < 16; ++i) sGc[(16 * sc_q + i) * LDG + sc_c] += add;
    }
    mbar_wait(bar_load, lph, abort_flag);                // every thread reads the K / Q tiles below
    // the previous item's Q~ / O_loc images have left the room of the operand copies written next
    if (tid == 0 && prev_cj >= 0) bulk_wait_read_all();
    bsync();
    PP(4);

    // ---- op #2 KKT and the masked Q K^T with per-channel decay:
    //   A_ij = beta_i sum_c k_ic k_jc 2^(G_ic - G_jc) (j < i),  P_ij = sum_c q_ic k_jc 2^(G_ic - G_jc) (j <= i).
    // Tokens are grouped in blocks of 16.  For i in block-row I the decay factors through the gate R_I at the
    // first token of block I:  2^(G_i - R_I) * 2^(R_I - G_j), so every block is a plain contraction of rescaled
    // bf16 operands on the tensor cores:
    //   K+_i = k_i 2^(G_i - R_I), Q+_i = q_i 2^(G_i - R_I)   (one copy),   K-_j^(I) = k_j 2^(R_I - G_j)  (per block-row I).
    // The first exponent is <= 0.  The second is <= 0 for j in an earlier block; inside the diagonal block it is
    // the decay accumulated since the start of the block, >= 0: it is clamped to kMaxUpExp, and a block where the
    // clamp was hit (a decay of more than 2^100 within 16 tokens in some channel) is evaluated again afterwards,
    // element by element in fp32.
    {
      // eight threads per token; thread t takes the 8-channel pieces t and t + 8, so that the eight threads of a
      // token read 256 contiguous bytes of a gate row and a whole 128-byte row of a K / Q tile (no bank conflicts)
      const int i = tid >> 3, bi16 = i >> 4;
      const int row_k = 32 * bi16 + (i & 15);
      bool clamped = false;
#pragma unroll 1
      for (int q = 0; q < 2; ++q) {
        const int cc = (tid & 7) + 8 * q;
        const uint8_t* kt = sm + OFF_KQ + (cc >> 3) * 16384;
        const uint32_t off = sw128_offset(i, cc & 7);
        float kf[8], qf[8], gi[8], gr[8], t8[8];
        unpack8(*reinterpret_cast<const uint4*>(kt + off), kf);
        unpack8(*reinterpret_cast<const uint4*>(kt + 8192 + off), qf);
        *reinterpret_cast<float4*>(gi) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8);
        *reinterpret_cast<float4*>(gi + 4) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8 + 4);
        *reinterpret_cast<float4*>(gr) = *reinterpret_cast<const float4*>(sGc + (bi16 * 16) * LDG + cc * 8);
        *reinterpret_cast<float4*>(gr + 4) = *reinterpret_cast<const float4*>(sGc + (bi16 * 16) * LDG + cc * 8 + 4);
        uint8_t* kqp = sm + OFF_KQP + (cc >> 3) * KQP_KB;
        uint8_t* km = sm + OFF_KM + (cc >> 3) * KM_KB;
        {                                                // K- for the token's own block-row (exponent >= 0)
          float up[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            up[e] = gr[e] - gi[e];
            clamped |= up[e] > kMaxUpExp;
            t8[e] = kf[e] * ex2(fminf(up[e], kMaxUpExp));
          }
          const int r0 = bi16 == 0 ? 0 : (bi16 == 1 ? 16 : (bi16 == 2 ? 48 : 96));
          *reinterpret_cast<uint4*>(km + sw128_offset(r0 + i, cc & 7)) = pack8(t8);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) { gr[e] = ex2(gi[e] - gr[e]); t8[e] = kf[e] * gr[e]; }
        *reinterpret_cast<uint4*>(kqp + sw128_offset(row_k, cc & 7)) = pack8(t8);
#pragma unroll
        for (int e = 0; e < 8; ++e) t8[e] = qf[e] * gr[e];
        *reinterpret_cast<uint4*>(kqp + sw128_offset(row_k + 16, cc & 7)) = pack8(t8);
        for (int I2 = bi16 + 1; I2 < 4; ++I2) {          // K- copies for the later block-rows
          float g2[8];
          *reinterpret_cast<float4*>(g2) = *reinterpret_cast<const float4*>(sGc + (I2 * 16) * LDG + cc * 8);
          *reinterpret_cast<float4*>(g2 + 4) = *reinterpret_cast<const float4*>(sGc + (I2 * 16) * LDG + cc * 8 + 4);
#pragma unroll
          for (int e = 0; e < 8; ++e) t8[e] = kf[e] * ex2(g2[e] - gi[e]);
          const int r0 = I2 == 1 ? 16 : (I2 == 2 ? 48 : 96);
          *reinterpret_cast<uint4*>(km + sw128_offset(r0 + i, cc & 7)) = pack8(t8);
        }
      }
      if (clamped) sFall[bi16] = 1;
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    bsync();
    // ---- operands rescaled in place: K <- K 2^G (for W), Q <- Q 2^G (for Q~); K e^{G_L - G} for the chain.
    // The tensor cores read the K+ / Q+ / K- copies, not these tiles, so this runs while they work (on the helper
    // warps) -- unless a diagonal block has to be evaluated again from the raw tiles first (then on the others).
    auto rescale_pass = [&](int t) {                     // by eight warps; t = 0..255 within them
    {
      const int i = t >> 2;
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        const int cc = (t & 3) + 4 * q;
        uint8_t* kt = sm + OFF_KQ + (cc >> 3) * 16384;
        const uint32_t off = sw128_offset(i, cc & 7);
        float kf[8], qf[8], gi[8], gl[8], kd[8];
        unpack8(*reinterpret_cast<const uint4*>(kt + off), kf);
        unpack8(*reinterpret_cast<const uint4*>(kt + 8192 + off), qf);
        *reinterpret_cast<float4*>(gi) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8);
        *reinterpret_cast<float4*>(gi + 4) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8 + 4);
        *reinterpret_cast<float4*>(gl) = *reinterpret_cast<const float4*>(sGc + 63 * LDG + cc * 8);
        *reinterpret_cast<float4*>(gl + 4) = *reinterpret_cast<const float4*>(sGc + 63 * LDG + cc * 8 + 4);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float eg = ex2(gi[e]);
          kd[e] = kf[e] * ex2(gl[e] - gi[e]);
          kf[e] *= eg;
          qf[e] *= eg;
        }
        *reinterpret_cast<uint4*>(kt + off) = pack8(kf);
        *reinterpret_cast<uint4*>(kt + 8192 + off) = pack8(qf);
        *reinterpret_cast<uint4*>(sm + OFF_KD + (cc >> 3) * 8192 + off) = pack8(kd);
      }
    }
    };
    PP(0);
    const bool anyfall = (sFall[0] | sFall[1] | sFall[2] | sFall[3]) != 0;
    // One product D[128 x 160] = [all K+ / Q+ rows] [K-^(0); K-^(1); K-^(2); K-^(3)]^T: the K- copies of the four
    // block-rows are stacked (16 + 32 + 48 + 64 rows), so block-row I's result is rows 32 I .. 32 I + 31 (K+_I, Q+_I)
    // of the columns where K-^(I) starts; the other row/column combinations are computed and never read (an MMA
    // costs the same whatever its rows: eight instructions instead of one set of eight per block-row).
    // Issued by a thread of the last helper warp, so that warp 0 starts its share of the rescaling pass at once.
    if (tid == kKdaThreads - 32) {
      tc_fence_after_sync();
      const uint32_t id = idesc_bf16(128, 160, false, false);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t a = smem_u32(sm + OFF_KQP) + (ks >> 2) * KQP_KB + (ks & 3) * 32;
        const uint32_t bb = smem_u32(sm + OFF_KM) + (ks >> 2) * KM_KB + (ks & 3) * 32;
        umma_ss(tmem, smem_desc(a, 16, 1024, kSwizzle128B), smem_desc(bb, 16, 1024, kSwizzle128B), id, ks > 0);
      }
      umma_commit(bar_mma);
    }
    if (tid < 128) sQt[tid] = sGc[63 * LDG + tid];       // the chunk's total decay, for the chain kernel's scalars
    if (!anyfall) {
      // The helper warps rescale the tiles on their own while the other warps take the first product's result and
      // solve (nothing there reads the tiles; the W / U products, much later, wait at barrier 10).  That is the
      // last use of the gate matrix (the scalars above are a copy), so the helpers then fetch the next item's gate
      // rows into it right away: a warp needs some 3 k cycles to issue its 64 row copies, which the whole group
      // used to wait for at the top of the next item.
      if (is_main) {
        asm volatile("bar.arrive 9, %0;" ::"r"(kKdaThreads) : "memory");
      } else {
        rescale_pass(tid - kPrepThreads);
        // the helpers' part of the rescaled K / Q / K e^{G_L-G} tiles: visible to the tensor cores and the bulk
        // stores (proxy fence) once the other warps have passed barrier 10, before the W / U products
        fence_proxy_async_smem();
        asm volatile("bar.arrive 10, %0;" ::"r"(kKdaThreads) : "memory");
        asm volatile("bar.sync 9, %0;" ::"r"(kKdaThreads) : "memory");   // every warp is done with the matrix
        helper_geom();
        if (warp == 8) __syncwarp();
        helper_fetch();
      }
    }
    if (is_main) {                                       // the helper warps are done with this item's arithmetic
    if (warp == 0) mbar_wait(bar_mma, mph, abort_flag);
    mph ^= 1;
    gsync();
    PP(1);
    tc_fence_after_sync();
    {
      // Block-row I sits in tensor-memory lanes 32 I .. 32 I + 31: lanes 0..15 the K+ rows (-> A), 16..31 the Q+
      // rows (-> P).  Warps I and I + 4 share its 16-column pieces.
      const int I = warp & 3, l16 = lane & 15;
      const bool isq = lane >= 16;
      const int i = 16 * I + l16;
      const uint32_t col = I == 0 ? 0 : (I == 1 ? 16 : (I == 2 ? 48 : 96));
      const uint32_t tl = tmem + (static_cast<uint32_t>(I * 32) << 16) + col;
      const float bi = sBeta[i];
      for (int cb = warp >> 2; cb < 4; cb += 2) {        // (pieces right of the diagonal block are zero)
        float v[16];
        if (cb <= I) {
          uint32_t r[16];
          tmem_ld16(tl + 16 * cb, r);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int jj = 16 * cb + c;
            const bool keep = isq ? jj <= i : jj < i;    // only the diagonal piece (cb == I) has entries to drop
            v[c] = keep ? __uint_as_float(r[c]) * (isq ? 1.f : bi) : 0.f;
          }
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) v[c] = 0.f;
        }
        if (!isq) {
          uint4* d = reinterpret_cast<uint4*>(sAh + i * LDH + 16 * cb);
          d[0] = make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]));
          d[1] = make_uint4(pack_f16(v[8], v[9]), pack_f16(v[10], v[11]), pack_f16(v[12], v[13]), pack_f16(v[14], v[15]));
        } else {
          *reinterpret_cast<uint4*>(sm + OFF_P + sw128_offset(i, 2 * cb)) = pack8(*reinterpret_cast<const float(*)[8]>(v));
          *reinterpret_cast<uint4*>(sm + OFF_P + sw128_offset(i, 2 * cb + 1)) = pack8(*reinterpret_cast<const float(*)[8]>(v + 8));
        }
      }
    }
    if (anyfall) {
      gsync();
      // diagonal blocks where the clamp was hit: element by element, 136 pairs (j <= i) per block
      for (int blk = 0; blk < 4; ++blk) {
        if (!sFall[blk]) continue;
        for (int qq = tid; qq < 136; qq += kPrepThreads) {   // (first 8 warps)
          int il = 0;
          while ((il + 1) * (il + 2) / 2 <= qq) ++il;
          const int jl = qq - il * (il + 1) / 2;
          const int i = blk * 16 + il, jj = blk * 16 + jl;
          float kk = 0.f, qk = 0.f;
  #pragma unroll 2
          for (int cc = 0; cc < 16; ++cc) {
            const uint8_t* kt = sm + OFF_KQ + (cc >> 3) * 16384;
            float kif[8], qif[8], kjf[8], gi[8], gj[8];
            unpack8(*reinterpret_cast<const uint4*>(kt + sw128_offset(i, cc & 7)), kif);
            unpack8(*reinterpret_cast<const uint4*>(kt + 8192 + sw128_offset(i, cc & 7)), qif);
            unpack8(*reinterpret_cast<const uint4*>(kt + sw128_offset(jj, cc & 7)), kjf);
            *reinterpret_cast<float4*>(gi) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8);
            *reinterpret_cast<float4*>(gi + 4) = *reinterpret_cast<const float4*>(sGc + i * LDG + cc * 8 + 4);
            *reinterpret_cast<float4*>(gj) = *reinterpret_cast<const float4*>(sGc + jj * LDG + cc * 8);
            *reinterpret_cast<float4*>(gj + 4) = *reinterpret_cast<const float4*>(sGc + jj * LDG + cc * 8 + 4);
  #pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float t = kjf[e] * ex2(gi[e] - gj[e]);
              kk = fmaf(kif[e], t, kk);
              qk = fmaf(qif[e], t, qk);
            }
          }
          if (jj < i) sAh[i * LDH + jj] = __float2half_rn(sBeta[i] * kk);
          *reinterpret_cast<__nv_bfloat16*>(sm + OFF_P + sw128_offset(i, jj >> 3) + (jj & 7) * 2) = __float2bfloat16_rn(qk);
        }
      }
      gsync();                                   // everyone is done with the raw K and Q tiles
      rescale_pass(tid);
    }
    }  // is_main

  } else {
    // ---- op #1 Gate: inclusive scan of the log-gate over the chunk (warp 1, tokens lane and lane + 32)
    if (warp == 1) {
      cp_async_wait_all();
      float x0 = sRaw[lane], x1 = sRaw[lane + 32];
      const float b0 = sRaw[64 + lane], b1 = sRaw[96 + lane];
  #pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float y0 = __shfl_up_sync(0xffffffffu, x0, o), y1 = __shfl_up_sync(0xffffffffu, x1, o);
        if (lane >= o) { x0 += y0; x1 += y1; }
      }
      x1 += __shfl_sync(0xffffffffu, x0, 31);
      const float e0 = __expf(x0), e1 = __expf(x1);
      sG[lane] = x0;             sG[lane + 32] = x1;
      sBeta[lane] = b0;          sBeta[lane + 32] = b1;
      sEG[lane] = e0;            sEG[lane + 32] = e1;
      sBE[lane] = e0 * b0;       sBE[lane + 32] = e1 * b1;
      sBE[64 + lane] = x0 * 1.4426950408889634f;           // G log2(e), for ex2 in the decay mask
      sBE[96 + lane] = x1 * 1.4426950408889634f;
    }

    // ---- op #2 KKT (+ Q K^T): S[0:64] = K K^T, S[64:128] = Q K^T
    if (tid == 0) {
      PP(2);
      publish_prev();                                    // (its wait for the stores overlaps the tiles' arrival)
      mbar_wait(bar_load, lph, abort_flag);
      PP(3);
      tc_fence_after_sync();
      const uint32_t id = idesc_bf16(128, 64, false, false);
      const uint32_t base = smem_u32(sm + OFF_KQ);
  #pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t a = base + (ks >> 2) * 16384 + (ks & 3) * 32;
        umma_ss(tmem, smem_desc(a, 16, 1024, kSwizzle128B), smem_desc(a, 16, 1024, kSwizzle128B), id, ks > 0);
      }
      umma_commit(bar_mma);
      // the previous item's last two images must have left before V lands on one and A is written over the other
      // (after the barrier below); the wait runs under the MMAs
      if (prev_cj >= 0) bulk_wait_read_all();
      issue_v(j, tok0);
    }
    if (warp == 0) mbar_wait(bar_mma, mph, abort_flag);  // one warp polls; the others sleep at the barrier
    mph ^= 1;
    gsync();                                     // (also makes sEG / sBE visible to everyone)
    PP(4);
    tc_fence_after_sync();
    {
      float v[32];
      ld32(my_tmem, v);
      const int i = rowq & 63;
      const float* sG2 = sBE + 64;                       // G log2(e)
      const float gi = sG2[i];
      if (rowq < 64) {                                     // row i of A (strictly lower, beta-scaled), fp16
        const float bi = sBeta[i];
  #pragma unroll
        for (int q = 0; q < 32; ++q) {
          const int jj = hf * 32 + q;
          const float e = ex2(gi - sG2[jj]);     // exponent <= 0 wherever the entry is kept
          v[q] = jj < i ? bi * e * v[q] : 0.f;
        }
  #pragma unroll
        for (int q = 0; q < 32; q += 8)
          *reinterpret_cast<uint4*>(sAh + i * LDH + hf * 32 + q) =
              make_uint4(pack_f16(v[q], v[q + 1]), pack_f16(v[q + 2], v[q + 3]), pack_f16(v[q + 4], v[q + 5]), pack_f16(v[q + 6], v[q + 7]));
      } else {                                             // row i of P (lower incl. diagonal), bf16 operand tile
  #pragma unroll
        for (int q = 0; q < 32; ++q) {
          const int jj = hf * 32 + q;
          const float e = ex2(gi - sG2[jj]);     // exponent <= 0 wherever the entry is kept
          v[q] = jj <= i ? e * v[q] : 0.f;
        }
        store_half_row(v, i, hf, sm + OFF_P);
      }
    }
  }
  const long long nxt = cjl + vstride;
  if (is_main) {                                         // ---- everything down to the Q~ image: the first 8 warps
  gsync();
  PP(5);

  // ---- op #3 Solve: T = (I + A)^-1
  {
    // Four 16x16 diagonal blocks, each as 2 x 2 blocks of 8 x 8:  [[X11, 0], [X21, X22]]  with
    // X11 = (I + A11)^-1, X22 = (I + A22)^-1 by fp32 forward substitution (64 threads: block, half, column; eight
    // steps instead of sixteen), then X21 = -X22 (A21 X11) by all threads, one element each.  The inverse goes to
    // a scratch copy first (other threads are still reading A).
    float* sM = reinterpret_cast<float*>(sD + 4 * 256);   // fp32 [4][8][8]: A21 X11
    if (tid < 64) {
      const int blk = tid >> 4, hb = (tid >> 3) & 1, c = tid & 7, o = blk * 16 + hb * 8;
      __half* dst = sD + blk * 256 + (hb * 8) * 16 + hb * 8 + c;
      float y[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float a[8];
        if (q > 0) unpack8h(*reinterpret_cast<const uint4*>(sAh + (o + q) * LDH + o), a);
        float s0 = q == c ? 1.f : 0.f, s1 = 0.f;
#pragma unroll
        for (int r = 0; r < q; ++r) {
          if (r & 1) s1 = fmaf(-a[r], y[r], s1);
          else s0 = fmaf(-a[r], y[r], s0);
        }
        y[q] = s0 + s1;
        dst[q * 16] = __float2half_rn(y[q]);
        if (hb == 0) sD[blk * 256 + q * 16 + 8 + c] = __float2half_rn(0.f);   // the block above the diagonal
      }
    }
    gsync();
    const int blk = tid >> 6, bi = (tid >> 3) & 7, bj = tid & 7, o = blk * 16;
    {
      float a[8];
      unpack8h(*reinterpret_cast<const uint4*>(sAh + (o + 8 + bi) * LDH + o), a);        // row bi of A21
      float m0 = 0.f, m1 = 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 2) {
        m0 = fmaf(a[k], __half2float(sD[blk * 256 + k * 16 + bj]), m0);                   // column bj of X11
        m1 = fmaf(a[k + 1], __half2float(sD[blk * 256 + (k + 1) * 16 + bj]), m1);
      }
      sM[tid] = m0 + m1;
    }
    gsync();
    {
      float x[8];
      unpack8h(*reinterpret_cast<const uint4*>(sD + blk * 256 + (8 + bi) * 16 + 8), x);   // row bi of X22
      float m0 = 0.f, m1 = 0.f;
#pragma unroll
      for (int k = 0; k < 8; k += 2) {
        m0 = fmaf(x[k], sM[blk * 64 + k * 8 + bj], m0);
        m1 = fmaf(x[k + 1], sM[blk * 64 + (k + 1) * 8 + bj], m1);
      }
      sD[blk * 256 + (8 + bi) * 16 + bj] = __float2half_rn(-(m0 + m1));
    }
  }
  gsync();
  PP(6);
  {
    // the diagonal inverses go back in place (for level 2 and the final read) ...
    const int blk = tid >> 6, r = (tid >> 2) & 15, c4 = (tid & 3) * 4;
    *reinterpret_cast<uint2*>(sAh + (blk * 16 + r) * LDH + blk * 16 + c4) =
        *reinterpret_cast<const uint2*>(sD + blk * 256 + r * 16 + c4);
    // ... while level 1 (blocks (1,0) and (3,2)) reads them from the scratch copy: one warp per block
    if (warp < 2) {
      const int lo = warp * 32, hi = lo + 16;
      float c2[2][4];
      merge_compute<16, 2>(c2, sD + (2 * warp) * 256, 16, sAh + hi * LDH + lo, LDH, sD + (2 * warp + 1) * 256, 16, 0, 0, lane);
      __syncwarp();
      merge_store<2>(c2, sAh + hi * LDH + lo, LDH, 0, 0, lane);
    }
  }
  gsync();
  PP(7);
  {
    // level 2: the 32x32 block (rows 32..63, columns 0..31); warp -> (16 columns, 8 rows) of the result
    const int mt = warp & 1, n2 = warp >> 1;
    float c2[1][4];
    merge_compute<32, 1>(c2, sAh, LDH, sAh + 32 * LDH, LDH, sAh + 32 * LDH + 32, LDH, mt, n2, lane);
    gsync();                                     // every warp has read A_10 before it is overwritten
    merge_store<1>(c2, sAh + 32 * LDH, LDH, mt, n2, lane);
  }
  gsync();
  PP(8);

  // ---- column-scaled copies of T as bf16 operand tiles: T^W = T diag(beta e^G), T^U = T diag(beta).
  // They overwrite T, so every thread first takes its part of T into registers.
  {
    const int i = tid >> 2, q4 = tid & 3;                // row, quarter (16 columns = two 16-byte pieces)
    const uint4 traw0 = *reinterpret_cast<const uint4*>(sAh + i * LDH + q4 * 16);
    const uint4 traw1 = *reinterpret_cast<const uint4*>(sAh + i * LDH + q4 * 16 + 8);
    {
      // T left the fp16 range (an exponent field of all ones: infinity or NaN) only for inputs far outside the
      // delta rule's stable range (beta |k|^2 <= 2): report it instead of returning wrong numbers silently.
      const uint32_t w[8] = {traw0.x, traw0.y, traw0.z, traw0.w, traw1.x, traw1.y, traw1.z, traw1.w};
      bool bad = false;
#pragma unroll
      for (int e = 0; e < 8; ++e)
        bad |= (w[e] & 0x7c000000u) == 0x7c000000u || (w[e] & 0x00007c00u) == 0x00007c00u;
      if (bad) report_status(p.status, HA_LA_ERR_DEVICE_CHECK);
    }
    gsync();
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int ch = q4 * 2 + q;
      float tv[8], tw[8], tu[8];
      unpack8h(q == 0 ? traw0 : traw1, tv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int jj = ch * 8 + e;
        tw[e] = tv[e] * sBE[jj];
        tu[e] = tv[e] * sBeta[jj];
      }
      const uint32_t off = sw128_offset(i, ch);
      *reinterpret_cast<uint4*>(sm + OFF_TW + off) = pack8(tw);
      *reinterpret_cast<uint4*>(sm + OFF_TU + off) = pack8(tu);
    }
  }
  if constexpr (KDA) {                                   // the helper warps' share of the rescaling pass is complete
    const int* fall = reinterpret_cast<const int*>(sm + OFF_FALL);
    if ((fall[0] | fall[1] | fall[2] | fall[3]) == 0) asm volatile("bar.sync 10, %0;" ::"r"(kKdaThreads) : "memory");
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  gsync();
  PP(9);
  if constexpr (KDA) {                                   // K e^{G_L-G} is complete (rescaling pass): its image leaves now,
    if (tid == 0) {                                      // in a bulk group of its own, well ahead of the W / U images
      bulk_store(p.ws.kd + (size_t)cj * kImgBytes, sm + OFF_KD, kImgBytes);
      bulk_commit();
    }
  }

  // ---- op #4 W/U: W^T = K^T (T^W)^T, U^T = V^T (T^U)^T  (A operands feature-major straight from the TMA tiles)
  if (tid == 0) {
    tc_fence_after_sync();
    const uint32_t id = idesc_bf16(128, 64, true, false);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(tmem, smem_desc(smem_u32(sm + OFF_KQ) + ks * 2048, 16384, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_TW) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
    mbar_wait(bar_v, lph, abort_flag);
    tc_fence_after_sync();
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(tmem + 64, smem_desc(smem_u32(sm + OFF_V) + ks * 2048, 8192, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_TU) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
    umma_commit(bar_mma);
  }
  if (warp == 0) mbar_wait(bar_mma, mph, abort_flag);
  mph ^= 1;
  gsync();
  PP(10);
  tc_fence_after_sync();
  {
    float v[32];
    ld32(my_tmem, v);                                    // row = key channel, columns = tokens
    store_half_row(v, rowq, hf, sm + OFF_WT);
    ld32(my_tmem + 64, v);
    store_half_row(v, rowq, hf, sm + OFF_UT);
    // E = diag(e^G) as an MMA operand: Q^T E puts (Q e^G)^T into the accumulator of the Q~ product.
    // It lies over the first K piece, which is dead now that the W product is complete.
    const int i = tid >> 2;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int ch = (tid & 3) * 2 + q;
      uint32_t ev[4] = {0u, 0u, 0u, 0u};
      if ((i >> 3) == ch) {
        const uint32_t bits = static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(sEG[i])));
        ev[(i & 7) >> 1] = (i & 1) ? (bits << 16) : bits;
      }
      *reinterpret_cast<uint4*>(sm + OFF_E + sw128_offset(i, ch)) = make_uint4(ev[0], ev[1], ev[2], ev[3]);
    }
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  gsync();
  PP(11);

  // ---- chunk-local halves of op #6: (P W)^T = W^T P^T, O_loc^T = U^T P^T; the W and U images leave meanwhile
  if (tid == 0) {
    tc_fence_after_sync();
    const uint32_t id = idesc_bf16(128, 64, false, false);
    const uint32_t id_q = idesc_bf16(128, 64, true, false);          // A = Q tile, feature-major
    const uint32_t id_neg = id | (1u << 13);                         // negate A: accumulate -W^T P^T
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)                                    // (Q e^G)^T = Q^T E
      umma_ss(tmem, smem_desc(smem_u32(sm + OFF_KQ) + 8192 + ks * 2048, 16384, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_E) + ks * 32, 16, 1024, kSwizzle128B), id_q, ks > 0);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)                                    // ... - W^T P^T  = Q~^T
      umma_ss(tmem, smem_desc(smem_u32(sm + OFF_WT) + ks * 32, 16, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_P) + ks * 32, 16, 1024, kSwizzle128B), id_neg, 1u);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks)
      umma_ss(tmem + 64, smem_desc(smem_u32(sm + OFF_UT) + ks * 32, 16, 1024, kSwizzle128B),
              smem_desc(smem_u32(sm + OFF_P) + ks * 32, 16, 1024, kSwizzle128B), id, ks > 0);
    umma_commit(bar_mma);
    // two bulk groups, so that the Q~ image can follow the W image before the U image has been read too
    bulk_store(p.ws.wq + (size_t)cj * 2 * kImgBytes, sm + OFF_WT, kImgBytes);
    bulk_commit();
    bulk_store(p.ws.u + (size_t)cj * kImgBytes, sm + OFF_UT, kImgBytes);
    bulk_commit();
  }
  if (!KDA && tid == 32) {                               // where the next item is (idle thread, under the MMAs)
    int jn = 0, jqn = 0, Ln = 0, tok0n = 0;
    bool hn = nxt < p.total;
    if (hn) { item_geom(nxt, jn, jqn, Ln, tok0n); hn = Ln > 0; }
    sNext[0] = hn ? 1 : 0; sNext[1] = jn; sNext[2] = jqn; sNext[3] = Ln; sNext[4] = tok0n;
  }
  if (tid >= 64) {                                       // per-chunk scalars for the chain kernel
    float* sc = p.ws.sc + (size_t)cj * kScFloats;
    const int t = tid - 64;                              // 0..191
    if constexpr (KDA) {
      sc[t] = t < 64 ? 1.f : ex2(reinterpret_cast<const float*>(sm + OFF_QT)[t - 64]);
    } else {
      const float gl = sG[63];
      sc[t] = t < 64 ? __expf(gl - sG[t]) : __expf(gl);
    }
  }
  }  // is_main
  // KDA: the helper warps have been waiting here.  Normally they fetched the next item's gate rows right after the
  // gate-dependent passes; if a diagonal block was evaluated again from the gate matrix, they do it now.  The
  // barrier also hands the next item's whereabouts (a helper thread's work) to the other warps.
  if constexpr (KDA) {
    const int* fall = reinterpret_cast<const int*>(sm + OFF_FALL);
    const bool late = (fall[0] | fall[1] | fall[2] | fall[3]) != 0;
    if (late) helper_geom();
    bsync();
    if (late && !is_main) helper_fetch();
    if (sNext[0]) stage_gates(sNext[1], sNext[3], sNext[4], false);   // (betas, by one of the other warps)
  }
  if (is_main) {
  if (warp == 0) mbar_wait(bar_mma, mph, abort_flag);
  // GDN: the W and U images must have been read, they receive the next two.  (KDA has room for those elsewhere.)
  if (!KDA && tid == 0) bulk_wait_read_all();
  mph ^= 1;
  gsync();
  PP(12);
  tc_fence_after_sync();
  // Every MMA of this item is done, so the K / Q tile regions are free: start the next item's loads now
  // (its V tiles follow at the top of the loop, once the O_loc image has left their room).
  // (Where the next item is was worked out meanwhile: KDA, by a helper thread; GDN, by thread 32 under the MMAs.
  // Two threads of different warps share the four tile loads, so that no warp starts the epilogue much later.)
  if (sNext[0]) {
    if (tid == 0) {
      mbar_expect_tx(bar_load, 4 * 8192);
      issue_tiles_kb(sNext[2], sNext[4], 0);
    } else if (tid == 32) {
      issue_tiles_kb(sNext[2], sNext[4], 1);
    }
  }
  {
    // Q~^T and O_loc^T are complete in the accumulators; their images go where W^T and U^T were.
    float v[32];
    ld32(my_tmem, v);
    store_half_row(v, rowq, hf, sm + OFF_QI);
    ld32(my_tmem + 64, v);
    store_half_row(v, rowq, hf, sm + OFF_OI);
  }
  // The accumulators were read: the next item's first MMA may overwrite them after this barrier.
  fence_proxy_async_smem();
  tc_fence_before_sync();
  gsync();
  if (tid == 0) {
    bulk_store(p.ws.wq + (size_t)cj * 2 * kImgBytes + kImgBytes, sm + OFF_QI, kImgBytes);
    bulk_store(p.ws.ol + (size_t)cj * kImgBytes, sm + OFF_OI, kImgBytes);
    bulk_commit();
  }
  if (!KDA && sNext[0]) stage_gates(sNext[1], sNext[3], sNext[4], false);   // (sNext: written before the barriers above)
  }  // is_main
  const bool have_n = sNext[0] != 0;
  const int jn = sNext[1], jqn = sNext[2], Ln = sNext[3], tok0n = sNext[4];
  PP(13);
  prev_cj = cjl;
  lph ^= 1;
  cjl = nxt; have = have_n; j = jn; jq = jqn; L = Ln; tok0 = tok0n;
  }  // work items

  if (tid == 0) {
    if (*abort_flag) report_status(p.status, HA_LA_ERR_TIMEOUT);
    if (prev_cj >= 0) {
      if (p.epoch != 0) {                                // hand-over to a concurrently running chain kernel
        bulk_wait_all();
        fence_proxy_async_all();
        __threadfence();
        st_release_gpu(p.ws.flags + prev_cj, p.epoch);
        if (prev_cj % p.HV == 0) HA_PROF_GT(prep, 512 + (int)(prev_cj / p.HV));
      } else {
        bulk_wait_read_all();                            // shared memory must outlive the bulk stores' reads
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();                                       // all groups are done with tensor memory
  if (threadIdx.x < 32) tmem_dealloc(tmem_cta, G == 1 ? 256 : 512);
  HA_PROF(prep, 14);
  if (threadIdx.x == 0) HA_PROF_GT(prep, 901);   // last writer wins: roughly the end of the kernel
}

}  // namespace

template <bool KDA>
static cudaError_t configure_prep_variant() {
  const int smem = KDA ? kPrepSmemKda : kGroups<KDA> * kGroupSmem;
  cudaError_t e = cudaFuncSetAttribute(tc_prep_kernel<KDA>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  // Same carve-out preference as the chain kernel: kernels that prefer different L1 / shared splits do not
  // run concurrently, and the two share SMs in the concurrent mode.
  return cudaFuncSetAttribute(tc_prep_kernel<KDA>, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxShared);
}

template <bool KDA>
static cudaError_t launch_prep_variant(const PrepParams& pp, const CUtensorMap& mq, const CUtensorMap& mk,
                                       const CUtensorMap& mv, long long grid, cudaStream_t stream) {
  const int smem = KDA ? kPrepSmemKda : kGroups<KDA> * kGroupSmem;
  timer_mark(stream, "tc_prep");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(KDA ? kKdaThreads : kPrepThreads * kGroups<KDA>);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_timer ? 0 : 1;                        // (per-kernel timing wants one kernel at a time)
  return cudaLaunchKernelEx(&cfg, tc_prep_kernel<KDA>, mq, mk, mv, pp);
}

// Sets the kernel's attributes, which also loads it.  Must run before ANY kernel of a concurrent launch is
// enqueued: loading a kernel for the first time can wait for the device, and the chain kernel would be spinning.
cudaError_t configure_tc_prep(const Problem& p) {
  return p.variant == HA_LA_KDA ? configure_prep_variant<true>() : configure_prep_variant<false>();
}

cudaError_t launch_tc_prep(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                           const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, int64_t epoch,
                           int reserved_sms, cudaStream_t stream) {
  PrepParams pp;
  pp.epoch = epoch;
  pp.g = a.g; pp.beta = a.beta;
  pp.chunk_tok0 = plan.chunk_tok0; pp.chunk_len = plan.chunk_len;
  pp.T_row = p.T_row; pp.cps = p.max_seq_chunks > 0 ? p.max_seq_chunks : 1;
  pp.ws = ws; pp.HK = p.HK; pp.HV = p.HV; pp.status = a.status_word;
  pp.total = (long long)p.max_chunks * p.HV;
  if (pp.total == 0) return cudaSuccess;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // one CTA per SM; in the concurrent mode the SMs that will hold a chain CTA are left out
  const int groups = p.variant == HA_LA_KDA ? 1 : 3;
  long long ctas = sms - reserved_sms;
  if (ctas < 1) ctas = 1;
  const long long need = (pp.total + groups - 1) / groups;
  const long long grid = need < ctas ? need : ctas;
  return p.variant == HA_LA_KDA ? launch_prep_variant<true>(pp, mq, mk, mv, grid, stream)
                                : launch_prep_variant<false>(pp, mq, mk, mv, grid, stream);
}

}  // namespace ha_la
