// Sequential part of the delta-rule prefill on tcgen05 tensor cores: operator #5 (state passing)
// with operator #6 (output) fused in the paper's chunk-first order.
//
// One CTA per (sequence, V-head, slice of NV value channels) walks the chunks of its sequence in
// order (there may be more CTAs than SMs; those of the longest sequences come first).  The d_k x NV slice of the state stays on chip for the whole sequence: fp32 in registers
// (thread t owns key channel t), plus a bf16 copy in shared memory as the MMA operand.  Value
// channels are independent (paper Section "Computation Splitting": the state splits column-wise
// into sub-heads with no cross-core reduction), so slices never communicate.
//
// Per chunk, with the operand images the prep kernel left in the workspace:
//   MMA1  D1[128 x NV] = [W ; Q~] h          rows 0..63: W h, rows 64..127: Q~ h      (M = 128)
//         threads 0..63  : U~_i = (U_i - (W h)_i) e^{G_L - G_i}  -> bf16 operand in shared memory
//         threads 64..127: o_i  = scale (O_loc,i + (Q~ h)_i)     -> global memory (op #6, uses the OLD state)
//                          (64- and 128-channel slices: through a swizzled tile and a TMA tile store)
//   MMA2  D2[128 x NV] = K^T U~              (A = the raw K tile, feature-major, by TMA)
//         all threads    : h <- e^{G_L} h + D2                   (op #5 update, in place)
//
// Warp roles: 4 CG compute warps (warp w <-> tensor-memory lanes 32 (w % 4).., column group w / 4 of the
// slice: CG groups of NV / CG value channels, so that wide slices do not lengthen the epilogues), then one
// producer warp (keeps the next chunks' operands in flight through a ring of shared-memory stages: 1-D
// bulk copies + one TMA tile) and one warp that issues the MMAs.  A tcgen05.mma costs the issuing thread
// some 45-80 cycles whatever its N <= 128, so issue runs on its own warp and is told "operand ready" with
// arrive-only named barriers; the compute warps never wait for issue, only for completion (mbarriers).
// In the concurrent mode the producer warp also watches the prep kernel's per-chunk flags (32 at a time).
// Every mbarrier wait and every flag wait is bounded.
#include <cuda.h>

#include "tc_common.cuh"
#include "tc_ptx.cuh"
#include "prof.cuh"

namespace ha_la {

using namespace ptx;

HA_PROF_DECL(chain)

namespace {

constexpr int chain_threads(int cg) { return (4 * cg + 2) * 32; }   // compute warps + producer warp + MMA warp

template <int NV, int S_> struct ChainCfg {
  static constexpr int kStages = S_;
  static constexpr uint32_t kRowB = NV * 2;                      // bytes of one operand row (NV bf16)
  static constexpr uint32_t kSliceB = NV * 128;                  // bytes of NV rows of a feature-major image
  static constexpr uint32_t OFF_WQ = 0;                          // 32 KiB
  static constexpr uint32_t OFF_K = 32768;                       // 16 KiB  [kb][64 tok][64 feat]
  static constexpr uint32_t OFF_U = 49152;                       // NV rows of the U image
  static constexpr uint32_t OFF_O = OFF_U + kSliceB;             // NV rows of the O_loc image
  static constexpr uint32_t OFF_SC = OFF_O + kSliceB;            // 192 floats
  static constexpr uint32_t kStageB = (OFF_SC + 768 + 1023) / 1024 * 1024;
  static constexpr uint32_t kTxBytes = 32768 + 16384 + 2 * kSliceB + 768;
  static constexpr uint32_t OFF_H = kStages * kStageB;           // bf16 h operand [128][NV]
  static constexpr uint32_t OFF_UT = OFF_H + 128 * kRowB;        // bf16 U~ operand [64][NV]
  static constexpr uint32_t OFF_OUT = OFF_UT + 64 * kRowB;       // bf16 output tile [64][NV], staged for the tile store
  static constexpr uint32_t kSmem = OFF_OUT + 64 * kRowB;
  static constexpr uint32_t OFF_BAR = OFF_SC + 768;              // barriers live in the unused tail of stage 0
  static_assert(kStageB - OFF_BAR >= (2 * S_ + 2) * 8 + 16, "room for the barriers");
  static constexpr uint32_t kTmemCols = 2 * NV < 32 ? 32 : 2 * NV;
};

struct ChainParams {
  const float* h0;
  float* hT;
  void* o;
  const int32_t* seq_tok0;     // per-sequence table of the plan kernel, or NULL for equal-length rows
  const int32_t* seq_len;      //   (then sequence n is tokens [n*T_row, (n+1)*T_row), cps chunk slots each)
  const int32_t* seq_chunk0;
  const int32_t* seq_order;    // launch order of the sequences (longest first), or NULL
  int T_row, cps;
  TcWorkspace ws;
  int HK, HV;
  float scale;
  int64_t epoch;               // != 0: the prep kernel runs concurrently; wait for ws.flags[cj] == epoch per chunk
                               // == 0: wait for the whole prep grid before the first workspace read
  int32_t* status;
};

// MN-major B operand with ROWS rows (K index) of NV bf16 each.  NV = 32: 64-byte rows, 64-byte swizzle.
// NV = 64: 128-byte rows, 128-byte swizzle.  NV = 128: two such 64-column blocks, ROWS*128 bytes apart.
template <int NV, int ROWS> __device__ __forceinline__ uint32_t brow_offset(int row, int ch) {
  if (NV == 32) return sw64_offset(row, ch);
  return static_cast<uint32_t>(ch >> 3) * (ROWS * 128u) + sw128_offset(row, ch & 7);
}
// Descriptor of k-step 0; k-step ks (16 rows further) adds ks * brow_step16<NV>() to the start-address field.
template <int NV, int ROWS> __device__ __forceinline__ uint64_t brow_desc0(uint32_t base) {
  if (NV == 32) return smem_desc(base, 16, 512, kSwizzle64B);
  return smem_desc(base, ROWS * 128, 1024, kSwizzle128B);
}
template <int NV> __host__ __device__ constexpr uint32_t brow_step16() { return (NV == 32 ? 16u * 64u : 2048u) >> 4; }

// 32 consecutive columns [c0, c0+32) of one operand row
template <int NV, int ROWS>
__device__ __forceinline__ void store_brow32(uint8_t* tile, int row, int c0, const float (&v)[32]) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 w;
    w.x = pack_bf16(v[q * 8 + 0], v[q * 8 + 1]);
    w.y = pack_bf16(v[q * 8 + 2], v[q * 8 + 3]);
    w.z = pack_bf16(v[q * 8 + 4], v[q * 8 + 5]);
    w.w = pack_bf16(v[q * 8 + 6], v[q * 8 + 7]);
    *reinterpret_cast<uint4*>(tile + brow_offset<NV, ROWS>(row, (c0 >> 3) + q)) = w;
  }
}
// 32 value channels [c0, c0+32) of token `i` from a slice of a feature-major image (row = channel,
// 128 swizzled bytes = 64 tokens).  Two-byte loads; a warp reads 64 contiguous bytes per channel.
__device__ __forceinline__ void load_img32(const uint8_t* slice, int i, int c0, float (&v)[32]) {
  const uint8_t* base = slice + (i & 7) * 2;
  const int ch = i >> 3;
#pragma unroll
  for (int q = 0; q < 32; ++q)
    v[q] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(base + sw128_offset(c0 + q, ch)));
}

__device__ __forceinline__ void ld32f(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  tmem_ld32(taddr, r);
  tmem_ld_wait();
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// named barriers (0 is __syncthreads)
constexpr int BAR_H_READY = 1;   // all compute threads arrive, MMA warp syncs: bf16 h is in shared memory
constexpr int BAR_U_READY = 2;   // the U~ writers (half of them) arrive, MMA warp syncs: U~ operand is in shared memory
constexpr int BAR_O_FREE = 3;    // output threads: the previous tile store has read the staging tile
constexpr int BAR_O_FULL = 4;    // output threads: the staging tile is written
__device__ __forceinline__ void named_arrive(int id, int count) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <int NV, bool KDA, int S, int CG>
__global__ void __launch_bounds__(chain_threads(CG), 1)
tc_chain_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_o, ChainParams p) {
  using Cfg = ChainCfg<NV, S>;
  constexpr int NSL = 128 / NV;
  constexpr int NVT = NV / CG;                           // value channels per compute thread
  constexpr int NCOMP = 128 * CG;                        // compute threads
  constexpr int W_PROD = 4 * CG, W_MMA = 4 * CG + 1;
  static_assert(NVT % 32 == 0, "column groups are multiples of 32 channels");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* sm = smem_raw;                                // no static shared memory in this kernel: 1024-aligned
  uint64_t* bar_full = reinterpret_cast<uint64_t*>(sm + Cfg::OFF_BAR);     // [S]  producer -> everyone
  uint64_t* bar_empty = bar_full + S;                                       // [S]  128 compute threads -> producer
  uint64_t* bar_mma1 = bar_empty + S;                                       // MMA1 complete
  uint64_t* bar_mma2 = bar_mma1 + 1;                                        // MMA2 complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mma2 + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int slice = blockIdx.x % NSL;
  const int nj = blockIdx.x / NSL;
  const int j = nj % p.HV;
  const int n = p.seq_order ? p.seq_order[nj / p.HV] : nj / p.HV;   // CTAs of the longest sequences come first
  const int jq = j / (p.HV / p.HK);
  const int tok0 = p.seq_tok0 ? p.seq_tok0[n] : n * p.T_row;
  const int len = p.seq_tok0 ? p.seq_len[n] : p.T_row;
  const int chunk0 = p.seq_tok0 ? p.seq_chunk0[n] : n * p.cps;
  const int nchunks = (len + kChunk - 1) / kChunk;

  if (blockIdx.x == 0 && threadIdx.x == 0) HA_PROF_GT(chain, 900);
  if (tid == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_empty[i], NCOMP); }
    mbar_init(bar_mma1, 1);
    mbar_init(bar_mma2, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tmap(&map_k);
    prefetch_tmap(&map_o);
  }
  if (warp == 0) tmem_alloc(tmem_slot, Cfg::kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t TM1 = tmem, TM2 = tmem + NV;
  // This kernel may be launched as a programmatic dependent of the prep kernel, i.e. start while that one is
  // still running.  Sequential mode: everything above overlapped the prep kernel's tail; wait for it here.
  if (p.epoch == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  uint8_t* sH = sm + Cfg::OFF_H;
  uint8_t* sUt = sm + Cfg::OFF_UT;
  uint8_t* sOut = sm + Cfg::OFF_OUT;

  if (warp == W_PROD) {
    // ------------------------------------------------------------ producer
    // Concurrent mode: the whole warp looks at the ready flags of the next 32 chunks at once (plain loads) and
    // remembers how far the prep kernel has got; the acquire fence and the proxy fence, which are what makes
    // the published images visible to this kernel's bulk copies, are then paid once per batch, not per chunk.
    const int lane = tid & 31;
    int ready_upto = p.epoch != 0 ? 0 : nchunks;         // chunks [0, ready_upto) are known to be published
    for (int c = 0; c < nchunks; ++c) {
      if (c >= ready_upto) {
        int got = 0;
        for (uint32_t it = 0; it < kSpinLimit && !*abort_flag; ++it) {
          const int cc = c + lane;
          bool ok = false;
          if (cc < nchunks)
            ok = *reinterpret_cast<const volatile int64_t*>(p.ws.flags + (size_t)(chunk0 + cc) * p.HV + j) == p.epoch;
          const unsigned m = __ballot_sync(0xffffffffu, ok);
          got = __ffs(~m) - 1;                           // leading published chunks (32 when all are)
          if (got < 0) got = 32;
          if (got > 0) break;
          __nanosleep(100);
        }
        if (got == 0) *abort_flag = 1;                   // gave up: carry on, the status word reports the time-out
        ready_upto = c + (got > 0 ? got : nchunks);
        __threadfence();                                 // acquire side of the prep kernel's release
        fence_proxy_async_all();
        if (blockIdx.x == 0 && lane == 0) HA_PROF_GT(chain, 600 + c);
      }
      if (lane == 0) {
        const int st = c % S;
        if (c >= S) mbar_wait(&bar_empty[st], ((c / S) - 1) & 1, abort_flag);
        uint8_t* stage = sm + st * Cfg::kStageB;
        const size_t cj = (size_t)(chunk0 + c) * p.HV + j;
        mbar_expect_tx(&bar_full[st], Cfg::kTxBytes);
        bulk_load(stage + Cfg::OFF_WQ, p.ws.wq + cj * 2 * kImgBytes, 32768, &bar_full[st]);
        bulk_load(stage + Cfg::OFF_U, p.ws.u + cj * kImgBytes + (size_t)slice * Cfg::kSliceB, Cfg::kSliceB, &bar_full[st]);
        bulk_load(stage + Cfg::OFF_O, p.ws.ol + cj * kImgBytes + (size_t)slice * Cfg::kSliceB, Cfg::kSliceB, &bar_full[st]);
        bulk_load(stage + Cfg::OFF_SC, p.ws.sc + cj * kScFloats, 768, &bar_full[st]);
        if constexpr (KDA) {   // K e^{G_L - G} from the prep kernel (per-channel decay cannot be applied to U~ rows)
          bulk_load(stage + Cfg::OFF_K, p.ws.kd + cj * kImgBytes, 16384, &bar_full[st]);
        } else {
          tma_load_3d(stage + Cfg::OFF_K, &map_k, &bar_full[st], 0, jq, tok0 + c * kChunk);
          tma_load_3d(stage + Cfg::OFF_K + 8192, &map_k, &bar_full[st], 64, jq, tok0 + c * kChunk);
        }
      }
      __syncwarp();
    }
  } else if (warp == W_MMA) {
    // ------------------------------------------------------------ MMA issue (lane 0 issues; the warp keeps the barriers)
    const uint32_t id = idesc_bf16(128, NV, true, true);
    const uint64_t dH = brow_desc0<NV, 128>(smem_u32(sH));
    const uint64_t dU = brow_desc0<NV, 64>(smem_u32(sUt));
    const bool lead = (tid & 31) == 0;
    for (int c = 0; c < nchunks; ++c) {
      const int st = c % S;
      const uint32_t stage = smem_u32(sm + st * Cfg::kStageB);
      const uint64_t dWQ = smem_desc(stage + Cfg::OFF_WQ, 16384, 1024, kSwizzle128B);
      const uint64_t dK = smem_desc(stage + Cfg::OFF_K, 8192, 1024, kSwizzle128B);
      if (lead) mbar_wait(&bar_full[st], (c / S) & 1, abort_flag);
      named_sync(BAR_H_READY, NCOMP + 32);               // h (bf16) of the previous chunk is in sH
      if (lead) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)                    // K = d_k: 16 feature rows (2048 B) per step
          umma_ss(TM1, dWQ + ks * (2048u >> 4), dH + ks * brow_step16<NV>(), id, ks > 0);
        umma_commit(bar_mma1);
      }
      named_sync(BAR_U_READY, NCOMP / 2 + 32);           // U~ is in sUt
      if (lead) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)                    // K = tokens: 16 token rows per step
          umma_ss(TM2, dK + ks * (2048u >> 4), dU + ks * brow_step16<NV>(), id, ks > 0);
        umma_commit(bar_mma2);
      }
    }
  } else {
    // ------------------------------------------------------------ compute
    const int row = tid & 127;                           // tensor-memory lane = state row (key channel) / D1 row
    const int cg0 = (warp >> 2) * NVT;                   // first value channel of this thread's column group
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    float h[NVT];                                        // state row `row`, NVT value channels
    {
      const size_t base = (((size_t)n * p.HV + j) * 128 + row) * 128 + (size_t)slice * NV + cg0;
#pragma unroll
      for (int q = 0; q < NVT; q += 4) {
        float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.h0) v4 = *reinterpret_cast<const float4*>(p.h0 + base + q);
        h[q] = v4.x; h[q + 1] = v4.y; h[q + 2] = v4.z; h[q + 3] = v4.w;
      }
    }
#pragma unroll
    for (int c0 = 0; c0 < NVT; c0 += 32) {
      float t[32];
#pragma unroll
      for (int q = 0; q < 32; ++q) t[q] = h[c0 + q];
      store_brow32<NV, 128>(sH, row, cg0 + c0, t);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    named_arrive(BAR_H_READY, NCOMP + 32);

    const int i = row & 63;                              // token row handled in the first epilogue
    for (int c = 0; c < nchunks; ++c) {
      const int st = c % S;
      const uint8_t* stage = sm + st * Cfg::kStageB;
      const int L = min(kChunk, len - c * kChunk);
      const uint32_t ph = c & 1;

      HA_PROF(chain, 8 * c + 0);
      mbar_wait(&bar_full[st], (c / S) & 1, abort_flag);
      HA_PROF(chain, 8 * c + 1);
      // operands of the first epilogue that do not depend on the MMA, fetched while it runs
      const float* sc = reinterpret_cast<const float*>(stage + Cfg::OFF_SC);
      const float dec = sc[i];
      const float gam = sc[64 + row];
      float pre[32];
      load_img32(stage + (row < 64 ? Cfg::OFF_U : Cfg::OFF_O), i, cg0, pre);

      mbar_wait(bar_mma1, ph, abort_flag);
      HA_PROF(chain, 8 * c + 2);
      tc_fence_after_sync();
      if (row < 64) {                                    // U~ rows: (U - W h) e^{G_L - G_i}, the MMA2 operand
#pragma unroll
        for (int c0 = 0; c0 < NVT; c0 += 32) {
          float d[32];
          ld32f(TM1 + lane_base + cg0 + c0, d);
          if (c0 > 0) load_img32(stage + Cfg::OFF_U, i, cg0 + c0, pre);
#pragma unroll
          for (int q = 0; q < 32; ++q) d[q] = (pre[q] - d[q]) * dec;
          if (c0 == 0) HA_PROF(chain, 8 * c + 6);
          store_brow32<NV, 64>(sUt, i, cg0 + c0, d);
        }
        HA_PROF(chain, 8 * c + 7);
        fence_proxy_async_smem();
        tc_fence_before_sync();
        named_arrive(BAR_U_READY, NCOMP / 2 + 32);
        HA_PROF(chain, 8 * c + 3);
      } else {                                           // output rows: o = scale (O_loc + Q~ h)  (op #6)
        // A full chunk leaves as one tile store per 64-channel block from a swizzled staging tile (a thread
        // holds one token row, so direct stores would touch 32 lines per instruction); the ragged last chunk
        // of a sequence is stored row by row, since a tile store could not stop at the sequence's end.
        // (32-channel slices keep the direct stores: four per thread, cheaper than the staging's two barriers.)
        const bool tile_out = NV > 32 && L == kChunk;
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) +
                              ((size_t)(tok0 + c * kChunk + i) * p.HV + j) * 128 + (size_t)slice * NV + cg0;
        if (tile_out) named_sync(BAR_O_FREE, NCOMP / 2);
#pragma unroll
        for (int c0 = 0; c0 < NVT; c0 += 32) {
          float d[32];
          ld32f(TM1 + lane_base + cg0 + c0, d);
          if (c0 > 0) load_img32(stage + Cfg::OFF_O, i, cg0 + c0, pre);
#pragma unroll
          for (int q = 0; q < 32; ++q) d[q] = p.scale * (pre[q] + d[q]);
          if (tile_out) {
            store_brow32<NV, 64>(sOut, i, cg0 + c0, d);
          } else if (i < L) {
#pragma unroll
            for (int q = 0; q < 32; q += 8) {
              uint4 w;
              w.x = pack_bf16(d[q + 0], d[q + 1]); w.y = pack_bf16(d[q + 2], d[q + 3]);
              w.z = pack_bf16(d[q + 4], d[q + 5]); w.w = pack_bf16(d[q + 6], d[q + 7]);
              *reinterpret_cast<uint4*>(orow + c0 + q) = w;
            }
          }
        }
        if (tile_out) {
          fence_proxy_async_smem();
          named_sync(BAR_O_FULL, NCOMP / 2);
          if (tid == 64) {                               // the first output thread issues and waits for the reads
#pragma unroll
            for (int b = 0; b < (NV + 63) / 64; ++b)
              tma_store_3d(&map_o, sOut + b * 8192, slice * NV + b * 64, j, tok0 + c * kChunk);
            bulk_commit();
            bulk_wait_read_all();
          }
        }
      }

      mbar_wait(bar_mma2, ph, abort_flag);
      HA_PROF(chain, 8 * c + 4);
      tc_fence_after_sync();
      mbar_arrive(&bar_empty[st]);                       // this thread and both MMAs are done with the stage
#pragma unroll
      for (int c0 = 0; c0 < NVT; c0 += 32) {
        float d[32];
        ld32f(TM2 + lane_base + cg0 + c0, d);
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          h[c0 + q] = fmaf(gam, h[c0 + q], d[q]);
          d[q] = h[c0 + q];
        }
        store_brow32<NV, 128>(sH, row, cg0 + c0, d);
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      named_arrive(BAR_H_READY, NCOMP + 32);
      HA_PROF(chain, 8 * c + 5);
      if (blockIdx.x == 0 && tid == 0 && (c == 0 || c == nchunks - 1)) HA_PROF_GT(chain, 700 + c);
    }

    if (p.hT) {
      const size_t base = (((size_t)n * p.HV + j) * 128 + row) * 128 + (size_t)slice * NV + cg0;
#pragma unroll
      for (int q = 0; q < NVT; q += 4)
        *reinterpret_cast<float4*>(p.hT + base + q) = make_float4(h[q], h[q + 1], h[q + 2], h[q + 3]);
    }
  }

  if (warp == W_MMA) named_sync(BAR_H_READY, NCOMP + 32);  // pairs with the compute warps' last arrival
  if (*abort_flag && tid == 0) report_status(p.status, HA_LA_ERR_TIMEOUT);
  // Concurrent mode: do not finish before the prep grid has (it has published its last chunk by now), so that
  // work queued behind this kernel is also behind the prep kernel.
  if (p.epoch != 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 64) bulk_wait_all();                        // this thread's tile stores have landed
  tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0) HA_PROF_GT(chain, 901);
  if (warp == 0) tmem_dealloc(tmem, Cfg::kTmemCols);
}

template <int NV, bool KDA, int S, int CG>
cudaError_t run_nv(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int grid, bool dependent,
                   cudaStream_t stream) {
  auto kern = tc_chain_kernel<NV, KDA, S, CG>;
  constexpr int smem = ChainCfg<NV, S>::kSmem;
  static_assert(smem <= 227 * 1024, "shared memory budget");
  if (!cp) {                                             // configure only (this also loads the kernel)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  }
  timer_mark(stream, "tc_chain");
  // `dependent`: programmatic dependent launch behind the prep kernel (same stream): the CTAs may start as soon
  // as every prep CTA is running, instead of after the prep grid has drained.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(chain_threads(CG));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, *mk, *mo, *cp);
}

// Slices of 64 and 128 value channels are worked on by two column groups of compute warps.
template <bool KDA>
cudaError_t run_variant(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int nv, int grid,
                        bool dependent, cudaStream_t stream) {
  if (nv == 32) return run_nv<32, KDA, 3, 1>(cp, mk, mo, grid, dependent, stream);
  if (nv == 64) return run_nv<64, KDA, 3, 2>(cp, mk, mo, grid, dependent, stream);
  return run_nv<128, KDA, 2, 2>(cp, mk, mo, grid, dependent, stream);
}

}  // namespace

cudaError_t launch_tc_chain(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                            const CUtensorMap& mk, const CUtensorMap& mo, int nv, int64_t epoch, bool dependent,
                            cudaStream_t stream) {
  ChainParams cp;
  cp.h0 = a.h0; cp.hT = a.hT; cp.o = a.o;
  cp.seq_tok0 = plan.seq_tok0; cp.seq_len = plan.seq_len; cp.seq_chunk0 = plan.seq_chunk0;
  cp.seq_order = plan.seq_tok0 ? plan.seq_order : nullptr;
  cp.T_row = p.T_row; cp.cps = p.max_seq_chunks > 0 ? p.max_seq_chunks : 1;
  cp.ws = ws; cp.HK = p.HK; cp.HV = p.HV; cp.scale = p.scale; cp.status = a.status_word;
  cp.epoch = epoch;
  const int grid = p.N * p.HV * (128 / nv);
  if (grid == 0) return cudaSuccess;
  return p.variant == HA_LA_KDA ? run_variant<true>(&cp, &mk, &mo, nv, grid, dependent, stream)
                                : run_variant<false>(&cp, &mk, &mo, nv, grid, dependent, stream);
}

// Attributes (and loading) of the chain kernel instance a launch will use; see configure_tc_prep.
cudaError_t configure_tc_chain(const Problem& p, int nv) {
  return p.variant == HA_LA_KDA ? run_variant<true>(nullptr, nullptr, nullptr, nv, 0, false, nullptr)
                                : run_variant<false>(nullptr, nullptr, nullptr, nv, 0, false, nullptr);
}

}  // namespace ha_la
