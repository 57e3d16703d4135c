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
#include <stdlib.h>

#include "tc_common.cuh"
#include "tc_ptx.cuh"
#include "prof.cuh"

namespace ha_la {

using namespace ptx;

HA_PROF_DECL(chain)

namespace {

// compute warps + producer warp + MMA warp (+ a clean-up warp in the instances that drop consumed images from L2)
constexpr int chain_threads(int cg, bool drop) { return (4 * cg + 2 + (drop ? 1 : 0)) * 32; }

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
  static_assert(kStageB - OFF_BAR >= (2 * S_ + 2) * 8 + 16, "room for the barriers and three words");
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
  uint32_t spin_limit;         // polls before a bounded wait gives up (kSpinLimit; a few thousand in the time-out test)
  int drop_consumed;           // concurrent mode, images larger than L2: drop consumed images from L2 (clean-up warp)
  // Segment-parallel state passing (sliced kernels, equal-length rows): a sequence's chunks are cut into `nseg`
  // segments that run at the same time.  Segment 0 starts from h0.  A later segment s runs twice over: its value
  // columns from a ZERO state (provisional outputs into o, end state b_s into seg_b) and 128 "transition" columns
  // from the IDENTITY with U = O_loc = 0 (end state Phi_s into seg_phi; its output rows are R = scale Q~ Phi,
  // written to r_out).  The true start state h_s of the segment then gives  o += R h_s  and  h_{s+1} = Phi_s h_s + b_s.
  int nseg;                    // 1: off
  float* seg_b;                // [N*HV][nseg][128][128] fp32
  float* seg_phi;              // [N*HV][nseg][128][128] fp32
  void* r_out;                 // [T][HV][128], dtype of o
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

// eight bf16 (16 bytes) -> fp32
__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8]) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(u[i] << 16);
    f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
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
                                 // (the whole-head kernel has two tiles: ids 3, 4 for tile 0 and 5, 6 for tile 1)
// A chain CTA lets the stream's next programmatic dependent be scheduled when it has this many chunks left (CTAs
// with fewer chunks: when they exit).  That kernel -- the next call's prep kernel, or the segment fix-up -- then
// gets through its launch and set-up under the tail of this one and waits at its griddepcontrol.wait for this
// grid to complete; only kernels launched with the programmatic attribute react.
constexpr int kTailChunks = 6;
__device__ __forceinline__ void launch_dependents_early() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void named_arrive(int id, int count) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <int NV, bool KDA, int S, int CG, bool DROP>
__global__ void __launch_bounds__(chain_threads(CG, DROP), 1)
tc_chain_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_o, ChainParams p) {
  using Cfg = ChainCfg<NV, S>;
  constexpr int NSL = 128 / NV;
  constexpr int NVT = NV / CG;                           // value channels per compute thread
  constexpr int NCOMP = 128 * CG;                        // compute threads
  constexpr int W_PROD = 4 * CG, W_MMA = 4 * CG + 1, W_CLEAN = 4 * CG + 2;
  static_assert(NVT % 32 == 0, "column groups are multiples of 32 channels");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* sm = smem_raw;                                // no static shared memory in this kernel: 1024-aligned
  uint64_t* bar_full = reinterpret_cast<uint64_t*>(sm + Cfg::OFF_BAR);     // [S]  producer -> everyone
  uint64_t* bar_empty = bar_full + S;                                       // [S]  128 compute threads -> producer
  uint64_t* bar_mma1 = bar_empty + S;                                       // MMA1 complete
  uint64_t* bar_mma2 = bar_mma1 + 1;                                        // MMA2 complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mma2 + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* consumed = reinterpret_cast<volatile int*>(tmem_slot + 2);   // chunks this CTA is done with

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int slice = blockIdx.x % NSL;
  const int unit_id = blockIdx.x / NSL;
  const int units = 2 * p.nseg - 1;                      // per (sequence, V-head): nseg value runs + (nseg - 1) transition runs
  const int unit = unit_id % units;
  const int nj = unit_id / units;
  const int seg = unit < p.nseg ? unit : unit - p.nseg + 1;
  const bool trans = unit >= p.nseg;                     // this CTA carries transition columns (see ChainParams)
  const int j = nj % p.HV;
  const int n = p.seq_order ? p.seq_order[nj / p.HV] : nj / p.HV;   // CTAs of the longest sequences come first
  const int jq = j / (p.HV / p.HK);
  const int tok0_seq = p.seq_tok0 ? p.seq_tok0[n] : n * p.T_row;
  const int len_seq = p.seq_tok0 ? p.seq_len[n] : p.T_row;
  const int chunk0_seq = p.seq_tok0 ? p.seq_chunk0[n] : n * p.cps;
  // this CTA's segment of the sequence, walked like a sequence of its own
  const int nch_seq = (len_seq + kChunk - 1) / kChunk;
  const int cpseg = (nch_seq + p.nseg - 1) / p.nseg;
  const int tok0 = tok0_seq + seg * cpseg * kChunk;
  const int len = max(0, min(len_seq - seg * cpseg * kChunk, cpseg * kChunk));
  const int chunk0 = chunk0_seq + seg * cpseg;
  const int nchunks = (len + kChunk - 1) / kChunk;

  if (blockIdx.x == 0 && threadIdx.x == 0) HA_PROF_GT(chain, 900);
  if (tid == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_empty[i], NCOMP); }
    mbar_init(bar_mma1, 1);
    mbar_init(bar_mma2, 1);
    *abort_flag = 0;
    if constexpr (DROP) *consumed = 0;
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
        for (uint32_t it = 0; it < p.spin_limit && !*abort_flag; ++it) {
          const int cc = c + lane;
          bool ok = false;
          if (cc < nchunks)
            ok = (*reinterpret_cast<const volatile int64_t*>(p.ws.flags + (size_t)(chunk0 + cc) * p.HV + j) & ~kFlagCountMask) == p.epoch;
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
        if (c >= S) mbar_wait(&bar_empty[st], ((c / S) - 1) & 1, abort_flag, p.spin_limit);
        uint8_t* stage = sm + st * Cfg::kStageB;
        const size_t cj = (size_t)(chunk0 + c) * p.HV + j;
        mbar_expect_tx(&bar_full[st], Cfg::kTxBytes - (trans ? 2 * Cfg::kSliceB : 0));
        bulk_load(stage + Cfg::OFF_WQ, p.ws.wq + cj * 2 * kImgBytes, 32768, &bar_full[st]);
        if (!trans) {                                    // (transition columns: U = O_loc = 0)
          bulk_load(stage + Cfg::OFF_U, p.ws.u + cj * kImgBytes + (size_t)slice * Cfg::kSliceB, Cfg::kSliceB, &bar_full[st]);
          bulk_load(stage + Cfg::OFF_O, p.ws.ol + cj * kImgBytes + (size_t)slice * Cfg::kSliceB, Cfg::kSliceB, &bar_full[st]);
        }
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
      if (lead) mbar_wait(&bar_full[st], (c / S) & 1, abort_flag, p.spin_limit);
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
  } else if (DROP && warp == W_CLEAN) {
    // ------------------------------------------------------------ clean-up (concurrent mode, images larger than L2)
    // The images were written microseconds ago and mostly still sit in L2 as dirty lines.  Once this CTA is done
    // with a chunk, the U and O_loc rows of its slice -- read by this CTA alone -- are dead, and so are the W / Q~
    // image (and KDA's K e^{G_L-G} image) when the last slice of the head is done with them: the low byte of the
    // chunk's flag counts the slices.  Dropping the lines from L2 spares their write-back to HBM.  (Back to back
    // the lines have long been written back, and a workspace that stays in L2 from call to call is never written
    // back at all: nothing to gain in either case.)  Nothing waits for this warp; if its wait runs out it stops.
    if (!trans) {
      const int lane = tid & 31;
      for (int c = 0; c < nchunks; ++c) {
        bool done = false;
        for (uint32_t it = 0; it < p.spin_limit && !*abort_flag; ++it) {
          if (*consumed > c) { done = true; break; }
          __nanosleep(200);
        }
        if (!done) break;
        const size_t cj = (size_t)(chunk0 + c) * p.HV + j;
        int last = 0;
        if (lane == 0)
          last = (atomicAdd(reinterpret_cast<unsigned long long*>(p.ws.flags + cj), 1ull) & kFlagCountMask) == NSL - 1;
        last = __shfl_sync(0xffffffffu, last, 0);
        const uint8_t* u0 = p.ws.u + cj * kImgBytes + (size_t)slice * Cfg::kSliceB;
        const uint8_t* o0 = p.ws.ol + cj * kImgBytes + (size_t)slice * Cfg::kSliceB;
        for (uint32_t off = lane * 128u; off < Cfg::kSliceB; off += 4096u) {
          discard_l2_line(u0 + off);
          discard_l2_line(o0 + off);
        }
        if (last) {
          const uint8_t* w0 = p.ws.wq + cj * 2 * kImgBytes;
          for (uint32_t off = lane * 128u; off < 2 * kImgBytes; off += 4096u) discard_l2_line(w0 + off);
          if constexpr (KDA) {
            const uint8_t* k0 = p.ws.kd + cj * kImgBytes;
            for (uint32_t off = lane * 128u; off < kImgBytes; off += 4096u) discard_l2_line(k0 + off);
          }
        }
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
        if (p.h0 && seg == 0) v4 = *reinterpret_cast<const float4*>(p.h0 + base + q);   // later segments: zero start
        h[q] = v4.x; h[q + 1] = v4.y; h[q + 2] = v4.z; h[q + 3] = v4.w;
      }
      if (trans) {                                       // identity columns slice * NV + cg0 .. of the transition
#pragma unroll
        for (int q = 0; q < NVT; ++q) h[q] = row == slice * NV + cg0 + q ? 1.f : 0.f;
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
      if (c == nchunks - kTailChunks) launch_dependents_early();

      HA_PROF(chain, 8 * c + 0);
      mbar_wait(&bar_full[st], (c / S) & 1, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 1);
      // operands of the first epilogue that do not depend on the MMA, fetched while it runs
      const float* sc = reinterpret_cast<const float*>(stage + Cfg::OFF_SC);
      const float dec = sc[i];
      const float gam = sc[64 + row];
      float pre[32];
      if (!trans) {
        load_img32(stage + (row < 64 ? Cfg::OFF_U : Cfg::OFF_O), i, cg0, pre);
      } else {
#pragma unroll
        for (int q = 0; q < 32; ++q) pre[q] = 0.f;
      }

      mbar_wait(bar_mma1, ph, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 2);
      tc_fence_after_sync();
      if (row < 64) {                                    // U~ rows: (U - W h) e^{G_L - G_i}, the MMA2 operand
#pragma unroll
        for (int c0 = 0; c0 < NVT; c0 += 32) {
          float d[32];
          ld32f(TM1 + lane_base + cg0 + c0, d);
          if (c0 > 0 && !trans) load_img32(stage + Cfg::OFF_U, i, cg0 + c0, pre);
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
        const bool tile_out = NV > 32 && L == kChunk && !trans;   // (the tensor map is o's: transition rows go out directly)
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(trans ? p.r_out : p.o) +
                              ((size_t)(tok0 + c * kChunk + i) * p.HV + j) * 128 + (size_t)slice * NV + cg0;
        if (tile_out) named_sync(BAR_O_FREE, NCOMP / 2);
#pragma unroll
        for (int c0 = 0; c0 < NVT; c0 += 32) {
          float d[32];
          ld32f(TM1 + lane_base + cg0 + c0, d);
          if (c0 > 0 && !trans) load_img32(stage + Cfg::OFF_O, i, cg0 + c0, pre);
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

      mbar_wait(bar_mma2, ph, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 4);
      tc_fence_after_sync();
      mbar_arrive(&bar_empty[st]);                       // this thread and both MMAs are done with the stage
      if constexpr (DROP) {
        if (tid == 0) *consumed = c + 1;
      }
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

    // where the end state goes: hT, or with segments the segment's offset b_s / transition Phi_s
    float* hdst = p.hT ? p.hT + ((size_t)n * p.HV + j) * 128 * 128 : nullptr;
    if (p.nseg > 1) hdst = (trans ? p.seg_phi : p.seg_b) + (((size_t)n * p.HV + j) * p.nseg + seg) * 128 * 128;
    if (hdst) {
      const size_t base = (size_t)row * 128 + (size_t)slice * NV + cg0;
#pragma unroll
      for (int q = 0; q < NVT; q += 4)
        *reinterpret_cast<float4*>(hdst + base + q) = make_float4(h[q], h[q + 1], h[q + 2], h[q + 3]);
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

// ---------------------------------------------------------------------------------------------------------
// Whole-head variant: one CTA owns all 128 value channels of a (sequence, V-head) and keeps the state TRANSPOSED
// in tensor memory: lane = value channel v, columns = key channels.  Both products of a chunk then take their
// state-dependent operand from tensor memory (the A operand of tcgen05.mma may live there), and the operand images
// of the workspace serve unchanged as B operands from shared memory:
//   MMA1  D1^T[v][0:64 | 64:128] = h^T [W ; Q~]^T      A = h^T (bf16 pairs, tensor memory), B = the W / Q~ images
//         U~^T[v][i] = (U^T[v][i] - D1^T[v][i]) e^{G_L - G_i}   -> bf16 pairs straight back into tensor memory
//   MMA2  D2^T[v][k] = U~^T K~                          A = U~^T (tensor memory), B = the K tile (K e^{G_L-G}: KDA)
//         h^T[v][k] <- gamma_k h^T[v][k] + D2^T[v][k]   fp32 in registers, bf16 pairs back into tensor memory
//         o[i][v]   = scale (O_loc^T[v][i] + D1^T[v][64 + i])   (after the update, under the next chunk's MMA1:
//                                                                D1 alternates between two accumulators)
// No operand goes through shared memory, so the two proxy fences per chunk of the sliced kernel (and its operand
// stores) are gone, and the twelve MMA instructions of a chunk serve 128 value channels instead of 32 or 64.
// Measured: about 1.5 us per chunk (the MMAs with a tensor-memory A operand and a 128-wide B run at about half
// of the tensor peak and are the limit), against 0.9 us on FOUR SMs for 32-channel slices: the cheapest way
// through a chunk in SM-time, the slowest in latency.
// Eight compute warps: warp w works on lanes 32 (w % 4).. and on half w / 4 of the columns of each accumulator;
// two more warps copy the output rows from a shared-memory tile to global memory.
constexpr int t_threads(int cg) { return (4 * cg + 4) * 32; }   // compute warps + producer, MMA and 2 output warps

struct ChainTCfg {
  static constexpr int kStages = 2;
  static constexpr uint32_t OFF_WQ = 0;                          // 32 KiB: W image, Q~ image
  static constexpr uint32_t OFF_K = 32768;                       // 16 KiB  [kb][64 tok][64 feat]
  static constexpr uint32_t OFF_U = 49152;                       // 16 KiB: U image
  static constexpr uint32_t OFF_O = 65536;                       // 16 KiB: O_loc image
  static constexpr uint32_t OFF_SC = 81920;                      // 192 floats
  static constexpr uint32_t kStageB = 82944;
  static constexpr uint32_t kTxBytes = 32768 + 16384 + 16384 + 16384 + 768;
  static constexpr uint32_t OFF_BAR = OFF_SC + 768 + 128;        // barriers: in the unused tail of stage 0
  static constexpr uint32_t OFF_OUT = kStages * kStageB;         // two bf16 output tiles [2 x 64 ch blocks][64 tok], swizzled
  static constexpr uint32_t kSmem = OFF_OUT + 2 * 16384;
  static constexpr uint32_t kTmemCols = 512;
  static constexpr uint32_t TM_D1 = 0, TM_D2 = 256, TM_H = 384, TM_UT = 448;   // D1: two accumulators of 128
};

template <bool KDA, int CG>
__global__ void __launch_bounds__(t_threads(CG), 1)
tc_chain_t_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_o, ChainParams p) {
  using Cfg = ChainTCfg;
  constexpr int S = Cfg::kStages;
  constexpr int NCOMP = 128 * CG;                        // compute threads: CG column groups of four warps
  constexpr int TOK = 64 / CG;                           // tokens per thread in the U~ and output epilogues
  constexpr int KC = 128 / CG;                           // key channels per thread in the state update
  constexpr int W_PROD = 4 * CG, W_MMA = 4 * CG + 1, W_OUT = 4 * CG + 2;   // the last two warps write o
  static_assert(CG == 2 || CG == 4, "two or four column groups");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* sm = smem_raw;
  uint64_t* bar_full = reinterpret_cast<uint64_t*>(sm + Cfg::OFF_BAR);
  uint64_t* bar_empty = bar_full + S;
  uint64_t* bar_mma1 = bar_empty + S;
  uint64_t* bar_mma2 = bar_mma1 + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mma2 + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int nj = blockIdx.x;
  const int j = nj % p.HV;
  const int n = p.seq_order ? p.seq_order[nj / p.HV] : nj / p.HV;
  const int jq = j / (p.HV / p.HK);
  const int tok0 = p.seq_tok0 ? p.seq_tok0[n] : n * p.T_row;
  const int len = p.seq_tok0 ? p.seq_len[n] : p.T_row;
  const int chunk0 = p.seq_tok0 ? p.seq_chunk0[n] : n * p.cps;
  const int nchunks = (len + kChunk - 1) / kChunk;

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
  if (p.epoch == 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // sequential mode: the prep grid is done

  if (warp == W_PROD) {
    // ------------------------------------------------------------ producer (as in the sliced kernel)
    int ready_upto = p.epoch != 0 ? 0 : nchunks;
    for (int c = 0; c < nchunks; ++c) {
      if (c >= ready_upto) {
        int got = 0;
        for (uint32_t it = 0; it < p.spin_limit && !*abort_flag; ++it) {
          const int cc = c + lane;
          bool ok = false;
          if (cc < nchunks)
            ok = (*reinterpret_cast<const volatile int64_t*>(p.ws.flags + (size_t)(chunk0 + cc) * p.HV + j) & ~kFlagCountMask) == p.epoch;
          const unsigned m = __ballot_sync(0xffffffffu, ok);
          got = __ffs(~m) - 1;
          if (got < 0) got = 32;
          if (got > 0) break;
          __nanosleep(100);
        }
        if (got == 0) *abort_flag = 1;
        ready_upto = c + (got > 0 ? got : nchunks);
        __threadfence();
        fence_proxy_async_all();
      }
      if (lane == 0) {
        const int st = c % S;
        if (c >= S) mbar_wait(&bar_empty[st], ((c / S) - 1) & 1, abort_flag, p.spin_limit);
        uint8_t* stage = sm + st * Cfg::kStageB;
        const size_t cj = (size_t)(chunk0 + c) * p.HV + j;
        mbar_expect_tx(&bar_full[st], Cfg::kTxBytes);
        bulk_load(stage + Cfg::OFF_WQ, p.ws.wq + cj * 2 * kImgBytes, 32768, &bar_full[st]);
        if constexpr (KDA) {
          bulk_load(stage + Cfg::OFF_K, p.ws.kd + cj * kImgBytes, 16384, &bar_full[st]);
        } else {
          tma_load_3d(stage + Cfg::OFF_K, &map_k, &bar_full[st], 0, jq, tok0 + c * kChunk);
          tma_load_3d(stage + Cfg::OFF_K + 8192, &map_k, &bar_full[st], 64, jq, tok0 + c * kChunk);
        }
        bulk_load(stage + Cfg::OFF_U, p.ws.u + cj * kImgBytes, 16384, &bar_full[st]);
        bulk_load(stage + Cfg::OFF_SC, p.ws.sc + cj * kScFloats, 768, &bar_full[st]);
        bulk_load(stage + Cfg::OFF_O, p.ws.ol + cj * kImgBytes, 16384, &bar_full[st]);
      }
      __syncwarp();
    }
  } else if (warp == W_MMA) {
    // ------------------------------------------------------------ MMA issue
    // A from tensor memory (K-major by construction), B from shared memory, MN-major (the images are feature-
    // major: rows = the K index of these products, 128 swizzled bytes of the N index each).
    const uint32_t id = idesc_bf16(128, 128, false, true);
    const bool lead = lane == 0;
    for (int c = 0; c < nchunks; ++c) {
      const int st = c % S;
      const uint32_t stage = smem_u32(sm + st * Cfg::kStageB);
      const uint64_t dWQ = smem_desc(stage + Cfg::OFF_WQ, 16384, 1024, kSwizzle128B);   // N = 64 W + 64 Q~ tokens
      const uint64_t dK = smem_desc(stage + Cfg::OFF_K, 8192, 1024, kSwizzle128B);      // N = 2 x 64 key channels
      const uint32_t d1 = tmem + Cfg::TM_D1 + (c & 1) * 128;
      if (lead) mbar_wait(&bar_full[st], (c / S) & 1, abort_flag, p.spin_limit);
      named_sync(BAR_H_READY, NCOMP + 32);               // h^T (bf16 pairs) of the previous chunk is in tensor memory
      if (lead) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)                    // K = d_k: 16 key channels = 8 columns of A, 2048 B of B
          umma_ts(d1, tmem + Cfg::TM_H + ks * 8, dWQ + ks * (2048u >> 4), id, ks > 0);
        umma_commit(bar_mma1);
      }
      named_sync(BAR_U_READY, NCOMP + 32);               // U~^T is in tensor memory
      if (lead) {
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)                    // K = tokens: 16 tokens = 8 columns of A, 2048 B of B
          umma_ts(tmem + Cfg::TM_D2, tmem + Cfg::TM_UT + ks * 8, dK + ks * (2048u >> 4), id, ks > 0);
        umma_commit(bar_mma2);
      }
    }
  } else if (warp >= W_OUT) {
    // ------------------------------------------------------------ output rows: the compute warps leave a chunk's o
    // as a token-major tile in shared memory (two tiles, used alternately); these two warps copy it out with plain
    // 16-byte loads and stores, two whole token rows (512 contiguous bytes) per store instruction.  Plain accesses
    // on both sides: no proxy fence (which takes thousands of cycles in this kernel, with 80 KiB of bulk loads per
    // chunk in flight), and no global stores on the compute warps (a warp there holds 32 channels of a token).
    const int ht = tid - W_OUT * 32;                     // 0..63
    named_arrive(BAR_O_FREE, NCOMP + 64);                // both tiles start out free
    named_arrive(BAR_O_FREE + 2, NCOMP + 64);
    for (int c = 0; c < nchunks; ++c) {
      const int b = c & 1;
      const int L = min(kChunk, len - c * kChunk);
      named_sync(BAR_O_FULL + 2 * b, NCOMP + 64);
      const uint8_t* tile = sm + Cfg::OFF_OUT + b * 16384;
      __nv_bfloat16* obase = reinterpret_cast<__nv_bfloat16*>(p.o) + ((size_t)(tok0 + c * kChunk) * p.HV + j) * 128;
      const int k = ht & 15;                             // 16-byte piece of a token row (8 channels)
#pragma unroll 4
      for (int it = 0; it < 16; ++it) {
        const int t = it * 4 + (ht >> 4);
        const uint4 w = *reinterpret_cast<const uint4*>(tile + (k >> 3) * 8192 + sw128_offset(t, k & 7));
        if (t < L) *reinterpret_cast<uint4*>(obase + (size_t)t * p.HV * 128 + k * 8) = w;
      }
      named_arrive(BAR_O_FREE + 2 * b, NCOMP + 64);
    }
  } else {
    // ------------------------------------------------------------ compute
    const int v = (warp & 3) * 32 + lane;                // value channel = tensor-memory lane
    const int g = warp >> 2;                             // column group
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    auto ld_cols = [&](uint32_t taddr, float (&d)[TOK]) {     // TOK consecutive fp32 columns of this lane
      if constexpr (TOK == 32) {
        ld32f(taddr, d);
      } else {
        uint32_t r[16];
        tmem_ld16(taddr, r);
        tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 16; ++q) d[q] = __uint_as_float(r[q]);
      }
    };
    auto img_row = [&](const uint8_t* img, float (&x)[TOK]) { // tokens TOK g .. of channel v of a feature-major image
#pragma unroll
      for (int q = 0; q < TOK / 8; ++q)
        unpack8(*reinterpret_cast<const uint4*>(img + sw128_offset(v, (TOK / 8) * g + q)),
                *reinterpret_cast<float(*)[8]>(x + 8 * q));
    };
    float h[KC];                                         // h^T[v][KC g .. KC g + KC - 1]
    {
      const size_t base = ((size_t)n * p.HV + j) * 128 * 128 + v;
#pragma unroll
      for (int q = 0; q < KC; ++q) h[q] = p.h0 ? p.h0[base + (size_t)(KC * g + q) * 128] : 0.f;
    }
    auto store_h = [&]() {                               // bf16 pairs of this thread's key channels -> A operand
#pragma unroll
      for (int c0 = 0; c0 < KC; c0 += 32) {
        uint32_t r[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) r[q] = pack_bf16(h[c0 + 2 * q], h[c0 + 2 * q + 1]);
        tmem_st16(tmem + Cfg::TM_H + lane_base + (KC / 2) * g + c0 / 2, r);
      }
      tmem_st_wait();
    };
    store_h();
    tc_fence_before_sync();
    named_arrive(BAR_H_READY, NCOMP + 32);

    // o of chunk c: after the state update, while the tensor cores work on the next chunk
    auto output_part = [&](int c) {
      const int st = c % S;
      const uint8_t* stage = sm + st * Cfg::kStageB;
      float d[TOK];
      ld_cols(tmem + Cfg::TM_D1 + (c & 1) * 128 + lane_base + 64 + TOK * g, d);
      float ol[TOK];
      img_row(stage + Cfg::OFF_O, ol);
      mbar_arrive(&bar_empty[st]);                       // last read of the stage by this thread
      // hand the tokens of this thread's channel to the output warps (token-major tile, 2-byte stores: a warp
      // writes 64 contiguous bytes of a token row per instruction)
      uint8_t* tile = sm + Cfg::OFF_OUT + (c & 1) * 16384 + (v >> 6) * 8192 + (v & 7) * 2;
      named_sync(BAR_O_FREE + 2 * (c & 1), NCOMP + 64);  // the output warps are done with this tile's last contents
#pragma unroll
      for (int q = 0; q < TOK; ++q) {
        const int t = TOK * g + q;
        *reinterpret_cast<__nv_bfloat16*>(tile + sw128_offset(t, (v & 63) >> 3)) =
            __float2bfloat16_rn(p.scale * (ol[q] + d[q]));
      }
      named_arrive(BAR_O_FULL + 2 * (c & 1), NCOMP + 64);
    };

    for (int c = 0; c < nchunks; ++c) {
      const int st = c % S;
      const uint8_t* stage = sm + st * Cfg::kStageB;
      const uint32_t ph = c & 1;
      if (c == nchunks - kTailChunks) launch_dependents_early();
      HA_PROF(chain, 8 * c + 0);
      mbar_wait(&bar_full[st], (c / S) & 1, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 1);
      const float* sc = reinterpret_cast<const float*>(stage + Cfg::OFF_SC);
      float u[TOK];                                      // U^T[v][TOK g ..], fetched while MMA1 runs
      img_row(stage + Cfg::OFF_U, u);
      mbar_wait(bar_mma1, ph, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 2);
      tc_fence_after_sync();
      {
        float d[TOK];
        ld_cols(tmem + Cfg::TM_D1 + (c & 1) * 128 + lane_base + TOK * g, d);
        uint32_t r[TOK / 2];
#pragma unroll
        for (int q = 0; q < TOK / 2; ++q) {
          const float2 dc = *reinterpret_cast<const float2*>(sc + TOK * g + 2 * q);   // e^{G_L - G_i}, two tokens
          r[q] = pack_bf16((u[2 * q] - d[2 * q]) * dc.x, (u[2 * q + 1] - d[2 * q + 1]) * dc.y);
        }
        if constexpr (TOK == 32) tmem_st16(tmem + Cfg::TM_UT + lane_base + 16 * g, r);
        else tmem_st8(tmem + Cfg::TM_UT + lane_base + 8 * g, r);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      named_arrive(BAR_U_READY, NCOMP + 32);
      HA_PROF(chain, 8 * c + 3);

      mbar_wait(bar_mma2, ph, abort_flag, p.spin_limit);
      HA_PROF(chain, 8 * c + 4);
      tc_fence_after_sync();
#pragma unroll
      for (int c0 = 0; c0 < KC; c0 += 32) {
        float d[32];
        ld32f(tmem + Cfg::TM_D2 + lane_base + KC * g + c0, d);
        if constexpr (KDA) {
#pragma unroll
          for (int q = 0; q < 32; q += 4) {
            const float4 gm = *reinterpret_cast<const float4*>(sc + 64 + KC * g + c0 + q);   // decay per key channel
            h[c0 + q] = fmaf(gm.x, h[c0 + q], d[q]);
            h[c0 + q + 1] = fmaf(gm.y, h[c0 + q + 1], d[q + 1]);
            h[c0 + q + 2] = fmaf(gm.z, h[c0 + q + 2], d[q + 2]);
            h[c0 + q + 3] = fmaf(gm.w, h[c0 + q + 3], d[q + 3]);
          }
        } else {
          const float gm = sc[64];                         // one decay for the whole chunk
#pragma unroll
          for (int q = 0; q < 32; ++q) h[c0 + q] = fmaf(gm, h[c0 + q], d[q]);
        }
      }
      store_h();
      tc_fence_before_sync();
      named_arrive(BAR_H_READY, NCOMP + 32);
      HA_PROF(chain, 8 * c + 5);
      output_part(c);
      HA_PROF(chain, 8 * c + 6);
    }

    if (p.hT) {
      const size_t base = ((size_t)n * p.HV + j) * 128 * 128 + v;
#pragma unroll
      for (int q = 0; q < KC; ++q) p.hT[base + (size_t)(KC * g + q) * 128] = h[q];
    }
  }

  if (warp == W_MMA) named_sync(BAR_H_READY, NCOMP + 32);  // pairs with the compute warps' last arrival
  if (*abort_flag && tid == 0) report_status(p.status, HA_LA_ERR_TIMEOUT);
  if (p.epoch != 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, Cfg::kTmemCols);
}

template <bool KDA, int CG>
cudaError_t run_t(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int grid, bool dependent,
                  cudaStream_t stream) {
  auto kern = tc_chain_t_kernel<KDA, CG>;
  constexpr int smem = ChainTCfg::kSmem;
  static_assert(smem <= 227 * 1024, "shared memory budget");
  if (!cp) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  }
  timer_mark(stream, "tc_chain");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(t_threads(CG));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, *mk, *mo, *cp);
}

template <int NV, bool KDA, int S, int CG, bool DROP>
cudaError_t run_nv_inst(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int grid, bool dependent,
                        cudaStream_t stream) {
  auto kern = tc_chain_kernel<NV, KDA, S, CG, DROP>;
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
  cfg.blockDim = dim3(chain_threads(CG, DROP));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, *mk, *mo, *cp);
}

// Two instances per width: with and without the clean-up warp (ChainParams::drop_consumed); both are configured.
template <int NV, bool KDA, int S, int CG>
cudaError_t run_nv(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int grid, bool dependent,
                   cudaStream_t stream) {
  if (!cp) {
    cudaError_t e = run_nv_inst<NV, KDA, S, CG, false>(cp, mk, mo, grid, dependent, stream);
    if (e != cudaSuccess) return e;
    return run_nv_inst<NV, KDA, S, CG, true>(cp, mk, mo, grid, dependent, stream);
  }
  return cp->drop_consumed ? run_nv_inst<NV, KDA, S, CG, true>(cp, mk, mo, grid, dependent, stream)
                           : run_nv_inst<NV, KDA, S, CG, false>(cp, mk, mo, grid, dependent, stream);
}

// Slices of 64 value channels are worked on by two column groups of compute warps.
template <bool KDA>
cudaError_t run_variant(const ChainParams* cp, const CUtensorMap* mk, const CUtensorMap* mo, int nv, int grid,
                        bool dependent, cudaStream_t stream) {
  if (nv == 32) return run_nv<32, KDA, 3, 1>(cp, mk, mo, grid, dependent, stream);
  if (nv == 64) return run_nv<64, KDA, 3, 2>(cp, mk, mo, grid, dependent, stream);
  // all 128 channels: the whole-head kernel (two column groups of compute warps; four measured no faster: its
  // products, slowed by the shared-memory traffic around them, are the limit, not the epilogues)
  return run_t<KDA, 2>(cp, mk, mo, grid, dependent, stream);
}

}  // namespace

cudaError_t launch_tc_chain(const Problem& p, const ha_la_prefill_args& a, PlanView plan, const TcWorkspace& ws,
                            const CUtensorMap& mk, const CUtensorMap& mo, int nv, int64_t epoch, bool dependent,
                            uint32_t spin_limit, const SegBuffers& sg, cudaStream_t stream) {
  ChainParams cp;
  cp.h0 = a.h0; cp.hT = a.hT; cp.o = a.o;
  cp.seq_tok0 = plan.seq_tok0; cp.seq_len = plan.seq_len; cp.seq_chunk0 = plan.seq_chunk0;
  cp.seq_order = plan.seq_tok0 ? plan.seq_order : nullptr;
  cp.T_row = p.T_row; cp.cps = p.max_seq_chunks > 0 ? p.max_seq_chunks : 1;
  cp.ws = ws; cp.HK = p.HK; cp.HV = p.HV; cp.scale = p.scale; cp.status = a.status_word;
  cp.epoch = epoch;
  cp.spin_limit = spin_limit;
  {
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev);
    const size_t images = (size_t)p.max_chunks * p.HV * 4 * kImgBytes;
    cp.drop_consumed = epoch != 0 && sg.nseg == 1 && images > (size_t)l2;
  }
  cp.nseg = sg.nseg; cp.seg_b = sg.seg_b; cp.seg_phi = sg.seg_phi; cp.r_out = sg.r;
  const int grid = p.N * p.HV * (128 / nv) * (2 * sg.nseg - 1);
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
