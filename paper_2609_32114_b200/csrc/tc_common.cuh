// Layout of the tensor-core path's workspace and the parameters shared by its two kernels.
//
// For every (chunk slot s, V-head j), cj = s * HV + j, the prep kernel writes
//   wq  [cj] : 32 KiB  W image (16 KiB) followed by the Q~ image (16 KiB)
//   u   [cj] : 16 KiB  U image
//   ol  [cj] : 16 KiB  O_loc image
//   kd  [cj] : 16 KiB  KDA only: K e^{G_L - G}, in the shared-memory layout of the TMA K tile
//   flg [cj] : int64   set to the call's epoch by the prep CTA once everything above is in memory; the
//                      chain kernel, when it runs concurrently with the prep kernel, waits for it per chunk.
//                      An epoch is a per-process random 32-bit tag and a call counter, so that whatever the
//                      caller's workspace held before cannot pass for "published" (nothing is ever cleared)
//   sc  [cj] : 192 floats  e^{G_L - G_i} for the 64 tokens, then e^{G_L} for the 128 key channels
// An "image" is a 128 x 64 bf16 matrix stored feature-major: row r (key or value channel) holds the
// 64 tokens of the chunk in 128 bytes, and the eight 16-byte pieces of a row are stored at piece
// index (p XOR (r mod 8)).  That is byte for byte the 128-byte-swizzled shared-memory layout that
// tcgen05.mma reads, so the chain kernel fetches images with plain 1-D bulk copies.
#pragma once

#include "common.cuh"

namespace ha_la {

constexpr size_t kImgBytes = 128 * 64 * 2;     // 16 KiB
constexpr int kScFloats = 192;

// A chunk's ready flag holds the call's epoch (low byte zero) when the prep kernel has published it; the chain
// kernel's slices then count themselves off in the low byte as they finish with the chunk.
constexpr long long kFlagCountMask = 0xff;

struct TcWorkspace {
  uint8_t* wq;
  uint8_t* u;
  uint8_t* ol;
  uint8_t* kd;      // KDA only
  int64_t* flags;
  float* sc;
};

inline __host__ size_t tc_ws_bytes_for(size_t ncj, bool kda) {
  return ncj * (2 * kImgBytes + kImgBytes + kImgBytes + (kda ? kImgBytes : 0)) +
         align_up(ncj * kScFloats * sizeof(float), 1024) + align_up(ncj * sizeof(int64_t), 1024);
}

inline __host__ TcWorkspace tc_ws_view(void* base, size_t ncj, bool kda) {
  TcWorkspace w;
  uint8_t* b = reinterpret_cast<uint8_t*>(base);
  w.wq = b;                      b += ncj * 2 * kImgBytes;
  w.u = b;                       b += ncj * kImgBytes;
  w.ol = b;                      b += ncj * kImgBytes;
  w.kd = kda ? b : nullptr;      b += kda ? ncj * kImgBytes : 0;
  w.sc = reinterpret_cast<float*>(b);  b += align_up(ncj * kScFloats * sizeof(float), 1024);
  w.flags = reinterpret_cast<int64_t*>(b);
  return w;
}

// Scratch of the segment-parallel state passing, behind the images: per (sequence, V-head) and segment the
// offset b_s and the transition Phi_s (fp32 128 x 128 each) and the segment's true start state as bf16; per
// token-head the transition output rows R (bf16 [T][HV][128]).
struct SegBuffers {
  int nseg;             // 1: segments are off and the pointers are null
  float* seg_b;
  float* seg_phi;
  __nv_bfloat16* hs;    // [N*HV][nseg][128][128]: start state of segment s (s >= 1)
  __nv_bfloat16* r;     // [T][HV][128]
};

inline __host__ size_t tc_seg_bytes(size_t nj, int nseg, size_t rows, int HV) {
  if (nseg <= 1) return 0;
  return nj * nseg * 128 * 128 * (4 + 4 + 2) + align_up(rows * HV * 128 * 2, 1024);
}

inline __host__ SegBuffers tc_seg_view(void* base, size_t nj, int nseg, size_t rows, int HV) {
  SegBuffers g{nseg, nullptr, nullptr, nullptr, nullptr};
  if (nseg <= 1) return g;
  uint8_t* b = reinterpret_cast<uint8_t*>(base);
  g.seg_b = reinterpret_cast<float*>(b);               b += nj * nseg * 128 * 128 * 4;
  g.seg_phi = reinterpret_cast<float*>(b);             b += nj * nseg * 128 * 128 * 4;
  g.hs = reinterpret_cast<__nv_bfloat16*>(b);          b += nj * nseg * 128 * 128 * 2;
  g.r = reinterpret_cast<__nv_bfloat16*>(b);
  (void)rows; (void)HV;
  return g;
}

}  // namespace ha_la
