// Shared declarations of the ha_la CUDA library (host launchers + plan layout).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ha_la.h"

namespace ha_la {

constexpr int kChunk = 64;

// Chunk table written by the plan kernel at the start of the workspace.  A "chunk slot" is one
// (sequence, chunk-in-sequence); slots of a sequence are consecutive.  All offsets in tokens are
// rows of the packed [B*T] token axis.
struct PlanView {
  int32_t* hdr;         // [8]: hdr[0] = chunk slots in use, hdr[1] = sequences
  int32_t* seq_tok0;    // [N]   first token row of sequence n
  int32_t* seq_len;     // [N]   tokens in sequence n (0 if the sequence failed a check)
  int32_t* seq_chunk0;  // [N+1] first chunk slot of sequence n (prefix sum)
  int32_t* seq_order;   // [N]   sequences by descending length (longest first), for launch order
  int32_t* chunk_seq;   // [MC]  sequence of chunk slot s
  int32_t* chunk_tok0;  // [MC]  first token row of chunk slot s
  int32_t* chunk_len;   // [MC]  tokens in chunk slot s (1..64), 0 for an unused slot
};

struct Problem {
  int variant, dtype;
  int N;            // sequences (batch rows or packed sequences)
  int T_total;      // rows of the token axis (B*T or packed total)
  int T_row;        // tokens per batch row when cu_seqlens == NULL
  int HK, HV, dk, dv;
  int max_len;      // bound on one sequence's length
  int max_chunks;   // bound on chunk slots (MC)
  int max_seq_chunks;
  float scale;
  int varlen;       // packed batch (cu_seqlens) rather than equal-length rows
};

inline __host__ size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline __host__ size_t plan_bytes(const Problem& p) {
  size_t ints = 8 + 3 * (size_t)p.N + ((size_t)p.N + 1) + 3 * (size_t)p.max_chunks;
  return align_up(ints * sizeof(int32_t), 1024);
}

inline __host__ PlanView plan_view(void* ws, const Problem& p) {
  PlanView v;
  int32_t* b = reinterpret_cast<int32_t*>(ws);
  v.hdr = b;                       b += 8;
  v.seq_tok0 = b;                  b += p.N;
  v.seq_len = b;                   b += p.N;
  v.seq_chunk0 = b;                b += p.N + 1;
  v.seq_order = b;                 b += p.N;
  v.chunk_seq = b;                 b += p.max_chunks;
  v.chunk_tok0 = b;                b += p.max_chunks;
  v.chunk_len = b;
  return v;
}

// Host launchers (each returns a cudaError_t from the launch).
cudaError_t launch_plan(const Problem& p, const int32_t* cu_seqlens, PlanView plan, int32_t* status,
                        cudaStream_t stream);
cudaError_t launch_simt(const Problem& p, const ha_la_prefill_args& a, PlanView plan, cudaStream_t stream);
bool simt_supported(const Problem& p);

// Tensor-core (tcgen05) path: bf16, d_k = d_v = 128.
bool tc_supported(const Problem& p);
size_t tc_workspace_bytes(const Problem& p);
int tc_num_launches(const Problem& p);
int tc_num_segments(const Problem& p);                                      // segments per sequence launch_tc would use
void tc_launch_plan(const Problem& p, int* slice_width, int* concurrent);   // what launch_tc would choose
cudaError_t launch_tc(const Problem& p, const ha_la_prefill_args& a, PlanView plan, void* tc_ws,
                      cudaStream_t stream);
cudaError_t launch_tc_chain_unpublished(const Problem& p, const ha_la_prefill_args& a, void* tc_ws, uint32_t spin_limit,
                                        cudaStream_t stream);

// Optional per-kernel event timing (ha_la_prefill_timed): every launcher marks the stream before its kernel.
struct KernelTimer {
  static constexpr int kMax = 8;
  cudaEvent_t ev[kMax + 1];
  const char* name[kMax];
  int n = 0;
};
extern thread_local KernelTimer* g_timer;
inline void timer_mark(cudaStream_t s, const char* name) {
  if (g_timer && g_timer->n < KernelTimer::kMax) {
    cudaEventRecord(g_timer->ev[g_timer->n], s);
    g_timer->name[g_timer->n++] = name;
  }
}

__device__ __forceinline__ void report_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

}  // namespace ha_la
