// Plan kernel: turns (batch, seqlen) or a packed cu_seqlens array into the chunk table that the
// compute kernels index by chunk slot.  Runs on the device so that a packed batch needs no host
// synchronisation.  Chunks restart at every sequence start; the last chunk of a sequence may be
// partial (paper Section 2.1, "Chunkwise Map-Reduce-Map Execution": inputs are partitioned into
// chunks; chunk length 64 in the paper's experimental setup).
#include "common.cuh"

namespace ha_la {

namespace {

struct PlanParams {
  int N, T_total, T_row, max_len, max_chunks;
};

__global__ void __launch_bounds__(256) plan_kernel(PlanParams p, const int32_t* __restrict__ cu, PlanView v,
                                                   int32_t* status) {
  __shared__ int s_warp[8];
  __shared__ int s_carry;
  const int tid = threadIdx.x;

  // 1. per-sequence start and length, checked
  for (int n = tid; n < p.N; n += blockDim.x) {
    int t0, len;
    if (cu) {
      const int a = cu[n], b = cu[n + 1];
      bool ok = a >= 0 && b >= a && b <= p.T_total && (b - a) <= p.max_len;
      if (n == 0 && a != 0) ok = false;
      if (n == p.N - 1 && b != p.T_total) ok = false;
      if (!ok) report_status(status, HA_LA_ERR_DEVICE_CHECK);
      t0 = ok ? a : 0;
      len = ok ? (b - a) : 0;
    } else {
      t0 = n * p.T_row;
      len = p.T_row;
    }
    v.seq_tok0[n] = t0;
    v.seq_len[n] = len;
  }
  if (tid == 0) s_carry = 0;
  __syncthreads();

  // 1b. sequences by descending length (ties: by index), so that a kernel with one CTA per sequence can start
  // the longest ones first.  Rank by counting; beyond a few thousand sequences the order is left as it is
  // (they are then short, and the count would be quadratic).
  for (int n = tid; n < p.N; n += blockDim.x) {
    int rank = n;
    if (p.N <= 4096) {
      const int len = v.seq_len[n];
      rank = 0;
      for (int k = 0; k < p.N; ++k) {
        const int lk = v.seq_len[k];
        rank += (lk > len || (lk == len && k < n)) ? 1 : 0;
      }
    }
    v.seq_order[rank] = n;
  }

  // 2. exclusive prefix sum of chunk counts over sequences, 256 at a time
  for (int base = 0; base < p.N; base += blockDim.x) {
    const int n = base + tid;
    const int cnt = n < p.N ? (v.seq_len[n] + kChunk - 1) / kChunk : 0;
    int x = cnt;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if ((tid & 31) >= o) x += y;
    }
    if ((tid & 31) == 31) s_warp[tid >> 5] = x;
    __syncthreads();
    int woff = 0;
    for (int w = 0; w < (tid >> 5); ++w) woff += s_warp[w];
    const int incl = x + woff + s_carry;
    if (n < p.N) v.seq_chunk0[n] = incl - cnt;
    __syncthreads();
    if (tid == blockDim.x - 1) s_carry = incl;
    __syncthreads();
  }
  int total = s_carry;
  if (total > p.max_chunks) {   // cannot happen for checked lengths; guard the table anyway
    if (tid == 0) report_status(status, HA_LA_ERR_DEVICE_CHECK);
    total = 0;
  }
  if (tid == 0) {
    v.seq_chunk0[p.N] = total;
    v.hdr[0] = total;
    v.hdr[1] = p.N;
  }
  __syncthreads();

  // 3. one entry per chunk slot (binary search for the owning sequence)
  for (int s = tid; s < p.max_chunks; s += blockDim.x) {
    if (s >= total) {
      v.chunk_seq[s] = -1;
      v.chunk_tok0[s] = 0;
      v.chunk_len[s] = 0;
      continue;
    }
    int lo = 0, hi = p.N - 1;   // last n with seq_chunk0[n] <= s
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (v.seq_chunk0[mid] <= s) lo = mid; else hi = mid - 1;
    }
    const int c = s - v.seq_chunk0[lo];
    const int L = v.seq_len[lo];
    v.chunk_seq[s] = lo;
    v.chunk_tok0[s] = v.seq_tok0[lo] + c * kChunk;
    v.chunk_len[s] = min(kChunk, L - c * kChunk);
  }
}

}  // namespace

cudaError_t launch_plan(const Problem& p, const int32_t* cu_seqlens, PlanView plan, int32_t* status,
                        cudaStream_t stream) {
  PlanParams pp{p.N, p.T_total, p.T_row, p.max_len, p.max_chunks};
  timer_mark(stream, "plan");
  plan_kernel<<<1, 256, 0, stream>>>(pp, cu_seqlens, plan, status);
  return cudaGetLastError();
}

}  // namespace ha_la
