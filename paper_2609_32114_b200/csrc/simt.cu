// fp32 CUDA-core implementation of the chunkwise delta-rule prefill (GDN and KDA).
//
// One CTA per (sequence, V-head) walks the chunks of its sequence in order and evaluates, per
// chunk, the six operators of the paper's chunkwise pipeline (Section 2.1, "Chunkwise
// Map-Reduce-Map Execution"): #1 Gate (cumulative log-gate), #2 KKT (beta-scaled, decay-masked
// K K^T), #3 Solve and #4 W/U (forward substitution of (I + A) [W | U] = diag(beta) [K e^G | V]),
// #5 H (state read U~ = U - W h and update h <- e^{G_L} h + (K e^{G_L - G})^T U~) and #6 O
// (o = scale [(Q e^G) h + P U~], P = decay-masked Q K^T with the diagonal).  The state stays in
// registers for the whole sequence; operator 6 runs between the read and the update of operator
// 5 (the paper's "chunk-first" order, Section "Lifetime-Aware Operator Reordering"), so the state
// is updated in place.
//
// This path serves fp32 inputs (where the 1e-4 tolerance rules out 16-bit tensor-core operands)
// and head dimensions / variants the tensor-core path does not cover.  All arithmetic is fp32.
#include "common.cuh"

namespace ha_la {

namespace {

constexpr int kThreads = 256;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

struct SimtParams {
  const void* q; const void* k; const void* v;
  const float* g; const float* beta; const float* h0;
  void* o; float* hT;
  const int32_t* seq_tok0; const int32_t* seq_len;
  int HK, HV;
  float scale;
};

template <int DK, int DV, bool KDA>
struct SimtSmem {
  static constexpr int SK = DK + 1;                       // padded row strides (bank spread)
  static constexpr int SV = DV + 1;
  static constexpr int SW = (DK > DV ? DK : DV) + 1;      // W rows; reused as the o accumulator
  static constexpr int SA = kChunk + 1;
  static constexpr int SG = KDA ? DK + 1 : 1;
  static constexpr size_t floats = (size_t)kChunk * (2 * SK + SV + SW + 2 * SA + SG) + 2 * kChunk;
  static constexpr size_t bytes = floats * sizeof(float);
};

template <typename In, int DK, int DV, bool KDA>
__global__ void __launch_bounds__(kThreads, 1) simt_prefill_kernel(SimtParams p) {
  using S = SimtSmem<DK, DV, KDA>;
  constexpr int C = kChunk;
  constexpr int NP = kThreads / DV;        // threads sharing one state column
  constexpr int RPT = DK / NP;             // state rows per thread
  constexpr int IB = 16;                   // chunk rows per register block
  static_assert(kThreads % DV == 0 && DK % NP == 0 && DK + DV <= kThreads, "unsupported head dims");

  extern __shared__ float smem[];
  float* sQ = smem;                        // [C][SK]
  float* sK = sQ + C * S::SK;              // [C][SK]
  float* sU = sK + C * S::SK;              // [C][SV]  beta*V -> U -> U~
  float* sW = sU + C * S::SV;              // [C][SW]  beta*K*e^G -> W ; later the o accumulator
  float* sA = sW + C * S::SW;              // [C][SA]
  float* sP = sA + C * S::SA;              // [C][SA]
  float* sG = sP + C * S::SA;              // GDN [C] ; KDA [C][SG]   (cumulative log-gate)
  float* sB = sG + C * S::SG;              // [C] beta
  float* sD = sB + C;                      // [C] GDN: e^{G_L - G_i}

  const int tid = threadIdx.x;
  const int n = blockIdx.x / p.HV;
  const int j = blockIdx.x % p.HV;
  const int jq = j / (p.HV / p.HK);
  const int x = tid % DV;                  // state column owned by this thread
  const int part = tid / DV;               // owns rows c = part + NP*r

  const In* gq = reinterpret_cast<const In*>(p.q);
  const In* gk = reinterpret_cast<const In*>(p.k);
  const In* gv = reinterpret_cast<const In*>(p.v);
  In* go = reinterpret_cast<In*>(p.o);

  float h[RPT];
  {
    const size_t base = ((size_t)n * p.HV + j) * DK * DV;
#pragma unroll
    for (int r = 0; r < RPT; ++r) h[r] = p.h0 ? p.h0[base + (size_t)(part + NP * r) * DV + x] : 0.f;
  }

  const int tok0 = p.seq_tok0[n];
  const int len = p.seq_len[n];

  for (int cs = 0; cs < len; cs += C) {
    const int L = min(C, len - cs);
    const size_t t0 = (size_t)tok0 + cs;

    // ---- load the chunk; rows >= L are no-op tokens (k = q = v = 0, beta = 0, g = 0)
    for (int idx = tid; idx < C * DK; idx += kThreads) {
      const int i = idx / DK, c = idx % DK;
      float qv = 0.f, kv = 0.f;
      if (i < L) {
        const size_t off = ((t0 + i) * p.HK + jq) * DK + c;
        qv = to_f32<In>(gq[off]);
        kv = to_f32<In>(gk[off]);
      }
      sQ[i * S::SK + c] = qv;
      sK[i * S::SK + c] = kv;
      if (KDA) sG[i * S::SG + c] = i < L ? p.g[((t0 + i) * p.HV + j) * DK + c] : 0.f;
    }
    for (int idx = tid; idx < C * DV; idx += kThreads) {
      const int i = idx / DV, c = idx % DV;
      sU[i * S::SV + c] = i < L ? to_f32<In>(gv[((t0 + i) * p.HV + j) * DV + c]) : 0.f;
    }
    if (tid < C) {
      sB[tid] = tid < L ? p.beta[(t0 + tid) * p.HV + j] : 0.f;
      if (!KDA) sG[tid] = tid < L ? p.g[(t0 + tid) * p.HV + j] : 0.f;
    }
    __syncthreads();

    // ---- op #1 Gate: chunk-local inclusive cumulative sum of the log-gate
    if (KDA) {
      if (tid < DK) {
        float acc = 0.f;
        for (int i = 0; i < C; ++i) { acc += sG[i * S::SG + tid]; sG[i * S::SG + tid] = acc; }
      }
    } else if (tid == 0) {
      float acc = 0.f;
      for (int i = 0; i < C; ++i) { acc += sG[i]; sG[i] = acc; }
    }
    __syncthreads();
    if (!KDA && tid < C) sD[tid] = expf(sG[C - 1] - sG[tid]);

    // ---- op #2 KKT and the masked Q K^T: A (strictly lower, beta-scaled) and P (lower incl. diagonal)
    for (int idx = tid; idx < C * C; idx += kThreads) {
      const int i = idx / C, jj = idx % C;
      float kk = 0.f, qk = 0.f;
      if (jj <= i) {
        if (KDA) {
          for (int c = 0; c < DK; ++c) {
            const float e = expf(sG[i * S::SG + c] - sG[jj * S::SG + c]);
            const float kj = sK[jj * S::SK + c] * e;
            kk = fmaf(sK[i * S::SK + c], kj, kk);
            qk = fmaf(sQ[i * S::SK + c], kj, qk);
          }
        } else {
          for (int c = 0; c < DK; ++c) {
            const float kj = sK[jj * S::SK + c];
            kk = fmaf(sK[i * S::SK + c], kj, kk);
            qk = fmaf(sQ[i * S::SK + c], kj, qk);
          }
          const float e = expf(sG[i] - sG[jj]);
          kk *= e;
          qk *= e;
        }
      }
      sA[i * S::SA + jj] = jj < i ? sB[i] * kk : 0.f;
      sP[i * S::SA + jj] = jj <= i ? qk : 0.f;
    }
    // right-hand sides: W <- beta * K * e^G, U <- beta * V
    for (int idx = tid; idx < C * DK; idx += kThreads) {
      const int i = idx / DK, c = idx % DK;
      const float e = KDA ? expf(sG[i * S::SG + c]) : expf(sG[i]);
      sW[i * S::SW + c] = sB[i] * sK[i * S::SK + c] * e;
    }
    for (int idx = tid; idx < C * DV; idx += kThreads) {
      const int i = idx / DV, c = idx % DV;
      sU[i * S::SV + c] *= sB[i];
    }
    __syncthreads();

    // ---- op #3 Solve + op #4 W/U: forward substitution, one thread per column of [W | U]
    if (tid < DK + DV) {
      float* col = tid < DK ? (sW + tid) : (sU + (tid - DK));
      const int st = tid < DK ? S::SW : S::SV;
      for (int i = 1; i < C; ++i) {
        float acc = col[i * st];
        for (int jj = 0; jj < i; ++jj) acc = fmaf(-sA[i * S::SA + jj], col[jj * st], acc);
        col[i * st] = acc;
      }
    }
    __syncthreads();

    // ---- op #5 (read part): U~ = U - W h   (rows in blocks of IB to bound the unrolled code)
    for (int ib = 0; ib < C; ib += IB) {
      float acc[IB];
#pragma unroll
      for (int i = 0; i < IB; ++i) acc[i] = 0.f;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        const int c = part + NP * r;
        const float hv = h[r];
#pragma unroll
        for (int i = 0; i < IB; ++i) acc[i] = fmaf(sW[(ib + i) * S::SW + c], hv, acc[i]);
      }
      for (int pp = 0; pp < NP; ++pp) {        // fixed order: deterministic rounding
        if (part == pp) {
#pragma unroll
          for (int i = 0; i < IB; ++i) sU[(ib + i) * S::SV + x] -= acc[i];
        }
        __syncthreads();
      }
    }

    // ---- op #6 O: o = scale [ (Q e^G) h + P U~ ]   (sW is free now and holds the accumulator)
    for (int ib = 0; ib < C; ib += IB) {
      float acc[IB];
#pragma unroll
      for (int i = 0; i < IB; ++i) acc[i] = 0.f;
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        const int c = part + NP * r;
        const float hv = h[r];
#pragma unroll
        for (int i = 0; i < IB; ++i) {
          const float qv = sQ[(ib + i) * S::SK + c];
          const float qg = KDA ? qv * expf(sG[(ib + i) * S::SG + c]) : qv;
          acc[i] = fmaf(qg, hv, acc[i]);
        }
      }
      if (!KDA) {
#pragma unroll
        for (int i = 0; i < IB; ++i) acc[i] *= expf(sG[ib + i]);
      }
      for (int jj = part; jj < ib + IB; jj += NP) {     // P is 0 above the diagonal: jj <= i < ib + IB
        const float u = sU[jj * S::SV + x];
#pragma unroll
        for (int i = 0; i < IB; ++i) acc[i] = fmaf(sP[(ib + i) * S::SA + jj], u, acc[i]);
      }
      for (int pp = 0; pp < NP; ++pp) {
        if (part == pp) {
#pragma unroll
          for (int i = 0; i < IB; ++i) {
            // the W rows of this block were consumed by the read part above
            if (pp == 0) sW[(ib + i) * S::SW + x] = acc[i]; else sW[(ib + i) * S::SW + x] += acc[i];
          }
        }
        __syncthreads();
      }
    }
    for (int idx = tid; idx < L * DV; idx += kThreads) {
      const int i = idx / DV, c = idx % DV;
      go[((t0 + i) * p.HV + j) * DV + c] = from_f32<In>(p.scale * sW[i * S::SW + c]);
    }

    // ---- op #5 (update part): h <- e^{G_L} h + (K e^{G_L - G})^T U~
    for (int idx = tid; idx < C * DK; idx += kThreads) {
      const int i = idx / DK, c = idx % DK;
      const float e = KDA ? expf(sG[(C - 1) * S::SG + c] - sG[i * S::SG + c]) : sD[i];
      sK[i * S::SK + c] *= e;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      const int c = part + NP * r;
      float acc = h[r] * (KDA ? expf(sG[(C - 1) * S::SG + c]) : expf(sG[C - 1]));
      for (int i = 0; i < C; ++i) acc = fmaf(sK[i * S::SK + c], sU[i * S::SV + x], acc);
      h[r] = acc;
    }
    __syncthreads();
  }

  if (p.hT) {
    const size_t base = ((size_t)n * p.HV + j) * DK * DV;
#pragma unroll
    for (int r = 0; r < RPT; ++r) p.hT[base + (size_t)(part + NP * r) * DV + x] = h[r];
  }
}

template <typename In, int DK, int DV, bool KDA>
cudaError_t launch_one(const SimtParams& sp, int grid, cudaStream_t stream) {
  auto kern = simt_prefill_kernel<In, DK, DV, KDA>;
  constexpr size_t bytes = SimtSmem<DK, DV, KDA>::bytes;
  static_assert(bytes <= 227 * 1024, "shared memory budget");
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  timer_mark(stream, "simt_prefill");
  kern<<<grid, kThreads, bytes, stream>>>(sp);
  return cudaGetLastError();
}

template <typename In, bool KDA>
cudaError_t launch_dims(const Problem& p, const SimtParams& sp, int grid, cudaStream_t stream) {
  if (p.dk == 128 && p.dv == 128) return launch_one<In, 128, 128, KDA>(sp, grid, stream);
  if (p.dk == 64 && p.dv == 64) return launch_one<In, 64, 64, KDA>(sp, grid, stream);
  return cudaErrorInvalidValue;
}

SimtParams make_params(const Problem& p, const ha_la_prefill_args& a, PlanView plan) {
  SimtParams sp;
  sp.q = a.q; sp.k = a.k; sp.v = a.v; sp.g = a.g; sp.beta = a.beta; sp.h0 = a.h0;
  sp.o = a.o; sp.hT = a.hT;
  sp.seq_tok0 = plan.seq_tok0; sp.seq_len = plan.seq_len;
  sp.HK = p.HK; sp.HV = p.HV; sp.scale = p.scale;
  return sp;
}

}  // namespace

// The kernel instantiations are spread over translation units (HA_LA_SIMT_UNIT = 0..3, one per
// dtype x variant) so that they compile in parallel; unit 4 holds the dispatcher.
#ifndef HA_LA_SIMT_UNIT
#error "compile with -DHA_LA_SIMT_UNIT=0..4"
#endif

#define HA_LA_SIMT_DEFINE(NAME, IN, KDA)                                                              \
  cudaError_t NAME(const Problem& p, const ha_la_prefill_args& a, PlanView plan, cudaStream_t stream) { \
    return launch_dims<IN, KDA>(p, make_params(p, a, plan), p.N * p.HV, stream);                      \
  }

#if HA_LA_SIMT_UNIT == 0
HA_LA_SIMT_DEFINE(simt_bf16_gdn, __nv_bfloat16, false)
#elif HA_LA_SIMT_UNIT == 1
HA_LA_SIMT_DEFINE(simt_bf16_kda, __nv_bfloat16, true)
#elif HA_LA_SIMT_UNIT == 2
HA_LA_SIMT_DEFINE(simt_f32_gdn, float, false)
#elif HA_LA_SIMT_UNIT == 3
HA_LA_SIMT_DEFINE(simt_f32_kda, float, true)
#else
cudaError_t simt_bf16_gdn(const Problem&, const ha_la_prefill_args&, PlanView, cudaStream_t);
cudaError_t simt_bf16_kda(const Problem&, const ha_la_prefill_args&, PlanView, cudaStream_t);
cudaError_t simt_f32_gdn(const Problem&, const ha_la_prefill_args&, PlanView, cudaStream_t);
cudaError_t simt_f32_kda(const Problem&, const ha_la_prefill_args&, PlanView, cudaStream_t);

bool simt_supported(const Problem& p) { return p.dk == p.dv && (p.dk == 64 || p.dk == 128); }

cudaError_t launch_simt(const Problem& p, const ha_la_prefill_args& a, PlanView plan, cudaStream_t stream) {
  if (p.N * p.HV == 0) return cudaSuccess;
  const bool kda = p.variant == HA_LA_KDA;
  if (p.dtype == HA_LA_BF16) return kda ? simt_bf16_kda(p, a, plan, stream) : simt_bf16_gdn(p, a, plan, stream);
  return kda ? simt_f32_kda(p, a, plan, stream) : simt_f32_gdn(p, a, plan, stream);
}
#endif

}  // namespace ha_la
