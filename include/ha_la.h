/*
 * ha_la.h -- C ABI of the B200 (sm_100a) delta-rule linear-attention prefill library.
 *
 * One operation: the chunkwise-parallel prefill of a Gated DeltaNet (GDN) layer
 * (scalar log-gate per head per token) or its Kimi-Delta-Attention (KDA)
 * variant (log-gate per key channel).
 *
 * Paper passages that define the operation:
 *   - Section 2.1, "Architecture of Linear-Attention Hybrids": a fixed-size
 *     recurrent state per head; at step t the previous state is updated with
 *     K_t, V_t and the output is formed from Q_t and the UPDATED state.
 *   - Section 2.1, "Chunkwise Map-Reduce-Map Execution": operators #1 Gate,
 *     #2 KKT, #3 Solve, #4 W/U (Map), #5 H (Reduce, sequential per head),
 *     #6 O (Map).  Chunk length 64 (Section "Experimental setup").
 *   - Section "HA-NPU overview": inputs are Q/K/V, gates and the initial state;
 *     outputs are the attention outputs and the updated state.
 *   - Precisions (Section "Experimental setup"): 16-bit Q/K/V, FP32 gates and states.
 *
 * Result, per sequence and V-head j (QK-head jq = j / (HV/HK)), with the state
 * h of shape d_k x d_v starting at h0 (or zero), for each token t in order:
 *     GDN:  h <- exp(g[t,j]) h            KDA:  h[c,:] <- exp(g[t,j,c]) h[c,:]
 *     h <- h + beta[t,j] k[t,jq] (v[t,j] - h^T k[t,jq])^T
 *     o[t,j] = scale * h^T q[t,jq]
 * and hT = h after the last token.  The library evaluates this chunk by chunk
 * (chunk = 64); the result does not depend on the chunking beyond rounding.
 *
 * Conventions
 *   - Every pointer in ha_la_prefill_args is a DEVICE pointer owned by the
 *     caller, valid until the work enqueued on the stream has finished.
 *   - ha_la_prefill enqueues kernels on the given CUDA stream and returns
 *     without synchronising.  It allocates no device memory and keeps no
 *     pointer after it returns; the args struct is read during the call only.
 *   - Stream order holds as for any kernel: the call sees what earlier work on the
 *     stream wrote, later work sees its outputs.  The tensor-core kernels use
 *     programmatic dependent launch among themselves and let the stream's next
 *     kernel be scheduled shortly before they end; that only concerns a following
 *     kernel launched with the programmatic-serialization attribute, which -- as
 *     CUDA requires of such kernels -- waits for its grid dependency before it
 *     touches anything this call reads or writes.
 *   - ha_la_prefill and ha_la_decode may be captured into a CUDA graph by stream
 *     capture and replayed on new contents of the same buffers; pointers, sizes
 *     and the launch plan are frozen at capture.  (ha_la_prefill_timed blocks and
 *     cannot be captured.)
 *   - Every entry point returns an ha_la_status; nothing throws or aborts.
 *   - Problems found on the device (a wait that ran out, an index out of
 *     range) are written as a non-zero code to *status_word, which the caller
 *     reads after its own synchronisation; the kernels then finish normally
 *     with unspecified outputs.
 *   - o must not overlap any input.  hT may be exactly the pointer h0
 *     (in-place state update) and must not partially overlap it.
 *   - The workspace is scratch for ONE call at a time: its contents on entry do
 *     not matter and nothing in it needs clearing, but calls that may overlap on
 *     the GPU (different streams without an ordering) need a workspace each.
 *   - Sequence lengths need not be multiples of 64; length-0 sequences are
 *     legal (hT = h0).
 *
 * What the inputs must satisfy
 *   - Every value is finite.  Log-gates are <= 0 (the kernels evaluate decays only
 *     as exp of non-positive numbers; a positive log-gate gives unspecified results).
 *   - d_k == d_v (64 or 128).
 *   - The tensor-core path (bf16, d = 128) holds (I + A)^-1 of operator #3 in fp16
 *     between the levels of its blocked solve.  That is exact enough whenever
 *     beta |k|^2 stays within the delta rule's own stability range (<= 2; keys of
 *     norm 0.5 .. 2 are tested).  Inputs far outside it can overflow the fp16 range;
 *     the kernel detects that and reports HA_LA_ERR_DEVICE_CHECK through status_word
 *     instead of returning wrong numbers silently.
 *
 * Environment switches (test hooks, read by the host launch code; they change how the
 * work is launched, never the result): HA_LA_FORCE_SIMT=1 (read once) sends every shape
 * to the fp32 CUDA-core kernel; HA_LA_TC_NV=32|64|128 fixes the slice width of the
 * sequential kernel; HA_LA_TC_OVERLAP=0|2 forbids / forces running the two tensor-core
 * kernels side by side; HA_LA_TC_SEGMENTS=1|2|4|8 fixes the number of segments a head's
 * chunk sequence is split into.  Production callers leave them unset; a caller that sets one
 * does so before it asks for the workspace size (the size follows the plan, and a call whose
 * plan needs more than it was given returns HA_LA_ERR_WORKSPACE).
 */
#ifndef HA_LA_H_
#define HA_LA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { HA_LA_GDN = 0, HA_LA_KDA = 1 } ha_la_variant;
typedef enum { HA_LA_BF16 = 0, HA_LA_FP32 = 1 } ha_la_dtype;   /* dtype of q, k, v and o */

typedef enum {
  HA_LA_OK = 0,
  HA_LA_ERR_INVALID_ARG = 1,   /* null pointer, bad size, bad enum                         */
  HA_LA_ERR_UNSUPPORTED = 2,   /* legal but not implemented (head dim, chunk, ...)         */
  HA_LA_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small               */
  HA_LA_ERR_CUDA = 4,          /* a CUDA runtime / driver call or a launch failed          */
  HA_LA_ERR_TIMEOUT = 5,       /* device side: a bounded wait ran out (status word only)   */
  HA_LA_ERR_DEVICE_CHECK = 6,  /* device side: an index or length check failed             */
  HA_LA_ERR_TOO_LARGE = 7      /* ha_la_prefill_noalloc only: problem exceeds its fixed scratch */
} ha_la_status;

typedef struct {
  int32_t variant;        /* ha_la_variant                                                   */
  int32_t dtype;          /* ha_la_dtype                                                     */
  int32_t batch;          /* B; must be 1 when cu_seqlens != NULL                            */
  int32_t seqlen;         /* T per batch row; TOTAL packed tokens when cu_seqlens != NULL    */
  int32_t num_qk_heads;   /* HK                                                              */
  int32_t num_v_heads;    /* HV, a multiple of HK; V-head j reads QK-head j / (HV/HK)        */
  int32_t d_k, d_v;       /* d_k == d_v, 64 or 128                                           */
  int32_t chunk;          /* must be 64                                                      */
  float   scale;          /* o = scale * h^T q                                               */
  const void*  q;         /* [B, T, HK, d_k] contiguous, token-major                         */
  const void*  k;         /* [B, T, HK, d_k]                                                 */
  const void*  v;         /* [B, T, HV, d_v]                                                 */
  const float* g;         /* GDN [B, T, HV]; KDA [B, T, HV, d_k] (16-byte aligned); log-gate */
  const float* beta;      /* [B, T, HV]                                                      */
  const float* h0;        /* [N, HV, d_k, d_v] fp32 or NULL (zeros); N = B or num_seqs       */
  const int32_t* cu_seqlens; /* device int32 [num_seqs+1], cu[0]=0, non-decreasing,
                                cu[num_seqs]=seqlen; or NULL for B equal-length rows        */
  int32_t num_seqs;       /* > 0 selects the packed mode and then cu_seqlens is required;
                             0 with cu_seqlens == NULL means B equal-length rows            */
  int32_t max_seqlen;     /* upper bound on any sequence length when cu_seqlens != NULL
                             (sizes the launch; a longer sequence is reported through
                             status_word as HA_LA_ERR_DEVICE_CHECK); 0 = use seqlen          */
  void*   o;              /* [B, T, HV, d_v], dtype as v                                     */
  float*  hT;             /* [N, HV, d_k, d_v] fp32 or NULL (not wanted)                     */
  void*   workspace;      /* >= ha_la_prefill_workspace_bytes(), 256-byte aligned            */
  size_t  workspace_bytes;
  int32_t* status_word;   /* optional device int32; the caller zeroes it before the call     */
} ha_la_prefill_args;

/* Host only: bytes of scratch ha_la_prefill needs for these shapes (pointers are ignored).
 * Returns HA_LA_OK and writes *out_bytes, or an error for invalid / unsupported shapes.     */
int ha_la_prefill_workspace_bytes(const ha_la_prefill_args* args, size_t* out_bytes);

/* Enqueue the prefill on `cuda_stream` (a cudaStream_t; NULL = the default stream).
 * Implements operators #1-#6 of "Chunkwise Map-Reduce-Map Execution" (Section 2.1) for
 * every sequence and V-head.  Asynchronous; see the conventions above.                     */
int ha_la_prefill(const ha_la_prefill_args* args, void* cuda_stream);

/* Name of the implementation ha_la_prefill would run for these shapes ("tc" = tcgen05
 * tensor-core kernels, "simt" = fp32 CUDA-core kernel), or NULL if unsupported.  Host only. */
const char* ha_la_prefill_path(const ha_la_prefill_args* args);

/* Number of kernels ha_la_prefill launches for these shapes (0 if unsupported).  Host only. */
int ha_la_prefill_num_launches(const ha_la_prefill_args* args);

/* How ha_la_prefill would launch the tensor-core kernels for these shapes (host only; pointers are
 * ignored).  *slice_width = value channels per CTA of the sequential (state-passing) kernel: 32, 64 or
 * 128 -- the "Computation Splitting" paragraph of Section 4: a head's state split into column sub-heads --
 * or 0 on the CUDA-core path; *concurrent = 1 if that kernel runs beside the chunk-local kernel and
 * takes each chunk as it is published, 0 if the two run back to back.  The choice comes from measured
 * per-chunk costs of the two kernels and the bounds in `args` (sequences, longest sequence, total
 * tokens); the environment switches HA_LA_TC_NV and HA_LA_TC_OVERLAP override it.
 * Returns HA_LA_OK, or an error for invalid / unsupported shapes or NULL outputs.               */
int ha_la_prefill_launch_plan(const ha_la_prefill_args* args, int* slice_width, int* concurrent);

/* Segments per sequence ha_la_prefill would use for these shapes (host only; 1 = the chunks of a sequence are
 * walked strictly in order; 0 if the shapes are unsupported).  With S > 1 a sequence's chunks are cut into S
 * runs that are walked at the same time -- the Chunk-Seg-Seg mapping the paper describes for its FlashQLA
 * baseline (Section "Head-Level Mapping with Cross-Operator Fusion"): later segments start from a zero state and from the identity, and their true start
 * states, final state and outputs follow from one affine fix-up per segment.  Chosen only for equal-length rows
 * with so few (sequence, head) pairs that every run still gets an SM; HA_LA_TC_SEGMENTS overrides it.            */
int ha_la_prefill_num_segments(const ha_la_prefill_args* args);

/* Profiling aid (the paper's "Metrics" paragraph times kernels with device events): the same work
 * as ha_la_prefill, with a CUDA event recorded on `cuda_stream` before every kernel and after the
 * last one.  Unlike ha_la_prefill it BLOCKS until the stream has drained, then writes the device
 * time of each kernel in launch order to ms_out[0..n) (milliseconds), a static name for each to
 * names_out (may be NULL) and n to *num_kernels_out (n <= max_kernels <= 8).                       */
int ha_la_prefill_timed(const ha_la_prefill_args* args, void* cuda_stream, int max_kernels, float* ms_out,
                        const char** names_out, int* num_kernels_out);

/* Prefill without a workspace, for callers that cannot allocate device memory or hand scratch to
 * this library (an operator hook that must stay out of its framework's allocator, a runtime whose
 * memory pool is frozen, a plug-in that only sees the operator's own tensors).  The paper has no
 * counterpart of this entry point; it computes exactly what ha_la_prefill computes.
 *
 *   - args->workspace and args->workspace_bytes are ignored.  The chunk table lives in a fixed
 *     array inside the library image (ha_la_prefill_noalloc_scratch_bytes() bytes, 209 KiB),
 *     which every GPU that loads the library holds until the process exits.
 *   - Limits: at most 1024 sequences (batch rows or packed sequences) and at most 16384 chunk
 *     slots ((seqlen + 63 * num_seqs) / 64 in packed mode, batch * ceil(seqlen / 64) otherwise);
 *     beyond that it returns HA_LA_ERR_TOO_LARGE and launches nothing.
 *   - It always runs the fp32 CUDA-core kernels (the tensor-core path needs megabytes of scratch),
 *     so it is meant for small and medium problems; results agree with ha_la_prefill within the
 *     library's tolerances.
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.  Its FIRST call on a
 *     device looks up the array's device address (cudaGetSymbolAddress, with that device current)
 *     and caches it; make that first call outside any stream capture.  The cached address belongs
 *     to the device's primary context: it does not survive cudaDeviceReset, and a context other
 *     than the primary one on the same device ordinal must not use this entry point.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (each call
 *     rewrites every entry it later reads), but two calls that overlap on the GPU -- different
 *     streams without an ordering between them -- race on it: serialise them.                     */
int ha_la_prefill_noalloc(const ha_la_prefill_args* args, void* cuda_stream);
size_t ha_la_prefill_noalloc_scratch_bytes(void);

/* One decoding step of the same layer: ONE new token per sequence, the recurrent state kept by the
 * caller between calls.  In the paper the prefill's online stage returns the updated state so that
 * later layers and the decoder can carry on from it (Section "HA-NPU overview"), and the decoding
 * step itself is left to the framework's native backend; this entry point is that step for the state
 * layout ha_la_prefill produces (hT), so that prefill and decode share one library.
 *
 * For every sequence n and V-head j (QK-head jq = j / (HV/HK)), with h = h_in[n,j] (zeros if NULL):
 *     GDN:  h <- exp(g[n,j]) h            KDA:  h[c,:] <- exp(g[n,j,c]) h[c,:]
 *     h <- h + beta[n,j] k[n,jq] (v[n,j] - h^T k[n,jq])^T
 *     o[n,j] = scale * h^T q[n,jq]         h_out[n,j] = h
 * All arithmetic is fp32.  Device pointers, asynchronous on the stream, no workspace, no allocation.
 * q, k, v, o, h_in, h_out 16-byte aligned; h_out may be exactly h_in (in place) and must not
 * partially overlap it; o must not overlap any input.                                             */
typedef struct {
  int32_t variant;        /* ha_la_variant                                                   */
  int32_t dtype;          /* ha_la_dtype of q, k, v and o                                    */
  int32_t num_seqs;       /* N >= 0: sequences, one token each                               */
  int32_t num_qk_heads;   /* HK                                                              */
  int32_t num_v_heads;    /* HV, a multiple of HK                                            */
  int32_t d_k, d_v;       /* d_k == d_v, 64 or 128                                           */
  float   scale;
  const void*  q;         /* [N, HK, d_k]                                                    */
  const void*  k;         /* [N, HK, d_k]                                                    */
  const void*  v;         /* [N, HV, d_v]                                                    */
  const float* g;         /* GDN [N, HV]; KDA [N, HV, d_k]; log-gate                         */
  const float* beta;      /* [N, HV]                                                         */
  const float* h_in;      /* [N, HV, d_k, d_v] fp32 or NULL (zeros)                          */
  float*       h_out;     /* [N, HV, d_k, d_v] fp32                                          */
  void*        o;         /* [N, HV, d_v], dtype as v                                        */
} ha_la_decode_args;

/* Enqueue one decoding step on `cuda_stream`.  Returns HA_LA_OK or an error code; launches one
 * kernel (none when N == 0).                                                                      */
int ha_la_decode(const ha_la_decode_args* args, void* cuda_stream);

/* Test hook for the device-side bounded waits (the paper has no counterpart).  Every wait inside the
 * kernels -- on an mbarrier, on another kernel's "chunk is ready" flag -- gives up after a fixed number
 * of polls, records HA_LA_ERR_TIMEOUT in *status_word and lets the kernel run to a normal exit with
 * unspecified outputs.  This call makes such a wait run out on purpose, without faulting or hanging
 * anything: it enqueues ONLY the sequential (state-passing) kernel, in the mode in which it waits per
 * chunk for the chunk-local kernel's flags, with a flag value that nothing publishes and `spin_limit`
 * (1 .. 2^20) polls per wait.  Arguments as for ha_la_prefill (bf16, d = 128, equal-length rows,
 * status_word required); o and hT receive meaningless numbers.  Returns HA_LA_OK once enqueued.       */
int ha_la_debug_wait_timeout(const ha_la_prefill_args* args, void* cuda_stream, unsigned int spin_limit);

const char* ha_la_status_string(int status);
int ha_la_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HA_LA_H_ */
