/*
 * gdn.h -- C ABI of the B200 (sm_100a) chunked gated delta-rule prefill library.
 *
 * The operation.  For every sequence n and head h (all independent), with a
 * recurrent state S in R^{d_k x d_v} per head (Section "The model": state
 * S in R^{H_k x H_v} per value head, updated token by token) the library
 * evaluates the gated delta-net recurrence of Section "A chunked delta-rule scan
 * for the recurrent layers", S_t = diag(gamma_t) S_{t-1} + k_t delta_t^T, read as
 *
 *     S      <- exp(log_alpha_t) * S                 (scalar gate per token, head)
 *     delta  <- beta_t * (v_t - S^T k_t)             (against the decayed state)
 *     S      <- S + k_t delta^T
 *     out_t  <- S^T q_t                              (updated state, no 1/sqrt(d_k))
 *
 * over a whole prompt, using the intra-/inter-chunk form of that section: per
 * 64-token chunk a cumulative log gate, the decay-masked token-token matrices,
 * a forward substitution of the unit lower triangular system, the WY factors,
 * and a short recurrence over chunks that carries the state.  The result does
 * not depend on the chunk size; `chunk` names the internal tiling and only 64
 * is supported.
 *
 * Layouts (row-major, last index fastest; every pointer is a DEVICE pointer
 * unless its name ends in _host, and must be 16-byte aligned):
 *     q, k                       [B, T, H, d_k]
 *     v, out                     [B, T, H, d_v]
 *     log_alpha, beta            [B, T, H]            fp32
 *     initial_state, final_state [B, H, d_k, d_v]     fp32
 * With cu_seqlens != NULL the tensors are packed [T, H, .] where T is the total
 * number of tokens, B is the number of sequences and sequence n owns tokens
 * [cu_seqlens[n], cu_seqlens[n+1]); cu_seqlens has B+1 int32 entries,
 * cu_seqlens[0] = 0, cu_seqlens[B] = T.  A sequence of length 0 passes its
 * state through.  initial_state == NULL means zeros; final_state == NULL means
 * "do not return it".  final_state may alias initial_state; no other input may
 * alias an output.
 *
 * Ownership and execution.  The caller owns every buffer.  The calls enqueue
 * work on `stream` and return without synchronising; they allocate no device
 * memory.  All functions return a gdn_status (0 = success) and never abort.
 * Nothing is launched when a non-zero status is returned for an argument error.
 */
#ifndef GDN_H_
#define GDN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GDN_OK = 0,
    GDN_ERR_INVALID_ARG = 1,  /* NULL required pointer, non-positive size, bad cu_seqlens_host */
    GDN_ERR_UNSUPPORTED = 2,  /* chunk != 64, unsupported (d_k, d_v), misaligned pointer */
    GDN_ERR_WORKSPACE = 3,    /* caller-provided scratch too small */
    GDN_ERR_CUDA = 4,         /* a CUDA runtime/driver call or a launch failed */
    GDN_ERR_TIMEOUT = 5,      /* a bounded device-side wait expired (see gdn_query_status) */
    GDN_ERR_TOO_LARGE = 6     /* problem exceeds the built-in scratch of gdn_chunk_prefill_noalloc */
} gdn_status;

/* Same handle as cudaStream_t / CUstream (NULL = the default stream). */
typedef struct CUstream_st* gdn_stream_t;

/*
 * The chunked prefill, bf16 q/k/v/out, fp32 gates and state (the main entry
 * point; steps: cumulative gate, decay-masked KK^T and QK^T, forward
 * substitution, WY factors, inter-chunk state recurrence, output -- Section "A
 * chunked delta-rule scan for the recurrent layers").  Supported: chunk = 64,
 * d_k = 128, d_v a multiple of 128 (tensor-core path); other d_k, d_v that are
 * multiples of 32 with d_k <= 128 fall back to the fp32-arithmetic kernel below.
 * The call makes no host-device copy and no synchronisation, so it can be
 * recorded into a CUDA graph and replayed on new contents of the same buffers
 * (set the workspace before the capture: gdn_set_workspace synchronises).
 */
int gdn_chunk_prefill(const void* q, const void* k, const void* v,
                      const float* log_alpha, const float* beta,
                      const float* initial_state,
                      void* out, float* final_state,
                      const int32_t* cu_seqlens,
                      int B, int T, int H, int d_k, int d_v, int chunk,
                      gdn_stream_t stream);

/*
 * Same operation and argument list with fp32 q/k/v/out and fp32 arithmetic
 * throughout (plain FMA kernels; the paper's own precision, Section "A chunked
 * delta-rule scan for the recurrent layers").  Supported: chunk = 64, d_k and d_v
 * multiples of 32, d_k <= 128.
 */
int gdn_chunk_prefill_f32(const float* q, const float* k, const float* v,
                          const float* log_alpha, const float* beta,
                          const float* initial_state,
                          float* out, float* final_state,
                          const int32_t* cu_seqlens,
                          int B, int T, int H, int d_k, int d_v, int chunk,
                          gdn_stream_t stream);

/*
 * bf16 q/k/v/out through the fp32-arithmetic kernel (inputs widened exactly, fp32
 * everywhere inside, one rounding at the output).  A slow cross-check of the
 * tensor-core path with the same chunked algorithm; same support as the f32 call.
 */
int gdn_chunk_prefill_bf16_simt(const void* q, const void* k, const void* v,
                                const float* log_alpha, const float* beta,
                                const float* initial_state,
                                void* out, float* final_state,
                                const int32_t* cu_seqlens,
                                int B, int T, int H, int d_k, int d_v, int chunk,
                                gdn_stream_t stream);

/*
 * The bf16 prefill with HOST buffers: copies the inputs to the device staging
 * area (cudaMemcpyAsync on `stream`; pinned host memory keeps it asynchronous),
 * runs gdn_chunk_prefill there and copies out/final_state back, all on `stream`,
 * without synchronising.  staging_dev is caller-owned device memory of at least
 * gdn_host_staging_bytes(...) bytes, 256-byte aligned.  cu_seqlens_host may be
 * NULL; initial_state_host / final_state_host may be NULL as above.
 * One long sequence (B = 1, no cu_seqlens, T >= 4096, d_k = 128) is processed in
 * pieces of 2048 tokens with the fp32 state carried from piece to piece: uploads,
 * kernels and downloads of different pieces overlap on two copy streams that the
 * library creates once (with their events; nothing else is ever allocated).  The
 * call is still complete on `stream` when everything has reached the host.
 * Errors: as gdn_chunk_prefill, plus GDN_ERR_WORKSPACE when staging is too small.
 */
int gdn_chunk_prefill_host(const void* q_host, const void* k_host, const void* v_host,
                           const float* log_alpha_host, const float* beta_host,
                           const float* initial_state_host,
                           void* out_host, float* final_state_host,
                           const int32_t* cu_seqlens_host,
                           int B, int T, int H, int d_k, int d_v, int chunk,
                           void* staging_dev, size_t staging_bytes,
                           gdn_stream_t stream);

/* Bytes of device staging gdn_chunk_prefill_host needs for these sizes (0 on bad sizes). */
size_t gdn_host_staging_bytes(int B, int T, int H, int d_k, int d_v);

/*
 * One decode step: the same recurrence for a single new token per sequence, continuing from
 * the state a prefill returned (Section "The model": the state advances by one token at a time;
 * Section "Decode, and why 4-bit is slower": decode is bandwidth-bound -- here the state is
 * read once and written once).  q, k [B, H, d_k] and v, out [B, H, d_v] are bf16; log_alpha,
 * beta [B, H] fp32; state [B, H, d_k, d_v] fp32 is updated IN PLACE (it is both the incoming
 * and the outgoing state).  Supported: d_k a multiple of 8 up to 128, d_v a multiple of 128.
 * Errors as gdn_chunk_prefill; asynchronous on `stream`; allocates nothing.
 */
int gdn_decode_step(const void* q, const void* k, const void* v,
                    const float* log_alpha, const float* beta,
                    float* state, void* out,
                    int B, int H, int d_k, int d_v,
                    gdn_stream_t stream);

/*
 * gdn_chunk_prefill that also returns the recurrent state at chunk boundaries: the material of a
 * position-indexed prefix-snapshot cache (Section "An All-GPU Engine for the Hybrid Backbone": the
 * serving process keeps snapshots of the recurrent state by position).  Batched input only (no
 * cu_seqlens).  snapshots is [B, n_snap, H, d_k, d_v] fp32 with n_snap = (T / 64) /
 * snapshot_every_chunks; entry i holds the state after token (i + 1) * snapshot_every_chunks * 64
 * of each sequence -- exactly what initial_state must be to resume the prefill there.  Needs the
 * scratch of gdn_set_workspace (GDN_ERR_WORKSPACE without it); other arguments, support and
 * errors as gdn_chunk_prefill with d_k = 128, d_v a multiple of 128.
 */
int gdn_chunk_prefill_snapshots(const void* q, const void* k, const void* v,
                                const float* log_alpha, const float* beta,
                                const float* initial_state,
                                void* out, float* final_state,
                                int B, int T, int H, int d_k, int d_v, int chunk,
                                int snapshot_every_chunks, float* snapshots,
                                gdn_stream_t stream);

/*
 * gdn_chunk_prefill with the per-position prologue fused in (Section "Prefill projections: dequantize, then call the vendor": the norms
 * and gating around the projections are batched over the chunk).  q_raw, k_raw are the raw bf16
 * projections and a_raw, b_raw the fp32 gate pre-activations, same shapes as q, k, log_alpha, beta
 * of gdn_chunk_prefill.  The call computes, per (token, head),
 *   q = q_raw / sqrt(sum_f q_raw_f^2 + norm_eps)      k likewise
 *   beta = 1 / (1 + e^{-b_raw})                        log_alpha = -ln(1 + e^{a_raw}) * gate_scale
 * and then the prefill of gdn_chunk_prefill on them; the normalised q, k are never written to
 * memory (the inverse norms are folded into the masks and gate vectors in fp32, so they see the
 * unrounded norm).  The paper names these kernels without printing formulas; these are the forms
 * the benchmark inputs are drawn with.  A row whose sum of squares plus norm_eps is zero counts
 * as a zero vector.  gate_scale >= 0, norm_eps >= 0 (else GDN_ERR_INVALID_ARG).  Needs the
 * scratch of gdn_set_workspace (GDN_ERR_WORKSPACE without it); other arguments, support and
 * errors as gdn_chunk_prefill with d_k = 128, d_v a multiple of 128.
 */
int gdn_chunk_prefill_raw(const void* q_raw, const void* k_raw, const void* v,
                          const float* a_raw, const float* b_raw,
                          float gate_scale, float norm_eps,
                          const float* initial_state,
                          void* out, float* final_state,
                          const int32_t* cu_seqlens,
                          int B, int T, int H, int d_k, int d_v, int chunk,
                          gdn_stream_t stream);

/*
 * gdn_chunk_prefill with the per-position output stage fused in (Section "Prefill projections:
 * dequantize, then call the vendor" names the norms and the gating that surround the scan among the
 * kernels batched over the chunk; the paper prints no formula, this library takes the gated
 * root-mean-square norm).  Per (token, head), with o the row gdn_chunk_prefill would return,
 *   out_j = o_j / sqrt(mean_j' o_j'^2 + norm_eps) * norm_weight_j * silu(gate_z_j),  silu(z) = z / (1 + e^{-z})
 * gate_z is bf16 with the shape of out, norm_weight is fp32 [d_v] (shared by all heads), norm_eps >= 0.
 * The norm is taken on the fp32 rows before they are rounded, inside the kernel that produces them, so
 * the un-normalised output is never written.  Supported: d_k = d_v = 128, chunk = 64.  Needs the scratch of
 * gdn_set_workspace (GDN_ERR_WORKSPACE without it).  final_state is the same as without the output stage.
 * Errors: as gdn_chunk_prefill; GDN_ERR_INVALID_ARG for a NULL gate_z or norm_weight or a negative norm_eps.
 */
int gdn_chunk_prefill_gated(const void* q, const void* k, const void* v,
                            const float* log_alpha, const float* beta,
                            const float* initial_state,
                            const void* gate_z, const float* norm_weight, float norm_eps,
                            void* out, float* final_state,
                            const int32_t* cu_seqlens,
                            int B, int T, int H, int d_k, int d_v, int chunk,
                            gdn_stream_t stream);

/*
 * Optional scratch memory.  Without it gdn_chunk_prefill runs one fused kernel per call in
 * which each (sequence, head) chain also does its own forward substitutions.  With scratch of
 * at least gdn_workspace_bytes(...) bytes the state-independent steps (cumulative gate,
 * token-token matrices, forward substitution, WY factor W) run first as a kernel over every
 * (chunk, head) on all SMs -- every position of a chunk is resolved at once, Section "A chunked
 * delta-rule scan for the recurrent layers" -- and leave their results in the scratch for the
 * chain kernel; this is the faster path.  The scratch stays owned by the caller, is 256-byte
 * aligned device memory, must outlive every call that uses it, and is shared by all calls
 * (calls on different streams must not overlap).  The scratch belongs to the device that is current
 * when gdn_set_workspace is called: every device has its own, and a call uses the one of the device
 * current at that call.  gdn_set_workspace zeroes the first 4096 bytes with a synchronous cudaMemset
 * (work counters that every call leaves at zero again; the caller must not write there between calls;
 * after a call that reported GDN_ERR_TIMEOUT set the workspace again before reusing it) and returns GDN_ERR_CUDA if that fails; a pointer that is
 * not 256-byte aligned gives GDN_ERR_UNSUPPORTED.  gdn_set_workspace(NULL, 0) removes it.
 * `packed` is 1 when cu_seqlens will be passed (T = total tokens), else 0.
 * gdn_workspace_bytes returns 0 for sizes the tensor-core path does not support (chunk other than 64 included).
 */
size_t gdn_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int packed);
int gdn_set_workspace(void* device_ptr, size_t bytes);

/*
 * gdn_chunk_prefill for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for how the library is embedded.)
 *
 * Who needs it: an operator that a host framework calls with nothing but its input and
 * output buffers has no allocator to turn to, and a serving process that carved up the
 * whole GPU into its own pools at start-up has nothing left to request.  Neither can hand
 * gdn_set_workspace a scratch buffer, and neither may have cudaMalloc called on its behalf.
 * This call needs none: it runs the two-kernel pipeline (prepare kernel, then chain kernel,
 * without the sequence split) on a scratch area of 64 MiB that is built into the library
 * image -- every GPU that loads the library carries those 64 MiB until the process ends.
 * It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Same arguments, layouts, support (d_k = 128, d_v a multiple of 128, chunk = 64) and
 * results as gdn_chunk_prefill.  Limit: (tokens / 64 + B) * H * 34048 bytes must not exceed
 * 64 MiB, tokens being T when cu_seqlens is given and B * T otherwise (for H = 16 that is
 * about 7800 tokens); beyond it the call launches nothing and returns GDN_ERR_TOO_LARGE.
 *
 * The first call made while a given device is current also looks up the device address of
 * the built-in scratch and sets kernel attributes for that device; make that first call
 * outside any stream capture.  All calls share the one scratch area and find in it what
 * the previous call left (nothing in it needs to be zero: each call overwrites every part
 * it later reads).  Calls that overlap on the GPU -- different streams, or different host
 * threads -- race on it; issue them one after another on one stream.
 */
int gdn_chunk_prefill_noalloc(const void* q, const void* k, const void* v,
                              const float* log_alpha, const float* beta,
                              const float* initial_state,
                              void* out, float* final_state,
                              const int32_t* cu_seqlens,
                              int B, int T, int H, int d_k, int d_v, int chunk,
                              gdn_stream_t stream);

/*
 * Waits for the device to finish (cudaDeviceSynchronize) and returns the status word of
 * the kernels: GDN_OK, or GDN_ERR_TIMEOUT if a bounded device-side wait (on a TMA copy,
 * a tensor-core completion or another warp role) ever expired, in which case the outputs
 * of that call are undefined.  GDN_ERR_CUDA if the device reports an error.
 */
int gdn_query_status(void);

/*
 * The same status, but waiting only for `stream` (cudaStreamSynchronize): everything enqueued on that
 * stream before this call has finished when it returns, other streams of the device keep running.  The
 * status word is shared by all streams of a device, so a time-out raised by a call on another stream that
 * has already run shows up here too.  (Failure reporting of the bounded device-side waits; the paper's
 * engine has no counterpart.)
 */
int gdn_query_status_stream(gdn_stream_t stream);

/* Number of kernels this library has launched in this process so far. */
unsigned long long gdn_launch_count(void);

/* Static description of a status code. */
const char* gdn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GDN_H_ */
