// Internal declarations shared by the translation units of libgdn (not installed).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "gdn.h"

namespace gdn {

constexpr int kChunk = 64;

// One prefill call, device pointers.  io_bf16 selects the storage type of q/k/v/out.
struct PrefillArgs {
    const void* q;
    const void* k;
    const void* v;
    const float* log_alpha;
    const float* beta;
    const float* initial_state;
    void* out;
    float* final_state;
    const int32_t* cu_seqlens;
    int B, T, H, d_k, d_v;
};

// fp32-arithmetic kernel (plain FMA); TIO = float or __nv_bfloat16 storage.
int launch_simt(const PrefillArgs& a, bool io_bf16, cudaStream_t stream);
bool simt_supported(int d_k, int d_v);

// Tensor-core (tcgen05) kernel for bf16 storage.
int launch_tc(const PrefillArgs& a, cudaStream_t stream);
bool tc_supported(int d_k, int d_v);
int tc_query_status();               // synchronises the device, returns the kernels' status word
// Enqueue, on `stream`, the copy of one translation unit's status word to *host_dst (read it after the stream
// has been synchronised).
int tc_status_async(int* host_dst, cudaStream_t stream);
int lean_status_async(int* host_dst, cudaStream_t stream);
int attn_status_async(int* host_dst, cudaStream_t stream);
void tc_set_debug_dump(float* p);    // tests only: stage dump of chunk 0 of CTA (0,0,0)

// [tokens, H, d] bf16 tensor map, box = 64 tokens x 1 head x 64 features, 128-byte swizzle
bool tc_make_map(CUtensorMap* map, const void* ptr, uint64_t tokens, uint64_t H, uint64_t d);

// Two-kernel pipeline (prepare on all SMs, then the chain) using caller-provided scratch.
size_t lean_workspace_bytes(int B, int T, int H, int d_k, int d_v, bool packed);
int lean_init_workspace(void* workspace);   // zeroes the header of a newly provided workspace (synchronous)
struct LeanOptions {
    float* snaps = nullptr;    // optional (batched input only): [B, (T/64)/snap_every, H, d_k, d_v], the state
    int snap_every = 1;        //   after every snap_every chunks
    bool raw = false;          // q, k are raw projections and log_alpha, beta pre-activations: the prepare
    float gate_scale = 1.f;    //   kernel L2-normalises q, k and applies -softplus(.) * gate_scale and sigmoid(.)
    float eps = 0.f;           //   (eps under the square root of the norms)
    // fused output stage (d_v = 128): out = o / sqrt(mean o^2 + norm_eps) * norm_w * silu(gate_z); nullptr = plain output
    const __nv_bfloat16* gate_z = nullptr;
    const float* norm_w = nullptr;
    float norm_eps = 0.f;
};
int launch_lean(const PrefillArgs& a, void* workspace, size_t workspace_bytes, cudaStream_t stream,
                const LeanOptions& opt = LeanOptions());
int launch_lean_static(const PrefillArgs& a, cudaStream_t stream);   // built-in scratch, allocates nothing
int lean_query_status();
void lean_force_segments(int nseg);   // tests only: 0 = automatic plan
void lean_set_drop_chunk(int c);      // tests only: make one TMA load never happen (bounded waits expire)
int lean_reset_status();              // tests only: clear the status word
void lean_set_debug(float* p);        // tests only: time stamps of the chain kernel
int lean_set_timing(int enable);      // benchmark only: record events around each kernel
int lean_get_timing(float* ms5);      // {prepare, summary, combine, chain, scan} of the last call
void lean_set_l2_hints(int enable);   // tests only: 0 = no L2 eviction-priority hints
void lean_set_scan(int enable);       // tests only: 0 = never merge summary, combine and chain into one launch

// Single-token decode step (bf16 q/k/v/out, fp32 state updated in place).
bool decode_supported(int d_k, int d_v);
int launch_decode(const void* q, const void* k, const void* v, const float* log_alpha, const float* beta,
                  float* state, void* out, int B, int H, int d_k, int d_v, cudaStream_t stream);

// Causal grouped-query softmax attention (bf16, d = 128).
bool attn_supported(int Hq, int Hkv, int d);
int launch_attn(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens, int B, int T,
                int Hq, int Hkv, int d, float scale, cudaStream_t stream);
int attn_query_status();

void count_launch(int n = 1);

}  // namespace gdn
