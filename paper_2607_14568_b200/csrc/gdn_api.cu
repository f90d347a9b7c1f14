// C-ABI entry points of libgdn: argument validation and dispatch.  See include/gdn.h.

#include <atomic>
#include <mutex>
#include <vector>

#include "gdn_internal.h"
#include "gdn_attn.h"

namespace gdn {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks shared by every prefill entry point.  Returns GDN_OK or the error to report.
int validate(const PrefillArgs& a, int chunk) {
    if (!a.q || !a.k || !a.v || !a.log_alpha || !a.beta || !a.out) return GDN_ERR_INVALID_ARG;
    if (a.B <= 0 || a.T < 0 || a.H <= 0 || a.d_k <= 0 || a.d_v <= 0) return GDN_ERR_INVALID_ARG;
    if (chunk != kChunk) return GDN_ERR_UNSUPPORTED;
    const void* ptrs[] = {a.q, a.k, a.v, a.log_alpha, a.beta, a.initial_state, a.out, a.final_state};
    for (const void* p : ptrs)
        if (p && !aligned16(p)) return GDN_ERR_UNSUPPORTED;
    if (a.cu_seqlens && (reinterpret_cast<uintptr_t>(a.cu_seqlens) & 3u)) return GDN_ERR_UNSUPPORTED;
    return GDN_OK;
}

PrefillArgs pack(const void* q, const void* k, const void* v, const float* log_alpha, const float* beta,
                 const float* initial_state, void* out, float* final_state, const int32_t* cu_seqlens,
                 int B, int T, int H, int d_k, int d_v) {
    return PrefillArgs{q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v};
}

// Caller-provided scratch (gdn_set_workspace), one per device: a pointer is only valid on the device that was
// current when it was set, so calls look up the scratch of the device that is current when they are made.
constexpr int kMaxDevices = 64;
struct Workspace {
    void* ptr = nullptr;
    size_t bytes = 0;
};
Workspace g_workspace_of_device[kMaxDevices];
std::mutex g_workspace_mutex;
Workspace current_workspace() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return Workspace{};
    std::lock_guard<std::mutex> lock(g_workspace_mutex);
    return g_workspace_of_device[dev];
}
int g_force_path = 0;   // tests: 0 = automatic, 1 = fused kernel, 2 = two-kernel pipeline

int dispatch_bf16(const PrefillArgs& a, cudaStream_t stream) {
    if (!tc_supported(a.d_k, a.d_v)) return launch_simt(a, /*io_bf16=*/true, stream);
    const uint64_t tokens = a.cu_seqlens ? (uint64_t)a.T : (uint64_t)a.B * a.T;
    if (tokens == 0 || g_force_path == 1) return launch_tc(a, stream);
    const size_t need = lean_workspace_bytes(a.B, a.T, a.H, a.d_k, a.d_v, a.cu_seqlens != nullptr);
    const Workspace ws = current_workspace();
    if (ws.ptr && ws.bytes >= need) return launch_lean(a, ws.ptr, ws.bytes, stream);
    if (g_force_path == 2) return GDN_ERR_WORKSPACE;
    return launch_tc(a, stream);
}

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

// Device staging area of the host-buffer entry point: offsets of each tensor.
struct Staging {
    size_t q, k, v, a, b, s0, out, sT, cu, total;
    size_t n_qk, n_v, n_gate, n_state, n_cu;   // byte sizes
};

bool staging_layout(int B, int T, int H, int d_k, int d_v, bool packed, Staging* L) {
    if (B <= 0 || T < 0 || H <= 0 || d_k <= 0 || d_v <= 0) return false;
    const size_t tok = packed ? (size_t)T : (size_t)B * T;
    L->n_qk = tok * H * d_k * sizeof(__nv_bfloat16);
    L->n_v = tok * H * d_v * sizeof(__nv_bfloat16);
    L->n_gate = tok * H * sizeof(float);
    L->n_state = (size_t)B * H * d_k * d_v * sizeof(float);
    L->n_cu = (size_t)(B + 1) * sizeof(int32_t);
    size_t o = 0;
    L->q = o;   o += up256(L->n_qk);
    L->k = o;   o += up256(L->n_qk);
    L->v = o;   o += up256(L->n_v);
    L->a = o;   o += up256(L->n_gate);
    L->b = o;   o += up256(L->n_gate);
    L->s0 = o;  o += up256(L->n_state);
    L->out = o; o += up256(L->n_v);
    L->sT = o;  o += up256(L->n_state);
    L->cu = o;  o += up256(L->n_cu);
    L->total = o;
    return true;
}

// One long sequence through the host-buffer entry point: the sequence is cut into pieces of kHostPiece
// tokens whose upload, prefill (the state carried from piece to piece, exactly, in fp32) and download run
// on three streams, so that the two PCIe directions and the kernels overlap instead of following each other.
constexpr int kHostPiece = 2048;

struct HostPipe {
    cudaStream_t s_in = nullptr, s_out = nullptr;
    std::vector<cudaEvent_t> ev;
    bool ensure(size_t n) {
        if (!s_in && cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) != cudaSuccess) return false;
        if (!s_out && cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) != cudaSuccess) return false;
        while (ev.size() < n) {
            cudaEvent_t e;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return false;
            ev.push_back(e);
        }
        return true;
    }
};
HostPipe g_host_pipe;

int host_pipelined(const void* q_host, const void* k_host, const void* v_host, const float* a_host, const float* b_host,
                   const float* s0_host, void* out_host, float* sT_host, int T, int H, int d_k, int d_v, char* base,
                   const Staging& L, cudaStream_t stream) {
    const int npieces = (T + kHostPiece - 1) / kHostPiece;
    HostPipe& hp = g_host_pipe;
    if (!hp.ensure(2 * (size_t)npieces + 2)) return GDN_ERR_CUDA;
    auto ok = [](cudaError_t e) { return e == cudaSuccess; };
    cudaEvent_t ev_start = hp.ev[0], ev_done = hp.ev[1];
    // the copy streams start after whatever the caller has already queued on `stream`
    if (!ok(cudaEventRecord(ev_start, stream)) || !ok(cudaStreamWaitEvent(hp.s_in, ev_start, 0)) ||
        !ok(cudaStreamWaitEvent(hp.s_out, ev_start, 0)))
        return GDN_ERR_CUDA;
    if (s0_host && !ok(cudaMemcpyAsync(base + L.s0, s0_host, L.n_state, cudaMemcpyHostToDevice, hp.s_in)))
        return GDN_ERR_CUDA;
    float* carry = reinterpret_cast<float*>(base + L.sT);           // the state between pieces, and the final state
    const size_t row_qk = (size_t)H * d_k * sizeof(__nv_bfloat16), row_v = (size_t)H * d_v * sizeof(__nv_bfloat16);
    const size_t row_g = (size_t)H * sizeof(float);
    for (int p = 0; p < npieces; ++p) {
        const size_t t0 = (size_t)p * kHostPiece;
        const int tl = (int)((size_t)T - t0 < (size_t)kHostPiece ? (size_t)T - t0 : (size_t)kHostPiece);
        auto up = [&](size_t off, const void* src, size_t row) {
            return ok(cudaMemcpyAsync(base + off + t0 * row, static_cast<const char*>(src) + t0 * row, (size_t)tl * row,
                                      cudaMemcpyHostToDevice, hp.s_in));
        };
        if (!up(L.q, q_host, row_qk) || !up(L.k, k_host, row_qk) || !up(L.v, v_host, row_v) ||
            !up(L.a, a_host, row_g) || !up(L.b, b_host, row_g))
            return GDN_ERR_CUDA;
        cudaEvent_t ev_in = hp.ev[2 + 2 * p], ev_c = hp.ev[3 + 2 * p];
        if (!ok(cudaEventRecord(ev_in, hp.s_in)) || !ok(cudaStreamWaitEvent(stream, ev_in, 0))) return GDN_ERR_CUDA;
        const float* s_in = p == 0 ? (s0_host ? reinterpret_cast<const float*>(base + L.s0) : nullptr) : carry;
        const PrefillArgs a = pack(base + L.q + t0 * row_qk, base + L.k + t0 * row_qk, base + L.v + t0 * row_v,
                                   reinterpret_cast<const float*>(base + L.a + t0 * row_g),
                                   reinterpret_cast<const float*>(base + L.b + t0 * row_g), s_in,
                                   base + L.out + t0 * row_v, carry, nullptr, 1, tl, H, d_k, d_v);
        if (int rc = validate(a, kChunk)) return rc;
        if (int rc = dispatch_bf16(a, stream)) return rc;
        if (!ok(cudaEventRecord(ev_c, stream)) || !ok(cudaStreamWaitEvent(hp.s_out, ev_c, 0)) ||
            !ok(cudaMemcpyAsync(static_cast<char*>(out_host) + t0 * row_v, base + L.out + t0 * row_v, (size_t)tl * row_v,
                                cudaMemcpyDeviceToHost, hp.s_out)))
            return GDN_ERR_CUDA;
    }
    if (sT_host && !ok(cudaMemcpyAsync(sT_host, carry, L.n_state, cudaMemcpyDeviceToHost, hp.s_out))) return GDN_ERR_CUDA;
    // the call is complete on `stream` when the last download is
    if (!ok(cudaEventRecord(ev_done, hp.s_out)) || !ok(cudaStreamWaitEvent(stream, ev_done, 0))) return GDN_ERR_CUDA;
    return GDN_OK;
}

}  // namespace
}  // namespace gdn

using namespace gdn;

extern "C" {

int gdn_chunk_prefill(const void* q, const void* k, const void* v, const float* log_alpha,
                      const float* beta, const float* initial_state, void* out, float* final_state,
                      const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v, int chunk,
                      gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    return dispatch_bf16(a, reinterpret_cast<cudaStream_t>(stream));
}

int gdn_chunk_prefill_f32(const float* q, const float* k, const float* v, const float* log_alpha,
                          const float* beta, const float* initial_state, float* out, float* final_state,
                          const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v, int chunk,
                          gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    return launch_simt(a, /*io_bf16=*/false, reinterpret_cast<cudaStream_t>(stream));
}

int gdn_chunk_prefill_bf16_simt(const void* q, const void* k, const void* v, const float* log_alpha,
                                const float* beta, const float* initial_state, void* out, float* final_state,
                                const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v, int chunk,
                                gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    return launch_simt(a, /*io_bf16=*/true, reinterpret_cast<cudaStream_t>(stream));
}

size_t gdn_host_staging_bytes(int B, int T, int H, int d_k, int d_v) {
    Staging L;
    // The packed and the batched layouts differ only in how many tokens T stands for; the
    // larger of the two (B*T) always suffices.
    return staging_layout(B, T, H, d_k, d_v, /*packed=*/false, &L) ? L.total : 0;
}

int gdn_chunk_prefill_host(const void* q_host, const void* k_host, const void* v_host,
                           const float* log_alpha_host, const float* beta_host,
                           const float* initial_state_host, void* out_host, float* final_state_host,
                           const int32_t* cu_seqlens_host, int B, int T, int H, int d_k, int d_v, int chunk,
                           void* staging_dev, size_t staging_bytes, gdn_stream_t stream_) {
    if (!q_host || !k_host || !v_host || !log_alpha_host || !beta_host || !out_host || !staging_dev)
        return GDN_ERR_INVALID_ARG;
    Staging L;
    if (!staging_layout(B, T, H, d_k, d_v, cu_seqlens_host != nullptr, &L)) return GDN_ERR_INVALID_ARG;
    if (chunk != kChunk) return GDN_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(staging_dev) & 255u) return GDN_ERR_UNSUPPORTED;
    if (staging_bytes < L.total) return GDN_ERR_WORKSPACE;
    if (cu_seqlens_host) {
        if (cu_seqlens_host[0] != 0 || cu_seqlens_host[B] != T) return GDN_ERR_INVALID_ARG;
        for (int n = 0; n < B; ++n)
            if (cu_seqlens_host[n + 1] < cu_seqlens_host[n]) return GDN_ERR_INVALID_ARG;
    }
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    char* base = static_cast<char*>(staging_dev);
    if (B == 1 && !cu_seqlens_host && T >= 2 * kHostPiece && tc_supported(d_k, d_v))
        return host_pipelined(q_host, k_host, v_host, log_alpha_host, beta_host, initial_state_host, out_host,
                              final_state_host, T, H, d_k, d_v, base, L, stream);
    auto h2d = [&](size_t off, const void* src, size_t bytes) {
        return bytes == 0 || cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    };
    bool ok = h2d(L.q, q_host, L.n_qk) && h2d(L.k, k_host, L.n_qk) && h2d(L.v, v_host, L.n_v) &&
              h2d(L.a, log_alpha_host, L.n_gate) && h2d(L.b, beta_host, L.n_gate);
    if (ok && initial_state_host) ok = h2d(L.s0, initial_state_host, L.n_state);
    if (ok && cu_seqlens_host) ok = h2d(L.cu, cu_seqlens_host, L.n_cu);
    if (!ok) return GDN_ERR_CUDA;
    const PrefillArgs a = pack(base + L.q, base + L.k, base + L.v, reinterpret_cast<const float*>(base + L.a),
                               reinterpret_cast<const float*>(base + L.b),
                               initial_state_host ? reinterpret_cast<const float*>(base + L.s0) : nullptr,
                               base + L.out, final_state_host ? reinterpret_cast<float*>(base + L.sT) : nullptr,
                               cu_seqlens_host ? reinterpret_cast<const int32_t*>(base + L.cu) : nullptr,
                               B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    if (int rc = dispatch_bf16(a, stream)) return rc;
    if (L.n_v && cudaMemcpyAsync(out_host, base + L.out, L.n_v, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    if (final_state_host &&
        cudaMemcpyAsync(final_state_host, base + L.sT, L.n_state, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GDN_ERR_CUDA;
    return GDN_OK;
}

int gdn_chunk_prefill_noalloc(const void* q, const void* k, const void* v, const float* log_alpha,
                              const float* beta, const float* initial_state, void* out, float* final_state,
                              const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v, int chunk,
                              gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    if (!tc_supported(d_k, d_v)) return GDN_ERR_UNSUPPORTED;
    const uint64_t tokens = cu_seqlens ? (uint64_t)T : (uint64_t)B * T;
    if (tokens == 0) return launch_tc(a, reinterpret_cast<cudaStream_t>(stream));   // states pass through; no scratch involved
    return launch_lean_static(a, reinterpret_cast<cudaStream_t>(stream));
}

int gdn_decode_step(const void* q, const void* k, const void* v, const float* log_alpha, const float* beta,
                    float* state, void* out, int B, int H, int d_k, int d_v, gdn_stream_t stream) {
    if (!q || !k || !v || !log_alpha || !beta || !state || !out) return GDN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || d_k <= 0 || d_v <= 0) return GDN_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, log_alpha, beta, state, out};
    for (const void* p : ptrs)
        if (!aligned16(p)) return GDN_ERR_UNSUPPORTED;
    return launch_decode(q, k, v, log_alpha, beta, state, out, B, H, d_k, d_v, reinterpret_cast<cudaStream_t>(stream));
}

int gdn_chunk_prefill_snapshots(const void* q, const void* k, const void* v, const float* log_alpha,
                                const float* beta, const float* initial_state, void* out, float* final_state,
                                int B, int T, int H, int d_k, int d_v, int chunk,
                                int snapshot_every_chunks, float* snapshots, gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, nullptr, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    if (snapshot_every_chunks <= 0) return GDN_ERR_INVALID_ARG;
    if ((T / kChunk) / snapshot_every_chunks == 0) snapshots = nullptr;   // no boundary reached: nothing to write
    else if (!snapshots) return GDN_ERR_INVALID_ARG;
    if (!aligned16(snapshots) || !tc_supported(d_k, d_v)) return GDN_ERR_UNSUPPORTED;
    if (T == 0) return launch_tc(a, reinterpret_cast<cudaStream_t>(stream));
    const size_t need = lean_workspace_bytes(B, T, H, d_k, d_v, false);
    const Workspace ws = current_workspace();
    if (!ws.ptr || ws.bytes < need) return GDN_ERR_WORKSPACE;
    LeanOptions opt;
    opt.snaps = snapshots;
    opt.snap_every = snapshot_every_chunks;
    return launch_lean(a, ws.ptr, ws.bytes, reinterpret_cast<cudaStream_t>(stream), opt);
}

int gdn_chunk_prefill_raw(const void* q_raw, const void* k_raw, const void* v, const float* a_raw, const float* b_raw,
                          float gate_scale, float norm_eps, const float* initial_state, void* out, float* final_state,
                          const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v, int chunk,
                          gdn_stream_t stream) {
    const PrefillArgs a = pack(q_raw, k_raw, v, a_raw, b_raw, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    if (!(gate_scale >= 0.f) || !(norm_eps >= 0.f)) return GDN_ERR_INVALID_ARG;
    if (!tc_supported(d_k, d_v)) return GDN_ERR_UNSUPPORTED;
    const long tokens = cu_seqlens ? (long)T : (long)B * T;
    if (tokens == 0) return launch_tc(a, reinterpret_cast<cudaStream_t>(stream));   // only copies the states
    const size_t need = lean_workspace_bytes(B, T, H, d_k, d_v, cu_seqlens != nullptr);
    const Workspace ws = current_workspace();
    if (!ws.ptr || ws.bytes < need) return GDN_ERR_WORKSPACE;
    LeanOptions opt;
    opt.raw = true;
    opt.gate_scale = gate_scale;
    opt.eps = norm_eps;
    return launch_lean(a, ws.ptr, ws.bytes, reinterpret_cast<cudaStream_t>(stream), opt);
}

int gdn_chunk_prefill_gated(const void* q, const void* k, const void* v, const float* log_alpha, const float* beta,
                            const float* initial_state, const void* gate_z, const float* norm_weight, float norm_eps,
                            void* out, float* final_state, const int32_t* cu_seqlens, int B, int T, int H, int d_k,
                            int d_v, int chunk, gdn_stream_t stream) {
    const PrefillArgs a = pack(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v);
    if (int rc = validate(a, chunk)) return rc;
    if (!gate_z || !norm_weight || !(norm_eps >= 0.f)) return GDN_ERR_INVALID_ARG;
    if (!aligned16(gate_z) || !aligned16(norm_weight) || d_k != 128 || d_v != 128) return GDN_ERR_UNSUPPORTED;
    const long tokens = cu_seqlens ? (long)T : (long)B * T;
    if (tokens == 0) return launch_tc(a, reinterpret_cast<cudaStream_t>(stream));   // only copies the states
    const size_t need = lean_workspace_bytes(B, T, H, d_k, d_v, cu_seqlens != nullptr);
    const Workspace ws = current_workspace();
    if (!ws.ptr || ws.bytes < need) return GDN_ERR_WORKSPACE;
    LeanOptions opt;
    opt.gate_z = static_cast<const __nv_bfloat16*>(gate_z);
    opt.norm_w = norm_weight;
    opt.norm_eps = norm_eps;
    return launch_lean(a, ws.ptr, ws.bytes, reinterpret_cast<cudaStream_t>(stream), opt);
}

size_t gdn_workspace_bytes(int B, int T, int H, int d_k, int d_v, int chunk, int packed) {
    if (chunk != kChunk) return 0;
    return lean_workspace_bytes(B, T, H, d_k, d_v, packed != 0);
}

int gdn_set_workspace(void* device_ptr, size_t bytes) {
    if (device_ptr && (reinterpret_cast<uintptr_t>(device_ptr) & 255u)) return GDN_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return device_ptr ? GDN_ERR_CUDA : GDN_OK;   // no device: nothing was set
    if (dev < 0 || dev >= kMaxDevices) return GDN_ERR_UNSUPPORTED;
    Workspace ws;
    if (device_ptr && bytes >= 4096) {
        if (int rc = lean_init_workspace(device_ptr)) return rc;
        ws.ptr = device_ptr;
        ws.bytes = bytes;
    }
    std::lock_guard<std::mutex> lock(g_workspace_mutex);
    g_workspace_of_device[dev] = ws;
    return GDN_OK;
}

int gdn_attn_causal_prefill(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens,
                            int B, int T, int Hq, int Hkv, int d, float scale, gdn_stream_t stream) {
    if (B < 0 || T < 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || !(scale >= 0.f) || scale - scale != 0.f)
        return GDN_ERR_INVALID_ARG;
    if ((B > 0 && T > 0) && (!q || !k || !v || !out)) return GDN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return GDN_ERR_UNSUPPORTED;
    return launch_attn(q, k, v, out, cu_seqlens, B, T, Hq, Hkv, d, scale, reinterpret_cast<cudaStream_t>(stream));
}

int gdn_query_status(void) {
    const int s = tc_query_status();      // synchronises the device
    return s ? s : attn_query_status();
}

int gdn_query_status_stream(gdn_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int words[3] = {0, 0, 0};
    if (tc_status_async(&words[0], stream) || lean_status_async(&words[1], stream) || attn_status_async(&words[2], stream))
        return GDN_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return GDN_ERR_CUDA;
    for (int w : words)
        if (w) return w;
    return GDN_OK;
}

// Not part of the public header: 0 = automatic, 1 = fused kernel only, 2 = two-kernel pipeline only.
void gdn_debug_force_path(int path) { g_force_path = path; }

// Not part of the public header: failure-path test hooks.  gdn_debug_drop_chunk(c) makes the chain
// kernel's TMA thread of one CTA skip chunk c, so the bounded waits on that data expire;
// gdn_debug_reset_status() clears the status word afterwards.
void gdn_debug_drop_chunk(int chunk) { lean_set_drop_chunk(chunk); }
int gdn_debug_reset_status(void) { return lean_reset_status(); }

// Not part of the public header: per-kernel event timing of the two-kernel pipeline (benchmark).
int gdn_debug_set_timing(int enable) { return lean_set_timing(enable); }
int gdn_debug_get_timing(float* ms5) { return ms5 ? lean_get_timing(ms5) : GDN_ERR_INVALID_ARG; }

// Not part of the public header: forces the number of sequence segments (0 = automatic); chooses between the
// merged scan kernel (1: used whenever its grid fits the GPU at once) and the three stand-alone kernels (0, default).
void gdn_debug_force_segments(int nseg) { lean_force_segments(nseg); }
void gdn_debug_set_scan(int enable) { lean_set_scan(enable); }
void gdn_debug_set_l2_hints(int enable) { lean_set_l2_hints(enable); }

// Not part of the public header: lets the tests capture per-stage intermediates.
void gdn_debug_set_dump(float* device_buffer) { tc_set_debug_dump(device_buffer); }
void gdn_debug_set_chain_stamps(float* device_buffer) { lean_set_debug(device_buffer); }

unsigned long long gdn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* gdn_status_string(int status) {
    switch (status) {
        case GDN_OK: return "ok";
        case GDN_ERR_INVALID_ARG: return "invalid argument";
        case GDN_ERR_UNSUPPORTED: return "unsupported size, chunk or alignment";
        case GDN_ERR_WORKSPACE: return "caller-provided scratch too small";
        case GDN_ERR_CUDA: return "CUDA call or launch failed";
        case GDN_ERR_TIMEOUT: return "bounded device-side wait expired";
        case GDN_ERR_TOO_LARGE: return "problem exceeds the 64 MiB built-in scratch of gdn_chunk_prefill_noalloc";
        default: return "unknown status";
    }
}

}  // extern "C"
