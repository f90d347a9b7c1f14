// Single-token decode step of the gated delta rule (the recurrence advanced by one token,
// Section "The model"; decode is bandwidth-bound, Section "Decode, and why 4-bit is slower").
//
// Per (sequence, head), state S in R^{d_k x d_v} (fp32, updated in place), one token:
//     S <- alpha S ;  delta <- beta (v - S^T k) ;  S <- S + k delta^T ;  o <- S^T q
// Every value column j is independent.  With u_j = sum_m S[m][j] k[m] and w_j = sum_m S[m][j] q[m]
// taken from the OLD state, delta_j = beta (v_j - alpha u_j) and o_j = alpha w_j + (k.q) delta_j,
// so the state is read once and written once: 8 d_k d_v bytes per (sequence, head), the floor.
//
// One CTA per (sequence, head, 128 value columns); a warp owns d_k/8 whole rows (512 contiguous
// bytes per row: one float4 per lane), all of a thread's loads are issued before any is used,
// the column sums are reduced across the 8 warps through shared memory, and the updated rows are
// written back from registers.

#include "gdn_internal.h"

namespace gdn {
namespace {

constexpr int DVB = 128;          // value columns per CTA
constexpr int NW = 8;             // warps per CTA
constexpr int MAX_ROWS = 16;      // rows per warp (d_k <= 128)

struct DecodeParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const float* a;
    const float* beta;
    float* state;
    __nv_bfloat16* out;
    int H, dk, dv;
};

__global__ void __launch_bounds__(NW * 32, 2) gdn_decode_kernel(DecodeParams p) {
    __shared__ float sk[128], sq[128];
    __shared__ float4 su[NW][32], sw[NW][32];
    __shared__ float skq[NW];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int dvb = blockIdx.x, h = blockIdx.y, n = blockIdx.z;
    const int dk = p.dk, dv = p.dv;
    const size_t nh = (size_t)n * p.H + h;
    const int rows = dk / NW;                                 // rows of this warp: warp * rows ...
    float* S = p.state + nh * dk * dv + (size_t)dvb * DVB + 4 * lane;

    // the state first: every load in flight before anything else is touched
    float4 s[MAX_ROWS];
#pragma unroll
    for (int i = 0; i < MAX_ROWS; ++i)
        if (i < rows) s[i] = *reinterpret_cast<const float4*>(S + (size_t)(warp * rows + i) * dv);
    if (tid < dk) {
        sk[tid] = __bfloat162float(p.k[nh * dk + tid]);
        sq[tid] = __bfloat162float(p.q[nh * dk + tid]);
    }
    const float alpha = expf(p.a[nh]), beta = p.beta[nh];
    const __nv_bfloat16* vp = p.v + nh * dv + (size_t)dvb * DVB + 4 * lane;
    const float v0 = __bfloat162float(vp[0]), v1 = __bfloat162float(vp[1]);
    const float v2 = __bfloat162float(vp[2]), v3 = __bfloat162float(vp[3]);
    __syncthreads();

    float4 u = make_float4(0.f, 0.f, 0.f, 0.f), wq = u;
    float kq = 0.f;
#pragma unroll
    for (int i = 0; i < MAX_ROWS; ++i)
        if (i < rows) {
            const float km = sk[warp * rows + i], qm = sq[warp * rows + i];
            u.x = fmaf(s[i].x, km, u.x); u.y = fmaf(s[i].y, km, u.y); u.z = fmaf(s[i].z, km, u.z); u.w = fmaf(s[i].w, km, u.w);
            wq.x = fmaf(s[i].x, qm, wq.x); wq.y = fmaf(s[i].y, qm, wq.y); wq.z = fmaf(s[i].z, qm, wq.z); wq.w = fmaf(s[i].w, qm, wq.w);
            kq = fmaf(km, qm, kq);
        }
    su[warp][lane] = u;
    sw[warp][lane] = wq;
    if (lane == 0) skq[warp] = kq;
    __syncthreads();
    u = su[0][lane]; wq = sw[0][lane]; kq = skq[0];
#pragma unroll
    for (int x = 1; x < NW; ++x) {                            // fixed order: deterministic
        const float4 a4 = su[x][lane], b4 = sw[x][lane];
        u.x += a4.x; u.y += a4.y; u.z += a4.z; u.w += a4.w;
        wq.x += b4.x; wq.y += b4.y; wq.z += b4.z; wq.w += b4.w;
        kq += skq[x];
    }
    float4 d;
    d.x = beta * (v0 - alpha * u.x); d.y = beta * (v1 - alpha * u.y);
    d.z = beta * (v2 - alpha * u.z); d.w = beta * (v3 - alpha * u.w);
#pragma unroll
    for (int i = 0; i < MAX_ROWS; ++i)
        if (i < rows) {
            const float km = sk[warp * rows + i];
            float4 o;
            o.x = fmaf(alpha, s[i].x, km * d.x); o.y = fmaf(alpha, s[i].y, km * d.y);
            o.z = fmaf(alpha, s[i].z, km * d.z); o.w = fmaf(alpha, s[i].w, km * d.w);
            *reinterpret_cast<float4*>(S + (size_t)(warp * rows + i) * dv) = o;
        }
    if (warp == 0) {
        __nv_bfloat16* op = p.out + nh * dv + (size_t)dvb * DVB + 4 * lane;
        const __nv_bfloat162 o01 = __floats2bfloat162_rn(fmaf(alpha, wq.x, kq * d.x), fmaf(alpha, wq.y, kq * d.y));
        const __nv_bfloat162 o23 = __floats2bfloat162_rn(fmaf(alpha, wq.z, kq * d.z), fmaf(alpha, wq.w, kq * d.w));
        *reinterpret_cast<__nv_bfloat162*>(op) = o01;
        *reinterpret_cast<__nv_bfloat162*>(op + 2) = o23;
    }
}

}  // namespace

bool decode_supported(int d_k, int d_v) { return d_k > 0 && d_k % NW == 0 && d_k <= NW * MAX_ROWS && d_v > 0 && d_v % DVB == 0; }

int launch_decode(const void* q, const void* k, const void* v, const float* log_alpha, const float* beta,
                  float* state, void* out, int B, int H, int d_k, int d_v, cudaStream_t stream) {
    if (!decode_supported(d_k, d_v)) return GDN_ERR_UNSUPPORTED;
    if (H > 65535 || B > 65535) return GDN_ERR_UNSUPPORTED;
    DecodeParams p{static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k),
                   static_cast<const __nv_bfloat16*>(v), log_alpha, beta, state, static_cast<__nv_bfloat16*>(out), H, d_k, d_v};
    dim3 grid(d_v / DVB, H, B);
    gdn_decode_kernel<<<grid, NW * 32, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

}  // namespace gdn
