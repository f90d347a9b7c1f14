// fp32-arithmetic chunked gated delta-rule prefill (plain FMA, no tensor cores).
//
// One CTA walks the chunks of one (sequence, head) chain for a 32-column slice of
// the value dimension; the slice of the state lives in shared memory for the whole
// chain.  Per 64-token chunk it runs the steps of the chunked scan (Section "A
// chunked delta-rule scan for the recurrent layers") in fp32:
//   a   g_r = sum_{i<=r} log_alpha_i                       (warp scan)
//   b1  A[r,i] = beta_r e^{g_r-g_i} (k_r.k_i), i <  r      (4x4 register tiles)
//       P[r,i] =        e^{g_r-g_i} (q_r.k_i), i <= r
//   b2  Tm = (I + A)^{-1}: forward substitution, one column per thread, reading
//       the matrix the previous step produced (never recomputing a dot product)
//       and needing no barrier inside the solve
//   b3  W = Tm diag(beta e^g) K ,  U = Tm diag(beta) V
//   c   v_new = U - W S ;  S <- e^{g_C} S + sum_i e^{g_C-g_i} k_i v_new_i^T
//   d   O = diag(e^g) Q S + P v_new            (S = the chunk's incoming state)
// Rows past the end of a sequence are identity tokens (beta = 0, log_alpha = 0,
// k = q = v = 0): they change nothing and are never stored.
//
// This kernel serves fp32 inputs (the paper's precision) and doubles as a slow
// cross-check of the tensor-core kernel for bf16 inputs.

#include "gdn_internal.h"

namespace gdn {
namespace {

constexpr int C = kChunk;   // 64
constexpr int DVT = 32;     // value columns per CTA
constexpr int NT = 256;     // threads per CTA
constexpr int LDA = C + 1;  // row stride of the 64x64 matrices

struct SimtParams {
    const void* q;
    const void* k;
    const void* v;
    const float* a;
    const float* beta;
    const float* s0;
    void* out;
    float* sT;
    const int32_t* cu;
    int B, T, H, dk, dv;
};

template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) {
    return __ldg(reinterpret_cast<const float4*>(p));
}
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
    float4 r;
    r.x = __uint_as_float(u.x << 16);
    r.y = __uint_as_float(u.x & 0xffff0000u);
    r.z = __uint_as_float(u.y << 16);
    r.w = __uint_as_float(u.y & 0xffff0000u);
    return r;
}
__device__ __forceinline__ void store1(float* p, float x) { *p = x; }
__device__ __forceinline__ void store1(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__host__ __device__ inline size_t simt_smem_floats(int dk) {
    const int ldk = dk + 4;
    return (size_t)3 * C * ldk + (size_t)dk * DVT + 3 * C * DVT + 3 * C * LDA + 4 * C;
}

template <typename TIO>
__global__ void __launch_bounds__(NT, 1) gdn_simt_kernel(SimtParams p) {
    extern __shared__ __align__(16) float smem[];
    const int dk = p.dk, dv = p.dv, H = p.H;
    const int ldk = dk + 4;
    float* sK = smem;
    float* sQ = sK + C * ldk;
    float* sW = sQ + C * ldk;
    float* sS = sW + C * ldk;      // [dk][DVT]
    float* sV = sS + dk * DVT;     // [C][DVT]
    float* sU = sV + C * DVT;
    float* sD = sU + C * DVT;      // v_new
    float* sA = sD + C * DVT;      // [C][LDA]
    float* sTm = sA + C * LDA;
    float* sP = sTm + C * LDA;
    float* sg = sP + C * LDA;      // g_r
    float* sb = sg + C;            // beta_r
    float* seg = sb + C;           // e^{g_r}
    float* sec = seg + C;          // e^{g_C - g_r}

    const int tid = threadIdx.x, lane = tid & 31, grp = tid >> 5;
    const int slice = blockIdx.x, h = blockIdx.y, n = blockIdx.z;
    long tok0;
    int len;
    if (p.cu) { tok0 = p.cu[n]; len = p.cu[n + 1] - p.cu[n]; }
    else      { tok0 = (long)n * p.T; len = p.T; }

    const TIO* gq = static_cast<const TIO*>(p.q);
    const TIO* gk = static_cast<const TIO*>(p.k);
    const TIO* gv = static_cast<const TIO*>(p.v);
    TIO* gout = static_cast<TIO*>(p.out);
    const size_t state_off = ((size_t)n * H + h) * dk * dv + (size_t)slice * DVT;

    for (int idx = tid; idx < dk * DVT; idx += NT) {
        const int m = idx / DVT, j = idx % DVT;
        sS[idx] = p.s0 ? p.s0[state_off + (size_t)m * dv + j] : 0.f;
    }

    const int dk4 = dk >> 2;
    for (int c0 = 0; c0 < len; c0 += C) {
        const int R = min(C, len - c0);
        __syncthreads();   // previous chunk fully consumed; state slice loaded
        // ---- load the chunk (zero rows past the end) ----
        for (int idx = tid; idx < C * dk4; idx += NT) {
            const int r = idx / dk4, m4 = idx % dk4;
            float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), qq = kk;
            if (r < R) {
                const size_t off = ((size_t)(tok0 + c0 + r) * H + h) * dk + (size_t)m4 * 4;
                kk = load4<TIO>(gk + off);
                qq = load4<TIO>(gq + off);
            }
            *reinterpret_cast<float4*>(sK + r * ldk + m4 * 4) = kk;
            *reinterpret_cast<float4*>(sQ + r * ldk + m4 * 4) = qq;
        }
        for (int idx = tid; idx < C * (DVT / 4); idx += NT) {
            const int r = idx / (DVT / 4), j4 = idx % (DVT / 4);
            float4 vv = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < R)
                vv = load4<TIO>(gv + ((size_t)(tok0 + c0 + r) * H + h) * dv + slice * DVT + j4 * 4);
            *reinterpret_cast<float4*>(sV + r * DVT + j4 * 4) = vv;
        }
        // ---- step a: chunk-local cumulative log gate (one warp) ----
        if (grp == 0) {
            const int r0 = lane, r1 = lane + 32;
            float x = 0.f, y = 0.f, b0 = 0.f, b1 = 0.f;
            if (r0 < R) { const size_t o = (size_t)(tok0 + c0 + r0) * H + h; x = p.a[o]; b0 = p.beta[o]; }
            if (r1 < R) { const size_t o = (size_t)(tok0 + c0 + r1) * H + h; y = p.a[o]; b1 = p.beta[o]; }
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const float xu = __shfl_up_sync(0xffffffffu, x, d);
                const float yu = __shfl_up_sync(0xffffffffu, y, d);
                if (lane >= d) { x += xu; y += yu; }
            }
            y += __shfl_sync(0xffffffffu, x, 31);
            const float gC = __shfl_sync(0xffffffffu, y, 31);
            sg[r0] = x; sg[r1] = y;
            sb[r0] = b0; sb[r1] = b1;
            seg[r0] = expf(x); seg[r1] = expf(y);
            sec[r0] = expf(gC - x); sec[r1] = expf(gC - y);
        }
        __syncthreads();
        // ---- step b1: decay-masked token-token matrices, 4x4 tile per thread ----
        {
            const int tr = tid >> 4, ti = tid & 15;
            if (ti <= tr) {
                float accA[4][4], accP[4][4];
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) { accA[x][y] = 0.f; accP[x][y] = 0.f; }
                for (int m = 0; m < dk; m += 4) {
                    float4 kr[4], qr[4], ki[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        kr[x] = *reinterpret_cast<const float4*>(sK + (tr * 4 + x) * ldk + m);
                        qr[x] = *reinterpret_cast<const float4*>(sQ + (tr * 4 + x) * ldk + m);
                        ki[x] = *reinterpret_cast<const float4*>(sK + (ti * 4 + x) * ldk + m);
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int y = 0; y < 4; ++y) {
                            accA[x][y] += kr[x].x * ki[y].x + kr[x].y * ki[y].y + kr[x].z * ki[y].z + kr[x].w * ki[y].w;
                            accP[x][y] += qr[x].x * ki[y].x + qr[x].y * ki[y].y + qr[x].z * ki[y].z + qr[x].w * ki[y].w;
                        }
                }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) {
                        const int r = tr * 4 + x, i = ti * 4 + y;
                        const float e = (i <= r) ? expf(sg[r] - sg[i]) : 0.f;   // mask before exp is used
                        sA[r * LDA + i] = (i < r) ? sb[r] * e * accA[x][y] : 0.f;
                        sP[r * LDA + i] = (i <= r) ? e * accP[x][y] : 0.f;
                    }
            } else {
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) {
                        sA[(tr * 4 + x) * LDA + ti * 4 + y] = 0.f;
                        sP[(tr * 4 + x) * LDA + ti * 4 + y] = 0.f;
                    }
            }
        }
        __syncthreads();
        // ---- step b2: Tm = (I + A)^{-1}; thread c owns column c, no barriers ----
        if (tid < C) {
            const int c = tid;
            for (int r = 0; r < C; ++r) {
                float x = (r == c) ? 1.f : 0.f;
                if (r > c) {
                    float x0 = 0.f, x1 = 0.f;
                    int i = c;
                    for (; i + 1 < r; i += 2) {
                        x0 += sA[r * LDA + i] * sTm[i * LDA + c];
                        x1 += sA[r * LDA + i + 1] * sTm[(i + 1) * LDA + c];
                    }
                    if (i < r) x0 += sA[r * LDA + i] * sTm[i * LDA + c];
                    x = -(x0 + x1);
                }
                sTm[r * LDA + c] = x;
            }
        }
        __syncthreads();
        // ---- step b3: W = Tm diag(beta e^g) K, U = Tm diag(beta) V ----
        const int r0 = grp * 8;
        for (int m4 = lane; m4 < dk4; m4 += 32) {
            float4 acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int i = 0; i <= r0 + 7; ++i) {
                float4 kv = *reinterpret_cast<const float4*>(sK + i * ldk + m4 * 4);
                const float bg = sb[i] * seg[i];
                kv.x *= bg; kv.y *= bg; kv.z *= bg; kv.w *= bg;
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float t = sTm[(r0 + x) * LDA + i];
                    acc[x].x += t * kv.x; acc[x].y += t * kv.y; acc[x].z += t * kv.z; acc[x].w += t * kv.w;
                }
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) *reinterpret_cast<float4*>(sW + (r0 + x) * ldk + m4 * 4) = acc[x];
        }
        {
            float acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = 0.f;
            for (int i = 0; i <= r0 + 7; ++i) {
                const float vv = sV[i * DVT + lane] * sb[i];
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] += sTm[(r0 + x) * LDA + i] * vv;
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) sU[(r0 + x) * DVT + lane] = acc[x];
        }
        __syncthreads();
        // ---- step c (first half): v_new = U - W S ----
        {
            float acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = sU[(r0 + x) * DVT + lane];
            for (int m = 0; m < dk; m += 4) {
                const float s0 = sS[(m + 0) * DVT + lane], s1 = sS[(m + 1) * DVT + lane];
                const float s2 = sS[(m + 2) * DVT + lane], s3 = sS[(m + 3) * DVT + lane];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float4 w = *reinterpret_cast<const float4*>(sW + (r0 + x) * ldk + m);
                    acc[x] -= w.x * s0 + w.y * s1 + w.z * s2 + w.w * s3;
                }
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) sD[(r0 + x) * DVT + lane] = acc[x];
        }
        __syncthreads();
        // ---- step d: O = diag(e^g) Q S + P v_new ----
        {
            float acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = 0.f;
            for (int m = 0; m < dk; m += 4) {
                const float s0 = sS[(m + 0) * DVT + lane], s1 = sS[(m + 1) * DVT + lane];
                const float s2 = sS[(m + 2) * DVT + lane], s3 = sS[(m + 3) * DVT + lane];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float4 qv = *reinterpret_cast<const float4*>(sQ + (r0 + x) * ldk + m);
                    acc[x] += qv.x * s0 + qv.y * s1 + qv.z * s2 + qv.w * s3;
                }
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] *= seg[r0 + x];
            for (int i = 0; i <= r0 + 7; ++i) {
                const float d = sD[i * DVT + lane];
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] += sP[(r0 + x) * LDA + i] * d;
            }
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                const int r = r0 + x;
                if (r < R)
                    store1(gout + ((size_t)(tok0 + c0 + r) * H + h) * dv + slice * DVT + lane, acc[x]);
            }
        }
        __syncthreads();   // every read of the incoming state is done
        // ---- step c (second half): S <- e^{g_C} S + sum_i e^{g_C-g_i} k_i v_new_i^T ----
        {
            const int rows = dk >> 3;   // state rows per warp (dk % 32 == 0 -> multiple of 4, <= 16)
            const int mb = grp * rows;
            float acc[16];
#pragma unroll
            for (int x = 0; x < 16; ++x) acc[x] = 0.f;
            for (int i = 0; i < C; ++i) {
                const float d = sD[i * DVT + lane] * sec[i];
#pragma unroll
                for (int x4 = 0; x4 < 4; ++x4) {
                    if (x4 * 4 < rows) {
                        const float4 kv = *reinterpret_cast<const float4*>(sK + i * ldk + mb + x4 * 4);
                        acc[x4 * 4 + 0] += kv.x * d; acc[x4 * 4 + 1] += kv.y * d;
                        acc[x4 * 4 + 2] += kv.z * d; acc[x4 * 4 + 3] += kv.w * d;
                    }
                }
            }
            const float gamma = seg[C - 1];
#pragma unroll
            for (int x = 0; x < 16; ++x)
                if (x < rows) sS[(mb + x) * DVT + lane] = gamma * sS[(mb + x) * DVT + lane] + acc[x];
        }
    }
    __syncthreads();
    if (p.sT)
        for (int idx = tid; idx < dk * DVT; idx += NT) {
            const int m = idx / DVT, j = idx % DVT;
            p.sT[state_off + (size_t)m * dv + j] = sS[idx];
        }
}

template <typename TIO>
int launch_typed(const SimtParams& p, cudaStream_t stream) {
    const size_t smem = simt_smem_floats(p.dk) * sizeof(float);
    static bool attr_done = false;   // per instantiation; the attribute is sticky per function
    if (!attr_done) {
        if (cudaFuncSetAttribute(gdn_simt_kernel<TIO>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(simt_smem_floats(128) * sizeof(float))) != cudaSuccess)
            return GDN_ERR_CUDA;
        attr_done = true;
    }
    dim3 grid(p.dv / DVT, p.H, p.B), block(NT);
    gdn_simt_kernel<TIO><<<grid, block, smem, stream>>>(p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

}  // namespace

bool simt_supported(int d_k, int d_v) {
    return d_k > 0 && d_v > 0 && d_k % 32 == 0 && d_k <= 128 && d_v % DVT == 0;
}

int launch_simt(const PrefillArgs& a, bool io_bf16, cudaStream_t stream) {
    if (!simt_supported(a.d_k, a.d_v)) return GDN_ERR_UNSUPPORTED;
    if (a.H > 65535 || a.B > 65535) return GDN_ERR_UNSUPPORTED;
    SimtParams p{a.q, a.k, a.v, a.log_alpha, a.beta, a.initial_state, a.out, a.final_state,
                 a.cu_seqlens, a.B, a.T, a.H, a.d_k, a.d_v};
    return io_bf16 ? launch_typed<__nv_bfloat16>(p, stream) : launch_typed<float>(p, stream);
}

}  // namespace gdn
