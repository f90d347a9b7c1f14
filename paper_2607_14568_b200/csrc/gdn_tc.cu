// Tensor-core chunked gated delta-rule prefill for bf16 storage (sm_100a).
//
// One CTA walks the 64-token chunks of one (sequence, head) chain for a 128-column
// block of the value dimension.  Everything is kept transposed so that the two
// quantities on the sequential chain -- the state and the per-chunk correction --
// are tensor-core A operands living in tensor memory, one lane per value column:
//
//   G    = [K;Q] K^T            M=128 (64 key rows, 64 query rows), N=64, K=d_k
//   W^T  = K^T (T diag(b e^g))^T   M=d_k,  N=64, K=64     (A = K tile, MN-major)
//   U^T  = V^T (T diag(b))^T       M=128,  N=64, K=64     (A = V tile, MN-major)
//   v^T  = U^T - S^T W^T           M=128,  N=64, K=d_k    (A = bf16 S^T in TMEM, accumulates onto U^T)
//   dS^T = (v e^{gC-g})^T K        M=128,  N=d_k, K=64    (A = bf16 v^T in TMEM, B = K tile, MN-major)
//   O1^T = S^T Q^T, O2^T = v^T P^T M=128,  N=64           (out = e^{g_r} O1 + O2)
//
// (steps a, b1, b2, b3, c, d of the chunked scan, Section "A chunked delta-rule scan
// for the recurrent layers").  The fp32 master copy of S^T stays in the registers of
// the chain warpgroup for the whole sequence (thread j holds column j of S).
//
// Warp roles (512 threads):
//   warpgroup 0  chain:    v_new and state update, the only sequential dependency
//   warpgroup 1  prepare:  cumulative gate, decay masks, forward substitution, WY images
//   warpgroup 2  epilogue: combines O1, O2 and stores the output rows
//   warp 12      issues every tcgen05.mma;  warp 13 issues the TMA loads
// Operands move HBM -> shared memory by TMA (128-byte swizzle, two stages); the
// token-token matrices, T and W never leave the SM.
//
// Every wait is bounded: after about a second a waiter raises an abort flag, records
// GDN_ERR_TIMEOUT in the library's status word, and all roles run to the end of their
// loops without blocking, release tensor memory and return.

#include <cuda.h>

#include <mutex>

#include "gdn_internal.h"
#include "sm100_ptx.cuh"

namespace gdn {

__device__ int g_tc_status = 0;            // first non-zero status raised by a kernel
static float* g_debug_dump = nullptr;      // optional stage dump (tests only)

namespace {

using namespace ptx;

constexpr int C = kChunk;
constexpr int DK = 128;
constexpr int DVB = 128;
constexpr int NTHREADS = 512;
constexpr float LOG2E = 1.4426950408889634f;
constexpr unsigned long long TIMEOUT_NS = 1000000000ull;

// ---- tensor memory columns (512 allocated) ----
constexpr uint32_t TM_DV = 0;     //  64: U^T, then v_new^T (fp32)
constexpr uint32_t TM_DS = 64;    // 128: state increment^T (fp32)
constexpr uint32_t TM_SBF = 192;  //  64: bf16 S^T, A operand
constexpr uint32_t TM_V = 256;    //  32: bf16 v_new^T, A operand
constexpr uint32_t TM_VT = 288;   //  32: bf16 decayed v_new^T, A operand
constexpr uint32_t TM_O1 = 320;   //  64
constexpr uint32_t TM_O2 = 384;   //  64
constexpr uint32_t TM_GW = 448;   //  64: G, then W^T
constexpr uint32_t TM_COLS = 512;

// ---- shared memory (bytes from a 1024-aligned base) ----
constexpr uint32_t SM_KQ = 0;                       // 2 stages x [K_lo | Q_lo | K_hi | Q_hi], 8 KiB each
constexpr uint32_t SM_V = SM_KQ + 2 * 32768;        // 2 stages x [V_lo | V_hi]
constexpr uint32_t SM_W = SM_V + 2 * 16384;         // 2 x (-W^T) image  [d_k rows][64 r]
constexpr uint32_t SM_P = SM_W + 2 * 16384;         // 2 x P image       [64 r][64 i]
constexpr uint32_t SM_T1 = SM_P + 2 * 8192;         // (T diag(b e^g))^T [64 i][64 r]
constexpr uint32_t SM_T2 = SM_T1 + 8192;            // (T diag(b))^T
constexpr uint32_t SM_A = SM_T2 + 8192;             // fp32 A [64][68]
constexpr uint32_t LDA = 68;
constexpr uint32_t SM_TF = SM_A + 64 * LDA * 4;     // fp32 T [64][68]
constexpr uint32_t SM_Y = SM_TF + 64 * LDA * 4;     // fp32 scratch of the blocked solve [32][36]
constexpr uint32_t LDY = 36;
constexpr uint32_t SM_OST = SM_Y + 32 * LDY * 4;    // bf16 output staging [64][128]
constexpr uint32_t SM_GATES = SM_OST + 64 * 128 * 2;  // 4 x {g log2e, beta, e^g, e^{gC-g}, e^{gC}}
constexpr uint32_t GATE_FLOATS = 320;
constexpr uint32_t SM_BARS = SM_GATES + 4 * GATE_FLOATS * 4;
constexpr uint32_t SM_MISC = SM_BARS + 32 * 8;      // tmem base, abort flag
constexpr uint32_t SM_TOTAL = SM_MISC + 64;
constexpr uint32_t SMEM_BYTES = SM_TOTAL + 1024;    // slack for the manual 1024-byte alignment

enum Bar : uint32_t {
    B_FULL0 = 0, B_FULL1, B_FREE0, B_FREE1, B_G, B_W, B_V, B_S, B_O,
    B_TREADY, B_WREADY0, B_WREADY1, B_SREADY, B_VREADY, B_OFREE,
    B_GREADY0, B_GREADY1, B_GREADY2, B_GREADY3, B_GFREE0, B_GFREE1, B_GFREE2, B_GFREE3, B_COUNT
};

struct TcParams {
    const float* a;
    const float* beta;
    const float* s0;
    __nv_bfloat16* out;
    float* sT;
    const int32_t* cu;
    float* dbg;
    int B, T, H, dv;
};

struct Cta {
    uint32_t base;          // shared address of the aligned region
    uint32_t tmem;          // tensor memory base address
    volatile int* abort_flag;
    __device__ __forceinline__ uint32_t bar(uint32_t i) const { return base + SM_BARS + i * 8; }
};

__device__ __forceinline__ void wait(const Cta& cta, uint32_t bar_idx, uint32_t parity) {
    const uint32_t bar = cta.bar(bar_idx);
    if (mbar_try_wait(bar, parity)) return;
    const unsigned long long t0 = globaltimer_ns();
    while (true) {
        if (mbar_try_wait_suspend(bar, parity, 100000u)) return;
        if (*cta.abort_flag) return;
        if (globaltimer_ns() - t0 > TIMEOUT_NS) {
            *cta.abort_flag = 1;
            atomicCAS(&g_tc_status, 0, (int)GDN_ERR_TIMEOUT);
            return;
        }
    }
}

// 16-byte chunk `chunk` (0..7) of 128-byte row `row` inside a 128B-swizzled image
__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t chunk) {
    return row * 128u + ((chunk ^ (row & 7u)) << 4);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// ------------------------------------------------------------------------------------------
// MMA issue helpers (one thread).  Descriptor offsets follow the image layouts above.
// ------------------------------------------------------------------------------------------
constexpr uint32_t ID_G = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_WU = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorMN, kMajorMN);
constexpr uint32_t ID_1 = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);
constexpr uint32_t ID_O = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_2 = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);

__device__ __forceinline__ void issue_G(const Cta& c, uint32_t stage) {
    const uint32_t kq = c.base + SM_KQ + stage * 32768;
#pragma unroll
    for (uint32_t ks = 0; ks < 8; ++ks) {
        const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
        mma_ss(c.tmem + TM_GW, make_smem_desc(kq + off, 16, 1024), make_smem_desc(kq + off, 16, 1024), ID_G, ks > 0);
    }
}
__device__ __forceinline__ void issue_Wt(const Cta& c, uint32_t stage) {
    const uint32_t kq = c.base + SM_KQ + stage * 32768, t1 = c.base + SM_T1;
#pragma unroll
    for (uint32_t ks = 0; ks < 4; ++ks)
        mma_ss(c.tmem + TM_GW, make_smem_desc(kq + ks * 2048, 16384, 1024), make_smem_desc(t1 + ks * 2048, 1024, 1024),
               ID_WU, ks > 0);
}
__device__ __forceinline__ void issue_U(const Cta& c, uint32_t stage) {
    const uint32_t vb = c.base + SM_V + stage * 16384, t2 = c.base + SM_T2;
#pragma unroll
    for (uint32_t ks = 0; ks < 4; ++ks)
        mma_ss(c.tmem + TM_DV, make_smem_desc(vb + ks * 2048, 8192, 1024), make_smem_desc(t2 + ks * 2048, 1024, 1024),
               ID_WU, ks > 0);
}
__device__ __forceinline__ void issue_1(const Cta& c, uint32_t buf) {
    const uint32_t w = c.base + SM_W + buf * 16384;
#pragma unroll
    for (uint32_t ks = 0; ks < 8; ++ks)
        mma_ts(c.tmem + TM_DV, c.tmem + TM_SBF + ks * 8, make_smem_desc(w + ks * 2048, 1024, 1024), ID_1, 1);
}
__device__ __forceinline__ void issue_o1(const Cta& c, uint32_t stage) {
    const uint32_t kq = c.base + SM_KQ + stage * 32768 + 8192;
#pragma unroll
    for (uint32_t ks = 0; ks < 8; ++ks)
        mma_ts(c.tmem + TM_O1, c.tmem + TM_SBF + ks * 8,
               make_smem_desc(kq + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024), ID_O, ks > 0);
}
__device__ __forceinline__ void issue_2(const Cta& c, uint32_t stage) {
    const uint32_t kq = c.base + SM_KQ + stage * 32768;
#pragma unroll
    for (uint32_t ks = 0; ks < 4; ++ks)
        mma_ts(c.tmem + TM_DS, c.tmem + TM_VT + ks * 8, make_smem_desc(kq + ks * 2048, 16384, 1024), ID_2, ks > 0);
}
__device__ __forceinline__ void issue_o2(const Cta& c, uint32_t buf) {
    const uint32_t pimg = c.base + SM_P + buf * 8192;
#pragma unroll
    for (uint32_t ks = 0; ks < 4; ++ks)
        mma_ts(c.tmem + TM_O2, c.tmem + TM_V + ks * 8, make_smem_desc(pimg + ks * 32, 16, 1024), ID_O, ks > 0);
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
template <bool DBG>
__global__ void __launch_bounds__(NTHREADS, 1)
gdn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_v, TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    Cta cta;
    cta.base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (cta.base - smem_u32(smem_raw));
    float* sA = reinterpret_cast<float*>(sm + SM_A);
    float* sGates = reinterpret_cast<float*>(sm + SM_GATES);
    float* sTf = reinterpret_cast<float*>(sm + SM_TF);
    float* sY = reinterpret_cast<float*>(sm + SM_Y);
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    cta.abort_flag = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int dvb = blockIdx.x, h = blockIdx.y, n = blockIdx.z;
    const int H = p.H, dv = p.dv;
    long tok0;
    int len;
    if (p.cu) { tok0 = p.cu[n]; len = p.cu[n + 1] - p.cu[n]; }
    else      { tok0 = (long)n * p.T; len = p.T; }
    const int nchunks = (len + C - 1) / C;

    if (tid == 0) {
        mbar_init(cta.bar(B_FULL0), 1); mbar_init(cta.bar(B_FULL1), 1);
        mbar_init(cta.bar(B_FREE0), 1); mbar_init(cta.bar(B_FREE1), 1);
        mbar_init(cta.bar(B_G), 1); mbar_init(cta.bar(B_W), 1); mbar_init(cta.bar(B_V), 1);
        mbar_init(cta.bar(B_S), 1); mbar_init(cta.bar(B_O), 1);
        mbar_init(cta.bar(B_TREADY), 128); mbar_init(cta.bar(B_WREADY0), 128); mbar_init(cta.bar(B_WREADY1), 128);
        mbar_init(cta.bar(B_SREADY), 128); mbar_init(cta.bar(B_VREADY), 128); mbar_init(cta.bar(B_OFREE), 128);
        for (uint32_t i = 0; i < 4; ++i) { mbar_init(cta.bar(B_GREADY0 + i), 32); mbar_init(cta.bar(B_GFREE0 + i), 128); }
        sMisc[1] = 0;   // abort flag
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(cta.base + SM_MISC, TM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    cta.tmem = sMisc[0];

    const bool dump = DBG && p.dbg != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
    const size_t state_off = ((size_t)n * H + h) * DK * dv + (size_t)dvb * DVB;
    // debug builds: per-role time stamps (ns since kernel start) of the first 16 chunks
    const unsigned long long t_start = DBG ? globaltimer_ns() : 0ull;
    auto stamp = [&](int role, int c, int ev) {
        if (DBG && dump && c < 16)
            p.dbg[7 * 16384 + (role * 16 + c) * 8 + ev] = (float)(globaltimer_ns() - t_start);
    };

    if (warp < 4) {
        // =============================== chain warpgroup ===============================
        setmaxnreg_inc<232>();
        const int j = tid;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float S[DK];
        if (p.s0) {
#pragma unroll
            for (int m = 0; m < DK; ++m) S[m] = __ldg(p.s0 + state_off + (size_t)m * dv + j);
        } else {
#pragma unroll
            for (int m = 0; m < DK; ++m) S[m] = 0.f;
        }
        if (nchunks > 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(S[32 * q + 2 * i], S[32 * q + 2 * i + 1]);
                tmem_st16(cta.tmem + lane_base + TM_SBF + 16 * q, pk);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(cta.bar(B_SREADY));
        }
        for (int c = 0; c < nchunks; ++c) {
            const float* gates = sGates + (c & 3) * GATE_FLOATS;
            // ---- v_new^T = U^T - S^T W^T is in TM_DV ----
            wait(cta, B_V, c & 1);
            tc_fence_after_sync();
            if (tid == 0) stamp(0, c, 0);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t x[32];
                tmem_ld32(cta.tmem + lane_base + TM_DV + 32 * hh, x);
                tmem_wait_ld();
                if (dump && c == 0)
#pragma unroll
                    for (int i = 0; i < 32; ++i) p.dbg[3 * 16384 + j * 64 + 32 * hh + i] = __uint_as_float(x[i]);
                uint32_t pv[16], pd[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float v0 = __uint_as_float(x[2 * i]), v1 = __uint_as_float(x[2 * i + 1]);
                    const float2 dec = *reinterpret_cast<const float2*>(gates + 192 + 32 * hh + 2 * i);
                    pv[i] = pack_bf16(v0, v1);
                    pd[i] = pack_bf16(v0 * dec.x, v1 * dec.y);
                }
                tmem_st16(cta.tmem + lane_base + TM_V + 16 * hh, pv);
                tmem_st16(cta.tmem + lane_base + TM_VT + 16 * hh, pd);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(cta.bar(B_VREADY));
            if (tid == 0) stamp(0, c, 1);
            // ---- S^T <- e^{gC} S^T + (v e^{gC-g})^T K ----
            wait(cta, B_S, c & 1);
            tc_fence_after_sync();
            if (tid == 0) stamp(0, c, 2);
            const float gamma = gates[256];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t d[32];
                tmem_ld32(cta.tmem + lane_base + TM_DS + 32 * q, d);
                tmem_wait_ld();
                if (dump && c == 0)
#pragma unroll
                    for (int i = 0; i < 32; ++i) p.dbg[4 * 16384 + j * 128 + 32 * q + i] = __uint_as_float(d[i]);
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; ++i) S[32 * q + i] = fmaf(gamma, S[32 * q + i], __uint_as_float(d[i]));
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(S[32 * q + 2 * i], S[32 * q + 2 * i + 1]);
                tmem_st16(cta.tmem + lane_base + TM_SBF + 16 * q, pk);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(cta.bar(B_SREADY));
            if (tid == 0) stamp(0, c, 3);
        }
        if (p.sT) {
#pragma unroll
            for (int m = 0; m < DK; ++m) p.sT[state_off + (size_t)m * dv + j] = S[m];
        }
    } else if (warp < 8) {
        // =============================== prepare warpgroup ===============================
        const int tp = tid - 128, wp = tp >> 5;
        const uint32_t lane_base = (uint32_t)(wp * 32) << 16;
        for (int c = 0; c < nchunks; ++c) {
            const uint32_t buf = c & 1;
            const int Rc = min(C, len - c * C);                // valid tokens of this chunk
            const float* gates = sGates + (c & 3) * GATE_FLOATS;
            if (tp == 0) stamp(1, c, 0);
            wait(cta, B_GREADY0 + (c & 3), (c >> 2) & 1);      // step a runs ahead in its own warp
            if (tp == 0) stamp(1, c, 1);
            // ---- step b1: decay masks on G = [K;Q] K^T ----
            wait(cta, B_G, c & 1);
            tc_fence_after_sync();
            if (tp == 0) stamp(1, c, 2);
            {
                const int r = tp & 63;
                const float gr = gates[r];
                const float br = gates[64 + r];
                const bool is_a = tp < 64;                 // warps 0,1: A rows; warps 2,3: P rows
                const int rmax = 32 * (wp & 1) + 31;       // largest row held by this warp
                const uint32_t pimg = cta.base + SM_P + buf * 8192;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    if (32 * hh <= rmax) {
                        uint32_t x[32];
                        tmem_ld32(cta.tmem + lane_base + TM_GW + 32 * hh, x);
                        tmem_wait_ld();
                        if (dump && c == 0)
#pragma unroll
                            for (int i = 0; i < 32; ++i) p.dbg[tp * 64 + 32 * hh + i] = __uint_as_float(x[i]);
                        float y[32];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const float4 gi = *reinterpret_cast<const float4*>(gates + 32 * hh + 4 * i4);
                            y[4 * i4 + 0] = ex2(gr - gi.x) * __uint_as_float(x[4 * i4 + 0]);
                            y[4 * i4 + 1] = ex2(gr - gi.y) * __uint_as_float(x[4 * i4 + 1]);
                            y[4 * i4 + 2] = ex2(gr - gi.z) * __uint_as_float(x[4 * i4 + 2]);
                            y[4 * i4 + 3] = ex2(gr - gi.w) * __uint_as_float(x[4 * i4 + 3]);
                        }
                        if (is_a) {
#pragma unroll
                            for (int i4 = 0; i4 < 8; ++i4) {
                                float o[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int i = 32 * hh + 4 * i4 + e;
                                    // rows of padded tokens by select too (their K rows need not be finite)
                                    o[e] = (i < r && r < Rc) ? br * y[4 * i4 + e] : 0.f;
                                }
                                st_shared_f4(cta.base + SM_A + (r * LDA + 32 * hh + 4 * i4) * 4, o[0], o[1], o[2], o[3]);
                            }
                        } else {
#pragma unroll
                            for (int ch = 0; ch < 4; ++ch) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int i0 = 32 * hh + 8 * ch + 2 * e;
                                    pk[e] = pack_bf16((i0 <= r) ? y[8 * ch + 2 * e] : 0.f,
                                                      (i0 + 1 <= r) ? y[8 * ch + 2 * e + 1] : 0.f);
                                }
                                st_shared_v4(pimg + swz(r, 4 * hh + ch), pk[0], pk[1], pk[2], pk[3]);
                            }
                        }
                    } else if (!is_a) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) st_shared_v4(pimg + swz(r, 4 * hh + ch), 0u, 0u, 0u, 0u);
                    }
                }
            }
            named_bar_sync(1, 128);
            if (tp == 0) stamp(1, c, 3);
            // ---- step b2: T = (I + A)^{-1} by blocked forward substitution (fp32, shared memory) ----
            // level 0: the four 16x16 diagonal blocks, one column per thread, no barrier inside
            if (tp < 64) {
                const int I = tp >> 4, cc = tp & 15;
                const float* Ab = sA + (16 * I) * LDA + 16 * I;
                float* Tb = sTf + (16 * I) * LDA + 16 * I;
                float xs[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                    for (int i4 = 0; i4 < (r + 3) / 4; ++i4) {
                        const float4 a4 = *reinterpret_cast<const float4*>(Ab + r * LDA + 4 * i4);
                        if (4 * i4 + 0 < r) acc0 = fmaf(a4.x, xs[4 * i4 + 0], acc0);
                        if (4 * i4 + 1 < r) acc1 = fmaf(a4.y, xs[4 * i4 + 1], acc1);
                        if (4 * i4 + 2 < r) acc0 = fmaf(a4.z, xs[4 * i4 + 2], acc0);
                        if (4 * i4 + 3 < r) acc1 = fmaf(a4.w, xs[4 * i4 + 3], acc1);
                    }
                    xs[r] = ((r == cc) ? 1.f : 0.f) - (acc0 + acc1);
                    Tb[r * LDA + cc] = xs[r];
                }
            }
            named_bar_sync(1, 128);
            // level 1: 16-blocks (1,0) and (3,2):  T21 = -T22 (A21 T11)
            {
                const int pr = tp >> 6, r = (tp >> 2) & 15, cg = tp & 3;
                const int lo = 32 * pr, hi = lo + 16;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
                for (int i4 = 0; i4 < 4; ++i4) {
                    const float4 a4 = *reinterpret_cast<const float4*>(sA + (hi + r) * LDA + lo + 4 * i4);
                    const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 t4 = *reinterpret_cast<const float4*>(sTf + (lo + 4 * i4 + e) * LDA + lo + 4 * cg);
                        acc[0] = fmaf(av[e], t4.x, acc[0]); acc[1] = fmaf(av[e], t4.y, acc[1]);
                        acc[2] = fmaf(av[e], t4.z, acc[2]); acc[3] = fmaf(av[e], t4.w, acc[3]);
                    }
                }
                *reinterpret_cast<float4*>(sY + (16 * pr + r) * LDY + 4 * cg) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                named_bar_sync(1, 128);
                float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
                for (int i4 = 0; i4 < 4; ++i4) {
                    const float4 a4 = *reinterpret_cast<const float4*>(sTf + (hi + r) * LDA + hi + 4 * i4);
                    const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 y4 = *reinterpret_cast<const float4*>(sY + (16 * pr + 4 * i4 + e) * LDY + 4 * cg);
                        t[0] = fmaf(av[e], y4.x, t[0]); t[1] = fmaf(av[e], y4.y, t[1]);
                        t[2] = fmaf(av[e], y4.z, t[2]); t[3] = fmaf(av[e], y4.w, t[3]);
                    }
                }
                *reinterpret_cast<float4*>(sTf + (hi + r) * LDA + lo + 4 * cg) = make_float4(-t[0], -t[1], -t[2], -t[3]);
                // the not-yet-written upper-right 16-blocks of the two 32-blocks are zero
                *reinterpret_cast<float4*>(sTf + (lo + r) * LDA + hi + 4 * cg) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            named_bar_sync(1, 128);
            // level 2: the 32-block (1,0):  T21 = -T22 (A21 T11)
            {
                const int r = tp >> 2, cg = tp & 3;
                float acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll 1
                for (int i4 = 0; i4 < 8; ++i4) {
                    const float4 a4 = *reinterpret_cast<const float4*>(sA + (32 + r) * LDA + 4 * i4);
                    const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float* trow = sTf + (4 * i4 + e) * LDA + 8 * cg;
                        const float4 t0 = *reinterpret_cast<const float4*>(trow);
                        const float4 t1 = *reinterpret_cast<const float4*>(trow + 4);
                        acc[0] = fmaf(av[e], t0.x, acc[0]); acc[1] = fmaf(av[e], t0.y, acc[1]);
                        acc[2] = fmaf(av[e], t0.z, acc[2]); acc[3] = fmaf(av[e], t0.w, acc[3]);
                        acc[4] = fmaf(av[e], t1.x, acc[4]); acc[5] = fmaf(av[e], t1.y, acc[5]);
                        acc[6] = fmaf(av[e], t1.z, acc[6]); acc[7] = fmaf(av[e], t1.w, acc[7]);
                    }
                }
                *reinterpret_cast<float4*>(sY + r * LDY + 8 * cg) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                *reinterpret_cast<float4*>(sY + r * LDY + 8 * cg + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
                named_bar_sync(1, 128);
                float t[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) t[e] = 0.f;
#pragma unroll 1
                for (int i4 = 0; i4 < 8; ++i4) {
                    const float4 a4 = *reinterpret_cast<const float4*>(sTf + (32 + r) * LDA + 32 + 4 * i4);
                    const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float* yrow = sY + (4 * i4 + e) * LDY + 8 * cg;
                        const float4 y0 = *reinterpret_cast<const float4*>(yrow);
                        const float4 y1 = *reinterpret_cast<const float4*>(yrow + 4);
                        t[0] = fmaf(av[e], y0.x, t[0]); t[1] = fmaf(av[e], y0.y, t[1]);
                        t[2] = fmaf(av[e], y0.z, t[2]); t[3] = fmaf(av[e], y0.w, t[3]);
                        t[4] = fmaf(av[e], y1.x, t[4]); t[5] = fmaf(av[e], y1.y, t[5]);
                        t[6] = fmaf(av[e], y1.z, t[6]); t[7] = fmaf(av[e], y1.w, t[7]);
                    }
                }
                *reinterpret_cast<float4*>(sTf + (32 + r) * LDA + 8 * cg) = make_float4(-t[0], -t[1], -t[2], -t[3]);
                *reinterpret_cast<float4*>(sTf + (32 + r) * LDA + 8 * cg + 4) = make_float4(-t[4], -t[5], -t[6], -t[7]);
            }
            named_bar_sync(1, 128);
            // ---- step b3 operands: rows i of (T diag(b e^g))^T and (T diag(b))^T; thread = (column, half) ----
            {
                const int cc = tp & 63, half = tp >> 6;
                const float b = gates[64 + cc], bg = b * gates[128 + cc];
                float t[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int r = 32 * half + i;
                    // rows above the 32-block of this column were never written: they are zero
                    t[i] = (half == 0 && cc >= 32) ? 0.f : sTf[r * LDA + cc];
                }
                if (dump && c == 0)
#pragma unroll
                    for (int i = 0; i < 32; ++i) p.dbg[1 * 16384 + (32 * half + i) * 64 + cc] = t[i];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t p1[4], p2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float t0 = t[8 * ch + 2 * e], t1 = t[8 * ch + 2 * e + 1];
                        p1[e] = pack_bf16(t0 * bg, t1 * bg);
                        p2[e] = pack_bf16(t0 * b, t1 * b);
                    }
                    st_shared_v4(cta.base + SM_T1 + swz(cc, 4 * half + ch), p1[0], p1[1], p1[2], p1[3]);
                    st_shared_v4(cta.base + SM_T2 + swz(cc, 4 * half + ch), p2[0], p2[1], p2[2], p2[3]);
                }
            }
            if (Rc < C) {
                // Tail chunk: the K and V tile rows behind the last token hold the first rows of whatever follows the
                // sequence in memory.  They only meet factors that are exactly zero, but zero times a non-finite value
                // is not zero: clear them before the products that contract over tokens (W, U, the state update).
                const uint32_t kq = cta.base + SM_KQ + buf * 32768, vb = cta.base + SM_V + buf * 16384;
                const uint32_t pieces = (uint32_t)(C - Rc) * 8u;
                for (uint32_t x = tp; x < 4 * pieces; x += 128) {
                    const uint32_t t4 = x / pieces, y = x - t4 * pieces;
                    const uint32_t tile = t4 == 0 ? kq : t4 == 1 ? kq + 16384 : t4 == 2 ? vb : vb + 8192;
                    st_shared_v4(tile + ((uint32_t)Rc + (y >> 3)) * 128 + ((y & 7) << 4), 0u, 0u, 0u, 0u);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            if (tp == 0) stamp(1, c, 4);
            mbar_arrive(cta.bar(B_TREADY));
            // ---- step b3 result: -W^T from tensor memory to its shared-memory image ----
            wait(cta, B_W, c & 1);
            tc_fence_after_sync();
            if (tp == 0) stamp(1, c, 5);
            {
                const uint32_t wimg = cta.base + SM_W + buf * 16384;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t w[32];
                    tmem_ld32(cta.tmem + lane_base + TM_GW + 32 * hh, w);
                    tmem_wait_ld();
                    if (dump && c == 0)
#pragma unroll
                        for (int i = 0; i < 32; ++i) p.dbg[2 * 16384 + tp * 64 + 32 * hh + i] = __uint_as_float(w[i]);
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            pk[e] = pack_bf16(-__uint_as_float(w[8 * ch + 2 * e]), -__uint_as_float(w[8 * ch + 2 * e + 1]));
                        st_shared_v4(wimg + swz(tp, 4 * hh + ch), pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(cta.bar(B_WREADY0 + buf));
            if (tp == 0) stamp(1, c, 6);
        }
    } else if (warp < 12) {
        // =============================== epilogue warpgroup ===============================
        setmaxnreg_dec<96>();
        const int j = tid - 256, we = j >> 5;
        const uint32_t lane_base = (uint32_t)(we * 32) << 16;
        __nv_bfloat16* ost = reinterpret_cast<__nv_bfloat16*>(sm + SM_OST);   // [64 rows][128 columns]
        for (int c = 0; c < nchunks; ++c) {
            const int R = min(C, len - c * C);
            const float* gates = sGates + (c & 3) * GATE_FLOATS;
            wait(cta, B_O, c & 1);
            tc_fence_after_sync();
            if (j == 0) stamp(2, c, 0);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t o1[32], o2[32];
                tmem_ld32(cta.tmem + lane_base + TM_O1 + 32 * hh, o1);
                tmem_ld32(cta.tmem + lane_base + TM_O2 + 32 * hh, o2);
                tmem_wait_ld();
                if (hh == 1) {
                    tc_fence_before_sync();
                    mbar_arrive(cta.bar(B_OFREE));
                }
                if (dump && c == 0)
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        p.dbg[5 * 16384 + j * 64 + 32 * hh + i] = __uint_as_float(o1[i]);
                        p.dbg[6 * 16384 + j * 64 + 32 * hh + i] = __uint_as_float(o2[i]);
                    }
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int r = 32 * hh + i;
                    const float o = fmaf(gates[128 + r], __uint_as_float(o1[i]), __uint_as_float(o2[i]));
                    ost[r * DVB + j] = __float2bfloat16_rn(o);      // transpose through shared memory
                }
            }
            named_bar_sync(2, 128);
            // coalesced 16-byte stores: 16 threads cover one 256-byte output row
            {
                __nv_bfloat16* obase = p.out + ((size_t)(tok0 + c * C) * H + h) * dv + (size_t)dvb * DVB;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int qd = it * 128 + j, r = qd >> 4, col = (qd & 15) * 8;
                    if (r < R) {
                        const uint4 val = *reinterpret_cast<const uint4*>(ost + r * DVB + col);
                        *reinterpret_cast<uint4*>(obase + (size_t)r * H * dv + col) = val;
                    }
                }
            }
            named_bar_sync(2, 128);
            mbar_arrive(cta.bar(B_GFREE0 + (c & 3)));          // last reader of this chunk's gate vectors
            if (j == 0) stamp(2, c, 1);
        }
    } else {
        // =============================== control warpgroup ===============================
        setmaxnreg_dec<56>();
        if (warp == 12 && lane == 0) {
            // ---- MMA issuer ----
            if (nchunks > 0) {
                wait(cta, B_FULL0, 0);
                tc_fence_after_sync();
                issue_G(cta, 0);
                mma_commit(cta.bar(B_G));
                wait(cta, B_TREADY, 0);
                tc_fence_after_sync();
                issue_Wt(cta, 0);
                mma_commit(cta.bar(B_W));
                issue_U(cta, 0);
            }
            for (int c = 0; c < nchunks; ++c) {
                const uint32_t buf = c & 1, par2 = (c >> 1) & 1;
                wait(cta, B_SREADY, c & 1);
                wait(cta, B_WREADY0 + buf, par2);
                tc_fence_after_sync();
                stamp(3, c, 0);
                issue_1(cta, buf);
                mma_commit(cta.bar(B_V));
                if (c > 0) { wait(cta, B_OFREE, (c - 1) & 1); tc_fence_after_sync(); }
                issue_o1(cta, buf);
                if (c + 1 < nchunks) {
                    const uint32_t nb = (c + 1) & 1;
                    wait(cta, B_FULL0 + nb, ((c + 1) >> 1) & 1);
                    issue_G(cta, nb);
                    mma_commit(cta.bar(B_G));
                }
                stamp(3, c, 1);
                wait(cta, B_VREADY, c & 1);
                tc_fence_after_sync();
                stamp(3, c, 2);
                issue_2(cta, buf);
                mma_commit(cta.bar(B_S));
                issue_o2(cta, buf);
                mma_commit(cta.bar(B_O));
                mma_commit(cta.bar(B_FREE0 + buf));
                if (c + 1 < nchunks) {
                    wait(cta, B_TREADY, (c + 1) & 1);
                    tc_fence_after_sync();
                    stamp(3, c, 3);
                    issue_Wt(cta, (c + 1) & 1);
                    mma_commit(cta.bar(B_W));
                    issue_U(cta, (c + 1) & 1);
                }
                stamp(3, c, 4);
            }
        } else if (warp == 14) {
            // ---- step a: chunk-local cumulative log gate, up to four chunks ahead ----
            for (int c = 0; c < nchunks; ++c) {
                const int R = min(C, len - c * C);
                float* gates = sGates + (c & 3) * GATE_FLOATS;
                const int r0 = lane, r1 = lane + 32;
                float x = 0.f, y = 0.f, b0 = 0.f, b1 = 0.f;
                if (r0 < R) { const size_t o = (size_t)(tok0 + c * C + r0) * H + h; x = __ldg(p.a + o); b0 = __ldg(p.beta + o); }
                if (r1 < R) { const size_t o = (size_t)(tok0 + c * C + r1) * H + h; y = __ldg(p.a + o); b1 = __ldg(p.beta + o); }
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const float xu = __shfl_up_sync(0xffffffffu, x, d);
                    const float yu = __shfl_up_sync(0xffffffffu, y, d);
                    if (lane >= d) { x += xu; y += yu; }
                }
                y += __shfl_sync(0xffffffffu, x, 31);
                const float gC = __shfl_sync(0xffffffffu, y, 31);
                if (c >= 4) wait(cta, B_GFREE0 + (c & 3), ((c >> 2) - 1) & 1);
                gates[r0] = x * LOG2E; gates[r1] = y * LOG2E;                        // g_r log2(e)
                gates[64 + r0] = b0; gates[64 + r1] = b1;                            // beta_r
                gates[128 + r0] = ex2(x * LOG2E); gates[128 + r1] = ex2(y * LOG2E);  // e^{g_r}
                gates[192 + r0] = ex2((gC - x) * LOG2E); gates[192 + r1] = ex2((gC - y) * LOG2E);
                if (lane == 0) gates[256] = ex2(gC * LOG2E);
                mbar_arrive(cta.bar(B_GREADY0 + (c & 3)));
            }
        } else if (warp == 13 && lane == 0) {
            // ---- TMA producer ----
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            for (int c = 0; c < nchunks; ++c) {
                const uint32_t stage = c & 1;
                if (c >= 2) wait(cta, B_FREE0 + stage, ((c - 2) >> 1) & 1);
                const uint32_t kq = cta.base + SM_KQ + stage * 32768, vb = cta.base + SM_V + stage * 16384;
                const uint32_t full = cta.bar(B_FULL0 + stage);
                const int tok = (int)(tok0 + (long)c * C);
                mbar_arrive_expect_tx(full, 49152);
                tma_load_3d(kq, &map_k, 0, h, tok, full);
                tma_load_3d(kq + 8192, &map_q, 0, h, tok, full);
                tma_load_3d(kq + 16384, &map_k, 64, h, tok, full);
                tma_load_3d(kq + 24576, &map_q, 64, h, tok, full);
                tma_load_3d(vb, &map_v, dvb * DVB, h, tok, full);
                tma_load_3d(vb + 8192, &map_v, dvb * DVB + 64, h, tok, full);
            }
            if (*cta.abort_flag) {
                // let copies in flight land before shared memory is released (bounded)
                for (int c = max(0, nchunks - 2); c < nchunks; ++c) {
                    const uint32_t bar = cta.bar(B_FULL0 + (c & 1));
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar, (c >> 1) & 1) && globaltimer_ns() - t0 < TIMEOUT_NS) {}
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(cta.tmem, TM_COLS);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// [tokens, H, d] bf16, box = 64 tokens x 1 head x 64 features, 128-byte swizzle.
// A map is a pure function of (address, tokens, H, d): a serving loop calls with the same few buffers again and
// again, so the last few encodings are kept per host thread and the driver call is skipped on a repeat.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t tokens, uint64_t H, uint64_t d) {
    struct Entry { const void* ptr; uint64_t tokens, H, d; CUtensorMap map; bool used; };
    constexpr int kEntries = 8;
    static thread_local Entry cache[kEntries] = {};
    static thread_local int next = 0;
    for (int i = 0; i < kEntries; ++i)
        if (cache[i].used && cache[i].ptr == ptr && cache[i].tokens == tokens && cache[i].H == H && cache[i].d == d) {
            *map = cache[i].map;
            return true;
        }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {d, H, tokens};
    const cuuint64_t strides[2] = {d * 2, H * d * 2};
    const cuuint32_t box[3] = {64, 1, 64};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    cache[next] = Entry{ptr, tokens, H, d, *map, true};
    next = (next + 1) % kEntries;
    return true;
}

}  // namespace

bool tc_supported(int d_k, int d_v) { return d_k == DK && d_v > 0 && d_v % DVB == 0; }

bool tc_make_map(CUtensorMap* map, const void* ptr, uint64_t tokens, uint64_t H, uint64_t d) {
    return make_map(map, ptr, tokens, H, d);
}

int launch_tc(const PrefillArgs& a, cudaStream_t stream) {
    if (!tc_supported(a.d_k, a.d_v)) return GDN_ERR_UNSUPPORTED;
    if (a.H > 65535 || a.B > 65535) return GDN_ERR_UNSUPPORTED;
    const uint64_t tokens = a.cu_seqlens ? (uint64_t)a.T : (uint64_t)a.B * a.T;
    if (tokens == 0) {
        // nothing to read: states pass through
        if (a.final_state && a.final_state != a.initial_state) {
            const size_t bytes = (size_t)a.B * a.H * a.d_k * a.d_v * sizeof(float);
            cudaError_t e = a.initial_state
                ? cudaMemcpyAsync(a.final_state, a.initial_state, bytes, cudaMemcpyDeviceToDevice, stream)
                : cudaMemsetAsync(a.final_state, 0, bytes, stream);
            if (e != cudaSuccess) return GDN_ERR_CUDA;
        }
        return GDN_OK;
    }
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, a.q, tokens, a.H, a.d_k) || !make_map(&mk, a.k, tokens, a.H, a.d_k) ||
        !make_map(&mv, a.v, tokens, a.H, a.d_v))
        return GDN_ERR_CUDA;
    auto kernel = g_debug_dump ? gdn_tc_kernel<true> : gdn_tc_kernel<false>;
    {   // the shared-memory opt-in is a per-device attribute of the kernel: set once per device and variant
        static std::mutex mu;
        static bool done[64][2] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return GDN_ERR_CUDA;
        if (dev < 0 || dev >= 64) return GDN_ERR_UNSUPPORTED;
        std::lock_guard<std::mutex> lock(mu);
        const int variant = g_debug_dump ? 1 : 0;
        if (!done[dev][variant]) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
                return GDN_ERR_CUDA;
            done[dev][variant] = true;
        }
    }
    TcParams p{a.log_alpha, a.beta, a.initial_state, static_cast<__nv_bfloat16*>(a.out), a.final_state,
               a.cu_seqlens, g_debug_dump, a.B, a.T, a.H, a.d_v};
    dim3 grid(a.d_v / DVB, a.H, a.B), block(NTHREADS);
    kernel<<<grid, block, SMEM_BYTES, stream>>>(mq, mk, mv, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

int tc_query_status() {
    int s = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return GDN_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&s, g_tc_status, sizeof(int)) != cudaSuccess) return GDN_ERR_CUDA;
    return s ? s : lean_query_status();
}

int tc_status_async(int* host_dst, cudaStream_t stream) {
    return cudaMemcpyFromSymbolAsync(host_dst, g_tc_status, sizeof(int), 0, cudaMemcpyDeviceToHost, stream) == cudaSuccess
               ? GDN_OK : GDN_ERR_CUDA;
}

void tc_set_debug_dump(float* p) { g_debug_dump = p; }

}  // namespace gdn
