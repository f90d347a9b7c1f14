// Causal softmax attention with grouped queries on the 5th-generation tensor core (sm_100a).
//
// Section "Batched attention" of the paper turns the prefill attention of the softmax layers
// into matrix products: scores for a whole block of queries at once, a softmax that normalises
// the causally valid prefix and leaves exact zeros beyond it, a second product with V, and
// grouped queries by pointing several query heads at one key/value block.  The paper materialises
// the score matrix in a buffer it already owned; here a tile of scores lives only in tensor
// memory: one CTA owns 128 queries of one head and walks the key/value tiles up to its diagonal,
//
//   S  = Q K^T                      tcgen05.mma, both operands from shared memory (TMA, 128-B swizzle)
//   P  = 2^(S c - m), l += sum P    one thread per query row, straight out of tensor memory
//   O += P V                        tcgen05.mma, P read back from tensor memory as the A operand
//
// with the running maximum m only raised when it grew by more than 8 (so O in tensor memory is
// rescaled rarely; the final division by l uses the same m, so the result is exact).  Score tiles
// are double buffered in tensor memory, so the next Q K^T runs under the current softmax.
//
// Every wait is bounded (about a second): a waiter that gives up raises the CTA's abort flag and
// GDN_ERR_TIMEOUT in the status word; all roles then fall through their loops and the kernel ends.

#include <cuda.h>

#include "gdn_internal.h"
#include "sm100_ptx.cuh"

namespace gdn {

__device__ int g_attn_status = 0;

namespace {

using namespace ptx;

constexpr int BM = 128;                 // queries per CTA
constexpr int BN = 128;                 // keys per tile
constexpr int HD = 128;                 // head dimension
constexpr int ATTN_THREADS = 192;       // warps 0-3 softmax (one thread per query), 4 MMA issue, 5 TMA
constexpr unsigned long long ATTN_TIMEOUT_NS = 1000000000ull;
constexpr float RESCALE_THRESHOLD = 8.f;   // in log2 units: P stays below 2^8

// tensor memory columns (512): two score tiles, the output accumulator, two probability tiles
constexpr uint32_t TM_S0 = 0, TM_O = 256, TM_P0 = 384;
constexpr uint32_t AT_COLS = 512;

// shared memory: a tile is [2 halves of the head dimension][128 rows][64 values], 128-byte rows
constexpr uint32_t TILE_BYTES = 32768;
constexpr uint32_t AS_Q = 0, AS_K = TILE_BYTES, AS_V = 3 * TILE_BYTES;          // K, V: two stages each
constexpr uint32_t AS_BARS = 5 * TILE_BYTES;
constexpr uint32_t AS_MISC = AS_BARS + 24 * 8;
constexpr uint32_t AS_TOTAL = AS_MISC + 64;
constexpr uint32_t ATTN_SMEM = AS_TOTAL + 1024;

enum ABar : uint32_t { AB_Q = 0, AB_KFULL0 = 1, AB_KFREE0 = 3, AB_VFULL0 = 5, AB_VFREE0 = 7, AB_SFULL0 = 9,
                       AB_SFREE0 = 11, AB_PFULL = 13, AB_PVDONE = 14 };

struct AWaiter {
    uint32_t bars;
    volatile int* abort_flag;
    __device__ __forceinline__ uint32_t bar(uint32_t i) const { return bars + i * 8; }
    __device__ __forceinline__ void wait(uint32_t idx, uint32_t parity) const {
        const uint32_t b = bar(idx);
#pragma unroll 1
        for (int i = 0; i < 2048; ++i)
            if (mbar_try_wait(b, parity)) return;
        const unsigned long long t0 = globaltimer_ns();
        while (true) {
            if (mbar_try_wait_suspend(b, parity, 100000u)) return;
            if (*abort_flag) return;
            if (globaltimer_ns() - t0 > ATTN_TIMEOUT_NS) {
                *abort_flag = 1;
                atomicCAS(&g_attn_status, 0, (int)GDN_ERR_TIMEOUT);
                return;
            }
        }
    }
};

struct AttnParams {
    __nv_bfloat16* out;      // [B, T, Hq, 128]
    int B, T, Hq, Hkv;
    float scale_log2e;       // scale * log2(e)
};

constexpr uint32_t ID_QK = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_PV = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);


__global__ void __launch_bounds__(ATTN_THREADS, 1)
attn_causal_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + AS_MISC);
    AWaiter w{base + AS_BARS, reinterpret_cast<volatile int*>(sm + AS_MISC + 4)};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nqt = (p.T + BM - 1) / BM;
    const int qt = nqt - 1 - (int)blockIdx.x;              // longest rows of tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int hk = h / (p.Hq / p.Hkv);                     // the key/value head this query head reads
    const int ntiles = qt + 1;                             // key tiles 0..qt (the last one is the diagonal)
    const int tok_q = b * p.T + qt * BM;

    if (tid == 0) {
        mbar_init(w.bar(AB_Q), 1);
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(w.bar(AB_KFULL0 + s), 1); mbar_init(w.bar(AB_KFREE0 + s), 1);
            mbar_init(w.bar(AB_VFULL0 + s), 1); mbar_init(w.bar(AB_VFREE0 + s), 1);
            mbar_init(w.bar(AB_SFULL0 + s), 1); mbar_init(w.bar(AB_SFREE0 + s), 128);
        }
        mbar_init(w.bar(AB_PFULL), 128); mbar_init(w.bar(AB_PVDONE), 1);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + AS_MISC, AT_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];

    if (warp < 4) {
        // =========================== softmax: thread = query row ===========================
        const int r = tid;                                 // row inside the tile = tensor-memory lane
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float m_ref = -INFINITY, l = 0.f;
        for (int j = 0; j < ntiles; ++j) {
            const uint32_t sb = j & 1;
            w.wait(AB_SFULL0 + sb, (j >> 1) & 1);
            tc_fence_after_sync();
            uint32_t x[4][32];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(tmem + lane_base + TM_S0 + sb * 128 + 32 * q4, x[q4]);
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(w.bar(AB_SFREE0 + sb));            // the next-but-one score tile may overwrite this one
            const bool diag = (j == qt);
            float mx = -INFINITY;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float s = __uint_as_float(x[q4][i]) * p.scale_log2e;
                    if (diag && 32 * q4 + i > r) s = -INFINITY;            // keys after the query
                    x[q4][i] = __float_as_uint(s);
                    mx = fmaxf(mx, s);
                }
            // raise the reference maximum only when it is first set or has grown by more than 2^8
            const bool grow = (mx > m_ref + RESCALE_THRESHOLD);
            const float m_new = grow ? mx : m_ref;
            const float alpha = grow ? ex2(m_ref - m_new) : 1.f;           // 0 on the first tile (m_ref = -inf)
            m_ref = m_new;
            float sum = 0.f;
            uint32_t pk[64];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = ex2(__uint_as_float(x[q4][i]) - m_new);
                    const float p1 = ex2(__uint_as_float(x[q4][i + 1]) - m_new);
                    sum += p0 + p1;
                    pk[16 * q4 + (i >> 1)] = pack_bf16(p0, p1);
                }
            l = l * alpha + sum;
            // O and this probability buffer are free once the previous P V product has completed
            if (j > 0) {
                w.wait(AB_PVDONE, (j - 1) & 1);
                tc_fence_after_sync();
                if (__any_sync(0xffffffffu, grow)) {       // rescale the accumulator rows of this warp
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t o[32];
                        tmem_ld32(tmem + lane_base + TM_O + 32 * q4, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tmem + lane_base + TM_O + 32 * q4, o);
                    }
                }
            }
#pragma unroll
            for (int q2 = 0; q2 < 2; ++q2) {
                uint32_t o[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = pk[32 * q2 + i];
                tmem_st32(tmem + lane_base + TM_P0 + sb * 64 + 32 * q2, o);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(w.bar(AB_PFULL));
        }
        // ---- epilogue: O / l -> bf16 -> global (one 256-byte row per thread) ----
        w.wait(AB_PVDONE, (ntiles - 1) & 1);
        tc_fence_after_sync();
        const float inv = 1.0f / l;
        const int row = qt * BM + r;
        __nv_bfloat16* dst = p.out + ((size_t)(b * p.T + row) * p.Hq + h) * HD;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t o[32];
            tmem_ld32(tmem + lane_base + TM_O + 32 * q4, o);
            tmem_wait_ld();
            if (row < p.T) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 val;
                    val.x = pack_bf16(__uint_as_float(o[8 * c + 0]) * inv, __uint_as_float(o[8 * c + 1]) * inv);
                    val.y = pack_bf16(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv);
                    val.z = pack_bf16(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv);
                    val.w = pack_bf16(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv);
                    *reinterpret_cast<uint4*>(dst + 32 * q4 + 8 * c) = val;
                }
            }
        }
    } else if (warp == 4) {
        // =========================== MMA issue (one thread) ===========================
        if (lane == 0) {
            const uint32_t qa = base + AS_Q;
            auto issue_qk = [&](int j) {                   // S[j & 1] = Q K_j^T
                const uint32_t s = j & 1, ka = base + AS_K + s * TILE_BYTES;
                w.wait(AB_KFULL0 + s, (j >> 1) & 1);
                if (j >= 2) w.wait(AB_SFREE0 + s, ((j >> 1) - 1) & 1);
                tc_fence_after_sync();
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
                    mma_ss(tmem + TM_S0 + s * 128, make_smem_desc(qa + off, 16, 1024), make_smem_desc(ka + off, 16, 1024),
                           ID_QK, ks > 0);
                }
                mma_commit(w.bar(AB_SFULL0 + s));
                mma_commit(w.bar(AB_KFREE0 + s));
            };
            w.wait(AB_Q, 0);
            issue_qk(0);
            for (int j = 0; j < ntiles; ++j) {
                if (j + 1 < ntiles) issue_qk(j + 1);
                const uint32_t s = j & 1, va = base + AS_V + s * TILE_BYTES;
                w.wait(AB_VFULL0 + s, (j >> 1) & 1);
                w.wait(AB_PFULL, j & 1);
                tc_fence_after_sync();
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks)        // O += P V_j, 16 keys per step
                    mma_ts(tmem + TM_O, tmem + TM_P0 + s * 64 + ks * 8, make_smem_desc(va + ks * 2048, 16384, 1024),
                           ID_PV, (j > 0 || ks > 0) ? 1u : 0u);
                mma_commit(w.bar(AB_PVDONE));
                mma_commit(w.bar(AB_VFREE0 + s));
            }
        }
    } else {
        // =========================== TMA producer (one thread) ===========================
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            auto load_tile = [&](uint32_t dst, const CUtensorMap* map, int head, int tok, uint32_t full) {
                mbar_arrive_expect_tx(full, TILE_BYTES);
                tma_load_3d(dst, map, 0, head, tok, full);
                tma_load_3d(dst + 8192, map, 0, head, tok + 64, full);
                tma_load_3d(dst + 16384, map, 64, head, tok, full);
                tma_load_3d(dst + 24576, map, 64, head, tok + 64, full);
            };
            load_tile(base + AS_Q, &map_q, h, tok_q, w.bar(AB_Q));
            for (int j = 0; j < ntiles; ++j) {
                const uint32_t s = j & 1;
                const int tok = b * p.T + j * BN;
                if (j >= 2) w.wait(AB_KFREE0 + s, ((j >> 1) - 1) & 1);
                load_tile(base + AS_K + s * TILE_BYTES, &map_k, hk, tok, w.bar(AB_KFULL0 + s));
                if (j >= 2) w.wait(AB_VFREE0 + s, ((j >> 1) - 1) & 1);
                load_tile(base + AS_V + s * TILE_BYTES, &map_v, hk, tok, w.bar(AB_VFULL0 + s));
            }
            if (*w.abort_flag) {
                // let copies in flight land before shared memory is released (bounded)
                const unsigned long long t0 = globaltimer_ns();
                for (uint32_t s = 0; s < 2; ++s)
                    for (uint32_t which = 0; which < 2; ++which) {
                        const uint32_t bar = w.bar((which ? AB_VFULL0 : AB_KFULL0) + s);
                        while (!mbar_try_wait(bar, 0) && !mbar_try_wait(bar, 1) &&
                               globaltimer_ns() - t0 < ATTN_TIMEOUT_NS) {}
                    }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, AT_COLS);
    }
}

}  // namespace

bool attn_supported(int Hq, int Hkv, int d) { return d == HD && Hkv > 0 && Hq > 0 && Hq % Hkv == 0; }

int attn_query_status() {
    int st = 0;
    if (cudaMemcpyFromSymbol(&st, g_attn_status, sizeof(int)) != cudaSuccess) return GDN_ERR_CUDA;
    return st;
}

int launch_attn(const void* q, const void* k, const void* v, void* out, int B, int T, int Hq, int Hkv, int d,
                float scale, cudaStream_t stream) {
    if (!attn_supported(Hq, Hkv, d)) return GDN_ERR_UNSUPPORTED;
    if (Hq > 65535 || B > 65535) return GDN_ERR_UNSUPPORTED;
    if (B == 0 || T == 0) return GDN_OK;
    const uint64_t tokens = (uint64_t)B * T;
    if (tokens > 0x7fffffffull) return GDN_ERR_TOO_LARGE;
    CUtensorMap mq, mk, mv;
    if (!tc_make_map(&mq, q, tokens, Hq, d) || !tc_make_map(&mk, k, tokens, Hkv, d) ||
        !tc_make_map(&mv, v, tokens, Hkv, d))
        return GDN_ERR_CUDA;
    if (cudaFuncSetAttribute(attn_causal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ATTN_SMEM) !=
        cudaSuccess)
        return GDN_ERR_CUDA;
    AttnParams p{static_cast<__nv_bfloat16*>(out), B, T, Hq, Hkv, scale * 1.4426950408889634f};
    dim3 grid((T + BM - 1) / BM, Hq, B);
    attn_causal_kernel<<<grid, ATTN_THREADS, ATTN_SMEM, stream>>>(mq, mk, mv, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

}  // namespace gdn
