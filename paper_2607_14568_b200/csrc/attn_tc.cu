// Causal softmax attention with grouped queries on the 5th-generation tensor core (sm_100a).
//
// Sections "The layout trick" and "Prefill attention: finding and removing the O(N^2) wall" of the
// paper turn the prefill attention of the softmax layers into matrix products: scores for a whole block of queries at once, a softmax that normalises
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

constexpr int BM = 128;                 // queries per tile (two tiles per CTA)
constexpr int BN = 128;                 // keys per tile
constexpr int HD = 128;                 // head dimension
constexpr int ATTN_THREADS = 320;       // warps 0-3 / 4-7: softmax of query tile A / B (thread = query), 8 MMA issue, 9 TMA
constexpr unsigned long long ATTN_TIMEOUT_NS = 1000000000ull;
constexpr float RESCALE_THRESHOLD = 8.f;   // in log2 units: P stays below 2^8

// tensor memory columns (512): scores of tile A and B (their bf16 probabilities overwrite the first
// 64 columns of the scores they came from), output accumulators of A and B
constexpr uint32_t TM_S = 0, TM_O = 256;
constexpr uint32_t AT_COLS = 512;

// shared memory: a tile is [2 halves of the head dimension][128 rows][64 values], 128-byte rows
constexpr uint32_t TILE_BYTES = 32768;
constexpr uint32_t AS_Q = 0, AS_K = 2 * TILE_BYTES, AS_V = 4 * TILE_BYTES;      // Q: A, B; K, V: two stages each
constexpr uint32_t AS_BARS = 6 * TILE_BYTES;
constexpr uint32_t AS_MISC = AS_BARS + 24 * 8;
constexpr uint32_t AS_TOTAL = AS_MISC + 64;
constexpr uint32_t ATTN_SMEM = AS_TOTAL + 1024;

enum ABar : uint32_t { AB_Q = 0, AB_KFULL0 = 1, AB_KFREE0 = 3, AB_VFULL0 = 5, AB_VFREE0 = 7, AB_SFULL0 = 9 /* A, B */,
                       AB_PFULL0 = 11 /* A, B */, AB_PVDONE0 = 13 /* A, B */ };

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
    __nv_bfloat16* out;      // [B, T, Hq, 128], or packed [T, Hq, 128]
    const int32_t* cu;       // packed input: B + 1 sequence boundaries (device), else nullptr
    int B, T, Hq, Hkv;
    float scale_log2e;       // scale * log2(e)
};

constexpr uint32_t ID_QK = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_PV = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);

// One CTA owns two neighbouring query tiles A = 2t, B = 2t + 1 of one head.  Both read the same key
// and value tiles, and their softmax warpgroups alternate: while one turns its scores into
// probabilities, the tensor core runs P V and the next Q K^T of the other.
__global__ void __launch_bounds__(ATTN_THREADS, 1)
attn_causal_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + AS_MISC);
    AWaiter w{base + AS_BARS, reinterpret_cast<volatile int*>(sm + AS_MISC + 4)};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // which sequence and which pair of query tiles: batched input takes them from the grid; packed input
    // walks the sequence boundaries (grid.y covers an upper bound of the pair count, the surplus CTAs leave)
    int tok0, len, t;
    if (p.cu) {
        int y = (int)blockIdx.y, n = 0;
        tok0 = 0; len = 0; t = -1;
        for (; n < p.B; ++n) {
            const int a = p.cu[n], l = p.cu[n + 1] - a;
            const int np = ((l + BM - 1) / BM + 1) / 2;
            if (y < np) { tok0 = a; len = l; t = np - 1 - y; break; }
            y -= np;
        }
        if (t < 0) return;                                 // uniform for the CTA; nothing has been set up yet
    } else {
        tok0 = (int)blockIdx.z * p.T;
        len = p.T;
        t = (((len + BM - 1) / BM + 1) / 2) - 1 - (int)blockIdx.y;   // CTAs start in x-major order: every head's
    }                                                      // longest pair of tiles first, the short ones fill the tail
    const int nqt = (len + BM - 1) / BM;
    const int h = blockIdx.x;
    const int hk = h / (p.Hq / p.Hkv);                     // the key/value head this query head reads
    const bool hasB = (2 * t + 1 < nqt);
    const int nA = 2 * t + 1;                              // key tiles of A: 0..2t (the last is its diagonal)
    const int nB = hasB ? 2 * t + 2 : 0;
    const int ntiles = hasB ? nB : nA;

    if (tid == 0) {
        mbar_init(w.bar(AB_Q), 1);
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(w.bar(AB_KFULL0 + s), 1); mbar_init(w.bar(AB_KFREE0 + s), 1);
            mbar_init(w.bar(AB_VFULL0 + s), 1); mbar_init(w.bar(AB_VFREE0 + s), 1);
            mbar_init(w.bar(AB_SFULL0 + s), 1); mbar_init(w.bar(AB_PFULL0 + s), 128);
            mbar_init(w.bar(AB_PVDONE0 + s), 1);
        }
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

    if (warp < 8) {
        // =========================== softmax: thread = query row ===========================
        const uint32_t X = warp >> 2;                      // 0 = tile A, 1 = tile B
        const int nX = X ? nB : nA;
        const int qt = 2 * t + (int)X;
        const int r = tid & 127;                           // row inside the tile = tensor-memory lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t ts = tmem + lane_base + TM_S + X * 128, to = tmem + lane_base + TM_O + X * 128;
        const float c = p.scale_log2e;
        float m_ref = -INFINITY, l = 0.f;
        for (int j = 0; j < nX; ++j) {
            // S_X of tile j is complete; so is every earlier MMA of the issuing thread (P V of tile j - 1)
            w.wait(AB_SFULL0 + X, j & 1);
            tc_fence_after_sync();
            // pass 1: row maximum of the raw scores (c >= 0, so max(c s) = c max(s)); the scores are read
            // again in pass 2 instead of being kept, so that both passes have registers to overlap their
            // loads, special-function operations and conversions
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            {
                uint32_t x[4][32];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(ts + 32 * q4, x[q4]);
                tmem_wait_ld();
                if (j == qt) {                             // diagonal tile: keys after the query do not count
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (32 * q4 + i > r) x[q4][i] = 0xff800000u;       // -inf
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                    for (int i = 0; i < 32; i += 2)
                        mx4[(i >> 1) & 3] = max3(mx4[(i >> 1) & 3], __uint_as_float(x[q4][i]), __uint_as_float(x[q4][i + 1]));
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * c;
            // raise the reference maximum only when it is first set or has grown by more than 2^8
            const bool grow = (mx > m_ref + RESCALE_THRESHOLD);
            const float m_new = grow ? mx : m_ref;
            const float alpha = grow ? ex2(m_ref - m_new) : 1.f;           // 0 on the first tile (m_ref = -inf)
            m_ref = m_new;
            // pass 2: P = 2^(c s - m) as bf16 over the first 64 columns of the scores it came from; the
            // next 32 columns are requested before the current 32 are worked on
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t xs[2][32];
            tmem_ld32(ts, xs[0]);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                tmem_wait_ld();
                if (q4 < 3) tmem_ld32(ts + 32 * (q4 + 1), xs[(q4 + 1) & 1]);
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int e = 32 * q4 + 2 * i;
                    float p0 = ex2(fmaf(__uint_as_float(xs[q4 & 1][2 * i]), c, -m_new));
                    float p1 = ex2(fmaf(__uint_as_float(xs[q4 & 1][2 * i + 1]), c, -m_new));
                    if (j == qt) {                         // exact zeros after the query's own position
                        if (e > r) p0 = 0.f;
                        if (e + 1 > r) p1 = 0.f;
                    }
                    sum[i & 1] += p0;
                    sum[2 + (i & 1)] += p1;
                    pk[i] = pack_bf16(p0, p1);
                }
                tmem_st16(ts + 16 * q4, pk);
            }
            const float sum0 = sum[0] + sum[1], sum1 = sum[2] + sum[3];
            l = l * alpha + (sum0 + sum1);
            if (j > 0 && __any_sync(0xffffffffu, grow)) {   // rescale the accumulator rows of this warp
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t o[32];
                    tmem_ld32(to + 32 * q4, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st32(to + 32 * q4, o);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(w.bar(AB_PFULL0 + X));
        }
        // ---- epilogue: O / l -> bf16 -> global (one 256-byte row per thread) ----
        if (nX > 0) {
            w.wait(AB_PVDONE0 + X, 0);
            tc_fence_after_sync();
            const float inv = 1.0f / l;
            const int row = qt * BM + r;
            __nv_bfloat16* dst = p.out + ((size_t)(tok0 + row) * p.Hq + h) * HD;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t o[32];
                tmem_ld32(to + 32 * q4, o);
                tmem_wait_ld();
                if (row < len) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 val;
                        val.x = pack_bf16(__uint_as_float(o[8 * cc + 0]) * inv, __uint_as_float(o[8 * cc + 1]) * inv);
                        val.y = pack_bf16(__uint_as_float(o[8 * cc + 2]) * inv, __uint_as_float(o[8 * cc + 3]) * inv);
                        val.z = pack_bf16(__uint_as_float(o[8 * cc + 4]) * inv, __uint_as_float(o[8 * cc + 5]) * inv);
                        val.w = pack_bf16(__uint_as_float(o[8 * cc + 6]) * inv, __uint_as_float(o[8 * cc + 7]) * inv);
                        *reinterpret_cast<uint4*>(dst + 32 * q4 + 8 * cc) = val;
                    }
                }
            }
        }
    } else if (warp == 8) {
        // =========================== MMA issue (one thread) ===========================
        if (lane == 0) {
            // operand descriptors are built once: issuing costs tens of nanoseconds per instruction and
            // sits on each tile's softmax -> P V -> Q K^T chain
            const uint64_t dq0 = make_smem_desc(base + AS_Q, 16, 1024), dk0 = make_smem_desc(base + AS_K, 16, 1024);
            const uint64_t dv0 = make_smem_desc(base + AS_V, 16384, 1024);
            auto issue_qk = [&](uint32_t X, int j) {       // S_X = Q_X K_j^T
                const uint64_t dq = dq0 + ((uint64_t)(X * TILE_BYTES) >> 4), dk = dk0 + ((uint64_t)((j & 1) * TILE_BYTES) >> 4);
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks) {
                    const uint64_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;   // the address field counts 16 bytes
                    mma_ss(tmem + TM_S + X * 128, dq + off, dk + off, ID_QK, ks > 0);
                }
                mma_commit(w.bar(AB_SFULL0 + X));
            };
            auto issue_pv = [&](uint32_t X, int j) {       // O_X += P_X V_j, 16 keys per step
                const uint64_t dv = dv0 + ((uint64_t)((j & 1) * TILE_BYTES) >> 4);
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks)
                    mma_ts(tmem + TM_O + X * 128, tmem + TM_S + X * 128 + ks * 8, dv + ((ks * 2048) >> 4), ID_PV,
                           (j > 0 || ks > 0) ? 1u : 0u);
            };
            w.wait(AB_Q, 0);
            w.wait(AB_KFULL0, 0);
            tc_fence_after_sync();
            issue_qk(0, 0);
            if (hasB) issue_qk(1, 0);
            mma_commit(w.bar(AB_KFREE0));
            for (int j = 0; j < ntiles; ++j) {
                const uint32_t s = j & 1, s1 = (j + 1) & 1;
                const bool more = (j + 1 < ntiles);
                // the tiles are normally there long before the probabilities: these waits come first, so that
                // nothing but the MMAs sits between "P ready" and "next scores ready"
                w.wait(AB_VFULL0 + s, (j >> 1) & 1);
                if (more) w.wait(AB_KFULL0 + s1, ((j + 1) >> 1) & 1);
                if (j < nA) {
                    w.wait(AB_PFULL0 + 0, j & 1);
                    tc_fence_after_sync();
                    issue_pv(0, j);
                    if (j + 1 < nA) {
                        issue_qk(0, j + 1);
                    } else {
                        mma_commit(w.bar(AB_PVDONE0 + 0));
                    }
                }
                if (hasB) {
                    w.wait(AB_PFULL0 + 1, j & 1);
                    tc_fence_after_sync();
                    issue_pv(1, j);
                    if (more) {
                        issue_qk(1, j + 1);
                    } else {
                        mma_commit(w.bar(AB_PVDONE0 + 1));
                    }
                }
                mma_commit(w.bar(AB_VFREE0 + s));
                if (more) mma_commit(w.bar(AB_KFREE0 + s1));
            }
        }
    } else {
        // =========================== TMA producer (one thread) ===========================
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            auto load_tile = [&](uint32_t dst, const CUtensorMap* map, int head, int tok, uint32_t full) {
                tma_load_3d(dst, map, 0, head, tok, full);
                tma_load_3d(dst + 8192, map, 0, head, tok + 64, full);
                tma_load_3d(dst + 16384, map, 64, head, tok, full);
                tma_load_3d(dst + 24576, map, 64, head, tok + 64, full);
            };
            const int tok_q = tok0 + 2 * t * BM;
            mbar_arrive_expect_tx(w.bar(AB_Q), hasB ? 2 * TILE_BYTES : TILE_BYTES);
            load_tile(base + AS_Q, &map_q, h, tok_q, w.bar(AB_Q));
            if (hasB) load_tile(base + AS_Q + TILE_BYTES, &map_q, h, tok_q + BM, w.bar(AB_Q));
            for (int j = 0; j < ntiles; ++j) {
                const uint32_t s = j & 1;
                const int tok = tok0 + j * BN;
                if (j >= 2) w.wait(AB_KFREE0 + s, ((j >> 1) - 1) & 1);
                mbar_arrive_expect_tx(w.bar(AB_KFULL0 + s), TILE_BYTES);
                load_tile(base + AS_K + s * TILE_BYTES, &map_k, hk, tok, w.bar(AB_KFULL0 + s));
                if (j >= 2) w.wait(AB_VFREE0 + s, ((j >> 1) - 1) & 1);
                mbar_arrive_expect_tx(w.bar(AB_VFULL0 + s), TILE_BYTES);
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

int attn_status_async(int* host_dst, cudaStream_t stream) {
    return cudaMemcpyFromSymbolAsync(host_dst, g_attn_status, sizeof(int), 0, cudaMemcpyDeviceToHost, stream) == cudaSuccess
               ? GDN_OK : GDN_ERR_CUDA;
}

int attn_query_status() {
    int st = 0;
    if (cudaMemcpyFromSymbol(&st, g_attn_status, sizeof(int)) != cudaSuccess) return GDN_ERR_CUDA;
    return st;
}

int launch_attn(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens, int B, int T,
                int Hq, int Hkv, int d, float scale, cudaStream_t stream) {
    if (!attn_supported(Hq, Hkv, d)) return GDN_ERR_UNSUPPORTED;
    if (B > 65535 || T / (2 * BM) + B + 1 > 65535) return GDN_ERR_UNSUPPORTED;
    if (B == 0 || T == 0) return GDN_OK;
    const uint64_t tokens = cu_seqlens ? (uint64_t)T : (uint64_t)B * T;
    if (tokens > 0x7fffffffull) return GDN_ERR_TOO_LARGE;
    CUtensorMap mq, mk, mv;
    if (!tc_make_map(&mq, q, tokens, Hq, d) || !tc_make_map(&mk, k, tokens, Hkv, d) ||
        !tc_make_map(&mv, v, tokens, Hkv, d))
        return GDN_ERR_CUDA;
    AttnParams p{static_cast<__nv_bfloat16*>(out), cu_seqlens, B, T, Hq, Hkv, scale * 1.4426950408889634f};
    // packed: sum over sequences of ceil(ceil(len / 128) / 2) <= T / 256 + B
    dim3 grid(Hq, cu_seqlens ? T / (2 * BM) + B : ((T + BM - 1) / BM + 1) / 2, cu_seqlens ? 1 : B);
    if (cudaFuncSetAttribute(attn_causal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ATTN_SMEM) !=
        cudaSuccess)
        return GDN_ERR_CUDA;
    attn_causal_kernel<<<grid, ATTN_THREADS, ATTN_SMEM, stream>>>(mq, mk, mv, p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

}  // namespace gdn
