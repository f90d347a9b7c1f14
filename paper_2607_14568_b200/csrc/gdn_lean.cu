// Two-kernel tensor-core pipeline for bf16 storage (sm_100a), used when the caller has
// provided scratch memory (gdn_set_workspace).
//
// The forward substitution is a latency-bound dependent chain; inside the fused kernel it
// sits, once per chunk, on one warpgroup of the few SMs that own a (sequence, head) chain.
// Here everything that does not depend on the incoming state is taken off those SMs:
//
//   gdn_prep_kernel    every (chunk, head) as an item handed out by a ticket, all SMs, four CTAs per SM:
//                      step a  cumulative log gate and the gate vectors,
//                      step b1 G = [K;Q] K^T on the tensor core, decay masks -> A (fp32), P (bf16),
//                      step b2 T = (I + A)^{-1}, blocked forward substitution in shared memory,
//                      step b3 W^T = K^T (T diag(b e^g))^T on the tensor core,
//                      and writes per (chunk, head) the operand images the chain needs:
//                      -W^T, (T diag(b))^T, P (each already in the 128-byte-swizzled
//                      shared-memory layout the MMA descriptors expect) and the gate vectors.
//   gdn_chain_kernel   one CTA per (sequence, head, 128 value columns[, segment]): steps c and d.
//                      TMA brings K, Q, V tiles and the images; U^T = V^T (T diag(b))^T,
//                      v^T = U^T - S^T W^T, dS^T = (v e^{gC-g})^T K, O^T = e^g S^T Q^T + v^T P^T
//                      run as tcgen05 MMAs with the state and v_new as TMEM A operands.
//
//   gdn_summary_kernel, gdn_combine_kernel   (few chains only) the sequence is cut into segments: per segment
//                      the map state-in -> state-out is formed from a zero and an identity state, the
//                      segments' incoming states follow by a short serial walk, and the chain kernel then
//                      runs all segments at once (see "sequence split" below).
//
// (Section "A chunked delta-rule scan for the recurrent layers": state-independent work
// for all positions at once, then a short recurrence over chunks.)
//
// Every wait is bounded (about a second); see gdn_tc.cu for the abort protocol.

#include <cuda.h>

#include <mutex>

#include "gdn_internal.h"
#include "sm100_ptx.cuh"

namespace gdn {

__device__ int g_lean_status = 0;         // first non-zero status raised by these kernels
static int g_lean_force_nseg = 0;         // tests: force a segment count (0 = automatic)
// optional per-kernel timing of the two-kernel pipeline (benchmark only): five events around the
// prepare, summary, combine and chain kernels of the most recent call
static bool g_lean_timing = false;
static cudaEvent_t g_lean_events[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
static bool g_lean_split_last = false;
static float* g_lean_dbg = nullptr;        // debug: time stamps of the chain kernel
static int g_lean_drop_chunk = -1;         // tests: chunk the chain kernel's TMA thread skips (-1 = none)
static int g_lean_l2_hints = 3;            // tests: bit 0 = L2 eviction-priority hints on the K, Q, V tile loads, bit 1 = on the
                                           // scratch images W and T2 (measured on the 10240-token workload, chain kernel:
                                           // 51.3 us without, 49.0 / 49.4 us with either, 47.2 us with both)
static bool g_lean_use_scan = false;       // true = summary, combination and chain of a split run as one resident launch (measured
                                           // slower than the three kernels under programmatic dependent launch: 0.162 vs 0.152 ms on
                                           // the 10240-token workload, 0.074 vs 0.060 ms at 2048 tokens, so it is off by default)
static bool g_lean_scan_last = false;

namespace {

using namespace ptx;

constexpr int C = kChunk;
constexpr int DK = 128;
constexpr int DVB = 128;
constexpr float LOG2E = 1.4426950408889634f;
constexpr unsigned long long TIMEOUT_NS = 1000000000ull;

// ---- per (chunk, head) scratch item ----
constexpr uint32_t IT_W = 0;          // 16384: -W^T image   [d_k rows][64 r]
constexpr uint32_t IT_T2 = 16384;     //  8192: (T diag(b))^T image [64 i][64 r]
constexpr uint32_t IT_P = 24576;      //  8192: P image      [64 r][64 i]
constexpr uint32_t IT_GATES = 32768;  //  1280: g log2e | beta | e^g | e^{gC-g} | e^{gC}
constexpr uint32_t GATE_FLOATS = 320;
constexpr uint32_t ITEM_BYTES = 34048;

constexpr uint32_t LDA = 68, LDY = 32;

// Bounded waits.  Their slow path is inlined at some thirty sites of kernels whose warp roles all run their
// loops at once, and the instruction footprint decides the chain kernel's speed (measured: with 82 KiB of code
// it ran at a 58 % instruction-cache hit rate and took 87 us on the 10240-token workload where 66 KiB took
// 51 us), so the slow path is a counted loop: every pass suspends the thread for up to a millisecond, 1024
// passes give the bound of about a second.  (An out-of-line function is not an option next to setmaxnreg.)
constexpr uint32_t WAIT_PASS_NS = 1000000u;
constexpr int WAIT_PASSES = 1024;
struct Waiter {
    uint32_t bars;              // shared address of barrier 0
    volatile int* abort_flag;
    __device__ __forceinline__ uint32_t bar(uint32_t i) const { return bars + i * 8; }
    __device__ __forceinline__ void wait_slow(uint32_t b, uint32_t parity) const {
#pragma unroll 1
        for (int i = 0; i < WAIT_PASSES; ++i) {
            if (mbar_try_wait_suspend(b, parity, WAIT_PASS_NS)) return;
            if (*abort_flag) return;
        }
        *abort_flag = 1;
        atomicCAS(&g_lean_status, 0, (int)GDN_ERR_TIMEOUT);
    }
    // For waits on the sequential chain: poll without suspending for a short while (a suspended
    // thread wakes up late), then fall back to the bounded suspending wait.
    __device__ __forceinline__ void wait_hot(uint32_t idx, uint32_t parity) const {
        const uint32_t b = bar(idx);
#pragma unroll 1
        for (int i = 0; i < 4096; ++i)
            if (mbar_try_wait(b, parity)) return;
        wait_slow(b, parity);
    }
    __device__ __forceinline__ void wait(uint32_t idx, uint32_t parity) const {
        const uint32_t b = bar(idx);
        if (mbar_try_wait(b, parity)) return;
        wait_slow(b, parity);
    }
};

__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t chunk) {
    return row * 128u + ((chunk ^ (row & 7u)) << 4);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_shared_f4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_global_v4(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    *reinterpret_cast<uint4*>(p) = make_uint4(a, b, c, d);
}
// warp-level TF32 MMA on register fragments: D (16 x 8, fp32) += A (16 x 8) * B (8 x 8)
__device__ __forceinline__ uint32_t tf32_rna(float x) {
    uint32_t y;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// plain (untiled) bulk copy global -> shared; both addresses 16-byte aligned, size % 16 == 0
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(bar) : "memory");
}

// plain bulk copy shared -> global (16-byte aligned, size % 16 == 0), tracked by bulk groups
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(reinterpret_cast<uint64_t>(gdst)), "r"(smem_src), "r"(bytes) : "memory");
}
// the same copies with an L2 eviction-priority hint
__device__ __forceinline__ void bulk_load_hint(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_store_hint(void* gdst, uint32_t smem_src, uint32_t bytes, uint64_t pol) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 ::"l"(reinterpret_cast<uint64_t>(gdst)), "r"(smem_src), "r"(bytes), "l"(pol) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// slot of chunk 0 of sequence n: disjoint ranges for any lengths, total <= tokens/64 + B
__device__ __forceinline__ long slot_base(long tok0, int n) { return (tok0 >> 6) + n; }

struct SeqInfo { long tok0; int len; };
__device__ __forceinline__ SeqInfo seq_info(const int32_t* cu, int n, int T) {
    SeqInfo s;
    if (cu) { s.tok0 = cu[n]; s.len = cu[n + 1] - cu[n]; }
    else    { s.tok0 = (long)n * T; s.len = T; }
    return s;
}

// =====================================================================================
// prepare kernel
// =====================================================================================
constexpr uint32_t PS_KQ = 0;                         // [K_lo | Q_lo | K_hi | Q_hi]
constexpr uint32_t PS_A = 32768;                      // fp32 A [64][68], turned into T = (I + A)^{-1} in place;
                                                      // later the staging space of the -W^T image
constexpr uint32_t PS_T1 = PS_KQ + 24576;             // (T diag(b e^g))^T image over the Q_hi tile (dead after G)
constexpr uint32_t PS_T2 = PS_KQ + 8192;              // (T diag(b))^T image over the Q_lo tile, after the P image
constexpr uint32_t PS_Y = PS_A + 64 * LDA * 4;
constexpr uint32_t PS_GATES = PS_Y + 32 * LDY * 4;
constexpr uint32_t PS_RN = PS_GATES + GATE_FLOATS * 4;     // raw inputs: 1/|k_i| (64), 1/|q_r| (64)
constexpr uint32_t PS_BARS = PS_RN + 128 * 4;
constexpr uint32_t PS_MISC = PS_BARS + 16 * 8;
constexpr uint32_t PS_TOTAL = PS_MISC + 64;
constexpr uint32_t PREP_SMEM = PS_TOTAL + 1024;
constexpr int PREP_THREADS = 192;
constexpr uint32_t PT_COLS = 64;

enum PBar : uint32_t { PB_FULL = 0, PB_G, PB_W, PB_TREADY, PB_GREADY, PB_DONE, PB_KQFREE, PB_ITEM };

struct PrepParams {
    const float* a;
    const float* beta;
    const int32_t* cu;
    uint8_t* items;
    long nslots;
    int B, T, H;
    float gate_scale, eps;     // raw inputs only
    int* ticket;               // {next item, CTAs done}: both zero before the launch, both zero again after it
    int l2;                    // bit 0: the K tiles are read again by later kernels of this call and fit in L2: keep them there;
                               // bit 1: the same for the W and T2 images this kernel writes
};

constexpr uint32_t ID_G = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_WU = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorMN, kMajorMN);
constexpr uint32_t ID_1 = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);
constexpr uint32_t ID_O = make_idesc(128, 64, kFmtBF16, kFmtBF16, kMajorK, kMajorK);
constexpr uint32_t ID_2 = make_idesc(128, 128, kFmtBF16, kFmtBF16, kMajorK, kMajorMN);

// item -> (head, first token, valid rows); false for a slot no sequence uses
__device__ __forceinline__ bool decode_item(const PrepParams& p, long item, int* h, long* tok, int* R) {
    const long slot = item / p.H;
    *h = (int)(item - slot * p.H);
    // which sequence owns this slot?  (largest n with slot_base(n) <= slot)
    int lo = 0, hi = p.B - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        const long t0 = p.cu ? (long)p.cu[mid] : (long)mid * p.T;
        if (slot_base(t0, mid) <= slot) lo = mid; else hi = mid - 1;
    }
    const SeqInfo sq = seq_info(p.cu, lo, p.T);
    const int c = (int)(slot - slot_base(sq.tok0, lo));
    if (c < 0 || c * C >= sq.len) return false;
    *R = min(C, sq.len - c * C);
    *tok = sq.tok0 + (long)c * C;
    return true;
}

// RAW: q and k are raw projections and a, beta pre-activations.  The norms and the gating
// (Section "Prefill projections: dequantize, then call the vendor": per-position kernels around the projections) are folded in here: the
// inverse row norms scale A, P and the columns of T diag(b e^g), and they ride to the chain kernels
// inside the gate vectors (e^g / |q| for the output rows, e^{gC-g} / |k| for the state update), so
// the K and Q tiles themselves are used as they are.
template <bool RAW>
__global__ void __launch_bounds__(PREP_THREADS, 4)
gdn_prep_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, PrepParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    float* sA = reinterpret_cast<float*>(sm + PS_A);
    float* sTf = sA;       // the solve overwrites A block by block
    float* gates = reinterpret_cast<float*>(sm + PS_GATES);
    float* sRN = reinterpret_cast<float*>(sm + PS_RN);
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + PS_MISC);
    Waiter w{base + PS_BARS, reinterpret_cast<volatile int*>(sm + PS_MISC + 4)};

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = p.H;
    pdl_trigger();                      // the next kernel of the call may set itself up while this one runs
    if (tid == 0) {
        mbar_init(w.bar(PB_FULL), 1); mbar_init(w.bar(PB_G), 1); mbar_init(w.bar(PB_W), 1);
        mbar_init(w.bar(PB_TREADY), 128); mbar_init(w.bar(PB_GREADY), 32); mbar_init(w.bar(PB_DONE), 128);
        mbar_init(w.bar(PB_KQFREE), 1); mbar_init(w.bar(PB_ITEM), 1);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + PS_MISC, PT_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];

    // Items are handed out through a global ticket: the time per item differs between SMs by a
    // quarter, so a fixed assignment would leave the fast ones idle at the end.  The issuing thread
    // draws the ticket one item ahead and publishes it in shared memory (slot it & 1, barrier PB_ITEM).
    const long nitems = p.nslots * H;
    int nh = 0, nR = 0;      // issuing thread: head, first token of the item it drew last
    long ntok = 0;
    auto draw = [&]() -> int {           // next ticket that names a used slot, or -1
        while (true) {
            const int t = atomicAdd(p.ticket, 1);
            if (t >= nitems) return -1;
            if (decode_item(p, t, &nh, &ntok, &nR)) return t;
        }
    };
    if (warp == 4 && lane == 0) {
        sMisc[2] = (uint32_t)draw();
        mbar_arrive(w.bar(PB_ITEM));
    }
    int it = 0;     // items this CTA has processed (barrier phases)
    while (true) {
        w.wait(PB_ITEM, it & 1);
        const long item = (int)sMisc[2 + (it & 1)];
        if (item < 0 || *w.abort_flag) break;
        int h, R;
        long tok;
        decode_item(p, item, &h, &tok, &R);
        uint8_t* out_item = p.items + (size_t)item * ITEM_BYTES;
        const uint32_t par = it & 1;

        if (warp < 4) {
            // ================= prepare warpgroup =================
            const int tp = tid;
            const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
            w.wait(PB_GREADY, par);
            if (RAW) {
                // inverse L2 norm of row tp of [K;Q] while the G MMA runs (the swizzle only permutes
                // the 16-byte pieces of a row, so the sum needs no un-swizzling)
                w.wait(PB_FULL, par);
                const uint32_t tile = base + PS_KQ + (uint32_t)(tp >> 6) * 8192 + (uint32_t)(tp & 63) * 128;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int cgi = 0; cgi < 16; ++cgi) {
                    const uint32_t addr = tile + (uint32_t)(cgi >> 3) * 16384 + (uint32_t)(((cgi & 7) ^ (tp & 7)) << 4);
                    uint32_t u[4];
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]) : "r"(addr));
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = __uint_as_float(u[e] << 16), hi = __uint_as_float(u[e] & 0xffff0000u);
                        s0 = fmaf(lo, lo, s0);
                        s1 = fmaf(hi, hi, s1);
                    }
                }
                const float ss = s0 + s1 + p.eps;
                sRN[tp] = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
                named_bar_sync(1, 128);
            }
            w.wait(PB_G, par);
            tc_fence_after_sync();
            // ---- step b1: decay masks on G = [K;Q] K^T ----
            {
                const int r = tp & 63;
                const float gr = gates[r];
                const float br = gates[64 + r];
                const float rnr = RAW ? sRN[tp] : 1.f;        // 1/|k_r| for the A rows, 1/|q_r| for the P rows
                const bool is_a = tp < 64;
                const int rmax = 32 * (warp & 1) + 31;
                const uint32_t pimg = base + PS_KQ + 8192;   // the Q_lo sub-tile is dead once G is complete
                // (one copy of the 32-column body: four CTAs per SM sit in different phases of this kernel, so all of
                //  its code is live at once and its size shows in the instruction cache)
#pragma unroll 1
                for (int hh = 0; hh < 2; ++hh) {
                    if (32 * hh <= rmax) {
                        uint32_t x[32];
                        tmem_ld32(tmem + lane_base + 32 * hh, x);
                        tmem_wait_ld();
                        float y[32];
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const float4 gi = *reinterpret_cast<const float4*>(gates + 32 * hh + 4 * i4);
                            y[4 * i4 + 0] = ex2(gr - gi.x) * __uint_as_float(x[4 * i4 + 0]);
                            y[4 * i4 + 1] = ex2(gr - gi.y) * __uint_as_float(x[4 * i4 + 1]);
                            y[4 * i4 + 2] = ex2(gr - gi.z) * __uint_as_float(x[4 * i4 + 2]);
                            y[4 * i4 + 3] = ex2(gr - gi.w) * __uint_as_float(x[4 * i4 + 3]);
                            if (RAW) {
                                const float4 rk = *reinterpret_cast<const float4*>(sRN + 32 * hh + 4 * i4);
                                y[4 * i4 + 0] *= rnr * rk.x; y[4 * i4 + 1] *= rnr * rk.y;
                                y[4 * i4 + 2] *= rnr * rk.z; y[4 * i4 + 3] *= rnr * rk.w;
                            }
                        }
                        if (is_a) {
#pragma unroll
                            for (int i4 = 0; i4 < 8; ++i4) {
                                float o[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int i = 32 * hh + 4 * i4 + e;
                                    // rows of padded tokens (r >= R) by select too: their K rows are whatever follows the
                                    // sequence in memory, possibly not finite, and 0 * NaN would spread through the merges
                                    o[e] = (i < r && r < R) ? br * y[4 * i4 + e] : 0.f;
                                }
                                st_shared_f4(base + PS_A + (r * LDA + 32 * hh + 4 * i4) * 4, o[0], o[1], o[2], o[3]);
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
            if (R < C) {
                // Tail chunk: the tile rows behind the sequence's last token hold the first rows of whatever follows
                // in memory.  They only ever meet factors that are exactly zero, but zero times a non-finite value
                // is not zero: clear the K rows (the W product contracts over them) now that G has been formed.
                const uint32_t pieces = (uint32_t)(C - R) * 8u;            // 16-byte pieces per 64-column half
                for (uint32_t x = tp; x < 2 * pieces; x += 128) {
                    const uint32_t half = x >= pieces ? 1u : 0u, y = x - half * pieces;
                    st_shared_v4(base + PS_KQ + half * 16384 + ((uint32_t)R + (y >> 3)) * 128 + ((y & 7) << 4), 0u, 0u, 0u, 0u);
                }
            }
            fence_proxy_async_smem();
            named_bar_sync(1, 128);
            // The images leave the SM as bulk copies from shared memory (a thread-per-row store would
            // touch 32 different lines per instruction); thread 0 issues them and later waits for their
            // shared-memory reads before the staging space is reused.
            if (tp == 0) { bulk_store(out_item + IT_P, base + PS_KQ + 8192, 8192); bulk_commit(); }
            // ---- step b2: T = (I + A)^{-1}, blocked forward substitution (fp32) ----
            if (tp < 64) {   // level 0: four 16x16 diagonal blocks, one column per thread
                const int I = tp >> 4, cc = tp & 15;
                const float* Ab = sA + (16 * I) * LDA + 16 * I;
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
                }
                named_bar_sync(1, 128);                    // every column has read the block: overwrite it
                float* Tb = sA + (16 * I) * LDA + 16 * I;
#pragma unroll
                for (int r = 0; r < 16; ++r) Tb[r * LDA + cc] = xs[r];
            } else {
                named_bar_sync(1, 128);
            }
            named_bar_sync(1, 128);
            // The merges T21 = -T22 A21 T11 are small dense products: they run as warp-level TF32 MMAs
            // (m16n8k8, fp32 accumulation) on fragments loaded straight from the fp32 matrix in shared memory.
            // The left product Z = T22 A21 stays in registers: an accumulator fragment holds columns 2t, 2t+1
            // of its row, which is what the next MMA wants as its A operand once the contraction index is
            // renumbered (position t <-> column 2t, position t+4 <-> column 2t+1) on both operands alike.
            // T (rounded to bf16 afterwards) keeps 11 significant bits through these products.
            {
                const int g = lane >> 2, t = lane & 3;
                if (warp < 2) {   // level 1: the 16-blocks (1,0) and (3,2), one warp each
                    const int lo = 32 * warp, hi = lo + 16;
                    float z[2][4] = {};
#pragma unroll 1
                    for (int ks = 0; ks < 2; ++ks) {
                        const float2 a01 = *reinterpret_cast<const float2*>(sTf + (hi + g) * LDA + hi + 8 * ks + 2 * t);
                        const float2 a23 = *reinterpret_cast<const float2*>(sTf + (hi + g + 8) * LDA + hi + 8 * ks + 2 * t);
                        const uint32_t af[4] = {tf32_rna(a01.x), tf32_rna(a23.x), tf32_rna(a01.y), tf32_rna(a23.y)};
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const uint32_t b0 = tf32_rna(sA[(hi + 8 * ks + 2 * t) * LDA + lo + 8 * q + g]);
                            const uint32_t b1 = tf32_rna(sA[(hi + 8 * ks + 2 * t + 1) * LDA + lo + 8 * q + g]);
                            mma_tf32(z[q], af, b0, b1);
                        }
                    }
                    float r[2][4] = {};
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        const uint32_t af[4] = {tf32_rna(z[ks][0]), tf32_rna(z[ks][2]), tf32_rna(z[ks][1]), tf32_rna(z[ks][3])};
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const uint32_t b0 = tf32_rna(sTf[(lo + 8 * ks + 2 * t) * LDA + lo + 8 * q + g]);
                            const uint32_t b1 = tf32_rna(sTf[(lo + 8 * ks + 2 * t + 1) * LDA + lo + 8 * q + g]);
                            mma_tf32(r[q], af, b0, b1);
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 2; ++q) {      // only this warp reads or writes this block
                        *reinterpret_cast<float2*>(sTf + (hi + g) * LDA + lo + 8 * q + 2 * t) = make_float2(-r[q][0], -r[q][1]);
                        *reinterpret_cast<float2*>(sTf + (hi + g + 8) * LDA + lo + 8 * q + 2 * t) = make_float2(-r[q][2], -r[q][3]);
                    }
                }
                named_bar_sync(1, 128);
                // level 2: the 32-block (1,0); warp = (16 rows mb, 16 columns nb) of the result.  The triangular
                // factors shorten the contractions: row block 0 of T22 ends at column 16, column block 1 of
                // T11 starts at row 16.
                const int mb = warp & 1, nb = warp >> 1;
                float z[4][4] = {};
#pragma unroll 1
                for (int ks = 0; ks < 4; ++ks) {
                    if (ks < 2 * (mb + 1)) {
                        const float2 a01 = *reinterpret_cast<const float2*>(sTf + (32 + 16 * mb + g) * LDA + 32 + 8 * ks + 2 * t);
                        const float2 a23 = *reinterpret_cast<const float2*>(sTf + (32 + 16 * mb + g + 8) * LDA + 32 + 8 * ks + 2 * t);
                        const uint32_t af[4] = {tf32_rna(a01.x), tf32_rna(a23.x), tf32_rna(a01.y), tf32_rna(a23.y)};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t b0 = tf32_rna(sA[(32 + 8 * ks + 2 * t) * LDA + 8 * q + g]);
                            const uint32_t b1 = tf32_rna(sA[(32 + 8 * ks + 2 * t + 1) * LDA + 8 * q + g]);
                            mma_tf32(z[q], af, b0, b1);
                        }
                    }
                }
                float r[2][4] = {};
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    if (ks >= 2 * nb) {
                        const uint32_t af[4] = {tf32_rna(z[ks][0]), tf32_rna(z[ks][2]), tf32_rna(z[ks][1]), tf32_rna(z[ks][3])};
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const uint32_t b0 = tf32_rna(sTf[(8 * ks + 2 * t) * LDA + 16 * nb + 8 * q + g]);
                            const uint32_t b1 = tf32_rna(sTf[(8 * ks + 2 * t + 1) * LDA + 16 * nb + 8 * q + g]);
                            mma_tf32(r[q], af, b0, b1);
                        }
                    }
                }
                named_bar_sync(1, 128);                    // every warp has read A21: overwrite it
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    *reinterpret_cast<float2*>(sTf + (32 + 16 * mb + g) * LDA + 16 * nb + 8 * q + 2 * t) = make_float2(-r[q][0], -r[q][1]);
                    *reinterpret_cast<float2*>(sTf + (32 + 16 * mb + g + 8) * LDA + 16 * nb + 8 * q + 2 * t) = make_float2(-r[q][2], -r[q][3]);
                }
            }
            if (tp == 0) bulk_wait_read_all();                 // the P image has left the Q_lo tile
            named_bar_sync(1, 128);
            // ---- step b3 operands: row i = cc of (T diag(b e^g))^T (shared) and (T diag(b))^T (scratch) ----
            {
                const int cc = tp & 63, half = tp >> 6;
                const float b = gates[64 + cc], bg = b * gates[128 + cc] * (RAW ? sRN[cc] : 1.f);
                float t[32];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    t[i] = (half == 0 && cc >= 32) ? 0.f : sTf[(32 * half + i) * LDA + cc];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t p1[4], p2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float t0 = t[8 * ch + 2 * e], t1 = t[8 * ch + 2 * e + 1];
                        p1[e] = pack_bf16(t0 * bg, t1 * bg);
                        p2[e] = pack_bf16(t0 * b, t1 * b);
                    }
                    st_shared_v4(base + PS_T1 + swz(cc, 4 * half + ch), p1[0], p1[1], p1[2], p1[3]);
                    st_shared_v4(base + PS_T2 + swz(cc, 4 * half + ch), p2[0], p2[1], p2[2], p2[3]);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(w.bar(PB_TREADY));
            named_bar_sync(1, 128);
            if (tp == 0) { bulk_store_hint(out_item + IT_T2, base + PS_T2, 8192, (p.l2 & 2) ? l2_policy_evict_last() : l2_policy_evict_normal()); bulk_commit(); }
            // ---- step b3 result: -W^T image to scratch; gate vectors to scratch ----
            if (tp < GATE_FLOATS / 4) {
                float4 gv = *reinterpret_cast<const float4*>(gates + 4 * tp);
                if (RAW && tp >= 32 && tp < 64) {      // e^g -> e^g / |q|   and   e^{gC-g} -> e^{gC-g} / |k|
                    const float4 rn = *reinterpret_cast<const float4*>(sRN + (tp < 48 ? 64 + 4 * (tp - 32) : 4 * (tp - 48)));
                    gv.x *= rn.x; gv.y *= rn.y; gv.z *= rn.z; gv.w *= rn.w;
                }
                *reinterpret_cast<float4*>(out_item + IT_GATES + tp * 16) = gv;
            }
            w.wait(PB_W, par);
            tc_fence_after_sync();
            if (tp == 0) {
                // The tensor core is done with the K tiles and the P and T2 copies have left shared
                // memory: the tiles of the next item may land while this one is finished.
                bulk_wait_read_all();
                mbar_arrive(w.bar(PB_KQFREE));
            }
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t x[32];
                tmem_ld32(tmem + lane_base + 32 * hh, x);
                tmem_wait_ld();
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t pk[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        pk[e] = pack_bf16(-__uint_as_float(x[8 * ch + 2 * e]), -__uint_as_float(x[8 * ch + 2 * e + 1]));
                    st_shared_v4(base + PS_A + (tp >> 6) * 8192 + swz(tp & 63, 4 * hh + ch), pk[0], pk[1], pk[2], pk[3]);
                }
            }
            fence_proxy_async_smem();
            named_bar_sync(1, 128);
            if (tp == 0) {                                     // staged over the fp32 T, which is dead by now
                bulk_store_hint(out_item + IT_W, base + PS_A, 16384, (p.l2 & 2) ? l2_policy_evict_last() : l2_policy_evict_normal());
                bulk_commit();
                bulk_wait_read_all();                          // the staging space may now be overwritten
            }
            tc_fence_before_sync();
            mbar_arrive(w.bar(PB_DONE));
        } else if (warp == 4) {
            // ================= TMA + MMA issue (one thread) =================
            if (lane == 0) {
                const uint32_t kq = base + PS_KQ, full = w.bar(PB_FULL);
                const uint64_t pol_k = (p.l2 & 1) ? l2_policy_evict_last() : l2_policy_evict_normal();
                auto load_tiles = [&](int hh, long tk) {
                    mbar_arrive_expect_tx(full, 32768);
                    tma_load_3d_hint(kq, &map_k, 0, hh, (int)tk, full, pol_k);
                    tma_load_3d_hint(kq + 16384, &map_k, 64, hh, (int)tk, full, pol_k);
                    tma_load_3d(kq + 8192, &map_q, 0, hh, (int)tk, full);
                    tma_load_3d(kq + 24576, &map_q, 64, hh, (int)tk, full);
                };
                if (it == 0) load_tiles(h, tok);                    // later items were requested one item ahead
                else w.wait(PB_DONE, (it - 1) & 1);                 // the accumulator columns of the last item are free
                tc_fence_after_sync();
                w.wait(PB_FULL, par);
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
                    mma_ss(tmem, make_smem_desc(kq + off, 16, 1024), make_smem_desc(kq + off, 16, 1024), ID_G, ks > 0);
                }
                mma_commit(w.bar(PB_G));
                const int nxt = draw();                             // the atomic's latency hides behind the solve
                w.wait(PB_TREADY, par);
                tc_fence_after_sync();
#pragma unroll
                for (uint32_t ks = 0; ks < 4; ++ks)
                    mma_ss(tmem, make_smem_desc(kq + ks * 2048, 16384, 1024),
                           make_smem_desc(base + PS_T1 + ks * 2048, 1024, 1024), ID_WU, ks > 0);
                mma_commit(w.bar(PB_W));
                // request the tiles of the next item as soon as the K/Q space is free, then publish it
                if (nxt >= 0) {
                    w.wait(PB_KQFREE, par);
                    load_tiles(nh, ntok);
                }
                sMisc[2 + ((it + 1) & 1)] = (uint32_t)nxt;
                mbar_arrive(w.bar(PB_ITEM));
            }
        } else {
            // ================= step a: chunk-local cumulative log gate (one warp) =================
            const int r0 = lane, r1 = lane + 32;
            float x = 0.f, y = 0.f, b0 = 0.f, b1 = 0.f;
            if (r0 < R) { const size_t o = (size_t)(tok + r0) * H + h; x = __ldg(p.a + o); b0 = __ldg(p.beta + o); }
            if (r1 < R) { const size_t o = (size_t)(tok + r1) * H + h; y = __ldg(p.a + o); b1 = __ldg(p.beta + o); }
            if (RAW) {   // log gate = -softplus(a) * scale, beta = sigmoid(b); padding rows stay the identity token
                if (r0 < R) { x = -(fmaxf(x, 0.f) + log1pf(expf(-fabsf(x)))) * p.gate_scale; b0 = 1.0f / (1.0f + expf(-b0)); }
                if (r1 < R) { y = -(fmaxf(y, 0.f) + log1pf(expf(-fabsf(y)))) * p.gate_scale; b1 = 1.0f / (1.0f + expf(-b1)); }
            }
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const float xu = __shfl_up_sync(0xffffffffu, x, d);
                const float yu = __shfl_up_sync(0xffffffffu, y, d);
                if (lane >= d) { x += xu; y += yu; }
            }
            y += __shfl_sync(0xffffffffu, x, 31);
            const float gC = __shfl_sync(0xffffffffu, y, 31);
            if (it > 0) w.wait(PB_DONE, (it - 1) & 1);
            gates[r0] = x * LOG2E; gates[r1] = y * LOG2E;
            gates[64 + r0] = b0; gates[64 + r1] = b1;
            gates[128 + r0] = ex2(x * LOG2E); gates[128 + r1] = ex2(y * LOG2E);
            gates[192 + r0] = ex2((gC - x) * LOG2E); gates[192 + r1] = ex2((gC - y) * LOG2E);
            gates[256 + lane] = (lane == 0) ? ex2(gC * LOG2E) : 0.f;
            gates[288 + lane] = 0.f;
            mbar_arrive(w.bar(PB_GREADY));
        }
        ++it;
    }
    if (tid == 0) bulk_wait_all();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, PT_COLS);
    }
    if (tid == 0) {      // the last CTA to leave re-arms the ticket for the next launch
        __threadfence();
        if (atomicAdd(p.ticket + 1, 1) == (int)gridDim.x - 1) {
            p.ticket[0] = 0;
            p.ticket[1] = 0;
            __threadfence();
        }
    }
}

// =====================================================================================
// chain kernel (steps c and d)
// =====================================================================================
constexpr int CHAIN_THREADS = 384;
// tensor memory columns
constexpr uint32_t TM_DV = 0, TM_DS = 64, TM_SBF = 192, TM_V = 256, TM_VT = 288, TM_O1 = 320, TM_O2 = 384;
constexpr uint32_t CT_COLS = 512;
// shared memory: two stages of {K/Q tiles, V tile, -W^T, T2, P, gates}
// shared memory: operands are staged in two rings with different lifetimes.
//   ring A (2 deep): K/Q tiles, -W^T, P   -- used from the v_new MMA of a chunk to its last output MMA
//   ring B (3 deep): V tile, (T diag b)^T -- used only by the U^T MMA, which is issued one chunk early
//   gate vectors (4 deep): read by threads, not by MMAs; a slot is reused four chunks later, when
//   every reader of its previous contents has provably finished (no barrier needed)
// A slot is released by the completion of the last MMA that reads it, so its refill starts early.
constexpr uint32_t ST_KQ = 0, ST_W = 32768, ST_P = 49152;
constexpr uint32_t STAGE_A = 57344, STAGE_A_TX = 32768 + 16384 + 8192 + 1280;   // + the gate vectors
constexpr uint32_t ST_V = 0, ST_T2 = 16384;
constexpr uint32_t STAGE_B = 24576, STAGE_B_TX = 16384 + 8192;
constexpr uint32_t CS_A = 0, CS_B = 2 * STAGE_A, CS_GATES = CS_B + 3 * STAGE_B;
constexpr uint32_t CS_OST = CS_GATES + 4 * 1280;       // bf16 output staging [64][128]
constexpr uint32_t CS_BARS = CS_OST + 16384;
constexpr uint32_t CS_MISC = CS_BARS + 24 * 8;
constexpr uint32_t CS_TOTAL = CS_MISC + 64;
constexpr uint32_t CHAIN_SMEM = CS_TOTAL + 1024;

enum CBar : uint32_t { CB_FULLA0 = 0, CB_FREEA0 = 2, CB_FULLB0 = 4, CB_FREEB0 = 7, CB_V = 10, CB_S, CB_O, CB_SREADY, CB_VREADY, CB_OFREE,
                       CB_U, CB_O1, CB_CLEAN };

struct ChainParams {
    const float* s0;          // [N,H,d_k,d_v] or nullptr
    __nv_bfloat16* out;
    float* sT;
    const int32_t* cu;
    const uint8_t* items;
    const float* seg_sin;     // [B*nseg, H, d_k, d_v] incoming states of segments 1.. (sequence split), or nullptr
    float* dbg;               // debug build: time stamps of CTA (0,0,0), [role][chunk < 32][event < 8], ns
    int drop_chunk;           // tests only: the TMA thread of CTA (0,0,0) never loads this chunk (-1 = off), so
                              // that the bounded waits on it expire and the abort path runs
    int B, T, H, dv;
    int nseg, seg_chunks;     // segments per sequence (1 = no split) and chunks per segment
    float* snaps;             // optional [B, nsnap, H, d_k, d_v]: the state after every snap_every chunks
    int snap_every, nsnap;
    int l2;                   // bit 0: the K, Q, V tiles are read for the last time here: mark them first to be evicted; bit 1: W, T2 too
    // optional fused output stage (d_v = 128): out = o / sqrt(mean_j o_j^2 + norm_eps) * norm_w * silu(gate_z)
    const __nv_bfloat16* gate_z;   // [.., H, d_v] like out, or nullptr
    const float* norm_w;           // [d_v]
    float norm_eps;
};

// One CTA's identity inside a kernel: aligned shared-memory base (address and pointer), tensor-memory base,
// and the grid coordinates the stand-alone kernels take from blockIdx.
struct Cta {
    uint32_t base;
    uint8_t* sm;
    uint32_t tmem;
    int dvb, h, z;
};
// Grid-level hand-over inside the merged scan kernel: `flag` is a counter in global memory that the CTAs of one
// (sequence, head) raise when their part of a phase is written; a consumer waits (bounded) until it reads
// `target`.  nullptr = no waiting (stand-alone kernels: the kernel boundary orders everything).
struct Handover {
    const int* flag;
    int target;
};
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// One thread polls; returns false when the wait was given up (abort flag set, status raised).
__device__ __forceinline__ bool handover_wait(const Handover& hv, volatile int* abort_flag) {
    if (!hv.flag) return true;
    const unsigned long long t0 = globaltimer_ns();
    while (ld_acquire_gpu(hv.flag) < hv.target) {
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > TIMEOUT_NS) {
            *abort_flag = 1;
            atomicCAS(&g_lean_status, 0, (int)GDN_ERR_TIMEOUT);
            return false;
        }
        __nanosleep(40);
    }
    // data written with ordinary stores by other SMs is about to be read by bulk copies as well
    asm volatile("fence.proxy.async;" ::: "memory");
    return true;
}

__device__ __forceinline__ void chain_init_bars(const Waiter& w) {
    for (uint32_t i = 0; i < 2; ++i) { mbar_init(w.bar(CB_FULLA0 + i), 1); mbar_init(w.bar(CB_FREEA0 + i), 2); }   // both issuers
    mbar_init(w.bar(CB_U), 1); mbar_init(w.bar(CB_O1), 1);
    for (uint32_t i = 0; i < 3; ++i) { mbar_init(w.bar(CB_FULLB0 + i), 1); mbar_init(w.bar(CB_FREEB0 + i), 1); }
    mbar_init(w.bar(CB_V), 1); mbar_init(w.bar(CB_S), 1); mbar_init(w.bar(CB_O), 1);
    mbar_init(w.bar(CB_SREADY), 128); mbar_init(w.bar(CB_VREADY), 128); mbar_init(w.bar(CB_OFREE), 128);
    mbar_init(w.bar(CB_CLEAN), 128);
}

// Steps c and d for one CTA.  SCAN: called from the merged scan kernel (register budgets are set there, the
// incoming state is awaited through `hv` and read past the L1 cache, since another SM wrote it in this launch).
template <bool DBG, bool SCAN, bool GATED>
__device__ __forceinline__ void chain_body(const CUtensorMap* map_q, const CUtensorMap* map_k, const CUtensorMap* map_v,
                                           const ChainParams& p, const Cta& cta, const Waiter& w, const Handover& hv) {
    const uint32_t base = cta.base, tmem = cta.tmem;
    uint8_t* sm = cta.sm;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int dvb = cta.dvb, h = cta.h;
    const int n = cta.z / p.nseg, seg = cta.z % p.nseg;
    const int H = p.H, dv = p.dv;
    const SeqInfo sq = seq_info(p.cu, n, p.T);
    // this CTA walks chunks [seg * seg_chunks, ...) of the sequence
    const int cbeg = seg * p.seg_chunks;
    const long tok0 = sq.tok0 + (long)cbeg * C;
    const int len = max(0, min(sq.len - cbeg * C, p.seg_chunks * C));
    const int nchunks = (len + C - 1) / C;
    const long slot0 = slot_base(sq.tok0, n) + cbeg;
    // A last chunk with fewer than 64 tokens: its K and V tile rows behind the last token hold the first rows of
    // whatever follows the sequence in memory.  They only meet factors that are exactly zero, but zero times a
    // non-finite value is not zero, so the epilogue warpgroup clears them once the tiles have landed and the MMAs
    // that contract over tokens (U, the state update) wait for that (barrier CB_CLEAN, used once per CTA).
    const int tail_c = (nchunks > 0 && (len & (C - 1)) != 0) ? nchunks - 1 : -1;
    const unsigned long long t_start = DBG ? globaltimer_ns() : 0ull;
    auto stamp = [&](int role, int c, int ev) {
        if (DBG && p.dbg && dvb == 0 && h == 0 && cta.z == 0 && c < 32)
            p.dbg[(role * 32 + c) * 8 + ev] = (float)(globaltimer_ns() - t_start);
    };
    const size_t state_off = ((size_t)n * H + h) * DK * dv + (size_t)dvb * DVB;
    // With a split every segment, the first included, takes its incoming state from seg_sin (the combine
    // kernel copied the caller's initial state there): nothing reads initial_state once this kernel runs,
    // so final_state may alias it.
    const float* s_in = p.seg_sin ? p.seg_sin + ((size_t)(n * p.nseg + seg) * H + h) * DK * dv + (size_t)dvb * DVB
                                  : (p.s0 ? p.s0 + state_off : nullptr);

    if (warp < 4) {
        // =============================== chain warpgroup ===============================
        if (!SCAN) setmaxnreg_inc<232>();
        const int j = tid;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float S[DK];
        if (SCAN) {                                     // the combine phase of every slice of this head has been written
            if (tid == 0) handover_wait(hv, w.abort_flag);
            named_bar_sync(3, 128);
        }
        if (s_in) {
#pragma unroll
            for (int m = 0; m < DK; ++m) S[m] = SCAN ? __ldcg(s_in + (size_t)m * dv + j) : __ldg(s_in + (size_t)m * dv + j);
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
                tmem_st16(tmem + lane_base + TM_SBF + 16 * q, pk);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(w.bar(CB_SREADY));
        }
        for (int c = 0; c < nchunks; ++c) {
            const float* gates = reinterpret_cast<const float*>(sm + CS_GATES + (c & 3) * 1280);
            if (c > 0) w.wait_hot(CB_O, (c - 1) & 1);     // O2 of the previous chunk no longer reads bf16 v_new
            w.wait_hot(CB_V, c & 1);
            tc_fence_after_sync();
            if (tid == 0) stamp(0, c, 0);
            {
                // v_new^T: the load of the second half is in flight while the first is converted
                uint32_t xa[32], xb[32];
                tmem_ld32(tmem + lane_base + TM_DV, xa);
                tmem_wait_ld();
                tmem_ld32(tmem + lane_base + TM_DV + 32, xb);
                uint32_t pv[16], pd[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float v0 = __uint_as_float(xa[2 * i]), v1 = __uint_as_float(xa[2 * i + 1]);
                    const float2 dec = *reinterpret_cast<const float2*>(gates + 192 + 2 * i);
                    pv[i] = pack_bf16(v0, v1);
                    pd[i] = pack_bf16(v0 * dec.x, v1 * dec.y);
                }
                tmem_st16(tmem + lane_base + TM_V, pv);
                tmem_st16(tmem + lane_base + TM_VT, pd);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float v0 = __uint_as_float(xb[2 * i]), v1 = __uint_as_float(xb[2 * i + 1]);
                    const float2 dec = *reinterpret_cast<const float2*>(gates + 224 + 2 * i);
                    pv[i] = pack_bf16(v0, v1);
                    pd[i] = pack_bf16(v0 * dec.x, v1 * dec.y);
                }
                tmem_st16(tmem + lane_base + TM_V + 16, pv);
                tmem_st16(tmem + lane_base + TM_VT + 16, pd);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(w.bar(CB_VREADY));
            if (tid == 0) stamp(0, c, 1);
            w.wait_hot(CB_O1, c & 1);                      // O1 of this chunk no longer reads the bf16 state
            w.wait_hot(CB_S, c & 1);
            tc_fence_after_sync();
            if (tid == 0) stamp(0, c, 2);
            const float gamma = gates[256];
            {
                // S^T <- e^{gC} S^T + dS^T, 32 columns at a time, the next load always in flight
                uint32_t da[32], db[32];
                tmem_ld32(tmem + lane_base + TM_DS, da);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t (&cur)[32] = (q & 1) ? db : da;
                    uint32_t (&nxt)[32] = (q & 1) ? da : db;
                    if (q < 3) tmem_ld32(tmem + lane_base + TM_DS + 32 * (q + 1), nxt);
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; ++i) S[32 * q + i] = fmaf(gamma, S[32 * q + i], __uint_as_float(cur[i]));
#pragma unroll
                    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(S[32 * q + 2 * i], S[32 * q + 2 * i + 1]);
                    tmem_st16(tmem + lane_base + TM_SBF + 16 * q, pk);
                    if (q < 3) tmem_wait_ld();
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(w.bar(CB_SREADY));
            if (tid == 0) stamp(0, c, 3);
            if (p.snaps) {                              // state snapshot at a chunk boundary (off the chain: plain stores)
                const int gc = cbeg + c + 1;            // chunks of the sequence consumed so far
                if (gc % p.snap_every == 0 && gc / p.snap_every <= p.nsnap && gc * C <= sq.len) {
                    float* dst = p.snaps + (((size_t)n * p.nsnap + (gc / p.snap_every - 1)) * H + h) * DK * dv +
                                 (size_t)dvb * DVB + j;
#pragma unroll
                    for (int m = 0; m < DK; ++m) dst[(size_t)m * dv] = S[m];
                }
            }
        }
        if (p.sT && seg == p.nseg - 1) {
#pragma unroll
            for (int m = 0; m < DK; ++m) p.sT[state_off + (size_t)m * dv + j] = S[m];
        }
    } else if (warp < 8) {
        // =============================== epilogue warpgroup ===============================
        const int j = tid - 128, we = j >> 5;
        const uint32_t lane_base = (uint32_t)(we * 32) << 16;
        __nv_bfloat16* ost = reinterpret_cast<__nv_bfloat16*>(sm + CS_OST);
        for (int c = 0; c < nchunks; ++c) {
            const int R = min(C, len - c * C);
            const float* gates = reinterpret_cast<const float*>(sm + CS_GATES + (c & 3) * 1280);
            if (tail_c >= 0 && c == max(tail_c - 1, 0)) {
                const int Rt = len - tail_c * C;
                const uint32_t sa = base + CS_A + (uint32_t)(tail_c & 1) * STAGE_A + ST_KQ;
                const uint32_t sv = base + CS_B + (uint32_t)(tail_c % 3) * STAGE_B + ST_V;
                w.wait(CB_FULLA0 + (tail_c & 1), (tail_c >> 1) & 1);
                w.wait(CB_FULLB0 + tail_c % 3, (tail_c / 3) & 1);
                const uint32_t pieces = (uint32_t)(C - Rt) * 8u;
                for (uint32_t x = j; x < 4 * pieces; x += 128) {             // K_lo, K_hi, V_lo, V_hi
                    const uint32_t t4 = x / pieces, y = x - t4 * pieces;
                    const uint32_t tile = t4 == 0 ? sa : t4 == 1 ? sa + 16384 : t4 == 2 ? sv : sv + 8192;
                    st_shared_v4(tile + ((uint32_t)Rt + (y >> 3)) * 128 + ((y & 7) << 4), 0u, 0u, 0u, 0u);
                }
                fence_proxy_async_smem();
                mbar_arrive(w.bar(CB_CLEAN));
            }
            w.wait_hot(CB_O, c & 1);
            tc_fence_after_sync();
            // take both accumulators out of tensor memory first and hand them back at once: the next
            // chunk's output MMAs wait for this
            uint32_t o1a[32], o1b[32], o2a[32], o2b[32];
            tmem_ld32(tmem + lane_base + TM_O1, o1a);
            tmem_ld32(tmem + lane_base + TM_O1 + 32, o1b);
            tmem_ld32(tmem + lane_base + TM_O2, o2a);
            tmem_ld32(tmem + lane_base + TM_O2 + 32, o2b);
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(w.bar(CB_OFREE));
            if (GATED) {
                // Fused output stage (the per-position kernels behind the scan, Section "Prefill projections:
                // dequantize, then call the vendor"): root-mean-square norm of each output row over the value
                // axis, weight vector, SiLU gate.  The rows go through shared memory in fp32, 32 tokens at a
                // time; sixteen neighbouring lanes hold one row and add up its squares by shuffles.
                float* fst = reinterpret_cast<float*>(sm + CS_OST);           // [32][128] fp32, the same 16 KiB
                const size_t row0 = (size_t)(tok0 + c * C) * H + h;
                const int col = (j & 15) * 8;
                const float4 w0 = __ldg(reinterpret_cast<const float4*>(p.norm_w + col));
                const float4 w1 = __ldg(reinterpret_cast<const float4*>(p.norm_w + col + 4));
                const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        fst[i * DVB + j] = half ? fmaf(gates[160 + i], __uint_as_float(o1b[i]), __uint_as_float(o2b[i]))
                                                : fmaf(gates[128 + i], __uint_as_float(o1a[i]), __uint_as_float(o2a[i]));
                    named_bar_sync(2, 128);
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int rr = (it * 128 + j) >> 4, r = 32 * half + rr;
                        const float4 x0 = *reinterpret_cast<const float4*>(fst + rr * DVB + col);
                        const float4 x1 = *reinterpret_cast<const float4*>(fst + rr * DVB + col + 4);
                        const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                        float ss = 0.f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) ss = fmaf(xv[e], xv[e], ss);
#pragma unroll
                        for (int d = 1; d < 16; d <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
                        const float inv = rsqrtf(ss * (1.0f / DVB) + p.norm_eps);
                        if (r < R) {
                            const size_t off = (row0 + (size_t)r * H) * dv + col;
                            const uint4 zz = *reinterpret_cast<const uint4*>(p.gate_z + off);
                            const uint32_t zu[4] = {zz.x, zz.y, zz.z, zz.w};
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float z0 = __uint_as_float(zu[e] << 16), z1 = __uint_as_float(zu[e] & 0xffff0000u);
                                const float y0 = xv[2 * e] * inv * wv[2 * e] * (z0 / (1.0f + __expf(-z0)));
                                const float y1 = xv[2 * e + 1] * inv * wv[2 * e + 1] * (z1 / (1.0f + __expf(-z1)));
                                pk[e] = pack_bf16(y0, y1);
                            }
                            *reinterpret_cast<uint4*>(p.out + off) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                    }
                    named_bar_sync(2, 128);
                }
                continue;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float oa = fmaf(gates[128 + i], __uint_as_float(o1a[i]), __uint_as_float(o2a[i]));
                const float ob = fmaf(gates[160 + i], __uint_as_float(o1b[i]), __uint_as_float(o2b[i]));
                ost[i * DVB + j] = __float2bfloat16_rn(oa);           // transpose through shared memory
                ost[(32 + i) * DVB + j] = __float2bfloat16_rn(ob);
            }
            named_bar_sync(2, 128);
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
        }
    } else {
        // =============================== control warpgroup ===============================
        if (!SCAN) setmaxnreg_dec<56>();
        if (warp == 8 && lane == 0) {
            // ---- MMA issuer of the sequential chain: v_new and the state update, nothing else ----
            // (issuing costs tens of nanoseconds per instruction; everything off the chain is
            //  issued by a second thread so that it does not sit between two dependent steps)
            // operand descriptors are built once per stage, outside the dependent chain: the address field
            // counts 16-byte units, so a k-step is a plain add
            const uint64_t dW0 = make_smem_desc(base + CS_A + ST_W, 1024, 1024);
            const uint64_t dK0 = make_smem_desc(base + CS_A + ST_KQ, 16384, 1024);
            for (int c = 0; c < nchunks; ++c) {
                const uint32_t s = c & 1;
                const uint64_t dW = dW0 + (uint64_t)((s * STAGE_A) >> 4), dK = dK0 + (uint64_t)((s * STAGE_A) >> 4);
                // the waits that are normally long satisfied come first: whatever follows the wait on the
                // state sits on the dependent chain
                w.wait_hot(CB_FULLA0 + s, (c >> 1) & 1);
                w.wait_hot(CB_U, c & 1);                       // U^T of this chunk is in the accumulator
                if (c == tail_c) w.wait_hot(CB_CLEAN, 0);      // padded K rows have been cleared
                w.wait_hot(CB_SREADY, c & 1);
                tc_fence_after_sync();
                stamp(1, c, 0);
#pragma unroll
                for (uint32_t ks = 0; ks < 8; ++ks)            // v^T = U^T - S^T W^T
                    mma_ts(tmem + TM_DV, tmem + TM_SBF + ks * 8, dW + ks * 128, ID_1, 1);
                mma_commit(w.bar(CB_V));
                stamp(1, c, 1);
                w.wait_hot(CB_VREADY, c & 1);
                tc_fence_after_sync();
                stamp(1, c, 3);
#pragma unroll
                for (uint32_t ks = 0; ks < 4; ++ks)            // dS^T = (v e^{gC-g})^T K
                    mma_ts(tmem + TM_DS, tmem + TM_VT + ks * 8, dK + ks * 128, ID_2, ks > 0);
                mma_commit(w.bar(CB_S));
                mma_commit(w.bar(CB_FREEA0 + s));
                stamp(1, c, 4);
            }
        } else if (warp == 10 && lane == 0) {
            // ---- MMA issuer of everything off the chain: U^T, O1^T, O2^T ----
            // (descriptors are built once; a stage or a k-step is an add on the 16-byte address field.  Every warp
            //  role runs its loop at the same time, so the size of these loops shows in the instruction cache.)
            const uint64_t dV0 = make_smem_desc(base + CS_B + ST_V, 8192, 1024), dT0 = make_smem_desc(base + CS_B + ST_T2, 1024, 1024);
            const uint64_t dQ0 = make_smem_desc(base + CS_A + ST_KQ + 8192, 16, 1024), dP0 = make_smem_desc(base + CS_A + ST_P, 16, 1024);
            for (int c = -1; c < nchunks; ++c) {
                const uint32_t s = c & 1;
                const uint64_t soff = (uint64_t)((s * STAGE_A) >> 4);
                if (c >= 0) {
                    w.wait(CB_SREADY, c & 1);
                    w.wait(CB_FULLA0 + s, (c >> 1) & 1);
                    if (c > 0) w.wait(CB_OFREE, (c - 1) & 1);  // the epilogue has read the previous O1, O2
                    w.wait_hot(CB_V, c & 1);                   // stay out of the tensor pipe until v_new is done
                    tc_fence_after_sync();
#pragma unroll
                    for (uint32_t ks = 0; ks < 8; ++ks)        // O1^T = S^T Q^T
                        mma_ts(tmem + TM_O1, tmem + TM_SBF + ks * 8, dQ0 + soff + (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                               ID_O, ks > 0);
                    mma_commit(w.bar(CB_O1));
                    w.wait(CB_VREADY, c & 1);
                    tc_fence_after_sync();
                }
                if (c + 1 < nchunks) {                         // U^T = V^T (T diag(b))^T of chunk c + 1: D_v is free,
                    const uint32_t sB = (c + 1) % 3;           // v_new of chunk c has been read
                    const uint64_t boff = (uint64_t)((sB * STAGE_B) >> 4);
                    w.wait(CB_FULLB0 + sB, ((c + 1) / 3) & 1);
                    if (c + 1 == tail_c) w.wait(CB_CLEAN, 0);  // padded V rows have been cleared
#pragma unroll
                    for (uint32_t ks = 0; ks < 4; ++ks)
                        mma_ss(tmem + TM_DV, dV0 + boff + ks * 128, dT0 + boff + ks * 128, ID_WU, ks > 0);
                    mma_commit(w.bar(CB_FREEB0 + sB));
                    mma_commit(w.bar(CB_U));
                }
                if (c >= 0) {
#pragma unroll
                    for (uint32_t ks = 0; ks < 4; ++ks)        // O2^T = v^T P^T
                        mma_ts(tmem + TM_O2, tmem + TM_V + ks * 8, dP0 + soff + ks * 2, ID_O, ks > 0);
                    mma_commit(w.bar(CB_O));
                    mma_commit(w.bar(CB_FREEA0 + s));
                }
            }
        } else if (warp == 9 && lane == 0) {
            // ---- TMA producer ----
            prefetch_tensormap(map_q);
            prefetch_tensormap(map_k);
            prefetch_tensormap(map_v);
            const uint64_t pol_done = (p.l2 & 1) ? l2_policy_evict_first() : l2_policy_evict_normal();
            const uint64_t pol_item = (p.l2 & 2) ? l2_policy_evict_first() : l2_policy_evict_normal();
            for (int c = 0; c < nchunks; ++c) {
                if (c == p.drop_chunk && dvb == 0 && h == 0 && cta.z == 0) continue;
                const int tok = (int)(tok0 + (long)c * C);
                const uint8_t* item = p.items + (size_t)((slot0 + c) * H + h) * ITEM_BYTES;
                {   // ring B: V tile and (T diag(b))^T
                    const uint32_t sB = c % 3, bb = base + CS_B + sB * STAGE_B, full = w.bar(CB_FULLB0 + sB);
                    if (c >= 3) w.wait(CB_FREEB0 + sB, ((c / 3) - 1) & 1);
                    mbar_arrive_expect_tx(full, STAGE_B_TX);
                    tma_load_3d_hint(bb + ST_V, map_v, dvb * DVB, h, tok, full, pol_done);
                    tma_load_3d_hint(bb + ST_V + 8192, map_v, dvb * DVB + 64, h, tok, full, pol_done);
                    bulk_load_hint(bb + ST_T2, item + IT_T2, 8192, full, pol_item);
                }
                {   // ring A: K/Q tiles, -W^T, P, and the gate vectors (own 4-deep ring, same barrier)
                    const uint32_t s = c & 1, sb = base + CS_A + s * STAGE_A, full = w.bar(CB_FULLA0 + s);
                    if (c >= 2) w.wait(CB_FREEA0 + s, ((c >> 1) - 1) & 1);
                    mbar_arrive_expect_tx(full, STAGE_A_TX);
                    bulk_load_hint(sb + ST_W, item + IT_W, 16384, full, pol_item);
                    tma_load_3d_hint(sb + ST_KQ, map_k, 0, h, tok, full, pol_done);
                    tma_load_3d_hint(sb + ST_KQ + 8192, map_q, 0, h, tok, full, pol_done);
                    tma_load_3d_hint(sb + ST_KQ + 16384, map_k, 64, h, tok, full, pol_done);
                    tma_load_3d_hint(sb + ST_KQ + 24576, map_q, 64, h, tok, full, pol_done);
                    bulk_load(sb + ST_P, item + IT_P, 8192, full);
                    bulk_load(base + CS_GATES + (c & 3) * 1280, item + IT_GATES, 1280, full);
                }
            }
            if (*w.abort_flag) {
                // let copies in flight land before shared memory is released (bounded)
                const unsigned long long t0 = globaltimer_ns();
                for (int c = max(0, nchunks - 3); c < nchunks; ++c) {
                    while (!mbar_try_wait(w.bar(CB_FULLB0 + c % 3), (c / 3) & 1) && globaltimer_ns() - t0 < TIMEOUT_NS) {}
                    if (c >= nchunks - 2)
                        while (!mbar_try_wait(w.bar(CB_FULLA0 + (c & 1)), (c >> 1) & 1) && globaltimer_ns() - t0 < TIMEOUT_NS) {}
                }
            }
        }
    }
}

template <bool DBG, bool GATED>
__global__ void __launch_bounds__(CHAIN_THREADS, 1)
gdn_chain_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + CS_MISC);
    Waiter w{base + CS_BARS, reinterpret_cast<volatile int*>(sm + CS_MISC + 4)};
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        chain_init_bars(w);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + CS_MISC, CT_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];
    pdl_wait();                         // scratch items and incoming states come from the kernels before this one
    const Cta cta{base, sm, tmem, (int)blockIdx.x, (int)blockIdx.y, (int)blockIdx.z};
    chain_body<DBG, false, GATED>(&map_q, &map_k, &map_v, p, cta, w, Handover{nullptr, 0});
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, CT_COLS);
    }
}


// =====================================================================================
// sequence split: segment summaries and their combination
//
// With few (sequence, head) chains the chain kernel leaves most SMs idle.  A sequence is
// then cut into segments; every column s of the state obeys, over a segment,
//     s_out = M_seg s_in + n_seg ,   M_seg = M_cL ... M_c1 ,  M_c = e^{gC} I - K~^T W
// (the S^(c+1) = M_c S^(c) + N_c form of Section "A chunked delta-rule scan for the
// recurrent layers", composed over the chunks of a segment).  gdn_summary_kernel runs,
// per segment, the chain from a zero state (giving N_seg = n_seg for all value columns)
// and the homogeneous chain from the identity (giving M_seg); gdn_combine_kernel walks
// the segments in fp32, S_in[p+1] = M_p S_in[p] + N_p; the chain kernel then runs every
// segment from its true incoming state.
// =====================================================================================
constexpr int SUM_THREADS = 384;
constexpr uint32_t CMB_IMG = 65536;                         // M_seg^T per (segment, head): leading bf16 image | remainder image
constexpr uint32_t SS_K = 0, SS_V = 16384, SS_W = 32768, SS_T2 = 49152, SS_GATES = 57344;
constexpr uint32_t SUM_STAGE = 59392;                       // 58 KiB
constexpr uint32_t SUM_STAGE_TX = 16384 + 16384 + 16384 + 8192 + 1280;
constexpr uint32_t SUM_STAGES = 3;
constexpr uint32_t SUS_BARS = SUM_STAGES * SUM_STAGE;
constexpr uint32_t SUS_MISC = SUS_BARS + 24 * 8;
constexpr uint32_t SUM_SMEM = SUS_MISC + 64 + 1024;
// tensor memory: instance 0 (values) and instance 1 (identity); bf16 state aliases the first
// 64 columns of its own dS accumulator (read by MMA1 strictly before MMA2 overwrites it)
__device__ __forceinline__ uint32_t sum_dv(int inst) { return inst ? 224u : 0u; }     // U^T / v_new^T
__device__ __forceinline__ uint32_t sum_ds(int inst) { return inst ? 288u : 64u; }    // dS^T and bf16 S^T
__device__ __forceinline__ uint32_t sum_vt(int inst) { return inst ? 416u : 192u; }   // bf16 decayed v_new^T
constexpr uint32_t SUM_COLS = 512;

enum SBar : uint32_t { SB_FULL0 = 0, SB_FREE0 = 3, SB_V0 = 6, SB_S0 = 8, SB_SREADY0 = 10, SB_VREADY0 = 12 };

struct SummaryParams {
    const int32_t* cu;
    const uint8_t* items;
    float* seg_n;             // [B*nseg, H, d_k, d_v]   N_seg
    float* seg_mt;            // [B*nseg, H] x 64 KiB: M_seg^T as two bf16 operand images (leading part | remainder)
    int B, T, H, dv;
    int nseg, seg_chunks;
    int l2;                   // bit 0: K and V are read again by the chain phase and fit in L2: keep them there; bit 1: W, T2 too
};

__device__ __forceinline__ void summary_init_bars(const Waiter& w, int ninst) {
    for (uint32_t i = 0; i < SUM_STAGES; ++i) {
        mbar_init(w.bar(SB_FULL0 + i), 1);
        mbar_init(w.bar(SB_FREE0 + i), 129 * ninst);         // per instance: its issue thread and its warpgroup
    }
    for (uint32_t i = 0; i < 2; ++i) {
        mbar_init(w.bar(SB_V0 + i), 1); mbar_init(w.bar(SB_S0 + i), 1);
        mbar_init(w.bar(SB_SREADY0 + i), 128); mbar_init(w.bar(SB_VREADY0 + i), 128);
    }
}

// Segment summary (M_seg, N_seg) of one CTA; cta.z = sequence * (nseg - 1) + segment.
template <bool SCAN>
__device__ __forceinline__ void summary_body(const CUtensorMap* map_k, const CUtensorMap* map_v, const SummaryParams& p,
                                             const Cta& cta, const Waiter& w) {
    const uint32_t base = cta.base, tmem = cta.tmem;
    uint8_t* sm = cta.sm;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int dvb = cta.dvb, h = cta.h;
    const int nsum = p.nseg - 1;                      // the last segment needs no summary
    const int n = cta.z / nsum, seg = cta.z % nsum;
    const int H = p.H, dv = p.dv;
    const SeqInfo sq = seq_info(p.cu, n, p.T);
    const int cbeg = seg * p.seg_chunks;
    const long tok0 = sq.tok0 + (long)cbeg * C;
    const int len = max(0, min(sq.len - cbeg * C, p.seg_chunks * C));
    const int nchunks = (len + C - 1) / C;
    const long slot0 = slot_base(sq.tok0, n) + cbeg;
    const bool with_m = (dvb == 0);                   // M_seg does not depend on the value columns
    const int ninst = with_m ? 2 : 1;

    if (warp < 8) {
        // ======================= two chain warpgroups: values (0) and identity (1) =======================
        if (!SCAN) setmaxnreg_inc<224>();
        const int inst = warp >> 2;
        const int j = tid & 127;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        if (inst < ninst) {
            float S[DK];
#pragma unroll
            for (int m = 0; m < DK; ++m) S[m] = (inst == 1 && m == j) ? 1.f : 0.f;
            if (nchunks > 0) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(S[32 * q + 2 * i], S[32 * q + 2 * i + 1]);
                    tmem_st16(tmem + lane_base + sum_ds(inst) + 16 * q, pk);
                }
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(w.bar(SB_SREADY0 + inst));
            }
            for (int c = 0; c < nchunks; ++c) {
                const uint32_t s = c % SUM_STAGES;
                const float* gates = reinterpret_cast<const float*>(sm + s * SUM_STAGE + SS_GATES);
                w.wait_hot(SB_V0 + inst, c & 1);
                tc_fence_after_sync();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t x[32];
                    tmem_ld32(tmem + lane_base + sum_dv(inst) + 32 * hh, x);
                    tmem_wait_ld();
                    uint32_t pd[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float2 dec = *reinterpret_cast<const float2*>(gates + 192 + 32 * hh + 2 * i);
                        pd[i] = pack_bf16(__uint_as_float(x[2 * i]) * dec.x, __uint_as_float(x[2 * i + 1]) * dec.y);
                    }
                    tmem_st16(tmem + lane_base + sum_vt(inst) + 16 * hh, pd);
                }
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(w.bar(SB_VREADY0 + inst));
                w.wait_hot(SB_S0 + inst, c & 1);
                tc_fence_after_sync();
                const float gamma = gates[256];
                mbar_arrive(w.bar(SB_FREE0 + s));
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t d[32];
                    tmem_ld32(tmem + lane_base + sum_ds(inst) + 32 * q, d);
                    tmem_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; ++i) S[32 * q + i] = fmaf(gamma, S[32 * q + i], __uint_as_float(d[i]));
#pragma unroll
                    for (int i = 0; i < 16; ++i) pk[i] = pack_bf16(S[32 * q + 2 * i], S[32 * q + 2 * i + 1]);
                    tmem_st16(tmem + lane_base + sum_ds(inst) + 16 * q, pk);   // columns already read
                }
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(w.bar(SB_SREADY0 + inst));
            }
            const size_t sidx = (size_t)(n * p.nseg + seg) * H + h;
            if (inst == 0) {
                float* dst = p.seg_n + sidx * DK * dv + (size_t)dvb * DVB + j;       // [m][j]
#pragma unroll
                for (int m = 0; m < DK; ++m) dst[(size_t)m * dv] = S[m];
            } else {
                // M_seg^T leaves as two bf16 operand images (leading part, remainder): row i = j holds
                // M_seg[m][i] for all m, in the layout the combine kernel's MMAs read (128-byte swizzle,
                // blocks of 64 rows x 64 columns).  Leading part + remainder carry 16 mantissa bits.
                uint8_t* img = reinterpret_cast<uint8_t*>(p.seg_mt) + sidx * CMB_IMG + (uint32_t)(j >> 6) * 16384;
                const uint32_t r = (uint32_t)j & 63u;
#pragma unroll
                for (int mh = 0; mh < 2; ++mh)
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float x0 = S[64 * mh + 8 * ch + 2 * e], x1 = S[64 * mh + 8 * ch + 2 * e + 1];
                            hi[e] = pack_bf16(x0, x1);
                            lo[e] = pack_bf16(x0 - __uint_as_float(hi[e] << 16), x1 - __uint_as_float(hi[e] & 0xffff0000u));
                        }
                        uint8_t* dst = img + mh * 8192 + swz(r, ch);
                        st_global_v4(dst, hi[0], hi[1], hi[2], hi[3]);
                        st_global_v4(dst + CMB_IMG / 2, lo[0], lo[1], lo[2], lo[3]);
                    }
            }
        }
    } else {
        // =============================== control warpgroup ===============================
        if (!SCAN) setmaxnreg_dec<56>();
        if ((warp == 8 || warp == 10) && lane == 0) {
            // ---- one MMA issue thread per chain instance (they are independent) ----
            const int inst = (warp == 8) ? 0 : 1;
            if (inst < ninst) {
                const uint64_t dW0 = make_smem_desc(base + SS_W, 1024, 1024), dK0 = make_smem_desc(base + SS_K, 8192, 1024);
                for (int c = 0; c < nchunks; ++c) {
                    const uint32_t s = c % SUM_STAGES, sb = base + s * SUM_STAGE;
                    const uint64_t dW = dW0 + (uint64_t)((s * SUM_STAGE) >> 4), dK = dK0 + (uint64_t)((s * SUM_STAGE) >> 4);
                    w.wait_hot(SB_FULL0 + s, (c / SUM_STAGES) & 1);
                    if (inst == 0) {
                        tc_fence_after_sync();
#pragma unroll
                        for (uint32_t ks = 0; ks < 4; ++ks)        // U^T = V^T (T diag(b))^T
                            mma_ss(tmem + sum_dv(0), make_smem_desc(sb + SS_V + ks * 2048, 8192, 1024),
                                   make_smem_desc(sb + SS_T2 + ks * 2048, 1024, 1024), ID_WU, ks > 0);
                    }
                    w.wait_hot(SB_SREADY0 + inst, c & 1);
                    tc_fence_after_sync();
#pragma unroll
                    for (uint32_t ks = 0; ks < 8; ++ks)            // v^T = U^T - S^T W^T   (U = 0 for the identity chain)
                        mma_ts(tmem + sum_dv(inst), tmem + sum_ds(inst) + ks * 8,
                               dW + ks * 128, ID_1, (inst == 0 || ks > 0) ? 1u : 0u);
                    mma_commit(w.bar(SB_V0 + inst));
                    w.wait_hot(SB_VREADY0 + inst, c & 1);
                    tc_fence_after_sync();
#pragma unroll
                    for (uint32_t ks = 0; ks < 4; ++ks)            // dS^T = (v e^{gC-g})^T K
                        mma_ts(tmem + sum_ds(inst), tmem + sum_vt(inst) + ks * 8,
                               dK + ks * 128, ID_2, ks > 0);
                    mma_commit(w.bar(SB_S0 + inst));
                    mma_commit(w.bar(SB_FREE0 + s));
                }
            }
        } else if (warp == 9 && lane == 0) {
            prefetch_tensormap(map_k);
            prefetch_tensormap(map_v);
            const uint64_t pol_keep = (p.l2 & 1) ? l2_policy_evict_last() : l2_policy_evict_normal();
            const uint64_t pol_item = (p.l2 & 2) ? l2_policy_evict_last() : l2_policy_evict_normal();
            for (int c = 0; c < nchunks; ++c) {
                const uint32_t s = c % SUM_STAGES, sb = base + s * SUM_STAGE;
                if (c >= (int)SUM_STAGES) w.wait(SB_FREE0 + s, ((c / SUM_STAGES) - 1) & 1);
                const uint32_t full = w.bar(SB_FULL0 + s);
                const int tok = (int)(tok0 + (long)c * C);
                const uint8_t* item = p.items + (size_t)((slot0 + c) * H + h) * ITEM_BYTES;
                mbar_arrive_expect_tx(full, SUM_STAGE_TX);
                tma_load_3d_hint(sb + SS_K, map_k, 0, h, tok, full, pol_keep);
                tma_load_3d_hint(sb + SS_K + 8192, map_k, 64, h, tok, full, pol_keep);
                tma_load_3d_hint(sb + SS_V, map_v, dvb * DVB, h, tok, full, pol_keep);
                tma_load_3d_hint(sb + SS_V + 8192, map_v, dvb * DVB + 64, h, tok, full, pol_keep);
                bulk_load_hint(sb + SS_W, item + IT_W, 16384, full, pol_item);
                bulk_load_hint(sb + SS_T2, item + IT_T2, 8192, full, pol_item);
                bulk_load(sb + SS_GATES, item + IT_GATES, 1280, full);
            }
            if (*w.abort_flag) {
                for (int c = max(0, nchunks - (int)SUM_STAGES); c < nchunks; ++c) {
                    const uint32_t bar = w.bar(SB_FULL0 + (c % SUM_STAGES));
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar, (c / SUM_STAGES) & 1) && globaltimer_ns() - t0 < TIMEOUT_NS) {}
                }
            }
        }
    }
}

__global__ void __launch_bounds__(SUM_THREADS, 1)
gdn_summary_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   SummaryParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + SUS_MISC);
    Waiter w{base + SUS_BARS, reinterpret_cast<volatile int*>(sm + SUS_MISC + 4)};
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        summary_init_bars(w, blockIdx.x == 0 ? 2 : 1);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + SUS_MISC, SUM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];
    pdl_trigger();
    pdl_wait();                         // the scratch items come from the prepare kernel
    const Cta cta{base, sm, tmem, (int)blockIdx.x, (int)blockIdx.y, (int)blockIdx.z};
    summary_body<false>(&map_k, &map_v, p, cta, w);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, SUM_COLS);
    }
}

// S_in[p+1] = M_p S_in[p] + N_p, p = 0 .. nseg-2; one CTA per (sequence, head, CMB_COLS value columns).
// Each hop is a 128 x CMB_COLS x 128 product on the tensor core with both factors split into a leading bf16
// part and a bf16 remainder (hi*hi + lo*hi + hi*lo, fp32 accumulation: 16 mantissa bits per factor), so
// the hops cost MMA round trips instead of fp32 FMAs.  A = M_p as the two operand images the summary kernel
// wrote (bulk copies, three segments ahead); B = the state slice, written to shared memory by the
// thread that owns each row; D in tensor memory.  The incoming state of segment 0 is copied to seg_sin as
// well, so that no later kernel reads the caller's initial_state (which final_state may alias).
constexpr int CMB_COLS = 16;                           // value columns per CTA.  Measured on the 10240-token workload: a hop takes
                                                       // about 1.0 us + 0.05 us per column (each thread converts, stores and
                                                       // reloads its own row), so narrow slices on many SMs win
constexpr int CMB_THREADS = 224;                       // warps 0-3: one state row per thread; warps 4-6: one MMA issue thread per partial product
constexpr uint32_t CMB_STAGES = 3;
constexpr uint32_t CMB_BIMG = CMB_COLS * 256;          // one image of the state slice: [column][row m], two 64-row blocks
constexpr uint32_t CM_B = CMB_STAGES * CMB_IMG;        // state slice images: leading part | remainder
constexpr uint32_t CM_BARS = CM_B + 2 * CMB_BIMG;
constexpr uint32_t CM_MISC = CM_BARS + 16 * 8;
constexpr uint32_t CMB_SMEM = CM_MISC + 64 + 1024;
constexpr uint32_t CMB_TCOLS = 64;                     // three accumulators of CMB_COLS columns (one per partial product)
static_assert(3 * CMB_COLS <= CMB_TCOLS, "accumulators of the three partial products");
enum MBar : uint32_t { MB_FULL0 = 0, MB_FREE0 = 3, MB_BREADY = 6, MB_D = 7 };
constexpr uint32_t ID_CMB = make_idesc(128, CMB_COLS, kFmtBF16, kFmtBF16, kMajorMN, kMajorK);

struct CombineParams {
    const float* s0;          // [B, H, d_k, d_v] or nullptr
    const float* seg_n;
    const float* seg_mt;      // per (sequence, segment, head): leading | remainder image of M_seg^T
    float* seg_sin;
    int H, dv, nseg;
};

__device__ __forceinline__ void combine_init_bars(const Waiter& w) {
    for (uint32_t i = 0; i < CMB_STAGES; ++i) { mbar_init(w.bar(MB_FULL0 + i), 1); mbar_init(w.bar(MB_FREE0 + i), 3); }
    mbar_init(w.bar(MB_BREADY), 128);
    mbar_init(w.bar(MB_D), 3);                             // one commit per issue thread
}

// The hops of one column slice (cta.dvb = slice, cta.z = sequence).  Warps 0-3 own the rows, lane 0 of warp
// `issue_warp` copies and issues.  SCAN: inside the merged scan kernel the summaries were written by other SMs
// during this launch, so they are read past the L1 cache and no programmatic-launch wait applies.
template <bool SCAN>
__device__ __forceinline__ void combine_body(const CombineParams& p, const Cta& cta, const Waiter& w, int issue_warp) {
    const uint32_t base = cta.base, tmem = cta.tmem;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j0 = cta.dvb * CMB_COLS, h = cta.h, n = cta.z;
    const int H = p.H, dv = p.dv, nhops = p.nseg - 1;
    auto seg_off = [&](int seg) { return ((size_t)(n * p.nseg + seg) * H + h) * DK * dv; };

    if (warp < 4) {
        // ---- thread m owns row m of the slice ----
        const int m = tid;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float s[CMB_COLS];
        if (p.s0) {   // the initial state is an input of the call: it may be read before the predecessor has finished
            const float4* src = reinterpret_cast<const float4*>(p.s0 + (((size_t)n * H + h) * DK + m) * dv + j0);
#pragma unroll
            for (int q = 0; q < CMB_COLS / 4; ++q) { const float4 x = __ldg(src + q); s[4 * q] = x.x; s[4 * q + 1] = x.y; s[4 * q + 2] = x.z; s[4 * q + 3] = x.w; }
        } else {
#pragma unroll
            for (int j = 0; j < CMB_COLS; ++j) s[j] = 0.f;
        }
        if (!SCAN) pdl_wait();          // M_seg, N_seg come from the summary kernel
        auto store_sin = [&](int seg) {
            float4* dst = reinterpret_cast<float4*>(p.seg_sin + seg_off(seg) + (size_t)m * dv + j0);
#pragma unroll
            for (int q = 0; q < CMB_COLS / 4; ++q) dst[q] = make_float4(s[4 * q], s[4 * q + 1], s[4 * q + 2], s[4 * q + 3]);
        };
        // element (column j, row m) of the K-major B images: the two 64-row blocks of m are CMB_COLS * 128 bytes apart
        const uint32_t bcol = base + CM_B + (uint32_t)(m >> 6) * (CMB_COLS * 128) + (uint32_t)(m & 7) * 2;
        const uint32_t bchunk = (uint32_t)(m & 63) >> 3;
        for (int seg = 0; seg < nhops; ++seg) {
            float4 nv[CMB_COLS / 4];
            const float4* nsrc = reinterpret_cast<const float4*>(p.seg_n + seg_off(seg) + (size_t)m * dv + j0);
#pragma unroll
            for (int q = 0; q < CMB_COLS / 4; ++q) nv[q] = SCAN ? __ldcg(nsrc + q) : __ldg(nsrc + q);
#pragma unroll
            for (int j = 0; j < CMB_COLS; ++j) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(s[j]);
                const __nv_bfloat16 lo = __float2bfloat16_rn(s[j] - __bfloat162float(hi));
                const uint32_t addr = bcol + (uint32_t)j * 128 + ((bchunk ^ ((uint32_t)j & 7u)) << 4);
                asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(*reinterpret_cast<const unsigned short*>(&hi)) : "memory");
                asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr + CMB_BIMG), "h"(*reinterpret_cast<const unsigned short*>(&lo)) : "memory");
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(w.bar(MB_BREADY));
            store_sin(seg);              // S_in of this segment drains while the product runs
            w.wait_hot(MB_D, seg & 1);
            tc_fence_after_sync();
#pragma unroll
            for (int q = 0; q < CMB_COLS / 16; ++q) {
                uint32_t d[16], e1[16], e2[16];              // hi*hi, lo*hi, hi*lo: one accumulator each
                tmem_ld16(tmem + lane_base + 16 * q, d);
                tmem_ld16(tmem + lane_base + CMB_COLS + 16 * q, e1);
                tmem_ld16(tmem + lane_base + 2 * CMB_COLS + 16 * q, e2);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float4 x = nv[4 * q + e];
                    const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        s[16 * q + 4 * e + u] = (__uint_as_float(d[4 * e + u]) +
                                                 (__uint_as_float(e1[4 * e + u]) + __uint_as_float(e2[4 * e + u]))) + xs[u];
                }
            }
        }
        store_sin(nhops);
    } else if (warp >= issue_warp && warp < issue_warp + 3 && lane == 0) {
        // ---- MMA issue, one thread per partial product (issuing costs tens of nanoseconds per instruction and the
        //      three products are independent); the first of them also copies the M images ----
        const uint32_t prod = (uint32_t)(warp - issue_warp);            // hi*hi, lo*hi, hi*lo
        const uint32_t aoff = (prod == 1) ? CMB_IMG / 2 : 0u, boff = (prod == 2) ? CMB_BIMG : 0u;
        if (!SCAN) pdl_wait();
        auto load_m = [&](int seg) {
            const uint32_t st = seg % CMB_STAGES, full = w.bar(MB_FULL0 + st);
            const uint8_t* src = reinterpret_cast<const uint8_t*>(p.seg_mt) + ((size_t)(n * p.nseg + seg) * H + h) * CMB_IMG;
            mbar_arrive_expect_tx(full, CMB_IMG);
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) bulk_load(base + st * CMB_IMG + q * 16384, src + q * 16384, 16384, full);
        };
        if (prod == 0)
            for (int sg = 0; sg < (int)CMB_STAGES && sg < nhops; ++sg) load_m(sg);
        const uint64_t dB0 = make_smem_desc(base + CM_B + boff, 16, 1024);
        for (int seg = 0; seg < nhops; ++seg) {
            const uint32_t st = seg % CMB_STAGES, ma = base + st * CMB_IMG + aoff;
            w.wait_hot(MB_FULL0 + st, (seg / CMB_STAGES) & 1);
            w.wait_hot(MB_BREADY, seg & 1);
            tc_fence_after_sync();
#pragma unroll
            for (uint32_t ks = 0; ks < 8; ++ks)
                mma_ss(tmem + prod * CMB_COLS, make_smem_desc(ma + (ks >> 2) * 16384 + (ks & 3) * 2048, 8192, 1024),
                       dB0 + (uint64_t)(((ks >> 2) * (CMB_COLS * 128) + (ks & 3) * 32) >> 4), ID_CMB, ks ? 1u : 0u);
            mma_commit(w.bar(MB_D));
            mma_commit(w.bar(MB_FREE0 + st));
            if (prod == 0 && seg + (int)CMB_STAGES < nhops) {
                w.wait(MB_FREE0 + st, (seg / CMB_STAGES) & 1);   // the tensor core has read this stage for all three products
                load_m(seg + CMB_STAGES);
            }
        }
        if (prod == 0 && *w.abort_flag) {   // let copies in flight land before shared memory is released (bounded)
            const unsigned long long t0 = globaltimer_ns();
            for (int seg = max(0, nhops - (int)CMB_STAGES); seg < nhops; ++seg)
                while (!mbar_try_wait(w.bar(MB_FULL0 + seg % CMB_STAGES), (seg / CMB_STAGES) & 1) &&
                       globaltimer_ns() - t0 < TIMEOUT_NS) {}
        }
    }
}

__global__ void __launch_bounds__(CMB_THREADS, 1) gdn_combine_kernel(CombineParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + CM_MISC);
    Waiter w{base + CM_BARS, reinterpret_cast<volatile int*>(sm + CM_MISC + 4)};
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        combine_init_bars(w);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + CM_MISC, CMB_TCOLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];
    pdl_trigger();
    const Cta cta{base, sm, tmem, (int)blockIdx.x, (int)blockIdx.y, (int)blockIdx.z};
    combine_body<false>(p, cta, w, 4);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, CMB_TCOLS);
    }
}

// =====================================================================================
// merged scan kernel: summary, combination and chain of a split sequence in ONE launch
//
// The three phases of the sequence split are latency chains of a few dozen microseconds each, and every
// kernel boundary between them costs a launch, a set-up (barriers, tensor memory, first loads) and a drain.
// Here one CTA per (sequence, head, segment) stays resident and runs all three phases; the hand-over between
// phases goes through two counters per (sequence, head) in global memory:
//   phase 1  segment summary (M_seg, N_seg) of its own segment           -> raises counter 0
//   phase 2  waits for counter 0 = nseg - 1, then runs the hops of one 16-column slice of the state
//            (CTAs seg, seg + nseg, ... take the slices)                   -> raises counter 1
//   phase 3  its operand ring is filled at once; the chain warpgroup waits for counter 1 = number of slice
//            owners, loads the incoming state of its segment and walks its chunks
// Every wait on a counter is bounded like the mbarrier waits (status GDN_ERR_TIMEOUT, abort flag, all roles
// fall through).  The grid must be co-resident (one CTA per SM): the host launches this kernel only when
// sequences x heads x segments <= #SMs, otherwise the three stand-alone kernels run.  The counters are zero
// before the launch and zero again after it (the last CTA of a head to get past both waits clears them), so a
// captured launch can be replayed.
// =====================================================================================
constexpr int SCAN_THREADS = 384;
constexpr uint32_t SC_BARS1 = CS_BARS;                 // behind the largest data layout (the chain phase's)
constexpr uint32_t SC_BARS2 = SC_BARS1 + 24 * 8;
constexpr uint32_t SC_BARS3 = SC_BARS2 + 16 * 8;
constexpr uint32_t SC_MISC = SC_BARS3 + 24 * 8;
constexpr uint32_t SCAN_SMEM = SC_MISC + 64 + 1024;
static_assert(SUS_BARS <= CS_BARS && CM_BARS <= CS_BARS, "phase layouts must end before the barrier area");
static_assert(SCAN_SMEM <= 232448, "shared memory per CTA");
constexpr int SCAN_FLAG_INTS = 4;                      // per (sequence, head): summaries, slices, CTAs done, pad

struct ScanParams {
    SummaryParams sp;
    CombineParams cb;
    ChainParams cp;
    int* flags;               // [B * H][4], zero before and after every launch
};

__device__ __forceinline__ void mbar_inval(uint32_t bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

template <bool DBG>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
gdn_scan_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, ScanParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* sMisc = reinterpret_cast<volatile uint32_t*>(sm + SC_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + SC_MISC + 4);
    const Waiter w1{base + SC_BARS1, abort_flag}, w2{base + SC_BARS2, abort_flag}, w3{base + SC_BARS3, abort_flag};

    const int tid = threadIdx.x, warp = tid >> 5;
    const int nseg = p.cp.nseg, H = p.cp.H;
    const int h = blockIdx.y, n = blockIdx.z / nseg, seg = blockIdx.z % nseg;
    int* fl = p.flags + (size_t)(n * H + h) * SCAN_FLAG_INTS;
    const int nslices = p.cp.dv / CMB_COLS;
    const int nowners = nseg < nslices ? nseg : nslices;

    if (tid == 0) {
        summary_init_bars(w1, 2);
        combine_init_bars(w2);
        chain_init_bars(w3);
        sMisc[1] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(base + SC_MISC, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sMisc[0];
    pdl_wait();                         // the scratch items come from the prepare kernel
    auto stamp = [&](int ev) {
        if (DBG && p.cp.dbg && tid == 0 && h == 0 && n == 0 && seg < 16)
            p.cp.dbg[512 + seg * 16 + ev] = (float)(globaltimer_ns() & 0xFFFFFFull);
    };
    // The three phases, run by every warp.  The code is instantiated once per warpgroup role below, each copy
    // behind that role's register budget, so the phase bodies (which branch on the warp index themselves)
    // reduce to the one role; CTA-wide synchronisation therefore uses a named barrier, not __syncthreads.
    auto cta_sync = [&]() { named_bar_sync(4, SCAN_THREADS); };
    auto phases = [&]() {
        stamp(0);
        // ---------------- phase 1: summary of this segment (the last segment needs none) ----------------
        if (seg < nseg - 1) {
            const Cta c1{base, sm, tmem, 0, h, n * (nseg - 1) + seg};
            summary_body<true>(&map_k, &map_v, p.sp, c1, w1);
            __threadfence();
            tc_fence_before_sync();
            cta_sync();
            tc_fence_after_sync();
            // (test hook: drop_chunk == -2 makes the first CTA keep its summary to itself, so that the
            //  bounded waits of its head on this counter expire)
            if (tid == 0 && !(p.cp.drop_chunk == -2 && blockIdx.y == 0 && blockIdx.z == 0)) { __threadfence(); atomicAdd(fl + 0, 1); }
        }
        stamp(1);
        // ---------------- phase 2: the hops of this CTA's column slices ----------------
        if (seg < nslices) {
            if (tid == 0) handover_wait(Handover{fl + 0, nseg - 1}, abort_flag);
            cta_sync();
            stamp(2);
            for (int slice = seg; slice < nslices; slice += nseg) {
                if (slice != seg) {     // barriers of the previous slice have advanced: start them afresh
                    cta_sync();
                    if (tid == 0) {
                        for (uint32_t i = 0; i < 8; ++i) mbar_inval(w2.bar(i));
                        combine_init_bars(w2);
                        fence_mbar_init();
                    }
                    cta_sync();
                }
                const Cta c2{base, sm, tmem, slice, h, n};
                combine_body<true>(p.cb, c2, w2, 8);
                tc_fence_before_sync();
            }
            __threadfence();
            cta_sync();
            tc_fence_after_sync();
            if (tid == 0) { __threadfence(); atomicAdd(fl + 1, 1); }
        }
        stamp(3);
        // ---------------- phase 3: chain over this segment's chunks ----------------
        const Cta c3{base, sm, tmem, 0, h, (int)blockIdx.z};
        chain_body<DBG, true, false>(&map_q, &map_k, &map_v, p.cp, c3, w3, Handover{fl + 1, nowners});
        stamp(4);
        tc_fence_before_sync();
        cta_sync();
    };
    // register budgets: warpgroup 0 holds a 128-value fp32 row per thread in all three phases (232), warpgroup 1
    // the identity chain of the summary and the epilogue of the chain phase (216), warpgroup 2 issues and copies (56)
    if (warp < 4) { setmaxnreg_inc<232>(); phases(); }
    else if (warp < 8) { setmaxnreg_inc<216>(); phases(); }
    else { setmaxnreg_dec<56>(); phases(); }
    if (tid == 0) {                     // the last CTA of this head to get here clears the counters
        __threadfence();
        if (atomicAdd(fl + 2, 1) == nseg - 1) {
            fl[0] = 0; fl[1] = 0; fl[2] = 0;
            __threadfence();
        }
    }
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
// Sequence split: only for batched (equal-length) input with few chains.  Returns the number
// of segments per sequence (1 = no split) and the chunks per segment.
static void plan_split(int B, int T, int H, int d_v, bool packed, int num_sms, int* nseg, int* seg_chunks) {
    const int nch = (T + C - 1) / C;
    *nseg = 1;
    *seg_chunks = nch > 0 ? nch : 1;
    if (packed || nch < 16) return;
    const long chains = (long)B * H * (d_v / DVB);
    if (chains * 2 > num_sms) return;
    int want = (int)(num_sms / chains);
    if (want > 16) want = 16;
    if (want > nch / 4) want = nch / 4;                 // at least four chunks per segment
    if (want < 2) return;
    const int sc = (nch + want - 1) / want;
    *seg_chunks = sc;
    *nseg = (nch + sc - 1) / sc;
}
constexpr int kMaxSeg = 16;

// In front of the items: the prepare kernel's item ticket (two ints) and, from int 16 on, the scan kernel's
// counters (four ints per (sequence, head)).  All of it reads zero before a call and zero again after it.
constexpr size_t kWorkspaceHeader = 4096;
constexpr int kScanFlagOffset = 16;
constexpr long kMaxScanChains = (long)(kWorkspaceHeader / sizeof(int) - kScanFlagOffset) / SCAN_FLAG_INTS;

// The ticket must read zero before the first launch; every launch leaves it zero again.
int lean_init_workspace(void* workspace) {
    return cudaMemset(workspace, 0, kWorkspaceHeader) == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

// Launch a kernel that may begin (set-up only, up to its pdl_wait) before the previous kernel in the stream ends.
template <typename... KArgs, typename... Args>
static void launch_after(void (*kernel)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_lean_timing ? 0 : 1;   // events between kernels: plain order
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Split scratch per segment and sequence batch: incoming state, N_seg (fp32 [d_k, d_v] each) and the two
// bf16 images of M_seg^T, per head.
static size_t split_scratch_bytes(int B, int H, int d_k, int d_v, int nseg) {
    return (size_t)nseg * B * H * (2 * (size_t)d_k * d_v * sizeof(float) + CMB_IMG);
}
static size_t items_bytes_aligned(uint64_t tokens, int B, int H) {
    const size_t slots = (size_t)(tokens >> 6) + (size_t)B;
    return (slots * H * ITEM_BYTES + 255) & ~(size_t)255;
}
// A split is planned only when 2 * chains <= #SMs; scratch for it is reserved for any GPU of up to this many SMs.
constexpr int kMaxSmsForSplit = 256;

size_t lean_workspace_bytes(int B, int T, int H, int d_k, int d_v, bool packed) {
    if (!tc_supported(d_k, d_v) || B <= 0 || T < 0 || H <= 0) return 0;
    const uint64_t tokens = packed ? (uint64_t)T : (uint64_t)B * T;
    size_t bytes = kWorkspaceHeader + items_bytes_aligned(tokens, B, H);
    if (!packed) {
        const size_t chains = (size_t)B * H * (d_v / DVB);
        if (chains * 2 <= (size_t)kMaxSmsForSplit) bytes += split_scratch_bytes(B, H, d_k, d_v, kMaxSeg);
    }
    return bytes;
}

// Set-up done once per device: the SM count and the kernels' dynamic shared-memory limits.
constexpr int kMaxDevices = 64;
static int device_setup(int* sms_out) {
    static std::mutex mu;
    static int sms_of_device[kMaxDevices] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GDN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GDN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (sms_of_device[dev] == 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return GDN_ERR_CUDA;
        if (cudaFuncSetAttribute(gdn_prep_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PREP_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_prep_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PREP_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_chain_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_chain_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_chain_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SUM_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_combine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CMB_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_scan_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCAN_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_scan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCAN_SMEM) != cudaSuccess)
            return GDN_ERR_CUDA;
        sms_of_device[dev] = sms;
    }
    *sms_out = sms_of_device[dev];
    return GDN_OK;
}

int launch_lean(const PrefillArgs& a, void* workspace, size_t workspace_bytes, cudaStream_t stream,
                const LeanOptions& opt) {
    float* const snaps = opt.snaps;
    const int snap_every = opt.snap_every;
    if (!tc_supported(a.d_k, a.d_v)) return GDN_ERR_UNSUPPORTED;
    if (opt.gate_z && a.d_v != DVB) return GDN_ERR_UNSUPPORTED;      // the fused norm sees one CTA's 128 value columns
    if (a.H > 65535 || a.B > 4095) return GDN_ERR_UNSUPPORTED;
    const bool packed = a.cu_seqlens != nullptr;
    const uint64_t tokens = packed ? (uint64_t)a.T : (uint64_t)a.B * a.T;
    const size_t items_bytes = items_bytes_aligned(tokens, a.B, a.H);
    if (!workspace || workspace_bytes < kWorkspaceHeader + items_bytes || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return GDN_ERR_WORKSPACE;
    int num_sms = 0;
    if (int rc = device_setup(&num_sms)) return rc;
    // ---- optional sequence split: planned here, before anything is launched, so that scratch that is too
    //      small is reported (forced plan) or avoided (automatic plan) instead of being overrun ----
    int nseg = 1, seg_chunks = 1;
    plan_split(a.B, a.T, a.H, a.d_v, packed, num_sms, &nseg, &seg_chunks);
    const bool forced = g_lean_force_nseg > 0 && !packed;
    if (forced) {                                     // tests: force a segment count
        const int nch = (a.T + C - 1) / C;
        nseg = g_lean_force_nseg > kMaxSeg ? kMaxSeg : g_lean_force_nseg;
        if (nseg > nch) nseg = nch > 0 ? nch : 1;
        seg_chunks = nch > 0 ? (nch + nseg - 1) / nseg : 1;
        nseg = nch > 0 ? (nch + seg_chunks - 1) / seg_chunks : 1;
    }
    if (nseg > 1 && kWorkspaceHeader + items_bytes + split_scratch_bytes(a.B, a.H, a.d_k, a.d_v, nseg) > workspace_bytes) {
        if (forced) return GDN_ERR_WORKSPACE;
        nseg = 1;
        seg_chunks = (a.T + C - 1) / C > 0 ? (a.T + C - 1) / C : 1;
    }
    CUtensorMap mq, mk, mv;
    if (!tc_make_map(&mq, a.q, tokens, a.H, a.d_k) || !tc_make_map(&mk, a.k, tokens, a.H, a.d_k) ||
        !tc_make_map(&mv, a.v, tokens, a.H, a.d_v))
        return GDN_ERR_CUDA;
    int* ticket = static_cast<int*>(workspace);                      // header, zeroed by lean_init_workspace
    uint8_t* ws = static_cast<uint8_t*>(workspace) + kWorkspaceHeader;
    const long nslots = (long)(tokens >> 6) + a.B;
    const long nitems = nslots * a.H;
    // ---- state-independent steps, every (chunk, head) ----
    // With a split, K (and V) are read by two or three kernels of the call; when they fit in L2 comfortably the
    // earlier readers ask L2 to keep them and the last reader releases them.
    const int l2 = (nseg > 1 && tokens * a.H * (uint64_t)(a.d_k + a.d_v) * 2 <= (96ull << 20)) ? (g_lean_l2_hints & 3) : 0;
    PrepParams pp{a.log_alpha, a.beta, a.cu_seqlens, ws, nslots, a.B, a.T, a.H, opt.gate_scale, opt.eps, ticket, l2};
    const int pgrid = (int)(nitems < 4L * num_sms ? nitems : 4L * num_sms);
    auto mark = [&](int i) { if (g_lean_timing && g_lean_events[i]) cudaEventRecord(g_lean_events[i], stream); };
    mark(0);
    if (opt.raw) gdn_prep_kernel<true><<<pgrid, PREP_THREADS, PREP_SMEM, stream>>>(mq, mk, pp);
    else gdn_prep_kernel<false><<<pgrid, PREP_THREADS, PREP_SMEM, stream>>>(mq, mk, pp);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return GDN_ERR_CUDA;
    mark(1);
    // ---- sequence split: segment summaries, their combination, per-segment chains ----
    float* seg_sin = nullptr;
    g_lean_split_last = nseg > 1;
    g_lean_scan_last = false;
    const int nsnap = snaps ? (a.T / C) / snap_every : 0;
    if (nseg > 1) {
        const size_t state_elems = (size_t)a.B * nseg * a.H * a.d_k * a.d_v;
        seg_sin = reinterpret_cast<float*>(ws + items_bytes);
        float* seg_n = seg_sin + state_elems;
        float* seg_mt = seg_n + state_elems;
        SummaryParams sp{a.cu_seqlens, ws, seg_n, seg_mt, a.B, a.T, a.H, a.d_v, nseg, seg_chunks, l2};
        CombineParams cb{a.initial_state, seg_n, seg_mt, seg_sin, a.H, a.d_v, nseg};
        // one resident CTA per (sequence, head, segment) runs all three phases when the grid fits the GPU at once
        if (g_lean_use_scan && !opt.gate_z && a.d_v == DVB && (long)a.B * a.H * nseg <= num_sms && (long)a.B * a.H <= kMaxScanChains) {
            ChainParams cp{a.initial_state, static_cast<__nv_bfloat16*>(a.out), a.final_state, a.cu_seqlens,
                           ws, seg_sin, g_lean_dbg, g_lean_drop_chunk, a.B, a.T, a.H, a.d_v, nseg, seg_chunks,
                           snaps, snap_every, nsnap, l2, opt.gate_z, opt.norm_w, opt.norm_eps};
            ScanParams scp{sp, cb, cp, static_cast<int*>(workspace) + kScanFlagOffset};
            dim3 grid(1, a.H, a.B * nseg);
            if (g_lean_dbg) launch_after(gdn_scan_kernel<true>, grid, SCAN_THREADS, SCAN_SMEM, stream, mq, mk, mv, scp);
            else launch_after(gdn_scan_kernel<false>, grid, SCAN_THREADS, SCAN_SMEM, stream, mq, mk, mv, scp);
            count_launch();
            g_lean_scan_last = true;
            mark(4);
            return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
        }
        dim3 sgrid(a.d_v / DVB, a.H, a.B * (nseg - 1));
        launch_after(gdn_summary_kernel, sgrid, SUM_THREADS, SUM_SMEM, stream, mk, mv, sp);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return GDN_ERR_CUDA;
        mark(2);
        dim3 cgrid(a.d_v / CMB_COLS, a.H, a.B);
        launch_after(gdn_combine_kernel, cgrid, CMB_THREADS, CMB_SMEM, stream, cb);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return GDN_ERR_CUDA;
        mark(3);
    }
    // ---- steps c, d ----
    ChainParams cp{a.initial_state, static_cast<__nv_bfloat16*>(a.out), a.final_state, a.cu_seqlens,
                   ws, seg_sin, g_lean_dbg, g_lean_drop_chunk, a.B, a.T, a.H, a.d_v, nseg, seg_chunks,
                   snaps, snap_every, nsnap, l2, opt.gate_z, opt.norm_w, opt.norm_eps};
    dim3 grid(a.d_v / DVB, a.H, a.B * nseg);
    if (opt.gate_z) launch_after(gdn_chain_kernel<false, true>, grid, CHAIN_THREADS, CHAIN_SMEM, stream, mq, mk, mv, cp);
    else if (g_lean_dbg) launch_after(gdn_chain_kernel<true, false>, grid, CHAIN_THREADS, CHAIN_SMEM, stream, mq, mk, mv, cp);
    else launch_after(gdn_chain_kernel<false, false>, grid, CHAIN_THREADS, CHAIN_SMEM, stream, mq, mk, mv, cp);
    count_launch();
    mark(4);
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

void lean_set_scan(int enable) { g_lean_use_scan = enable != 0; }
void lean_set_l2_hints(int enable) { g_lean_l2_hints = enable; }
void lean_force_segments(int nseg) { g_lean_force_nseg = nseg; }
void lean_set_debug(float* p) { g_lean_dbg = p; }
void lean_set_drop_chunk(int c) { g_lean_drop_chunk = c; }
int lean_reset_status() {
    const int zero = 0;
    return cudaMemcpyToSymbol(g_lean_status, &zero, sizeof(int)) == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

int lean_set_timing(int enable) {
    if (enable)
        for (auto& e : g_lean_events)
            if (!e && cudaEventCreate(&e) != cudaSuccess) return GDN_ERR_CUDA;
    g_lean_timing = enable != 0;
    return GDN_OK;
}

// milliseconds of {prepare, summary, combine, chain, scan} of the most recent call (0 for kernels not run)
int lean_get_timing(float* ms5) {
    for (int i = 0; i < 5; ++i) ms5[i] = 0.f;
    if (!g_lean_events[0]) return GDN_ERR_INVALID_ARG;
    if (cudaEventSynchronize(g_lean_events[4]) != cudaSuccess) return GDN_ERR_CUDA;
    bool ok = cudaEventElapsedTime(&ms5[0], g_lean_events[0], g_lean_events[1]) == cudaSuccess;
    if (g_lean_scan_last) {
        ok = ok && cudaEventElapsedTime(&ms5[4], g_lean_events[1], g_lean_events[4]) == cudaSuccess;
    } else if (g_lean_split_last) {
        ok = ok && cudaEventElapsedTime(&ms5[1], g_lean_events[1], g_lean_events[2]) == cudaSuccess;
        ok = ok && cudaEventElapsedTime(&ms5[2], g_lean_events[2], g_lean_events[3]) == cudaSuccess;
        ok = ok && cudaEventElapsedTime(&ms5[3], g_lean_events[3], g_lean_events[4]) == cudaSuccess;
    } else {
        ok = ok && cudaEventElapsedTime(&ms5[3], g_lean_events[1], g_lean_events[4]) == cudaSuccess;
    }
    return ok ? GDN_OK : GDN_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------
// Entry point for callers that cannot allocate device memory.
//
// Some users of this library own no allocator: an operator plugged into a host framework is
// handed its input and output buffers and nothing else, and a serving process that sized its
// memory pools at start-up has no device memory left to ask for.  They cannot provide the
// scratch the two-kernel pipeline wants, so that scratch lives here, in a fixed array inside
// the library image.  Every GPU that loads the library holds these bytes until the process
// exits, whether or not this entry point is ever called.
//
// The array name below is only a host-side handle; the address a kernel may use is obtained
// with cudaGetSymbolAddress, once per device, by the first call made while that device is
// current (make that first call outside any stream capture).  All calls share the array and
// it keeps whatever the previous call left in it.  Nothing in it has to start at zero: the
// prepare kernel writes every item the chain kernel reads before it is read, and items of
// unused slots are never read.  Two calls that overlap on the GPU would race on it.
// ------------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = 64ull << 20;            // 64 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static __device__ int g_static_ticket[2];                      // the prepare kernel's item ticket (zero at load)

int launch_lean_static(const PrefillArgs& a, cudaStream_t stream) {
    if (!tc_supported(a.d_k, a.d_v)) return GDN_ERR_UNSUPPORTED;
    if (a.H > 65535 || a.B > 65535) return GDN_ERR_UNSUPPORTED;
    const bool packed = a.cu_seqlens != nullptr;
    const uint64_t tokens = packed ? (uint64_t)a.T : (uint64_t)a.B * a.T;
    const uint64_t nslots = (tokens >> 6) + (uint64_t)a.B;
    const uint64_t need = nslots * (uint64_t)a.H * ITEM_BYTES;
    if (need > kStaticScratchBytes) return GDN_ERR_TOO_LARGE;
    // ---- set-up, once per device: the device address of the built-in scratch ----
    static void* scratch_of_device[kMaxDevices] = {nullptr};
    static void* ticket_of_device[kMaxDevices] = {nullptr};
    static int sms_of_device[kMaxDevices] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GDN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GDN_ERR_UNSUPPORTED;
    if (!scratch_of_device[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return GDN_ERR_CUDA;
        if (cudaGetSymbolAddress(&ticket_of_device[dev], g_static_ticket) != cudaSuccess || !ticket_of_device[dev])
            return GDN_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            return GDN_ERR_CUDA;
        if (cudaFuncSetAttribute(gdn_prep_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PREP_SMEM) != cudaSuccess ||
        cudaFuncSetAttribute(gdn_prep_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PREP_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(gdn_chain_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)CHAIN_SMEM) != cudaSuccess)
            return GDN_ERR_CUDA;
        sms_of_device[dev] = sms;
        scratch_of_device[dev] = ptr;
    }
    uint8_t* ws = static_cast<uint8_t*>(scratch_of_device[dev]);
    CUtensorMap mq, mk, mv;
    if (!tc_make_map(&mq, a.q, tokens, a.H, a.d_k) || !tc_make_map(&mk, a.k, tokens, a.H, a.d_k) ||
        !tc_make_map(&mv, a.v, tokens, a.H, a.d_v))
        return GDN_ERR_CUDA;
    const long nitems = (long)nslots * a.H;
    const long cap = 4L * sms_of_device[dev];
    PrepParams pp{a.log_alpha, a.beta, a.cu_seqlens, ws, (long)nslots, a.B, a.T, a.H, 1.f, 0.f, static_cast<int*>(ticket_of_device[dev])};
    gdn_prep_kernel<false><<<(int)(nitems < cap ? nitems : cap), PREP_THREADS, PREP_SMEM, stream>>>(mq, mk, pp);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return GDN_ERR_CUDA;
    const int nch = packed ? 1 : (a.T + C - 1) / C;            // one segment: the whole sequence
    ChainParams cp{a.initial_state, static_cast<__nv_bfloat16*>(a.out), a.final_state, a.cu_seqlens,
                   ws, nullptr, nullptr, -1, a.B, a.T, a.H, a.d_v, 1, packed ? (1 << 24) : (nch > 0 ? nch : 1),
                   nullptr, 1, 0};
    dim3 grid(a.d_v / DVB, a.H, a.B);
    gdn_chain_kernel<false, false><<<grid, CHAIN_THREADS, CHAIN_SMEM, stream>>>(mq, mk, mv, cp);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

int lean_status_async(int* host_dst, cudaStream_t stream) {
    return cudaMemcpyFromSymbolAsync(host_dst, g_lean_status, sizeof(int), 0, cudaMemcpyDeviceToHost, stream) == cudaSuccess
               ? GDN_OK : GDN_ERR_CUDA;
}

int lean_query_status() {
    int s = 0;
    if (cudaMemcpyFromSymbol(&s, g_lean_status, sizeof(int)) != cudaSuccess) return GDN_ERR_CUDA;
    return s;
}

}  // namespace gdn
