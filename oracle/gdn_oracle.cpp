// fp64 CPU oracle for the gated delta-rule prefill.  TEST INFRASTRUCTURE ONLY.
//
// This file is the yardstick the CUDA library is measured against.  It shares no
// code with the CUDA path, is never linked into it, and must not be called from
// the product: only the tests, the smoke check and the CPU-baseline leg of the
// benchmark may build or run it.
//
// Three independent formulations of the same map are given, so that each can be
// checked against the others and against closed forms:
//
//   gdn_oracle_sequential  the definition: the token-by-token recurrence of the
//                          recurrent layer (Section "A chunked delta-rule scan for
//                          the recurrent layers": S_t = diag(gamma_t) S_{t-1} +
//                          k_t delta_t^T; state S in R^{H_k x H_v} per value head,
//                          Section "The model").
//   gdn_oracle_chunked     the intra-/inter-chunk form of the same section, in the order of
//                          steps the section gives: (1) K K^T and Q K^T of a chunk with
//                          their decay masks, (2) row-by-row solve of the unit lower
//                          triangular system, (3) the factors W, U and from them the
//                          chunk's correction and output, (4) the state carried to the
//                          next chunk.  form=1 precomputes M_c, N_c per chunk and steps
//                          with S^(c+1) = M_c S^(c) + N_c, as the section also does.
//   gdn_oracle_dense       brute force: the whole sequence as one T x T system
//                          solved by general Gaussian elimination with pivoting
//                          (it does not know the matrix is triangular).
//   gdn_oracle_chunked_stages  gdn_oracle_chunked (form 0) for ONE (sequence, head)
//                          chain that also hands out what it computes on the way,
//                          chunk by chunk: g, A, P, T, W, U, Delta and the state each
//                          chunk starts from -- so that a GPU path can be compared
//                          stage by stage, each stage with its own reference (Section
//                          "Porting the Vision Tower, Stage by Stage").  Same code,
//                          same arithmetic; the extra outputs are copies.
//
// Pins (tests/test_oracle_pins.py): every function here is pinned by closed
// forms and invariants (pure decay, exact key overwrite, one-token closed form,
// masked linear attention, split/padding/chunk-size invariance, linearity) and by
// agreement of the three formulations to 1e-12.
//
// Conventions (all arrays row-major, last index fastest, fp64):
//   q, k            [B, T, H, d_k]      v, out   [B, T, H, d_v]
//   log_alpha, beta [B, T, H]           log_alpha is the natural log of the gate
//   initial_state, final_state [N, H, d_k, d_v]   (NULL initial = zeros,
//                                                   NULL final = not returned)
//   cu_seqlens == NULL : N = B sequences of T tokens each.
//   cu_seqlens != NULL : packed; tensors are [T_total, H, .], B is the number of
//                        sequences, sequence n owns tokens
//                        [cu_seqlens[n], cu_seqlens[n+1]).
// Per token (gate is a scalar per token and head; the delta sees the decayed
// state; the output reads the updated state; no 1/sqrt(d_k) scale):
//   S <- exp(a_t) S ; delta <- beta_t (v_t - S^T k_t) ; S <- S + k_t delta^T ;
//   o_t <- S^T q_t.
// Return value: 0 on success, 1 on an invalid argument.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

struct Problem {
    const double *q, *k, *v, *a, *beta, *s0;
    double *out, *sT;
    const int32_t* cu;
    int B, T, H, dk, dv;
};

// token range of sequence n and the flat index of its first token
inline void seq_range(const Problem& p, int n, long& tok0, int& len) {
    if (p.cu) { tok0 = p.cu[n]; len = p.cu[n + 1] - p.cu[n]; }
    else      { tok0 = (long)n * p.T; len = p.T; }
}

bool valid(const Problem& p) {
    if (!p.q || !p.k || !p.v || !p.a || !p.beta || !p.out) return false;
    if (p.B <= 0 || p.T < 0 || p.H <= 0 || p.dk <= 0 || p.dv <= 0) return false;
    if (p.cu) {
        if (p.cu[0] != 0 || p.cu[p.B] != p.T) return false;
        for (int n = 0; n < p.B; ++n) if (p.cu[n + 1] < p.cu[n]) return false;
    }
    return true;
}

// ---------------------------------------------------------------------------
// (1) the definition
// ---------------------------------------------------------------------------
void sequential_chain(const Problem& p, int n, int h) {
    const int dk = p.dk, dv = p.dv, H = p.H;
    long tok0; int len; seq_range(p, n, tok0, len);
    std::vector<double> S((size_t)dk * dv, 0.0), delta(dv);
    if (p.s0) std::memcpy(S.data(), p.s0 + ((size_t)n * H + h) * dk * dv, sizeof(double) * dk * dv);
    for (int t = 0; t < len; ++t) {
        const size_t th = (size_t)(tok0 + t) * H + h;
        const double* kt = p.k + th * dk;
        const double* qt = p.q + th * dk;
        const double* vt = p.v + th * dv;
        double* ot = p.out + th * dv;
        const double alpha = std::exp(p.a[th]);
        const double bt = p.beta[th];
        for (size_t i = 0; i < S.size(); ++i) S[i] *= alpha;          // decay first
        for (int j = 0; j < dv; ++j) delta[j] = 0.0;
        for (int m = 0; m < dk; ++m)                                   // S^T k
            for (int j = 0; j < dv; ++j) delta[j] += S[(size_t)m * dv + j] * kt[m];
        for (int j = 0; j < dv; ++j) delta[j] = bt * (vt[j] - delta[j]);
        for (int m = 0; m < dk; ++m)                                   // rank-1 write
            for (int j = 0; j < dv; ++j) S[(size_t)m * dv + j] += kt[m] * delta[j];
        for (int j = 0; j < dv; ++j) ot[j] = 0.0;
        for (int m = 0; m < dk; ++m)                                   // read updated state
            for (int j = 0; j < dv; ++j) ot[j] += S[(size_t)m * dv + j] * qt[m];
    }
    if (p.sT) std::memcpy(p.sT + ((size_t)n * H + h) * dk * dv, S.data(), sizeof(double) * dk * dv);
}

// ---------------------------------------------------------------------------
// (2) chunked form.  Within a chunk with incoming state S0, local index r,
// g_r = sum_{i<=r} a_i (restarting at every chunk):
//   A[r,i] = beta_r e^{g_r-g_i} (k_r.k_i)   (i <  r)   strictly lower
//   P[r,i] =        e^{g_r-g_i} (q_r.k_i)   (i <= r)   diagonal included
//   (I + A) Delta = diag(beta) V - diag(beta e^{g}) K S0
//   S_C = e^{g_C} S0 + sum_i e^{g_C-g_i} k_i delta_i^T
//   O   = diag(e^{g}) Q S0 + P Delta
// A tail chunk simply has fewer rows.
// ---------------------------------------------------------------------------
// Optional per-chunk copies of the intermediates of chunked_chain (any pointer may be null).
// Layouts, ci = chunk index: g [ci][C]; A, P, T [ci][C][C]; W [ci][C][dk]; U, D [ci][C][dv];
// Sin [ci][dk][dv].  Rows beyond a tail chunk's length are left untouched.
struct Stages {
    double *g, *A, *P, *T, *W, *U, *D, *Sin;
};

void chunked_chain(const Problem& p, int n, int h, int C, int form, const Stages* st = nullptr) {
    const int dk = p.dk, dv = p.dv, H = p.H;
    long tok0; int len; seq_range(p, n, tok0, len);
    std::vector<double> S((size_t)dk * dv, 0.0), Snew((size_t)dk * dv);
    if (p.s0) std::memcpy(S.data(), p.s0 + ((size_t)n * H + h) * dk * dv, sizeof(double) * dk * dv);
    std::vector<double> g(C), A((size_t)C * C), P((size_t)C * C), Tm((size_t)C * C);
    std::vector<double> W((size_t)C * dk), U((size_t)C * dv), D((size_t)C * dv);
    std::vector<double> M((size_t)dk * dk), Nn((size_t)dk * dv), Qp((size_t)C * dk), O0((size_t)C * dv);

    for (int c0 = 0; c0 < len; c0 += C) {
        const int R = std::min(C, len - c0);
        const size_t ci = (size_t)(c0 / C);
        if (st && st->Sin) std::memcpy(st->Sin + ci * dk * dv, S.data(), sizeof(double) * dk * dv);
        auto K = [&](int r) { return p.k + ((size_t)(tok0 + c0 + r) * H + h) * dk; };
        auto Q = [&](int r) { return p.q + ((size_t)(tok0 + c0 + r) * H + h) * dk; };
        auto V = [&](int r) { return p.v + ((size_t)(tok0 + c0 + r) * H + h) * dv; };
        auto Bt = [&](int r) { return p.beta[(size_t)(tok0 + c0 + r) * H + h]; };
        // chunk-local cumulative log gate
        double acc = 0.0;
        for (int r = 0; r < R; ++r) { acc += p.a[(size_t)(tok0 + c0 + r) * H + h]; g[r] = acc; }
        // the two token-token interaction matrices
        for (int r = 0; r < R; ++r)
            for (int i = 0; i < R; ++i) {
                double kk = 0.0, qk = 0.0;
                for (int m = 0; m < dk; ++m) { kk += K(r)[m] * K(i)[m]; qk += Q(r)[m] * K(i)[m]; }
                A[(size_t)r * C + i] = (i <  r) ? Bt(r) * std::exp(g[r] - g[i]) * kk : 0.0;
                P[(size_t)r * C + i] = (i <= r) ?          std::exp(g[r] - g[i]) * qk : 0.0;
            }
        // forward substitution: rows of Tm = (I + A)^{-1}, top to bottom
        for (int r = 0; r < R; ++r)
            for (int c = 0; c < R; ++c) {
                double x = (r == c) ? 1.0 : 0.0;
                for (int i = 0; i < r; ++i) x -= A[(size_t)r * C + i] * Tm[(size_t)i * C + c];
                Tm[(size_t)r * C + c] = x;
            }
        // W = Tm diag(beta e^g) K ,  U = Tm diag(beta) V
        for (int r = 0; r < R; ++r) {
            for (int m = 0; m < dk; ++m) {
                double x = 0.0;
                for (int i = 0; i < R; ++i) x += Tm[(size_t)r * C + i] * Bt(i) * std::exp(g[i]) * K(i)[m];
                W[(size_t)r * dk + m] = x;
            }
            for (int j = 0; j < dv; ++j) {
                double x = 0.0;
                for (int i = 0; i < R; ++i) x += Tm[(size_t)r * C + i] * Bt(i) * V(i)[j];
                U[(size_t)r * dv + j] = x;
            }
        }
        if (st) {
            for (int r = 0; r < R; ++r) {
                if (st->g) st->g[ci * C + r] = g[r];
                if (st->A) std::memcpy(st->A + (ci * C + r) * C, &A[(size_t)r * C], sizeof(double) * R);
                if (st->P) std::memcpy(st->P + (ci * C + r) * C, &P[(size_t)r * C], sizeof(double) * R);
                if (st->T) std::memcpy(st->T + (ci * C + r) * C, &Tm[(size_t)r * C], sizeof(double) * R);
                if (st->W) std::memcpy(st->W + (ci * C + r) * dk, &W[(size_t)r * dk], sizeof(double) * dk);
                if (st->U) std::memcpy(st->U + (ci * C + r) * dv, &U[(size_t)r * dv], sizeof(double) * dv);
            }
        }
        const double gC = g[R - 1];
        if (form == 0) {
            // correction Delta = U - W S0, output, state
            for (int r = 0; r < R; ++r)
                for (int j = 0; j < dv; ++j) {
                    double x = U[(size_t)r * dv + j];
                    for (int m = 0; m < dk; ++m) x -= W[(size_t)r * dk + m] * S[(size_t)m * dv + j];
                    D[(size_t)r * dv + j] = x;
                }
            if (st && st->D)
                for (int r = 0; r < R; ++r) std::memcpy(st->D + (ci * C + r) * dv, &D[(size_t)r * dv], sizeof(double) * dv);
            for (int r = 0; r < R; ++r) {
                double* o = p.out + ((size_t)(tok0 + c0 + r) * H + h) * dv;
                for (int j = 0; j < dv; ++j) {
                    double x = 0.0;
                    for (int m = 0; m < dk; ++m) x += Q(r)[m] * S[(size_t)m * dv + j];
                    x *= std::exp(g[r]);
                    for (int i = 0; i <= r; ++i) x += P[(size_t)r * C + i] * D[(size_t)i * dv + j];
                    o[j] = x;
                }
            }
            for (int m = 0; m < dk; ++m)
                for (int j = 0; j < dv; ++j) {
                    double x = std::exp(gC) * S[(size_t)m * dv + j];
                    for (int i = 0; i < R; ++i) x += std::exp(gC - g[i]) * K(i)[m] * D[(size_t)i * dv + j];
                    Snew[(size_t)m * dv + j] = x;
                }
        } else {
            // state-independent chunk summaries, then one affine step:
            //   M = e^{gC} I - Kt^T W ,  N = Kt^T U ,  Kt[i,:] = e^{gC-g_i} k_i
            //   S' = M S + N ;  O = (Qt - P W) S + P U ,  Qt[r,:] = e^{g_r} q_r
            for (int m = 0; m < dk; ++m) {
                for (int m2 = 0; m2 < dk; ++m2) {
                    double x = (m == m2) ? std::exp(gC) : 0.0;
                    for (int i = 0; i < R; ++i) x -= std::exp(gC - g[i]) * K(i)[m] * W[(size_t)i * dk + m2];
                    M[(size_t)m * dk + m2] = x;
                }
                for (int j = 0; j < dv; ++j) {
                    double x = 0.0;
                    for (int i = 0; i < R; ++i) x += std::exp(gC - g[i]) * K(i)[m] * U[(size_t)i * dv + j];
                    Nn[(size_t)m * dv + j] = x;
                }
            }
            for (int r = 0; r < R; ++r) {
                for (int m = 0; m < dk; ++m) {
                    double x = std::exp(g[r]) * Q(r)[m];
                    for (int i = 0; i <= r; ++i) x -= P[(size_t)r * C + i] * W[(size_t)i * dk + m];
                    Qp[(size_t)r * dk + m] = x;
                }
                for (int j = 0; j < dv; ++j) {
                    double x = 0.0;
                    for (int i = 0; i <= r; ++i) x += P[(size_t)r * C + i] * U[(size_t)i * dv + j];
                    O0[(size_t)r * dv + j] = x;
                }
            }
            for (int r = 0; r < R; ++r) {
                double* o = p.out + ((size_t)(tok0 + c0 + r) * H + h) * dv;
                for (int j = 0; j < dv; ++j) {
                    double x = O0[(size_t)r * dv + j];
                    for (int m = 0; m < dk; ++m) x += Qp[(size_t)r * dk + m] * S[(size_t)m * dv + j];
                    o[j] = x;
                }
            }
            for (int m = 0; m < dk; ++m)
                for (int j = 0; j < dv; ++j) {
                    double x = Nn[(size_t)m * dv + j];
                    for (int m2 = 0; m2 < dk; ++m2) x += M[(size_t)m * dk + m2] * S[(size_t)m2 * dv + j];
                    Snew[(size_t)m * dv + j] = x;
                }
        }
        S.swap(Snew);
    }
    if (p.sT) std::memcpy(p.sT + ((size_t)n * H + h) * dk * dv, S.data(), sizeof(double) * dk * dv);
}

// ---------------------------------------------------------------------------
// (3) dense brute force: the sequence is one L x L system; general elimination.
// ---------------------------------------------------------------------------
// Solves Mx X = Rhs in place (Rhs is L x nr, overwritten by X); partial pivoting.
bool gauss_solve(std::vector<double>& Mx, std::vector<double>& Rhs, int L, int nr) {
    for (int c = 0; c < L; ++c) {
        int piv = c; double best = std::fabs(Mx[(size_t)c * L + c]);
        for (int r = c + 1; r < L; ++r)
            if (std::fabs(Mx[(size_t)r * L + c]) > best) { best = std::fabs(Mx[(size_t)r * L + c]); piv = r; }
        if (best == 0.0) return false;
        if (piv != c) {
            for (int j = 0; j < L; ++j) std::swap(Mx[(size_t)c * L + j], Mx[(size_t)piv * L + j]);
            for (int j = 0; j < nr; ++j) std::swap(Rhs[(size_t)c * nr + j], Rhs[(size_t)piv * nr + j]);
        }
        for (int r = 0; r < L; ++r) {
            if (r == c) continue;
            const double f = Mx[(size_t)r * L + c] / Mx[(size_t)c * L + c];
            if (f == 0.0) continue;
            for (int j = c; j < L; ++j) Mx[(size_t)r * L + j] -= f * Mx[(size_t)c * L + j];
            for (int j = 0; j < nr; ++j) Rhs[(size_t)r * nr + j] -= f * Rhs[(size_t)c * nr + j];
        }
    }
    for (int r = 0; r < L; ++r) {
        const double d = Mx[(size_t)r * L + r];
        for (int j = 0; j < nr; ++j) Rhs[(size_t)r * nr + j] /= d;
    }
    return true;
}

bool dense_chain(const Problem& p, int n, int h) {
    const int dk = p.dk, dv = p.dv, H = p.H;
    long tok0; int L; seq_range(p, n, tok0, L);
    std::vector<double> S0((size_t)dk * dv, 0.0);
    if (p.s0) std::memcpy(S0.data(), p.s0 + ((size_t)n * H + h) * dk * dv, sizeof(double) * dk * dv);
    if (L > 0) {
        std::vector<double> G(L), IA((size_t)L * L), Rhs((size_t)L * dv);
        double acc = 0.0;
        for (int t = 0; t < L; ++t) { acc += p.a[(size_t)(tok0 + t) * H + h]; G[t] = acc; }
        auto K = [&](int r) { return p.k + ((size_t)(tok0 + r) * H + h) * dk; };
        auto Q = [&](int r) { return p.q + ((size_t)(tok0 + r) * H + h) * dk; };
        auto V = [&](int r) { return p.v + ((size_t)(tok0 + r) * H + h) * dv; };
        auto Bt = [&](int r) { return p.beta[(size_t)(tok0 + r) * H + h]; };
        for (int r = 0; r < L; ++r) {
            for (int i = 0; i < L; ++i) {
                double x = (i == r) ? 1.0 : 0.0;
                if (i < r) {
                    double kk = 0.0;
                    for (int m = 0; m < dk; ++m) kk += K(r)[m] * K(i)[m];
                    x = Bt(r) * std::exp(G[r] - G[i]) * kk;
                }
                IA[(size_t)r * L + i] = x;
            }
            for (int j = 0; j < dv; ++j) {
                double ks = 0.0;
                for (int m = 0; m < dk; ++m) ks += K(r)[m] * S0[(size_t)m * dv + j];
                Rhs[(size_t)r * dv + j] = Bt(r) * (V(r)[j] - std::exp(G[r]) * ks);
            }
        }
        if (!gauss_solve(IA, Rhs, L, dv)) return false;          // Rhs now holds Delta
        for (int r = 0; r < L; ++r) {
            double* o = p.out + ((size_t)(tok0 + r) * H + h) * dv;
            for (int j = 0; j < dv; ++j) {
                double x = 0.0;
                for (int m = 0; m < dk; ++m) x += Q(r)[m] * S0[(size_t)m * dv + j];
                x *= std::exp(G[r]);
                for (int i = 0; i <= r; ++i) {
                    double qk = 0.0;
                    for (int m = 0; m < dk; ++m) qk += Q(r)[m] * K(i)[m];
                    x += std::exp(G[r] - G[i]) * qk * Rhs[(size_t)i * dv + j];
                }
                o[j] = x;
            }
        }
        for (int m = 0; m < dk; ++m)
            for (int j = 0; j < dv; ++j) {
                double x = std::exp(G[L - 1]) * S0[(size_t)m * dv + j];
                for (int i = 0; i < L; ++i) x += std::exp(G[L - 1] - G[i]) * K(i)[m] * Rhs[(size_t)i * dv + j];
                S0[(size_t)m * dv + j] = x;
            }
    }
    if (p.sT) std::memcpy(p.sT + ((size_t)n * H + h) * dk * dv, S0.data(), sizeof(double) * dk * dv);
    return true;
}

} // namespace

extern "C" {

int gdn_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int gdn_oracle_sequential(const double* q, const double* k, const double* v,
                          const double* log_alpha, const double* beta,
                          const double* initial_state, double* out, double* final_state,
                          const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v) {
    Problem p{q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v};
    if (!valid(p)) return 1;
    const int chains = B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < chains; ++c) sequential_chain(p, c / H, c % H);
    return 0;
}

int gdn_oracle_chunked(const double* q, const double* k, const double* v,
                       const double* log_alpha, const double* beta,
                       const double* initial_state, double* out, double* final_state,
                       const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v,
                       int chunk, int form) {
    Problem p{q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v};
    if (!valid(p) || chunk <= 0 || (form != 0 && form != 1)) return 1;
    const int chains = B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < chains; ++c) chunked_chain(p, c / H, c % H, chunk, form);
    return 0;
}

// One chain (sequence n, head h), form 0, with the per-chunk intermediates copied out.  out and final_state
// are written for that chain only (same layouts as above; other chains' entries are left untouched).
int gdn_oracle_chunked_stages(const double* q, const double* k, const double* v,
                              const double* log_alpha, const double* beta,
                              const double* initial_state, double* out, double* final_state,
                              const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v,
                              int chunk, int n, int h,
                              double* g, double* A, double* P, double* Tm, double* W, double* U, double* D,
                              double* Sin) {
    Problem p{q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v};
    if (!valid(p) || chunk <= 0 || n < 0 || n >= B || h < 0 || h >= H) return 1;
    const Stages st{g, A, P, Tm, W, U, D, Sin};
    chunked_chain(p, n, h, chunk, 0, &st);
    return 0;
}

int gdn_oracle_dense(const double* q, const double* k, const double* v,
                     const double* log_alpha, const double* beta,
                     const double* initial_state, double* out, double* final_state,
                     const int32_t* cu_seqlens, int B, int T, int H, int d_k, int d_v) {
    Problem p{q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, B, T, H, d_k, d_v};
    if (!valid(p)) return 1;
    const int chains = B * H;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad)
    for (int c = 0; c < chains; ++c) bad += dense_chain(p, c / H, c % H) ? 0 : 1;
    return bad ? 1 : 0;
}

} // extern "C"
