// TEST INFRASTRUCTURE -- CPU oracle for the DecentLaM / DmSGD / PmSGD update rules.
//
// Plain, slow, double-precision restatement of what the paper defines, written so a
// reader can check every loop against the cited equation by eye.  It shares no code,
// header, table or constant with the CUDA library; only tests, the smoke check and the
// benchmark's CPU-baseline leg may call it.  The product never does.
//
// Conventions
//   * n nodes, d coordinates; every [n, d] array is row-major double, row i = node i.
//   * W is a dense row-major [n, n] double matrix, W[i*n+j] = w_ij = weight on what
//     flows from node j to node i (Sec. 3, "Network topology and weights").
//   * Indices are 0-based here (the paper counts from 1).
//   * "threads" splits the coordinate range [0, d) into disjoint contiguous pieces, one
//     per std::thread.  Coordinates never interact (every rule below is coordinate-wise),
//     so this changes no arithmetic.
//
// Reading of the row-sum condition (Assumption A.3, W 1 = 1): weights stored as fp32 do
// not add up to exactly one.  Wherever the paper's algebra needs (I - W) to annihilate
// the all-ones vector, the rules below form that product from the off-diagonal weights
// only,  ((I - W) x)_i = sum_{j != i} w_ij (x_i - x_j),  which is (I - W) x for a W whose
// diagonal is exactly 1 - sum_{j != i} w_ij.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <thread>
#include <vector>

namespace {

// Run body(c0, c1) over disjoint coordinate ranges covering [0, d).
void for_column_ranges(int64_t d, int threads, const std::function<void(int64_t, int64_t)>& body) {
    if (threads < 1) threads = 1;
    if ((int64_t)threads > d) threads = (int)(d > 0 ? d : 1);
    if (threads == 1) { body(0, d); return; }
    std::vector<std::thread> pool;
    for (int t = 0; t < threads; ++t) {
        int64_t c0 = d * t / threads, c1 = d * (t + 1) / threads;
        pool.emplace_back([=, &body] { body(c0, c1); });
    }
    for (auto& th : pool) th.join();
}

// floor(log2(v)) for v >= 1
int floor_log2(int v) { int l = 0; while ((v >> (l + 1)) > 0) ++l; return l; }

// Off-diagonal weight for an integer denominator q: 1/q rounded once to fp32.
double w32(int q) { return (double)(float)(1.0 / (double)q); }

}  // namespace

extern "C" {

// Topology kinds understood by the oracle.
enum { ORC_RING = 0, ORC_STATIC_EXP = 1, ORC_ONE_PEER_EXP = 2, ORC_COMPLETE = 3, ORC_ADJ_MH = 4,
       ORC_SYM_EXP = 5, ORC_MESH = 6 };

// Number of distinct weight matrices the topology cycles through (slot = k mod period).
// One-peer exponential graph: one hop 2^t per iteration, t = 0 .. floor(log2(n-1)).
int orc_topology_period(int kind, int n) {
    if (kind == ORC_ONE_PEER_EXP) return n >= 2 ? floor_log2(n - 1) + 1 : 1;
    return 1;
}

// Dense W for (kind, n, slot).  adj is an n*n 0/1 symmetric adjacency without self loops,
// used only by ORC_ADJ_MH.  Returns 0 on success, -1 on a bad argument.
//
// Every off-diagonal weight is 1/q for an integer q, rounded once to fp32 and promoted
// back to double.  The diagonal entry is the fp32 rounding of (1 - sum_{j != i} 1/q_ij),
// that sum taken in double over ascending j with the *unrounded* 1/q_ij.  This diagonal is
// what multiplies g_i in W g; the x-mixing never uses it (see the header comment).
//
//   RING          Sec. "Network topologies" (App. G): each node talks to its two direct
//                 neighbours; N_i = {i-1, i, i+1} mod n, all weights 1/3 (n >= 3).
//   STATIC_EXP    directed exponential graph: node i receives from (i + 2^t) mod n for
//                 t = 0 .. L-1, L = floor(log2(n-1)) + 1; all L+1 weights equal 1/(L+1).
//   ONE_PEER_EXP  slot t: node i receives from (i + 2^t) mod n only; weights 1/2, 1/2.
//   COMPLETE      w_ij = 1/n (Sec. 3: DSGD then reduces to parallel SGD).
//   ADJ_MH        Metropolis-Hastings rule (Assumption A.3 and App. G cite it without
//                 printing it): w_ij = 1 / (1 + max(deg_i, deg_j)) on every edge, the
//                 diagonal takes the remainder.
//   SYM_EXP       symmetric exponential graph of App. G: every odd rank i is joined to the even
//                 ranks (i + 2^t - 1) mod n, t = 1 .. floor(log2(n-1)) (the t = 0 term of the
//                 printed list is i itself, and its last term is read with the "- 1" the others
//                 carry); undirected; Metropolis-Hastings weights.  n even, n >= 4.
//   MESH          logical mesh of App. G: nodes on an r x c grid (row-major ranks), r the largest
//                 divisor of n not above sqrt(n), joined to their direct horizontal and
//                 vertical neighbours, no wrap-around; Metropolis-Hastings weights.  n >= 2.
int orc_topology_dense(int kind, int n, int slot, const uint8_t* adj, double* W) {
    if (n < 1 || !W) return -1;
    std::vector<int> q((size_t)n * n, 0);  // integer denominators, 0 = no edge
    auto Q = [&](int i, int j) -> int& { return q[(size_t)i * n + j]; };
    switch (kind) {
    case ORC_RING:
        if (n < 3) return -1;
        for (int i = 0; i < n; ++i) { Q(i, (i + 1) % n) = 3; Q(i, (i + n - 1) % n) = 3; }
        break;
    case ORC_STATIC_EXP: {
        if (n < 2) return -1;
        int L = floor_log2(n - 1) + 1;
        for (int i = 0; i < n; ++i)
            for (int t = 0; t < L; ++t) Q(i, (int)(((int64_t)i + ((int64_t)1 << t)) % n)) = L + 1;
        for (int i = 0; i < n; ++i) Q(i, i) = 0;
        break;
    }
    case ORC_ONE_PEER_EXP: {
        if (n < 2) return -1;
        int L = floor_log2(n - 1) + 1;
        if (slot < 0 || slot >= L) return -1;
        for (int i = 0; i < n; ++i) Q(i, (int)(((int64_t)i + ((int64_t)1 << slot)) % n)) = 2;
        for (int i = 0; i < n; ++i) Q(i, i) = 0;
        break;
    }
    case ORC_COMPLETE:
        for (int i = 0; i < n; ++i) for (int j = 0; j < n; ++j) if (i != j) Q(i, j) = n;
        break;
    case ORC_SYM_EXP:
    case ORC_MESH:
    case ORC_ADJ_MH: {
        std::vector<uint8_t> built;
        if (kind == ORC_SYM_EXP) {
            if (n < 4 || n % 2) return -1;
            built.assign((size_t)n * n, 0);
            const int T = floor_log2(n - 1);
            for (int i = 1; i < n; i += 2)
                for (int t = 1; t <= T; ++t) {
                    const int j = (int)(((int64_t)i + ((int64_t)1 << t) - 1) % n);
                    built[(size_t)i * n + j] = built[(size_t)j * n + i] = 1;
                }
            adj = built.data();
        } else if (kind == ORC_MESH) {
            if (n < 2) return -1;
            built.assign((size_t)n * n, 0);
            int r = 1;
            for (int c = 1; c * c <= n; ++c) if (n % c == 0) r = c;
            const int cols = n / r;
            for (int a = 0; a < r; ++a)
                for (int b = 0; b < cols; ++b) {
                    const int i = a * cols + b;
                    if (b + 1 < cols) built[(size_t)i * n + i + 1] = built[(size_t)(i + 1) * n + i] = 1;
                    if (a + 1 < r) built[(size_t)i * n + i + cols] = built[(size_t)(i + cols) * n + i] = 1;
                }
            adj = built.data();
        }
        if (!adj) return -1;
        std::vector<int> deg(n, 0);
        for (int i = 0; i < n; ++i) {
            if (adj[(size_t)i * n + i]) return -1;
            for (int j = 0; j < n; ++j) {
                if (adj[(size_t)i * n + j] != adj[(size_t)j * n + i]) return -1;
                if (adj[(size_t)i * n + j]) ++deg[i];
            }
        }
        for (int i = 0; i < n; ++i) for (int j = 0; j < n; ++j)
            if (adj[(size_t)i * n + j]) Q(i, j) = 1 + (deg[i] > deg[j] ? deg[i] : deg[j]);
        break;
    }
    default: return -1;
    }
    for (int i = 0; i < n; ++i) {
        double off = 0.0;
        for (int j = 0; j < n; ++j) {
            if (j == i) continue;
            W[(size_t)i * n + j] = Q(i, j) ? w32(Q(i, j)) : 0.0;
            if (Q(i, j)) off += 1.0 / (double)Q(i, j);
        }
        W[(size_t)i * n + i] = (double)(float)(1.0 - off);
    }
    return 0;
}

// DecentLaM, one iteration (Sec. 5, Eqs. decentLaM-x-1..3; Algorithm 2):
//   g~ = W g + (1/gamma) (I - W) x ;  m' = beta m + g~ ;  x' = x - gamma m'.
// All right-hand sides are iteration-k values (every node updates at once).
void orc_decentlam_step(int n, int64_t d, const double* W, const double* x, const double* m,
                        const double* g, double beta, double gamma, double* x_out, double* m_out,
                        int threads) {
    for_column_ranges(d, threads, [&](int64_t c0, int64_t c1) {
        for (int i = 0; i < n; ++i)
            for (int64_t c = c0; c < c1; ++c) {
                double mixg = 0.0;  // (W g)_i
                for (int j = 0; j < n; ++j) mixg += W[(size_t)i * n + j] * g[(size_t)j * d + c];
                double cons = 0.0;  // ((I - W) x)_i
                for (int j = 0; j < n; ++j)
                    if (j != i) cons += W[(size_t)i * n + j] * (x[(size_t)i * d + c] - x[(size_t)j * d + c]);
                double gt = mixg + cons / gamma;
                double mn = beta * m[(size_t)i * d + c] + gt;
                m_out[(size_t)i * d + c] = mn;
                x_out[(size_t)i * d + c] = x[(size_t)i * d + c] - gamma * mn;
            }
    });
}

// DecentLaM written the way each node evaluates it (Eq. DecentLaM-gi; App. A matrix form):
//   g~_i = x_i/gamma - (1/gamma) sum_{j in N_i} w_ij (x_j - gamma g_j).
// In the self term the weight on x_i is exactly 1 - sum_{j != i} w_ij (unit row sum) and the
// weight on g_i is the stored diagonal, so this names the same numbers as
// orc_decentlam_step.  Used only to cross-check the two printed forms against each other.
void orc_decentlam_step_pernode(int n, int64_t d, const double* W, const double* x, const double* m,
                                const double* g, double beta, double gamma, double* x_out, double* m_out) {
    for (int i = 0; i < n; ++i) {
        double off = 0.0;
        for (int j = 0; j < n; ++j) if (j != i) off += W[(size_t)i * n + j];
        double wii_exact = 1.0 - off, wii_stored = W[(size_t)i * n + i];
        for (int64_t c = 0; c < d; ++c) {
            double avg = 0.0;  // sum_j w_ij (x_j - gamma g_j)
            for (int j = 0; j < n; ++j) {
                if (j == i) avg += wii_exact * x[(size_t)i * d + c] - wii_stored * gamma * g[(size_t)i * d + c];
                else avg += W[(size_t)i * n + j] * (x[(size_t)j * d + c] - gamma * g[(size_t)j * d + c]);
            }
            double gt = x[(size_t)i * d + c] / gamma - avg / gamma;
            double mn = beta * m[(size_t)i * d + c] + gt;
            m_out[(size_t)i * d + c] = mn;
            x_out[(size_t)i * d + c] = x[(size_t)i * d + c] - gamma * mn;
        }
    }
}

// DmSGD, one iteration (Algorithm 1; App. A matrix form):
//   m' = beta m + g ;  y = x - gamma m' ;  x'_i = sum_j w_ij y_j = y_i + sum_{j != i} w_ij (y_j - y_i).
void orc_dmsgd_step(int n, int64_t d, const double* W, const double* x, const double* m,
                    const double* g, double beta, double gamma, double* x_out, double* m_out,
                    int threads) {
    for_column_ranges(d, threads, [&](int64_t c0, int64_t c1) {
        std::vector<double> y(n);
        for (int64_t c = c0; c < c1; ++c) {
            for (int i = 0; i < n; ++i) {
                double mn = beta * m[(size_t)i * d + c] + g[(size_t)i * d + c];
                m_out[(size_t)i * d + c] = mn;
                y[i] = x[(size_t)i * d + c] - gamma * mn;
            }
            for (int i = 0; i < n; ++i) {
                double acc = 0.0;
                for (int j = 0; j < n; ++j) if (j != i) acc += W[(size_t)i * n + j] * (y[j] - y[i]);
                x_out[(size_t)i * d + c] = y[i] + acc;
            }
        }
    });
}

// Decentralized SGD without momentum.
//   variant 0, adapt-then-combine (Sec. 3, Eqs. dsgd-1, dsgd-2):  y = x - gamma g ;  x' = W y
//   variant 1, adapt-with-combine (Remark in Sec. 5):             x' = W x - gamma g
// W is applied with exact unit row sums: (W y)_i = y_i + sum_{j != i} w_ij (y_j - y_i).
void orc_dsgd_step(int n, int64_t d, const double* W, const double* x, const double* g, double gamma, int variant,
                   double* x_out, int threads) {
    for_column_ranges(d, threads, [&](int64_t c0, int64_t c1) {
        std::vector<double> y(n);
        for (int64_t c = c0; c < c1; ++c) {
            for (int i = 0; i < n; ++i)
                y[i] = variant == 0 ? x[(size_t)i * d + c] - gamma * g[(size_t)i * d + c] : x[(size_t)i * d + c];
            for (int i = 0; i < n; ++i) {
                double acc = 0.0;
                for (int j = 0; j < n; ++j) if (j != i) acc += W[(size_t)i * n + j] * (y[j] - y[i]);
                double v = y[i] + acc;
                if (variant == 1) v -= gamma * g[(size_t)i * d + c];
                x_out[(size_t)i * d + c] = v;
            }
        }
    });
}

// Parallel momentum SGD (Sec. 1 and Sec. 7: every node applies momentum SGD to the
// globally averaged gradient):  gbar = (1/n) sum_i g_i ;  m'_i = beta m_i + gbar ;
// x'_i = x_i - gamma m'_i.
void orc_pmsgd_step(int n, int64_t d, const double* x, const double* m, const double* g,
                    double beta, double gamma, double* x_out, double* m_out, int threads) {
    for_column_ranges(d, threads, [&](int64_t c0, int64_t c1) {
        for (int64_t c = c0; c < c1; ++c) {
            double s = 0.0;
            for (int i = 0; i < n; ++i) s += g[(size_t)i * d + c];
            double gbar = s / (double)n;
            for (int i = 0; i < n; ++i) {
                double mn = beta * m[(size_t)i * d + c] + gbar;
                m_out[(size_t)i * d + c] = mn;
                x_out[(size_t)i * d + c] = x[(size_t)i * d + c] - gamma * mn;
            }
        }
    });
}

// Momentum-free form of DecentLaM (App. B.2):  x^{k+1} = W (x^k - gamma g^k) + beta (x^k - x^{k-1}).
// W x is taken as x_i + sum_{j != i} w_ij (x_j - x_i) (exact unit row sum), W g with the stored diagonal.
void orc_decentlam_two_term(int n, int64_t d, const double* W, const double* xk, const double* xkm1,
                            const double* g, double beta, double gamma, double* x_next) {
    for (int i = 0; i < n; ++i)
        for (int64_t c = 0; c < d; ++c) {
            double Wx = xk[(size_t)i * d + c], Wg = 0.0;
            for (int j = 0; j < n; ++j) {
                if (j != i) Wx += W[(size_t)i * n + j] * (xk[(size_t)j * d + c] - xk[(size_t)i * d + c]);
                Wg += W[(size_t)i * n + j] * g[(size_t)j * d + c];
            }
            x_next[(size_t)i * d + c] = Wx - gamma * Wg + beta * (xk[(size_t)i * d + c] - xkm1[(size_t)i * d + c]);
        }
}

// Momentum-free form of DmSGD for a constant W (Sec. 4 Eq. (DSGD + momentum); App. B.1):
//   x^{k+1} = W (x^k - gamma g^k) + beta (x^k - W x^{k-1}),  W applied with exact unit row sum.
void orc_dmsgd_two_term(int n, int64_t d, const double* W, const double* xk, const double* xkm1,
                        const double* g, double beta, double gamma, double* x_next) {
    std::vector<double> z(n), p(n);
    for (int64_t c = 0; c < d; ++c) {
        for (int i = 0; i < n; ++i) { z[i] = xk[(size_t)i * d + c] - gamma * g[(size_t)i * d + c]; p[i] = xkm1[(size_t)i * d + c]; }
        for (int i = 0; i < n; ++i) {
            double Wz = z[i], Wp = p[i];
            for (int j = 0; j < n; ++j) if (j != i) {
                Wz += W[(size_t)i * n + j] * (z[j] - z[i]);
                Wp += W[(size_t)i * n + j] * (p[j] - p[i]);
            }
            x_next[(size_t)i * d + c] = Wz + beta * (xk[(size_t)i * d + c] - Wp);
        }
    }
}

// Full-batch least-squares gradient of node i (App. G, linear-regression experiment):
//   f_i(x) = (scale/2) ||A_i x - b_i||^2 ,  g_i = scale * A_i^T (A_i x_i - b_i).
// A is [n, p, q] row-major fp32, b is [n, p] fp32 (the same bits the GPU reads), x and g are [n, q] double.
// "threads" splits the node range.
void orc_lsq_grad(int n, int p, int q, const float* A, const float* b, const double* x,
                  double scale, double* g, int threads) {
    for_column_ranges(n, threads, [&](int64_t i0, int64_t i1) {
        std::vector<double> r(p);
        for (int64_t i = i0; i < i1; ++i) {
            const float* Ai = A + (size_t)i * p * q;
            for (int a = 0; a < p; ++a) {
                double s = 0.0;
                for (int c = 0; c < q; ++c) s += (double)Ai[(size_t)a * q + c] * x[(size_t)i * q + c];
                r[a] = s - (double)b[(size_t)i * p + a];
            }
            for (int c = 0; c < q; ++c) {
                double s = 0.0;
                for (int a = 0; a < p; ++a) s += (double)Ai[(size_t)a * q + c] * r[a];
                g[(size_t)i * q + c] = scale * s;
            }
        }
    });
}

}  // extern "C"
