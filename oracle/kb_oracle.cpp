// CPU oracle for the batched bandit step (KernelBand decision layer).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
// definition of what the CUDA library must compute.  It is called from the
// tests, from the smoke check and from the benchmark's CPU-baseline leg, and
// from nowhere else; the product path never routes through it.  It shares no
// code, header, table or helper with the CUDA sources.
//
// Arithmetic: inputs and stored outputs are fp32 (the library's types); every
// sum, distance, mean, ratio and index is evaluated in double and rounded to
// fp32 only when it is stored in an fp32 output.  Every decision (argmin,
// argmax, threshold test) is taken on the double values.  Ties go to the
// lowest index.  One thread, no blocking, no fusion, no reordering.
//
// Parity pins: every function below is pinned by the CPU test-suite against
// closed forms, worked values, invariants, brute force and a library K-Means
// with a fixed initialisation.
//
// Arrays are dense, row-major, batch-major: X[B][N][D], C[B][K][D],
// labels[B][N], pulls[B][N][S], hsig[B][K][R].

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <limits>
#include <vector>

namespace {
inline size_t ix2(size_t a, size_t b, size_t nb) { return a * nb + b; }
inline size_t ix3(size_t a, size_t b, size_t c, size_t nb, size_t nc) { return (a * nb + b) * nc + c; }
const double kInf = std::numeric_limits<double>::infinity();
}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// Feature normalisation: per instance and column, population z-score.
// The paper only says the features are "normalized"/"log-transformed"
// (Sec. 3.2, App. A.1); the workloads fix the reading: z = (x - mean) / std
// with the population std (divide by N); a column whose std is below 1e-12
// gets scale 1 (so it becomes all zeros).
// ---------------------------------------------------------------------------
int kbo_normalize(int B, int N, int D, const float* x, float* z, float* mean, float* scale) {
    for (int b = 0; b < B; ++b) {
        for (int d = 0; d < D; ++d) {
            double sum = 0.0;
            for (int k = 0; k < N; ++k) sum += (double)x[ix3(b, k, d, N, D)];
            double m = N > 0 ? sum / (double)N : 0.0;
            double ss = 0.0;
            for (int k = 0; k < N; ++k) {
                double e = (double)x[ix3(b, k, d, N, D)] - m;
                ss += e * e;
            }
            double sd = N > 0 ? std::sqrt(ss / (double)N) : 0.0;
            double sc = sd < 1e-12 ? 1.0 : sd;
            for (int k = 0; k < N; ++k)
                z[ix3(b, k, d, N, D)] = (float)(((double)x[ix3(b, k, d, N, D)] - m) / sc);
            if (mean) mean[ix2(b, d, D)] = (float)m;
            if (scale) scale[ix2(b, d, D)] = (float)sc;
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Hardware-aware pruning.
//  roofline floor   T_lb(k,s) = max(F_k / P_s, Q_k / W_s)      (the roofline
//      model Assumption 1 cites for its bounding function)
//  roofline keep    T_lb(k,s) < T_inc     (an arm whose floor cannot beat the
//      incumbent, the best runtime found so far in Algorithm 1's return line)
//  saturation keep  h_c[label(k)][Target(s)] < theta_sat   (mask equation of
//      Sec. 3.4, strict <; applied only when labels/hsig/target are given)
//  bound            B(k,s) = clip((T_k - T_lb) / T_k, 0, 1)   (Assumption 1:
//      the gap between current performance and the limit, in reward units of
//      the reward definition in Sec. 2.2)
// keep[b][k] bit s = roofline keep AND saturation keep.
// margin (optional, [B][N][S]): the relative distance from its threshold of the
// comparison(s) that DECIDE the bit, for near-tie accounting in the tests:
//   |T_lb - T_inc| / T_inc  and  |h - theta_sat| / theta_sat  per comparison;
//   a kept arm passes both, and either one flipping prunes it: the smaller;
//   an arm pruned by one comparison only: that comparison's;
//   an arm pruned by both: both must flip to keep it: the larger.
// (Without the saturation inputs only the roofline comparison exists.)
// ---------------------------------------------------------------------------
int kbo_prune(int B, int N, int S, int K, int R, const float* flops, const float* bytes,
              const float* peak_flops, const float* peak_bw, const float* t_incumbent,
              const float* t_cur, const int32_t* labels, const float* hsig, const int32_t* target,
              float theta_sat, uint32_t* keep, uint32_t* kept_count, float* bound, double* margin) {
    if (S > 32) return 1;
    const bool sat = labels && hsig && target;
    for (int b = 0; b < B; ++b) {
        uint64_t kept = 0;
        const double tinc = (double)t_incumbent[b];
        for (int k = 0; k < N; ++k) {
            uint32_t bits = 0;
            for (int s = 0; s < S; ++s) {
                double tf = (double)flops[ix2(b, k, N)] / (double)peak_flops[s];
                double tq = (double)bytes[ix2(b, k, N)] / (double)peak_bw[s];
                double tlb = tf > tq ? tf : tq;
                const bool roof_ok = tlb < tinc;
                const double m_roof = std::fabs(tlb - tinc) / std::fabs(tinc);
                bool ok = roof_ok;
                double mg = m_roof;
                if (sat) {
                    int lab = labels[ix2(b, k, N)];
                    if (lab < 0 || lab >= K) return 2;
                    int r = target[s];
                    if (r < 0 || r >= R) return 3;
                    double h = (double)hsig[ix3(b, lab, r, K, R)];
                    const bool sat_ok = h < (double)theta_sat;
                    const double m_sat = std::fabs(h - (double)theta_sat) / std::fabs((double)theta_sat);
                    ok = roof_ok && sat_ok;
                    if (roof_ok && sat_ok) mg = m_sat < m_roof ? m_sat : m_roof;        // the first to flip prunes
                    else if (!roof_ok && !sat_ok) mg = m_sat > m_roof ? m_sat : m_roof; // the last to flip keeps
                    else mg = roof_ok ? m_sat : m_roof;                                 // the one failing comparison
                }
                if (ok) { bits |= (1u << s); ++kept; }
                if (margin) margin[ix3(b, k, s, N, S)] = mg;
                if (bound) {
                    double tk = (double)t_cur[ix2(b, k, N)];
                    double g = (tk - tlb) / tk;
                    if (!(g > 0.0)) g = 0.0;
                    if (g > 1.0) g = 1.0;
                    bound[ix3(b, k, s, N, S)] = (float)g;
                }
            }
            keep[ix2(b, k, N)] = bits;
        }
        if (kept_count) kept_count[b] = (uint32_t)kept;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// K-Means assignment (Sec. 3.3; Algorithm 1 "KMeans" line): nearest centroid
// in squared Euclidean distance (the L2 norm of Assumption 2), direct form
// sum_d (z_d - c_d)^2.  label = lowest j attaining the minimum.
// inertia[b] = sum_k dist2.  rep[b][i] = the member of cluster i nearest its
// centroid (the "centroid kernel" that Sec. 3.3 profiles), lowest k on ties,
// -1 for an empty cluster.
// best/second (optional, double [B][N]): smallest and second smallest d^2.
// ---------------------------------------------------------------------------
int kbo_cluster_assign(int B, int N, int D, int K, const float* z, const float* centroids,
                       int32_t* labels, float* dist2, float* inertia, int32_t* rep,
                       double* best_out, double* second_out) {
    std::vector<double> repd((size_t)(K > 0 ? K : 1));
    for (int b = 0; b < B; ++b) {
        double total = 0.0;
        if (rep) for (int i = 0; i < K; ++i) { rep[ix2(b, i, K)] = -1; repd[i] = kInf; }
        for (int k = 0; k < N; ++k) {
            double best = kInf, second = kInf;
            int arg = -1;
            for (int j = 0; j < K; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) {
                    double e = (double)z[ix3(b, k, d, N, D)] - (double)centroids[ix3(b, j, d, K, D)];
                    acc += e * e;
                }
                if (acc < best) { second = best; best = acc; arg = j; }
                else if (acc < second) { second = acc; }
            }
            labels[ix2(b, k, N)] = arg;
            if (dist2) dist2[ix2(b, k, N)] = (float)best;
            if (best_out) best_out[ix2(b, k, N)] = best;
            if (second_out) second_out[ix2(b, k, N)] = second;
            total += best;
            if (rep && arg >= 0 && best < repd[arg]) { repd[arg] = best; rep[ix2(b, arg, K)] = k; }
        }
        if (inertia) inertia[b] = (float)total;
    }
    return 0;
}

// d^2 of every row to the centroid named by `labels` (double), so a test can
// judge a disagreeing label by how far from optimal it is.
int kbo_dist2_at(int B, int N, int D, int K, const float* z, const float* centroids,
                 const int32_t* labels, double* out) {
    for (int b = 0; b < B; ++b)
        for (int k = 0; k < N; ++k) {
            int j = labels[ix2(b, k, N)];
            if (j < 0 || j >= K) { out[ix2(b, k, N)] = kInf; continue; }
            double acc = 0.0;
            for (int d = 0; d < D; ++d) {
                double e = (double)z[ix3(b, k, d, N, D)] - (double)centroids[ix3(b, j, d, K, D)];
                acc += e * e;
            }
            out[ix2(b, k, N)] = acc;
        }
    return 0;
}

// ---------------------------------------------------------------------------
// K-Means centroid update (Sec. 3.3; Algorithm 1 "Update centroids"): each
// centroid becomes the arithmetic mean of its members; an empty cluster keeps
// its previous centroid and reports count 0.
// ---------------------------------------------------------------------------
int kbo_cluster_update(int B, int N, int D, int K, const float* z, const int32_t* labels,
                       float* centroids, int32_t* counts) {
    std::vector<double> sum((size_t)K * (size_t)D);
    std::vector<int64_t> cnt((size_t)(K > 0 ? K : 1));
    for (int b = 0; b < B; ++b) {
        for (size_t i = 0; i < sum.size(); ++i) sum[i] = 0.0;
        for (int i = 0; i < K; ++i) cnt[i] = 0;
        for (int k = 0; k < N; ++k) {
            int j = labels[ix2(b, k, N)];
            if (j < 0 || j >= K) return 2;
            ++cnt[j];
            for (int d = 0; d < D; ++d) sum[ix2(j, d, D)] += (double)z[ix3(b, k, d, N, D)];
        }
        for (int i = 0; i < K; ++i) {
            if (counts) counts[ix2(b, i, K)] = (int32_t)cnt[i];
            if (cnt[i] > 0)
                for (int d = 0; d < D; ++d)
                    centroids[ix3(b, i, d, K, D)] = (float)(sum[ix2(i, d, D)] / (double)cnt[i]);
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Cluster-level statistics, optimistic index, arm selection.
//  statistics (Algorithm 1 initialisation N=1, mu=0.5 and its running-mean
//  lines, applied pull by pull, give exactly):
//      N_{i,s}  = n0 + sum_{k in C_i} pulls[k][s]
//      mu_{i,s} = (n0*mu0 + sum_{k in C_i} reward_sum[k][s]) / N_{i,s}
//  cluster index (masked-UCB equation, Sec. 3.4):
//      U_cl(i,s) = mu_{i,s} + c * sqrt(ln t / N_{i,s})
//  arm index (Assumption 2: mu(k,s) <= mu(centre,s) + L*||phi(k) - centre||):
//      U(k,s) = U_cl(label(k), s) + L * sqrt(dist2(k)),
//      optionally capped by B(k,s) (Assumption 1).
//  selection: best_arm = lowest flat index k*S+s maximising U over kept arms
//  (-1 and -inf if none); best_cluster_arm = lowest i*S+s maximising U_cl over
//  pairs with at least one kept member arm (the paper's M_{i,s} when the mask
//  is constant within a cluster), -1 if none.
//  arm_index holds -inf for a pruned arm.
// ---------------------------------------------------------------------------
int kbo_score_select(int B, int N, int K, int S, float c, float lipschitz_L, float prior_pulls,
                     float prior_mean, int cap_with_bound, const int32_t* labels, const float* dist2,
                     const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                     const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean,
                     float* cl_index, float* arm_index, int32_t* best_arm, float* best_val,
                     int32_t* best_cluster_arm) {
    if (S > 32) return 1;
    const size_t KS = (size_t)K * (size_t)S;
    std::vector<int64_t> np_(KS ? KS : 1);
    std::vector<double> rs(KS ? KS : 1), ucl(KS ? KS : 1);
    std::vector<char> anyk(KS ? KS : 1);
    for (int b = 0; b < B; ++b) {
        for (size_t i = 0; i < KS; ++i) { np_[i] = 0; rs[i] = 0.0; anyk[i] = 0; }
        for (int k = 0; k < N; ++k) {
            int lab = labels[ix2(b, k, N)];
            if (lab < 0 || lab >= K) return 2;
            uint32_t bits = keep ? keep[ix2(b, k, N)] : 0xffffffffu;
            for (int s = 0; s < S; ++s) {
                np_[ix2(lab, s, S)] += (int64_t)pulls[ix3(b, k, s, N, S)];
                rs[ix2(lab, s, S)] += (double)reward_sum[ix3(b, k, s, N, S)];
                if ((bits >> s) & 1u) anyk[ix2(lab, s, S)] = 1;
            }
        }
        const double lnt = std::log((double)t[b]);
        double cbest = -kInf;
        int carg = -1;
        for (int i = 0; i < K; ++i)
            for (int s = 0; s < S; ++s) {
                double n = (double)prior_pulls + (double)np_[ix2(i, s, S)];
                double mu = ((double)prior_pulls * (double)prior_mean + rs[ix2(i, s, S)]) / n;
                double u = mu + (double)c * std::sqrt(lnt / n);
                ucl[ix2(i, s, S)] = u;
                cl_pulls[ix3(b, i, s, K, S)] = (float)n;
                cl_mean[ix3(b, i, s, K, S)] = (float)mu;
                cl_index[ix3(b, i, s, K, S)] = (float)u;
                if (anyk[ix2(i, s, S)]) {
                    if (u > cbest) { cbest = u; carg = i * S + s; }
                }
            }
        best_cluster_arm[b] = carg;

        double abest = -kInf;
        int64_t aarg = -1;
        for (int k = 0; k < N; ++k) {
            int lab = labels[ix2(b, k, N)];
            uint32_t bits = keep ? keep[ix2(b, k, N)] : 0xffffffffu;
            double smooth = 0.0;
            if (lipschitz_L != 0.0f) smooth = (double)lipschitz_L * std::sqrt((double)dist2[ix2(b, k, N)]);
            for (int s = 0; s < S; ++s) {
                double u = ucl[ix2(lab, s, S)] + smooth;
                if (cap_with_bound && bound) {
                    double cap = (double)bound[ix3(b, k, s, N, S)];
                    if (cap < u) u = cap;
                }
                bool ok = (bits >> s) & 1u;
                if (arm_index) arm_index[ix3(b, k, s, N, S)] = ok ? (float)u : -std::numeric_limits<float>::infinity();
                if (!ok) continue;
                if (u > abest) { abest = u; aarg = (int64_t)k * S + s; }
            }
        }
        best_arm[b] = (int32_t)aarg;
        best_val[b] = aarg >= 0 ? (float)abest : -std::numeric_limits<float>::infinity();
    }
    return 0;
}

// Gather of initial centroids: C[b][i][:] = Z[b][rows[b][i]][:] (plain Lloyd
// started from K data rows supplied by the caller).
// rows[b][i] == -1 names no row: cluster i of that instance is UNUSED -- its centroid is put at 1e18 in every
// coordinate, farther from any data than any other centroid, so no row is ever assigned to it, it stays empty and
// keeps that centroid through every update.  This is how instances with fewer than K clusters share a batch (the
// K in {1, 2, 3, 5} sensitivity study of Sec. 4 as four instances of one call with K = 5).
int kbo_init_centroids(int B, int N, int D, int K, const float* z, const int32_t* rows, float* centroids) {
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < K; ++i) {
            int r = rows[ix2(b, i, K)];
            if (r < -1 || r >= N) return 2;
            for (int d = 0; d < D; ++d) centroids[ix3(b, i, d, K, D)] = r < 0 ? 1e18f : z[ix3(b, r, d, N, D)];
        }
    return 0;
}

// ---------------------------------------------------------------------------
// Lloyd's iteration with a tolerance stop (the `tol` of the "scikit-learn's KMeans" of Sec. 3.5): per instance,
//   repeat: assign, update, shift = sum_j ||c_j(new) - c_j(old)||^2;  stop after this update if shift <= tol
//   or max_iter updates are done;  then one more assign, so that labels and dist2 belong to the returned centroids.
// (Unchanged labels give unchanged centroids, shift = 0 <= tol: the rule also covers "labels did not change".)
// n_iter[b] = updates done for instance b;  last_shift[b] (optional) = the shift of its last update.
// Instances stop independently of one another.
// ---------------------------------------------------------------------------
int kbo_lloyd_tol(int B, int N, int D, int K, int max_iter, float tol, const float* z, float* centroids,
                  int32_t* labels, float* dist2, float* inertia, int32_t* rep, int32_t* counts, int32_t* n_iter,
                  double* last_shift) {
    std::vector<float> old((size_t)K * (size_t)D);
    for (int b = 0; b < B; ++b) {
        const float* zb = z + (size_t)b * N * D;
        float* cb = centroids + (size_t)b * K * D;
        int32_t* lb = labels + (size_t)b * N;
        int32_t* nb = counts ? counts + (size_t)b * K : nullptr;
        int it = 0;
        double shift = 0.0;
        if (nb) for (int i = 0; i < K; ++i) nb[i] = 0;
        while (it < max_iter) {
            int rc = kbo_cluster_assign(1, N, D, K, zb, cb, lb, nullptr, nullptr, nullptr, nullptr, nullptr);
            if (rc) return rc;
            for (size_t e = 0; e < old.size(); ++e) old[e] = cb[e];
            rc = kbo_cluster_update(1, N, D, K, zb, lb, cb, nb);
            if (rc) return rc;
            ++it;
            shift = 0.0;
            for (size_t e = 0; e < old.size(); ++e) {
                const double dlt = (double)cb[e] - (double)old[e];
                shift += dlt * dlt;
            }
            if (shift <= (double)tol) break;
        }
        int rc = kbo_cluster_assign(1, N, D, K, zb, cb, lb, dist2 ? dist2 + (size_t)b * N : nullptr,
                                    inertia ? inertia + b : nullptr, rep ? rep + (size_t)b * K : nullptr, nullptr, nullptr);
        if (rc) return rc;
        n_iter[b] = it;
        if (last_shift) last_shift[b] = shift;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Counter-based random numbers: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, "Parallel random
// numbers: as easy as 1, 2, 3", SC'11), written out from the published round function: two 32x32 -> 64 bit
// products by the constants below, a word permutation with the key mixed in, and a Weyl bump of the key
// between rounds.  Pinned by the known-answer vectors of the generator's reference distribution.
// ---------------------------------------------------------------------------
void kbo_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---------------------------------------------------------------------------
// Within-cluster sampling of the kernel k_t (Sec. 3.4, "Action selection"; Algorithm 1, the line
// "Sample k_t in C_{I_t}"): once the pair (I_t, S_t) is chosen, k_t is drawn from the members of
// cluster I_t with P(k) proportional to exp(V_hw(k, S_t)), V_hw(k, s) = theta_sat - h(k)[Target(s)].
//
// The draw uses the Gumbel-max rule, which samples exactly that distribution: every member gets
// V_hw + G, G = -ln(-ln u) with u uniform in (0, 1), and the largest perturbed value wins (lowest
// index on ties).  u comes from the counter-based generator above so that a parallel
// implementation draws the same numbers in any order:
//     counter = (candidate index, instance index, t[b], 0),  key = (low, high word of seed),
//     u = ((first output word >> 9) + 0.5) * 2^-23          (23 bits: exact in fp32 and in double).
// Readings: h(k) is given per candidate (h_cand[B][N][R]); the paper profiles only
// the cluster representatives, so a caller without per-candidate profiles passes its estimate.  The
// paper states no temperature: none is applied.  A member whose signature entry is NaN is never drawn.
//
// cluster_arm[b] = I_t * S + S_t as kbo_score_select returns it, or negative: no draw.
// member[b]: the drawn candidate, or -1 (no pair chosen, or the cluster has no drawable member).
// pert (optional, double [B][N]): the perturbed value of every drawable member of the chosen
// cluster, -inf elsewhere (lets a test rank the members itself).
// prob (optional, double [B][N]): the softmax probabilities by their plain definition
// exp(V - max V) / sum, 0 for non-members (what the draw must follow in distribution).
// ---------------------------------------------------------------------------
int kbo_sample_member(int B, int N, int K, int S, int R, const int32_t* labels, const int32_t* cluster_arm,
                      const float* h_cand, const int32_t* target, float theta_sat, uint64_t seed,
                      const int32_t* t, int32_t* member, double* member_val, double* pert, double* prob) {
    const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    for (int b = 0; b < B; ++b) {
        member[b] = -1;
        if (member_val) member_val[b] = -kInf;
        if (pert) for (int k = 0; k < N; ++k) pert[ix2(b, k, N)] = -kInf;
        if (prob) for (int k = 0; k < N; ++k) prob[ix2(b, k, N)] = 0.0;
        const int ca = cluster_arm[b];
        if (ca < 0) continue;
        if (ca >= K * S) return 2;
        const int I = ca / S, s = ca % S;
        const int col = target[s];
        if (col < 0 || col >= R) return 2;
        double best = -kInf, vmax = -kInf;
        int arg = -1;
        for (int k = 0; k < N; ++k) {
            if (labels[ix2(b, k, N)] != I) continue;
            const double h = (double)h_cand[ix3(b, k, col, N, R)];
            if (std::isnan(h)) continue;
            const double V = (double)theta_sat - h;
            if (V > vmax) vmax = V;
            const uint32_t ctr[4] = {(uint32_t)k, (uint32_t)b, (uint32_t)t[b], 0u};
            uint32_t rnd[4];
            kbo_philox4x32_10(ctr, key, rnd);
            const double u = ((double)(rnd[0] >> 9) + 0.5) * (1.0 / 8388608.0);
            const double G = -std::log(-std::log(u));
            const double v = V + G;
            if (pert) pert[ix2(b, k, N)] = v;
            if (v > best) { best = v; arg = k; }
        }
        member[b] = arg;
        if (member_val && arg >= 0) member_val[b] = best;
        if (prob && arg >= 0) {
            double sum = 0.0;
            for (int k = 0; k < N; ++k) {
                if (labels[ix2(b, k, N)] != I) continue;
                const double h = (double)h_cand[ix3(b, k, col, N, R)];
                if (std::isnan(h)) continue;
                sum += std::exp(((double)theta_sat - h) - vmax);
            }
            for (int k = 0; k < N; ++k) {
                if (labels[ix2(b, k, N)] != I) continue;
                const double h = (double)h_cand[ix3(b, k, col, N, R)];
                if (std::isnan(h)) continue;
                prob[ix2(b, k, N)] = std::exp(((double)theta_sat - h) - vmax) / sum;
            }
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Outcome of one iteration (Sec. 2.2 "Formal Model": r_t = Clip((L(k_t) - L(k'_t)) / L(k_t), 0, 1);
// Algorithm 1, "Generation & update": if Verify(k'_t): N_{I,S} <- N_{I,S} + 1,
// mu_{I,S} <- mu_{I,S} + (r_t - mu_{I,S}) / N_{I,S}).
//
// The statistics are kept per arm as (pulls, reward_sum), from which kbo_score_select forms
// N_{i,s} and mu_{i,s} per cluster in closed form (so that a re-clustering re-aggregates them);
// the update of the pair (I_t, S_t) through its drawn member k_t is therefore
//     pulls[k_t][S_t] += 1,  reward_sum[k_t][S_t] += r_t,
// which gives exactly the running mean above for the cluster that holds k_t.
// Readings: Algorithm 1 skips the update when verification fails, the formal model assigns
// zero reward to failures; `failures_count` = 0 takes Algorithm 1's line (no update), non-zero
// the other (one pull with reward 0).  A runtime L(k_t) <= 0 or a NaN ratio gives reward 0.
// The iteration counter t[b] advances in every case (it is the loop index of Algorithm 1).
//
// member [B]: k_t (negative: nothing was drawn, only t advances); cluster_arm [B]: I_t*S + S_t;
// t_cur [B][N]: L(k) of every candidate; t_new [B]: L(k'_t); verified [B] (nullable = all pass).
// reward [B] (optional out): r_t as used (0 where nothing was updated).
// ---------------------------------------------------------------------------
int kbo_record_outcome(int B, int N, int S, int failures_count, const int32_t* member, const int32_t* cluster_arm,
                       const float* t_cur, const float* t_new, const int32_t* verified, int32_t* pulls,
                       float* reward_sum, int32_t* t, float* reward) {
    for (int b = 0; b < B; ++b) {
        if (reward) reward[b] = 0.0f;
        t[b] += 1;
        const int k = member[b];
        if (k < 0) continue;
        if (k >= N || cluster_arm[b] < 0) return 2;
        const int s = cluster_arm[b] % S;
        const bool ok = verified ? verified[b] != 0 : true;
        if (!ok && !failures_count) continue;
        double r = 0.0;
        if (ok) {
            const double L = (double)t_cur[ix2(b, k, N)], Ln = (double)t_new[b];
            r = L > 0.0 ? (L - Ln) / L : 0.0;
            if (!(r > 0.0)) r = 0.0;          // regressions and NaN
            if (r > 1.0) r = 1.0;
        }
        pulls[ix3(b, k, s, N, S)] += 1;
        reward_sum[ix3(b, k, s, N, S)] = (float)((double)reward_sum[ix3(b, k, s, N, S)] + r);
        if (reward) reward[b] = (float)r;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// k-means++ seeding (Arthur & Vassilvitskii, "k-means++: the advantages of careful seeding", SODA'07;
// what "scikit-learn's KMeans" of Sec. 3.5 starts from by default, here without its extra greedy
// trials): the first centre is a row drawn uniformly; every further centre is a row drawn with
// probability D(x)^2 / sum D^2, D(x) = distance of x to the nearest centre chosen so far.
//
// Each draw is a Gumbel-max over the weights w (1 in round 0, D^2 afterwards): the row with the
// largest ln(w) + G wins, G = -ln(-ln u), u from the counter-based generator at
//     counter = (row, instance, round, 1),  key = (low, high word of seed),
//     u = ((first output word >> 9) + 0.5) * 2^-23;
// rows of weight 0 (chosen rows and their duplicates) are never drawn.  If every weight is 0 (fewer
// distinct rows than K) the round draws uniformly among all rows instead (weights 1, same G).
//
// One round, given the centres chosen so far (so that a test can follow another implementation's
// choices round by round): chosen[B][round] in; row[B] out; pert (optional, double [B][N]) the
// perturbed value of every drawable row (-inf elsewhere); mind2 (optional, double [B][N]) the
// weights D^2 of the round (1 in round 0).
// ---------------------------------------------------------------------------
int kbo_kmeanspp_round(int B, int N, int D, int round, const float* z, const int32_t* chosen, int chosen_stride,
                       uint64_t seed, int32_t* row, double* pert, double* mind2) {
    if (N < 1) return 1;
    const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    std::vector<double> w(N);
    for (int b = 0; b < B; ++b) {
        bool any = false;
        for (int k = 0; k < N; ++k) {
            double m = round == 0 ? 1.0 : kInf;
            for (int j = 0; j < round; ++j) {
                const int c = chosen[(size_t)b * chosen_stride + j];
                if (c < 0 || c >= N) return 2;
                double d2 = 0.0;
                for (int d = 0; d < D; ++d) {
                    const double e = (double)z[ix3(b, k, d, N, D)] - (double)z[ix3(b, c, d, N, D)];
                    d2 += e * e;
                }
                if (d2 < m) m = d2;
            }
            w[k] = m;
            if (m > 0.0) any = true;
        }
        double best = -kInf;
        int arg = -1;
        for (int k = 0; k < N; ++k) {
            const double wk = any ? w[k] : 1.0;
            if (mind2) mind2[ix2(b, k, N)] = wk;
            if (pert) pert[ix2(b, k, N)] = -kInf;
            if (!(wk > 0.0)) continue;
            const uint32_t ctr[4] = {(uint32_t)k, (uint32_t)b, (uint32_t)round, 1u};
            uint32_t rnd[4];
            kbo_philox4x32_10(ctr, key, rnd);
            const double u = ((double)(rnd[0] >> 9) + 0.5) * (1.0 / 8388608.0);
            const double v = std::log(wk) - std::log(-std::log(u));
            if (pert) pert[ix2(b, k, N)] = v;
            if (v > best) { best = v; arg = k; }
        }
        row[b] = arg;
    }
    return 0;
}

// All K rounds, each fed the rows this function chose before: rows[B][K].
int kbo_kmeanspp(int B, int N, int D, int K, const float* z, uint64_t seed, int32_t* rows) {
    std::vector<int32_t> r(B > 0 ? B : 1);
    for (int j = 0; j < K; ++j) {
        const int rc = kbo_kmeanspp_round(B, N, D, j, z, rows, K, seed, r.data(), nullptr, nullptr);
        if (rc) return rc;
        for (int b = 0; b < B; ++b) rows[(size_t)b * K + j] = r[b];
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Cluster radius: radius[b][i] = max over the members k of cluster i of ||z_k - c_i|| = sqrt(dist2[k])
// (0 for an empty cluster).  Theorem 1's bound carries the term L * max_i diam(C_i); by the triangle
// inequality through the centroid diam(C_i) <= 2 radius_i, so 2 L max_i radius_i bounds that term with one
// pass over the candidates instead of all pairs.
// ---------------------------------------------------------------------------
int kbo_cluster_radius(int B, int N, int K, const int32_t* labels, const float* dist2, float* radius) {
    for (int b = 0; b < B; ++b) {
        for (int i = 0; i < K; ++i) radius[ix2(b, i, K)] = 0.0f;
        for (int k = 0; k < N; ++k) {
            const int lab = labels[ix2(b, k, N)];
            if (lab < 0 || lab >= K) return 2;
            const double d2 = (double)dist2[ix2(b, k, N)];
            if (!(d2 > 0.0)) continue;
            const float r = (float)std::sqrt(d2);
            if (r > radius[ix2(b, lab, K)]) radius[ix2(b, lab, K)] = r;
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Top-M arms of an instance by the per-arm index U(k, s) (the masked argmax of Sec. 3.4 generalised from
// one arm to M, for generating M candidates per iteration; Sec. 5 mentions batched generation): the M arms
// with the largest arm_index, larger value first, lower flat index k*S + s first among equal values.  Pruned
// arms (-inf) and NaN entries never appear; when fewer than M arms are valid the tail is -1 / -inf.
// Written as its definition: order all valid arms, take the first M.
// ---------------------------------------------------------------------------
int kbo_top_m(int B, int NS, int M, const float* arm_index, int32_t* top_arm, float* top_val) {
    std::vector<int32_t> order;
    for (int b = 0; b < B; ++b) {
        const float* v = arm_index + (size_t)b * NS;
        order.clear();
        for (int i = 0; i < NS; ++i)
            if (v[i] > -std::numeric_limits<float>::infinity()) order.push_back(i);     // false for NaN too
        // insertion of one arm at a time into the first M places (plain selection, no library sort)
        std::vector<int32_t> top;
        for (int32_t i : order) {
            size_t pos = top.size();
            while (pos > 0 && (v[top[pos - 1]] < v[i])) --pos;      // equal values keep the earlier (lower) index first
            if (pos < (size_t)M) {
                top.insert(top.begin() + pos, i);
                if (top.size() > (size_t)M) top.pop_back();
            }
        }
        for (int j = 0; j < M; ++j) {
            const bool have = (size_t)j < top.size();
            top_arm[(size_t)b * M + j] = have ? top[j] : -1;
            top_val[(size_t)b * M + j] = have ? v[top[j]] : -std::numeric_limits<float>::infinity();
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Algorithm 1's loop kept on the cluster tables themselves (no pass over the candidates):
//
// kbo_select_pair: the masked-UCB choice (Sec. 3.4, masked-UCB equation; Algorithm 1 "Select (I_t, S_t)")
//     (I_t, S_t) = argmax over pairs with M_{i,s} = 1 of  mu_{i,s} + c sqrt(ln t / N_{i,s}),
//     M_{i,s} = [ h_c^(i)[Target(s)] < theta_sat ]  (Algorithm 1, "Hardware-constrained selection";
//     hsig null: no pair is masked).  Lowest i*S + s on ties; -1 when every pair is masked.
// kbo_update_pair: Algorithm 1's two statistics lines for the chosen pair, literally:
//     N <- N + 1,  mu <- mu + (r - mu) / N.
// ---------------------------------------------------------------------------
int kbo_select_pair(int B, int K, int S, int R, float c, const float* cl_pulls, const float* cl_mean, const int32_t* t,
                    const float* hsig, const int32_t* target, float theta_sat, float* cl_index, int32_t* pair) {
    for (int b = 0; b < B; ++b) {
        const double lnt = std::log((double)t[b]);
        double best = -kInf;
        int arg = -1;
        for (int i = 0; i < K; ++i)
            for (int s = 0; s < S; ++s) {
                const double n = (double)cl_pulls[ix3(b, i, s, K, S)];
                const double u = (double)cl_mean[ix3(b, i, s, K, S)] + (double)c * std::sqrt(lnt / n);
                if (cl_index) cl_index[ix3(b, i, s, K, S)] = (float)u;
                bool valid = true;
                if (hsig) {
                    const int col = target[s];
                    if (col < 0 || col >= R) return 2;
                    valid = (double)hsig[ix3(b, i, col, K, R)] < (double)theta_sat;
                }
                if (valid && u > best) { best = u; arg = i * S + s; }
            }
        pair[b] = arg;
    }
    return 0;
}

int kbo_update_pair(int B, int K, int S, const int32_t* pair, const float* reward, float* cl_pulls, float* cl_mean) {
    for (int b = 0; b < B; ++b) {
        const int p = pair[b];
        if (p < 0) continue;
        if (p >= K * S) return 2;
        const size_t i = (size_t)b * K * S + p;
        const double n = (double)cl_pulls[i] + 1.0;
        const double mu = (double)cl_mean[i] + ((double)reward[b] - (double)cl_mean[i]) / n;
        cl_pulls[i] = (float)n;
        cl_mean[i] = (float)mu;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// The expanding frontier (Sec. 2.2: the action space A_t = P_t x S grows with the frontier; Algorithm 1:
// "P <- {k_0}, C <- {P}" (one initial cluster), and inside "if Verify(k'_t)": "P <- P ∪ {k'_t}").
//
// The frontier of every search lives in arrays of a fixed capacity N_cap per instance, of which the first
// n_active[b] rows are candidates; the rest is padding whose label is -1.
//
// kbo_append_candidate: where the new kernel k'_t passed verification (verified[b] != 0; null = all passed) it
// becomes row j = n_active[b] of its instance:
//     x[b][j] = x_new[b] (its raw features),  t_cur[b][j] = t_new[b] (its runtime T(k'_t)),
//     flops / bytes / h_cand rows likewise (each array pair nullable together),
//     pulls[b][j][.] = 0, reward_sum[b][j][.] = 0   (an arm nobody has played),
//     labels[b][j] = labels[b][parent[b]], dist2[b][j] = dist2[b][parent[b]]
//         (Reading: until the next re-clustering the new kernel sits in the cluster of the kernel k_t it was
//          generated from -- Algorithm 1 re-partitions only every tau iterations, and a candidate outside
//          every cluster could never be drawn),
//     t_inc[b] = min(t_inc[b], t_new[b])   (the incumbent of Algorithm 1's return line, argmin T(k)),
//     n_active[b] += 1;   appended[b] = j.
// Nothing happens (appended[b] = -1) where verification failed, where nothing was drawn (parent[b] < 0), or
// where the frontier is full (n_active[b] == N_cap; full[b] = 1 reports it).  parent[b] >= n_active[b] is an error.
//
// kbo_recluster_due: Algorithm 1's test "t mod tau = 0 and |P| >= 2K" per search.
// ---------------------------------------------------------------------------
int kbo_append_candidate(int B, int N_cap, int D, int S, int R, const int32_t* verified, const int32_t* parent,
                         const float* x_new, const float* t_new, const float* flops_new, const float* bytes_new,
                         const float* h_new, int32_t* n_active, float* x, float* t_cur, float* flops, float* bytes,
                         float* h_cand, int32_t* labels, float* dist2, int32_t* pulls, float* reward_sum, float* t_inc,
                         int32_t* appended, int32_t* full) {
    for (int b = 0; b < B; ++b) {
        if (appended) appended[b] = -1;
        if (full) full[b] = 0;
        const int p = parent[b];
        if (p < 0) continue;
        const int n = n_active[b];
        if (n < 0 || n > N_cap || p >= n) return 2;
        if (verified && verified[b] == 0) continue;
        if (n == N_cap) { if (full) full[b] = 1; continue; }
        for (int d = 0; d < D; ++d) x[ix3(b, n, d, N_cap, D)] = x_new[ix2(b, d, D)];
        t_cur[ix2(b, n, N_cap)] = t_new[b];
        if (flops && flops_new) flops[ix2(b, n, N_cap)] = flops_new[b];
        if (bytes && bytes_new) bytes[ix2(b, n, N_cap)] = bytes_new[b];
        if (h_cand && h_new)
            for (int r = 0; r < R; ++r) h_cand[ix3(b, n, r, N_cap, R)] = h_new[ix2(b, r, R)];
        for (int s = 0; s < S; ++s) { pulls[ix3(b, n, s, N_cap, S)] = 0; reward_sum[ix3(b, n, s, N_cap, S)] = 0.0f; }
        labels[ix2(b, n, N_cap)] = labels[ix2(b, p, N_cap)];
        if (dist2) dist2[ix2(b, n, N_cap)] = dist2[ix2(b, p, N_cap)];
        if (t_inc && t_new[b] < t_inc[b]) t_inc[b] = t_new[b];
        n_active[b] = n + 1;
        if (appended) appended[b] = n;
    }
    return 0;
}

int kbo_recluster_due(int B, int tau, int K, const int32_t* t, const int32_t* n_active, int32_t* due) {
    if (tau < 1) return 1;
    for (int b = 0; b < B; ++b) due[b] = (t[b] % tau == 0 && n_active[b] >= 2 * K) ? 1 : 0;
    return 0;
}

// The profile of every cluster's representative (Algorithm 1: "profile h_c^(i) <- NCU(k_c^(i))", with the
// per-candidate signatures standing in for the profiler): hsig[b][i][:] = h_cand[b][rep[b][i]][:], and +inf for an
// empty cluster (rep = -1), whose mask entry M_{i,s} = [h < theta_sat] is then 0: an empty cluster is never
// selected.  run (nullable): instances with run[b] == 0 are left as they are.
int kbo_signatures_from_reps(int B, int N, int K, int R, const int32_t* rep, const float* h_cand, const int32_t* run,
                             float* hsig) {
    for (int b = 0; b < B; ++b) {
        if (run && run[b] == 0) continue;
        for (int i = 0; i < K; ++i) {
            const int k = rep[ix2(b, i, K)];
            if (k >= N) return 2;
            for (int r = 0; r < R; ++r)
                hsig[ix3(b, i, r, K, R)] = k < 0 ? std::numeric_limits<float>::infinity() : h_cand[ix3(b, k, r, N, R)];
        }
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Restarts (the n_init of the "scikit-learn's KMeans" of Sec. 3.5): a search instance is clustered n_init
// times from different seeds, as n_init consecutive instances of the batch; the run with the smallest
// inertia is kept.  best[g] = the index in [0, n_init) of the smallest inertia[g][.], lowest index on ties;
// NaN inertias are never chosen (-1 if all are NaN).
// ---------------------------------------------------------------------------
int kbo_best_restart(int G, int n_init, const float* inertia, int32_t* best) {
    for (int g = 0; g < G; ++g) {
        int arg = -1;
        double v = kInf;
        for (int r = 0; r < n_init; ++r) {
            const double x = (double)inertia[(size_t)g * n_init + r];
            if (std::isnan(x)) continue;
            if (arg < 0 || x < v) { v = x; arg = r; }
        }
        best[g] = arg;
    }
    return 0;
}

}  // extern "C"
