// EcoSpa CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-pass fp64 statement of what the coupled-sparsity hot
// path computes, written from the paper's definitions.  It shares no code with
// the CUDA library and is only ever called from the tests, the smoke check and
// the benchmark's CPU-baseline leg.
//
// What each function follows:
//   eco_sumsq_shared / _hadamard : squared column / row l2 norms of Eq. "l2norm"
//                                  (numerator), SwiGLU W_1 = W_gate (.) W_up
//                                  from the footnote to Eq. "importance".
//   eco_upsilon                  : Eq. "l2norm" (per coupled pair = per segment).
//   eco_upsilon_rope / eco_select_rotation_pairs_f32 : the same score and removal with rotary position
//                                  embedding (Eq. "self-attention-rope", footnote to Eq. "l2norm"): rotation
//                                  pairs of shared indices as the unit.
//   eco_fisher_pair              : Eq. "importance".
//   eco_select_topk_*            : Definition 1 (aligned removal) applied to
//                                  the (seg_len - k) lowest-scored indices.
//   eco_threshold_counts_f32     : Algorithm 1, the "while sum of scores > theta: remove smallest" loop
//                                  (how many aligned indices of each pair stay).
//   eco_choose_pairs_f32         : Algorithm 1, the top-K pairs with the smallest importance.
//   eco_compact_bytes            : Definition 1, the physical removal.
//   eco_coupled_single / eco_individual_single / eco_frob_removed :
//                                  Definitions 1 and 2, Propositions 1 and 2.
//   eco_proj_* / eco_ffn_*       : Eq. 2, 3 and 5 on the compacted matrices and
//                                  their textbook reverse-mode derivatives.
//   eco_attn_fwd / eco_attn_bwd  : the head of Eq. 2, phi(Q_i K_i^T / sqrt(d_h)) V_i, on compacted heads whose
//                                  Q/K width and V width differ from head to head (the "Coupled Weight Matrix in
//                                  MHA" reformulation with W_i^QK, W_i^VO restricted to the kept indices), and its
//                                  textbook reverse mode.
//
// Parity unpinned (conventions the paper does not fix):
//   - the SwiGLU slot of eco_fisher_pair (W_1 = gate (.) up is not a parameter),
//   - the choice between the erf and tanh GELU forms,
//   - in eco_threshold_counts_f32, whether theta is a share of the score mass (l1 = 1) or is compared with the
//     l2-normalised scores as stored (l1 = 0): the paper prints the l2 normaliser and thresholds of 85-95 %;
//   - the causal flag of eco_attn_*: Eq. 2 prints no mask (causal = 0 is the equation as printed); the decoder
//     models of the experiments mask keys after the query, which causal = 1 restates.
//
// Layout vocabulary: a matrix that owns a shared dimension D and another
// dimension `other` is stored row-major either as  other x D  ("shared cols",
// layout 0; W_1-like: column j belongs to shared index j) or as  D x other
// ("shared rows", layout 1; W_2-like: row j belongs to shared index j).
// dtype 0 = IEEE fp32, 1 = bfloat16 (upper 16 bits of an fp32), 2 = fp64.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

namespace {

inline double load_elem(const void* p, int dtype, int64_t i) {
    if (dtype == 0) return static_cast<double>(static_cast<const float*>(p)[i]);
    if (dtype == 1) {
        uint32_t bits = static_cast<uint32_t>(static_cast<const uint16_t*>(p)[i]) << 16;
        float f;
        std::memcpy(&f, &bits, 4);
        return static_cast<double>(f);
    }
    return static_cast<const double*>(p)[i];
}

// View of a matrix with a shared axis.  at(i, j): i in [0, other), j in [0, D).
struct SharedMat {
    const void* p;
    int dtype, layout;
    int64_t other, D, ld;
    double at(int64_t i, int64_t j) const {
        return layout == 0 ? load_elem(p, dtype, i * ld + j) : load_elem(p, dtype, j * ld + i);
    }
};

// Plain row-major activation matrix T x n with leading dimension ld.
struct Act {
    const void* p;
    int dtype;
    int64_t rows, cols, ld;
    double at(int64_t r, int64_t c) const { return load_elem(p, dtype, r * ld + c); }
};

const double kInvSqrt2 = 0.70710678118654752440;
const double kInvSqrt2Pi = 0.39894228040143267794;
const double kSqrt2OverPi = 0.79788456080286535588;

// act: 1 = GELU (erf form), 2 = GELU (tanh form)
double gelu(double x, int act) {
    if (act == 1) return 0.5 * x * (1.0 + std::erf(x * kInvSqrt2));
    double u = kSqrt2OverPi * (x + 0.044715 * x * x * x);
    return 0.5 * x * (1.0 + std::tanh(u));
}
double gelu_grad(double x, int act) {
    if (act == 1) return 0.5 * (1.0 + std::erf(x * kInvSqrt2)) + x * kInvSqrt2Pi * std::exp(-0.5 * x * x);
    double u = kSqrt2OverPi * (x + 0.044715 * x * x * x);
    double t = std::tanh(u);
    double du = kSqrt2OverPi * (1.0 + 3.0 * 0.044715 * x * x);
    return 0.5 * (1.0 + t) + 0.5 * x * (1.0 - t * t) * du;
}
double sigmoid(double x) { return 1.0 / (1.0 + std::exp(-x)); }
double silu(double x) { return x * sigmoid(x); }
double silu_grad(double x) {
    double s = sigmoid(x);
    return s * (1.0 + x * (1.0 - s));
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// Scores
// ---------------------------------------------------------------------------

// out[j] = sum over the other axis of W[., j]^2        (j = shared index)
void eco_sumsq_shared(const void* w, int dtype, int layout, int64_t other, int64_t D, int64_t ld, double* out) {
    SharedMat m{w, dtype, layout, other, D, ld};
    for (int64_t j = 0; j < D; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < other; ++i) {
            double v = m.at(i, j);
            s += v * v;
        }
        out[j] = s;
    }
}

// out[j] = sum_i (gate[i, j] * up[i, j])^2 : squared column norms of W_gate (.) W_up
void eco_sumsq_shared_hadamard(const void* gate, const void* up, int dtype, int layout, int64_t other, int64_t D,
                               int64_t ld_gate, int64_t ld_up, double* out) {
    SharedMat g{gate, dtype, layout, other, D, ld_gate};
    SharedMat u{up, dtype, layout, other, D, ld_up};
    for (int64_t j = 0; j < D; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < other; ++i) {
            double v = g.at(i, j) * u.at(i, j);
            s += v * v;
        }
        out[j] = s;
    }
}

// raw[j] = ||w1_j||_2 * ||w2_j||_2 ;  upsilon = raw / ||raw||_2 taken per segment (one
// segment = one coupled pair).  A segment whose raw vector is all zero gets upsilon = 0.
void eco_upsilon(const double* c1, const double* c2, int n_seg, int seg_len, double* raw, double* upsilon) {
    for (int s = 0; s < n_seg; ++s) {
        const int64_t o = static_cast<int64_t>(s) * seg_len;
        double nrm2 = 0.0;
        for (int j = 0; j < seg_len; ++j) {
            raw[o + j] = std::sqrt(c1[o + j]) * std::sqrt(c2[o + j]);
            nrm2 += raw[o + j] * raw[o + j];
        }
        const double nrm = std::sqrt(nrm2);
        for (int j = 0; j < seg_len; ++j) upsilon[o + j] = nrm > 0.0 ? raw[o + j] / nrm : 0.0;
    }
}

// With rotary position embedding (Eq. "self-attention-rope") W_Q P_t and W_K P_s rotate the shared index in
// 2 x 2 blocks, and the footnote to Eq. "l2norm" removes on W_Q / W_K and shrinks the position matrices with them:
// the removable unit is a rotation pair {a, b} of shared indices.  Its score is the Eq. "l2norm" score of the pair
// taken as one unit: raw = ||W_1[:, {a,b}]||_F * ||W_2[{a,b}, :]||_F = sqrt(c1[a] + c1[b]) * sqrt(c2[a] + c2[b])
// (a rotation of the two columns does not change it), normalised over the segment's seg_len/2 units.  Both
// members of a pair carry the pair's value.  mode 1: pairs (2u, 2u+1); mode 2: pairs (u, u + seg_len/2).
void eco_upsilon_rope(const double* c1, const double* c2, int n_seg, int seg_len, int mode, double* raw, double* upsilon) {
    const int half = seg_len / 2;
    for (int s = 0; s < n_seg; ++s) {
        const int64_t o = static_cast<int64_t>(s) * seg_len;
        double nrm2 = 0.0;
        for (int u = 0; u < half; ++u) {
            const int a = mode == 1 ? 2 * u : u, b = mode == 1 ? 2 * u + 1 : u + half;
            const double r = std::sqrt(c1[o + a] + c1[o + b]) * std::sqrt(c2[o + a] + c2[o + b]);
            raw[o + a] = raw[o + b] = r;
            nrm2 += r * r;
        }
        const double nrm = std::sqrt(nrm2);
        for (int j = 0; j < seg_len; ++j) upsilon[o + j] = nrm > 0.0 ? raw[o + j] / nrm : 0.0;
    }
}

// Aligned removal of whole rotation pairs: per segment the k/2 units with the largest score stay (equal scores:
// lower unit first; a unit's score is read at its first member); kept indices ascending.
void eco_select_rotation_pairs_f32(const float* upsilon, int n_seg, int seg_len, const int32_t* k, int mode, int32_t* kept) {
    const int half = seg_len / 2;
    int64_t w = 0;
    for (int s = 0; s < n_seg; ++s) {
        const int64_t o = static_cast<int64_t>(s) * seg_len;
        std::vector<int32_t> order(half);
        std::iota(order.begin(), order.end(), 0);
        auto unit_score = [&](int32_t u) { return upsilon[o + (mode == 1 ? 2 * u : u)]; };
        std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return unit_score(a) > unit_score(b); });
        std::vector<int32_t> idx;
        for (int i = 0; i < k[s] / 2; ++i) {
            const int32_t u = order[i];
            idx.push_back(mode == 1 ? 2 * u : u);
            idx.push_back(mode == 1 ? 2 * u + 1 : u + half);
        }
        std::sort(idx.begin(), idx.end());
        for (int32_t c : idx) kept[w++] = static_cast<int32_t>(o) + c;
    }
}

// I_hat[seg] = 1/2 * sum_{k=1,2} (1/|W_k|) (1/|D|) sum_{ij} G_k[i,j]^2 over the segment's block.
// For a SwiGLU pair (g1b != NULL) the W_1 slot is the mean of the gate and up terms.
void eco_fisher_pair(const void* g1, const void* g1b, const void* g2, int dtype, int layout1, int layout2,
                     int64_t other1, int64_t other2, int64_t ld1, int64_t ld1b, int64_t ld2, int n_seg, int seg_len,
                     double n_samples, double* fisher) {
    const int64_t D = static_cast<int64_t>(n_seg) * seg_len;
    SharedMat a{g1, dtype, layout1, other1, D, ld1};
    SharedMat ab{g1b, dtype, layout1, other1, D, ld1b};
    SharedMat b{g2, dtype, layout2, other2, D, ld2};
    for (int s = 0; s < n_seg; ++s) {
        double ss1 = 0.0, ss1b = 0.0, ss2 = 0.0;
        for (int64_t j = static_cast<int64_t>(s) * seg_len; j < static_cast<int64_t>(s + 1) * seg_len; ++j) {
            for (int64_t i = 0; i < other1; ++i) {
                double v = a.at(i, j);
                ss1 += v * v;
                if (g1b) {
                    double vb = ab.at(i, j);
                    ss1b += vb * vb;
                }
            }
            for (int64_t i = 0; i < other2; ++i) {
                double v = b.at(i, j);
                ss2 += v * v;
            }
        }
        const double numel1 = static_cast<double>(other1) * seg_len;
        const double numel2 = static_cast<double>(other2) * seg_len;
        double term1 = ss1 / numel1;
        if (g1b) term1 = 0.5 * (ss1 / numel1 + ss1b / numel1);
        const double term2 = ss2 / numel2;
        fisher[s] = 0.5 * (term1 + term2) / n_samples;
    }
}

// ---------------------------------------------------------------------------
// Aligned selection
// ---------------------------------------------------------------------------

// Keep the k[s] highest-scored indices of every segment (i.e. remove the lowest-scored
// seg_len - k[s], aligned in both matrices); equal scores: the lower index is kept.
// kept receives global shared indices, ascending, segment after segment.
static void select_impl(const double* score, int n_seg, int seg_len, const int32_t* k, int32_t* kept) {
    int64_t w = 0;
    for (int s = 0; s < n_seg; ++s) {
        const int64_t o = static_cast<int64_t>(s) * seg_len;
        std::vector<int32_t> order(seg_len);
        std::iota(order.begin(), order.end(), 0);
        std::stable_sort(order.begin(), order.end(),
                         [&](int32_t a, int32_t b) { return score[o + a] > score[o + b]; });
        std::vector<int32_t> chosen(order.begin(), order.begin() + k[s]);
        std::sort(chosen.begin(), chosen.end());
        for (int32_t c : chosen) kept[w++] = static_cast<int32_t>(o) + c;
    }
}

void eco_select_topk_f64(const double* upsilon, int n_seg, int seg_len, const int32_t* k, int32_t* kept) {
    select_impl(upsilon, n_seg, seg_len, k, kept);
}

// Same decision taken on fp32 score values exactly as stored (fp32 -> fp64 is exact and
// order preserving, so ties are exactly the fp32 ties).
void eco_select_topk_f32(const float* upsilon, int n_seg, int seg_len, const int32_t* k, int32_t* kept) {
    std::vector<double> tmp(static_cast<size_t>(n_seg) * seg_len);
    for (size_t i = 0; i < tmp.size(); ++i) tmp[i] = static_cast<double>(upsilon[i]);
    select_impl(tmp.data(), n_seg, seg_len, k, kept);
}

// ---------------------------------------------------------------------------
// Algorithm 1, inner loop: "while the sum of the scores exceeds theta, remove the smallest score".
// ---------------------------------------------------------------------------
// Per segment (= per coupled pair): the scores that are still there are summed in fp64, largest first
// (equal scores: lower index first); while that sum exceeds theta * total and more than k_min indices are
// left, the smallest remaining score goes (among equal scores the higher index goes first, the same rule as
// the top-k tie-break).  total = the sum of all scores of the segment when `l1` is set (theta is then the
// fraction of the score mass that stays), 1 otherwise (the scores are compared with theta as stored).
// chosen == nullptr: every segment is processed; otherwise segments with chosen[s] == 0 keep everything.
// Output: how many indices stay per segment.  Scores are taken as stored fp32 values (exactly widened).
// rope != 0 (rotation pairs, see eco_upsilon_rope): the units are the seg_len/2 pairs, each with the score stored at
// its first member and counted once; whole pairs leave; the result counts indices (even) and does not go below
// k_min rounded up to whole pairs.
void eco_threshold_counts_f32(const float* upsilon, int n_seg, int seg_len_idx, int rope, double theta, int l1, int k_min_idx,
                              const int32_t* chosen, int32_t* k_out) {
    const int unit = rope ? 2 : 1;
    const int seg_len = seg_len_idx / unit;
    const int k_min = std::min((k_min_idx + unit - 1) / unit, seg_len);
    std::vector<float> units(seg_len);
    for (int s = 0; s < n_seg; ++s) {
        if (chosen && !chosen[s]) {
            k_out[s] = seg_len_idx;
            continue;
        }
        for (int j = 0; j < seg_len; ++j) units[j] = upsilon[static_cast<int64_t>(s) * seg_len_idx + (rope == 1 ? 2 * j : j)];
        const float* u = units.data();
        std::vector<int32_t> order(seg_len);
        std::iota(order.begin(), order.end(), 0);
        std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return u[a] > u[b]; });
        double total = 1.0;
        if (l1) {
            total = 0.0;
            for (int i = 0; i < seg_len; ++i) total += static_cast<double>(u[order[i]]);
        }
        const double budget = theta * total;
        int left = seg_len;
        while (left > k_min) {
            double sum = 0.0;                       // sum of what is left, largest first
            for (int i = 0; i < left; ++i) sum += static_cast<double>(u[order[i]]);
            if (!(sum > budget)) break;
            --left;                                 // order[left] was the smallest one left
        }
        k_out[s] = left * unit;
    }
}

// Algorithm 1, "select the top-K coupled matrices with the smallest importance": the m smallest values of
// `fisher` are marked (equal values: lower index first).
void eco_choose_pairs_f32(const float* fisher, int n, int m, int32_t* chosen) {
    std::vector<int32_t> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return fisher[a] < fisher[b]; });
    for (int i = 0; i < n; ++i) chosen[i] = 0;
    for (int i = 0; i < m && i < n; ++i) chosen[order[i]] = 1;
}

// ---------------------------------------------------------------------------
// Physical removal (gather of what is kept); byte exact, pad columns zeroed.
// ---------------------------------------------------------------------------
// layout 0 (other x D): out is other x n_kept with leading dimension ld_out >= n_kept,
//                       columns [n_kept, ld_out) are written as zero bytes.
// layout 1 (D x other): out is n_kept x other with leading dimension ld_out >= other,
//                       columns [other, ld_out) are written as zero bytes.
// A kept entry of -1 stands for "no index": the output gets a zero column (row) there.  It lets a caller give
// every head's block of a compacted tensor a padded width; zero columns add nothing to any product they enter.
void eco_compact_bytes(const uint8_t* in, int elem_bytes, int layout, int64_t other, int64_t ld_in,
                       const int32_t* kept, int64_t n_kept, uint8_t* out, int64_t ld_out) {
    if (layout == 0) {
        for (int64_t i = 0; i < other; ++i) {
            for (int64_t c = 0; c < n_kept; ++c) {
                if (kept[c] < 0) std::memset(out + (i * ld_out + c) * elem_bytes, 0, elem_bytes);
                else std::memcpy(out + (i * ld_out + c) * elem_bytes, in + (i * ld_in + kept[c]) * elem_bytes, elem_bytes);
            }
            std::memset(out + (i * ld_out + n_kept) * elem_bytes, 0, (ld_out - n_kept) * elem_bytes);
        }
    } else {
        for (int64_t r = 0; r < n_kept; ++r) {
            if (kept[r] < 0) std::memset(out + r * ld_out * elem_bytes, 0, other * elem_bytes);
            else std::memcpy(out + r * ld_out * elem_bytes, in + static_cast<int64_t>(kept[r]) * ld_in * elem_bytes,
                             other * elem_bytes);
            std::memset(out + (r * ld_out + other) * elem_bytes, 0, (ld_out - other) * elem_bytes);
        }
    }
}

// ---------------------------------------------------------------------------
// Appendix A: single removal, coupled vs individual.  A is m x n (row-major,
// columns a_j), B is n x p (row-major, rows b_j^T).
// ---------------------------------------------------------------------------

// j* = argmin_j ||a_j|| ||b_j||   (first minimum)
int32_t eco_coupled_single(const double* A, const double* B, int64_t m, int64_t n, int64_t p) {
    int32_t best = 0;
    double bestv = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        double sa = 0.0, sb = 0.0;
        for (int64_t i = 0; i < m; ++i) sa += A[i * n + j] * A[i * n + j];
        for (int64_t c = 0; c < p; ++c) sb += B[j * p + c] * B[j * p + c];
        double v = std::sqrt(sa) * std::sqrt(sb);
        if (j == 0 || v < bestv) {
            bestv = v;
            best = static_cast<int32_t>(j);
        }
    }
    return best;
}

// k* = argmin_k ||a_k||, l* = argmin_l ||b_l||   (first minima)
void eco_individual_single(const double* A, const double* B, int64_t m, int64_t n, int64_t p, int32_t* kstar,
                           int32_t* lstar) {
    double bestA = 0.0, bestB = 0.0;
    *kstar = 0;
    *lstar = 0;
    for (int64_t j = 0; j < n; ++j) {
        double sa = 0.0, sb = 0.0;
        for (int64_t i = 0; i < m; ++i) sa += A[i * n + j] * A[i * n + j];
        for (int64_t c = 0; c < p; ++c) sb += B[j * p + c] * B[j * p + c];
        if (j == 0 || sa < bestA) {
            bestA = sa;
            *kstar = static_cast<int32_t>(j);
        }
        if (j == 0 || sb < bestB) {
            bestB = sb;
            *lstar = static_cast<int32_t>(j);
        }
    }
}

// || A B - A[:, keptA] B[keptB, :] ||_F with the kept columns/rows re-paired in order
// (p-th kept column of A with p-th kept row of B), as in Definitions 1 and 2.
double eco_frob_removed(const double* A, const double* B, int64_t m, int64_t n, int64_t p, const int32_t* keptA,
                        const int32_t* keptB, int64_t n_kept) {
    double acc = 0.0;
    for (int64_t i = 0; i < m; ++i) {
        for (int64_t c = 0; c < p; ++c) {
            double full = 0.0, part = 0.0;
            for (int64_t j = 0; j < n; ++j) full += A[i * n + j] * B[j * p + c];
            for (int64_t q = 0; q < n_kept; ++q) part += A[i * n + keptA[q]] * B[static_cast<int64_t>(keptB[q]) * p + c];
            acc += (full - part) * (full - part);
        }
    }
    return std::sqrt(acc);
}

// ---------------------------------------------------------------------------
// Layer math on compacted pairs (fp64 throughout; outputs dense row-major).
// Weight operands are SharedMat views: element (i, j) = (model-dim index, shared index).
// Weight gradients are returned in "math orientation": other x D row-major (dW[i*D + j]).
// ---------------------------------------------------------------------------

// Y[t, j] = sum_i X[t, i] W[i, j] + b[j]         (Q^c, K^c, V^c projections; W^c is d_m x n)
void eco_proj_fwd(const void* X, int xdtype, int64_t T, int64_t d_m, int64_t ldx, const void* W, int wdtype,
                  int wlayout, int64_t n, int64_t ldw, const void* bias, double* Y) {
    Act x{X, xdtype, T, d_m, ldx};
    SharedMat w{W, wdtype, wlayout, d_m, n, ldw};
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < n; ++j) {
            double s = bias ? load_elem(bias, wdtype, j) : 0.0;
            for (int64_t i = 0; i < d_m; ++i) s += x.at(t, i) * w.at(i, j);
            Y[t * n + j] = s;
        }
}

// Reverse of eco_proj_fwd:  dX[t,i] = sum_j dY[t,j] W[i,j];  dW[i,j] = sum_t X[t,i] dY[t,j];  db[j] = sum_t dY[t,j]
// dX is accumulated into (caller zeroes it), so that Q and K (or several projections) can share it.
void eco_proj_bwd(const void* X, int xdtype, int64_t T, int64_t d_m, int64_t ldx, const void* W, int wdtype,
                  int wlayout, int64_t n, int64_t ldw, const void* dY, int64_t lddy, double* dX, double* dW,
                  double* db) {
    Act x{X, xdtype, T, d_m, ldx};
    Act dy{dY, xdtype, T, n, lddy};
    SharedMat w{W, wdtype, wlayout, d_m, n, ldw};
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < d_m; ++i) {
            double s = 0.0;
            for (int64_t j = 0; j < n; ++j) s += dy.at(t, j) * w.at(i, j);
            dX[t * d_m + i] += s;
        }
    for (int64_t i = 0; i < d_m; ++i)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += x.at(t, i) * dy.at(t, j);
            dW[i * n + j] = s;
        }
    if (db)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += dy.at(t, j);
            db[j] = s;
        }
}

// Out[t, c] = sum_j Ctx[t, j] W_O[j, c] + b[c]     (W_O^c is n x d_m: shared index j, model index c)
void eco_outproj_fwd(const void* Ctx, int xdtype, int64_t T, int64_t n, int64_t ldc, const void* W, int wdtype,
                     int wlayout, int64_t d_m, int64_t ldw, const void* bias, double* Out) {
    Act ctx{Ctx, xdtype, T, n, ldc};
    SharedMat w{W, wdtype, wlayout, d_m, n, ldw};
    for (int64_t t = 0; t < T; ++t)
        for (int64_t c = 0; c < d_m; ++c) {
            double s = bias ? load_elem(bias, wdtype, c) : 0.0;
            for (int64_t j = 0; j < n; ++j) s += ctx.at(t, j) * w.at(c, j);
            Out[t * d_m + c] = s;
        }
}

// Reverse: dCtx[t,j] = sum_c dOut[t,c] W_O[j,c];  dW_O[c,j] (math orientation: other=c, shared=j) = sum_t Ctx[t,j] dOut[t,c]
void eco_outproj_bwd(const void* Ctx, int xdtype, int64_t T, int64_t n, int64_t ldc, const void* W, int wdtype,
                     int wlayout, int64_t d_m, int64_t ldw, const void* dOut, int64_t lddo, double* dCtx,
                     double* dW, double* db) {
    Act ctx{Ctx, xdtype, T, n, ldc};
    Act dout{dOut, xdtype, T, d_m, lddo};
    SharedMat w{W, wdtype, wlayout, d_m, n, ldw};
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t c = 0; c < d_m; ++c) s += dout.at(t, c) * w.at(c, j);
            dCtx[t * n + j] = s;
        }
    for (int64_t c = 0; c < d_m; ++c)
        for (int64_t j = 0; j < n; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += ctx.at(t, j) * dout.at(t, c);
            dW[c * n + j] = s;
        }
    if (db)
        for (int64_t c = 0; c < d_m; ++c) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += dout.at(t, c);
            db[c] = s;
        }
}

// FFN forward on a compacted pair with k hidden units.
//   act 1/2 (GELU erf/tanh): H = X W_1 + b_1, A = GELU(H), Y = A W_2 + b_2
//   act 3 (SwiGLU):          H = X W_gate, Hb = X W_up, A = silu(H) (.) Hb, Y = A W_2
// W_1 (and W_1b) are views with other = d_m; W_2 is a view with other = d_m too
// (element (c, j) = W_2[j, c] in the paper's k x d_m orientation).
void eco_ffn_fwd(const void* X, int xdtype, int64_t T, int64_t d_m, int64_t ldx, int act, const void* W1,
                 const void* W1b, const void* W2, int wdtype, int layout1, int layout2, int64_t k, int64_t ld1,
                 int64_t ld1b, int64_t ld2, const void* b1, const void* b2, double* Y, double* H, double* Hb,
                 double* A) {
    Act x{X, xdtype, T, d_m, ldx};
    SharedMat w1{W1, wdtype, layout1, d_m, k, ld1};
    SharedMat w1b{W1b, wdtype, layout1, d_m, k, ld1b};
    SharedMat w2{W2, wdtype, layout2, d_m, k, ld2};
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < k; ++j) {
            double h = b1 ? load_elem(b1, wdtype, j) : 0.0;
            for (int64_t i = 0; i < d_m; ++i) h += x.at(t, i) * w1.at(i, j);
            H[t * k + j] = h;
            if (act == 3) {
                double hb = 0.0;
                for (int64_t i = 0; i < d_m; ++i) hb += x.at(t, i) * w1b.at(i, j);
                Hb[t * k + j] = hb;
                A[t * k + j] = silu(h) * hb;
            } else {
                A[t * k + j] = gelu(h, act);
            }
        }
    for (int64_t t = 0; t < T; ++t)
        for (int64_t c = 0; c < d_m; ++c) {
            double y = b2 ? load_elem(b2, wdtype, c) : 0.0;
            for (int64_t j = 0; j < k; ++j) y += A[t * k + j] * w2.at(c, j);
            Y[t * d_m + c] = y;
        }
}

// FFN backward.  Recomputes H, Hb, A in fp64 from X (the oracle keeps nothing rounded).
// Outputs: dX (T x d_m), dW1, dW1b, dW2 in math orientation (d_m x k each; dW2[c*k + j] = dL/dW_2[j, c]),
// db1 (k), db2 (d_m).  Any of db1/db2/dW1b may be NULL.
void eco_ffn_bwd(const void* X, int xdtype, int64_t T, int64_t d_m, int64_t ldx, int act, const void* W1,
                 const void* W1b, const void* W2, int wdtype, int layout1, int layout2, int64_t k, int64_t ld1,
                 int64_t ld1b, int64_t ld2, const void* b1, const void* dY, int64_t lddy, double* dX, double* dW1,
                 double* dW1b, double* dW2, double* db1, double* db2) {
    Act x{X, xdtype, T, d_m, ldx};
    Act dy{dY, xdtype, T, d_m, lddy};
    SharedMat w1{W1, wdtype, layout1, d_m, k, ld1};
    SharedMat w1b{W1b, wdtype, layout1, d_m, k, ld1b};
    SharedMat w2{W2, wdtype, layout2, d_m, k, ld2};
    std::vector<double> H(T * k), Hb(act == 3 ? T * k : 0), A(T * k), dH(T * k), dHb(act == 3 ? T * k : 0);
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < k; ++j) {
            double h = b1 ? load_elem(b1, wdtype, j) : 0.0;
            for (int64_t i = 0; i < d_m; ++i) h += x.at(t, i) * w1.at(i, j);
            H[t * k + j] = h;
            if (act == 3) {
                double hb = 0.0;
                for (int64_t i = 0; i < d_m; ++i) hb += x.at(t, i) * w1b.at(i, j);
                Hb[t * k + j] = hb;
                A[t * k + j] = silu(h) * hb;
            } else {
                A[t * k + j] = gelu(h, act);
            }
        }
    // dA = dY W_2^T, then through the activation
    for (int64_t t = 0; t < T; ++t)
        for (int64_t j = 0; j < k; ++j) {
            double da = 0.0;
            for (int64_t c = 0; c < d_m; ++c) da += dy.at(t, c) * w2.at(c, j);
            if (act == 3) {
                dH[t * k + j] = da * Hb[t * k + j] * silu_grad(H[t * k + j]);
                dHb[t * k + j] = da * silu(H[t * k + j]);
            } else {
                dH[t * k + j] = da * gelu_grad(H[t * k + j], act);
            }
        }
    // dW_2[j, c] = sum_t A[t, j] dY[t, c]
    for (int64_t c = 0; c < d_m; ++c)
        for (int64_t j = 0; j < k; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += A[t * k + j] * dy.at(t, c);
            dW2[c * k + j] = s;
        }
    if (db2)
        for (int64_t c = 0; c < d_m; ++c) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += dy.at(t, c);
            db2[c] = s;
        }
    // dW_1 = X^T dH (and dW_up = X^T dHb)
    for (int64_t i = 0; i < d_m; ++i)
        for (int64_t j = 0; j < k; ++j) {
            double s = 0.0, sb = 0.0;
            for (int64_t t = 0; t < T; ++t) {
                s += x.at(t, i) * dH[t * k + j];
                if (act == 3) sb += x.at(t, i) * dHb[t * k + j];
            }
            dW1[i * k + j] = s;
            if (act == 3 && dW1b) dW1b[i * k + j] = sb;
        }
    if (db1)
        for (int64_t j = 0; j < k; ++j) {
            double s = 0.0;
            for (int64_t t = 0; t < T; ++t) s += dH[t * k + j];
            db1[j] = s;
        }
    // dX = dH W_1^T (+ dHb W_up^T)
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < d_m; ++i) {
            double s = 0.0;
            for (int64_t j = 0; j < k; ++j) {
                s += dH[t * k + j] * w1.at(i, j);
                if (act == 3) s += dHb[t * k + j] * w1b.at(i, j);
            }
            dX[t * d_m + i] = s;
        }
}

// ---------------------------------------------------------------------------
// Attention on compacted heads.  Q, K (T x ..., pitch ldq / ldk) hold head h in columns [qk_off[h], qk_off[h] +
// qk_w[h]); V (pitch ldv) holds it in columns [vo_off[h], vo_off[h] + vo_w[h]).  T = batch * seq: sequence b is
// rows [b*seq, (b+1)*seq).  For every sequence and head, Eq. 2:
//     S = scale * Q_h K_h^T,   P = phi(S) (softmax over the keys of each query row),   Ctx_h = P V_h
// `scale` is the caller's 1/sqrt(d_h) with the architectural d_h of Eq. 2 (removal does not change it: the logits of
// the compacted head are the full head's logits restricted to the kept indices).  causal != 0: query i sees keys
// j <= i only.  Outputs in fp64: Ctx (T x ldc, head h in the V columns of head h), lse[h*T + t] = log sum_j exp(S_tj)
// (may be NULL), P (n_heads x batch x seq x seq, may be NULL: for the tests on small sizes).
// ---------------------------------------------------------------------------
void eco_attn_fwd(const void* Q, const void* K, const void* V, int dtype, int64_t batch, int64_t seq, int n_heads,
                  const int32_t* qk_off, const int32_t* qk_w, const int32_t* vo_off, const int32_t* vo_w, int64_t ldq,
                  int64_t ldk, int64_t ldv, double scale, int causal, double* Ctx, int64_t ldc, double* lse, double* P) {
    const int64_t T = batch * seq;
    std::vector<double> srow(seq);
    for (int h = 0; h < n_heads; ++h)
        for (int64_t b = 0; b < batch; ++b)
            for (int64_t i = 0; i < seq; ++i) {
                const int64_t ti = b * seq + i;
                const int64_t n_keys = causal ? i + 1 : seq;
                double mx = -INFINITY;
                for (int64_t j = 0; j < n_keys; ++j) {
                    const int64_t tj = b * seq + j;
                    double s = 0.0;
                    for (int c = 0; c < qk_w[h]; ++c)
                        s += load_elem(Q, dtype, ti * ldq + qk_off[h] + c) * load_elem(K, dtype, tj * ldk + qk_off[h] + c);
                    srow[j] = s * scale;
                    mx = std::max(mx, srow[j]);
                }
                double z = 0.0;
                for (int64_t j = 0; j < n_keys; ++j) z += std::exp(srow[j] - mx);
                if (lse) lse[static_cast<int64_t>(h) * T + ti] = mx + std::log(z);
                for (int64_t j = 0; j < seq; ++j) {
                    const double p = j < n_keys ? std::exp(srow[j] - mx) / z : 0.0;
                    srow[j] = p;
                    if (P) P[((static_cast<int64_t>(h) * batch + b) * seq + i) * seq + j] = p;
                }
                for (int c = 0; c < vo_w[h]; ++c) {
                    double o = 0.0;
                    for (int64_t j = 0; j < n_keys; ++j) o += srow[j] * load_elem(V, dtype, (b * seq + j) * ldv + vo_off[h] + c);
                    Ctx[ti * ldc + vo_off[h] + c] = o;
                }
            }
}

// Reverse mode of eco_attn_fwd for L = <Ctx, dCtx>.  With P recomputed as above, per sequence and head:
//     dV = P^T dCtx_h,   dP = dCtx_h V_h^T,   dS_ij = P_ij (dP_ij - sum_j' P_ij' dP_ij'),
//     dQ_h = scale * dS K_h,   dK_h = scale * dS^T Q_h.
// dCtx has the dtype and column layout of V (pitch lddc).  dQ, dK (T x ldq_out), dV (T x ldv_out) in fp64, same
// column layout as Q, K, V; only the heads' columns are written.
void eco_attn_bwd(const void* Q, const void* K, const void* V, const void* dCtx, int dtype, int64_t batch, int64_t seq,
                  int n_heads, const int32_t* qk_off, const int32_t* qk_w, const int32_t* vo_off, const int32_t* vo_w,
                  int64_t ldq, int64_t ldk, int64_t ldv, int64_t lddc, double scale, int causal, double* dQ, double* dK,
                  int64_t ldq_out, double* dV, int64_t ldv_out) {
    std::vector<double> p(seq), dp(seq);
    for (int h = 0; h < n_heads; ++h)
        for (int64_t b = 0; b < batch; ++b) {
            for (int64_t t = b * seq; t < (b + 1) * seq; ++t) {
                for (int c = 0; c < qk_w[h]; ++c) dQ[t * ldq_out + qk_off[h] + c] = dK[t * ldq_out + qk_off[h] + c] = 0.0;
                for (int c = 0; c < vo_w[h]; ++c) dV[t * ldv_out + vo_off[h] + c] = 0.0;
            }
            for (int64_t i = 0; i < seq; ++i) {
                const int64_t ti = b * seq + i;
                const int64_t n_keys = causal ? i + 1 : seq;
                double mx = -INFINITY;
                for (int64_t j = 0; j < n_keys; ++j) {
                    double s = 0.0;
                    for (int c = 0; c < qk_w[h]; ++c)
                        s += load_elem(Q, dtype, ti * ldq + qk_off[h] + c) * load_elem(K, dtype, (b * seq + j) * ldk + qk_off[h] + c);
                    p[j] = s * scale;
                    mx = std::max(mx, p[j]);
                }
                double z = 0.0;
                for (int64_t j = 0; j < n_keys; ++j) z += std::exp(p[j] - mx);
                double dot = 0.0;
                for (int64_t j = 0; j < n_keys; ++j) {
                    p[j] = std::exp(p[j] - mx) / z;
                    double d = 0.0;
                    for (int c = 0; c < vo_w[h]; ++c)
                        d += load_elem(dCtx, dtype, ti * lddc + vo_off[h] + c) * load_elem(V, dtype, (b * seq + j) * ldv + vo_off[h] + c);
                    dp[j] = d;
                    dot += p[j] * d;
                }
                for (int64_t j = 0; j < n_keys; ++j) {
                    const int64_t tj = b * seq + j;
                    for (int c = 0; c < vo_w[h]; ++c)
                        dV[tj * ldv_out + vo_off[h] + c] += p[j] * load_elem(dCtx, dtype, ti * lddc + vo_off[h] + c);
                    const double ds = p[j] * (dp[j] - dot) * scale;
                    for (int c = 0; c < qk_w[h]; ++c) {
                        dQ[ti * ldq_out + qk_off[h] + c] += ds * load_elem(K, dtype, tj * ldk + qk_off[h] + c);
                        dK[tj * ldq_out + qk_off[h] + c] += ds * load_elem(Q, dtype, ti * ldq + qk_off[h] + c);
                    }
                }
            }
        }
}

}  // extern "C"
