/*
 * SpecKV oracle -- TEST INFRASTRUCTURE ONLY (see speckv_oracle.h).
 *
 * Plain C++17, double precision, sequential loops over the vocabulary; std::thread
 * is used across batch rows only (rows are independent).  No blocking, fusion or
 * reordering beyond what each definition states:
 *
 *   signals      paper Sec. 4.2: H(q_i) = -sum_v q_i(v) log q_i(v), c_i = max_v q_i(v),
 *                Hbar, cbar = means over the gamma drafted positions, Hmax, cmin.
 *   controller   paper Sec. 4.3: context vector -> 16 hidden units -> one predicted
 *                acceptance rate per candidate gamma; Eq. 1: E = a_hat * gamma + 1;
 *                gamma* = argmax.
 *   verification paper Sec. 3.1 (greedy: accept while the target's top prediction equals
 *                the draft token; the target's prediction replaces the first mismatch; a
 *                bonus prediction follows a fully accepted draft; tokens per step = k + 1),
 *                and, for temperature > 0, the lossless speculative-sampling rule the
 *                paper cites (Sec. 1, 2.1): accept x_i while u_i < min(1, p(x_i)/q(x_i));
 *                the first rejected position is resampled from norm(max(0, p - q)); a
 *                fully accepted draft gets a bonus token from p.
 *
 * Readings fixed where the paper is silent (the same list is kept in the design notes):
 *   - entropy in nats by default, bits on request (the paper writes log2);
 *   - signals use the draft softmax at the row's temperature; greedy rows (T = 0) use T = 1;
 *   - accept test evaluated as ln u + ln q(x) < ln p(x); q(x) = 0 accepts iff p(x) > 0;
 *   - uniforms are indexed by position: u[b,i,0] accept test, u[b,n,1] resample / bonus;
 *   - inverse CDF in vocabulary order: smallest v with cumulative weight > u * total,
 *     falling back to the last v with positive weight;
 *   - argmax ties go to the lowest index (token id, and candidate gamma);
 *   - -inf logits are legal (probability 0); NaN, +inf or an all -inf row flag the row;
 *   - target rows behind the stop position are not part of the step: not read, not checked.
 */
#include "speckv_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double load_logit(const void* base, int32_t dtype, int64_t idx) {
    if (dtype == ORACLE_DT_F32) {
        return static_cast<double>(static_cast<const float*>(base)[idx]);
    }
    uint16_t h = static_cast<const uint16_t*>(base)[idx];
    uint32_t w = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &w, sizeof f);
    return static_cast<double>(f);
}

struct RowRef {
    const void* base;
    int32_t dtype;
    int64_t off;
    double at(int64_t v) const { return load_logit(base, dtype, off + v); }
};

/* max and log-sum-exp of x_v / T; returns false when the row is unusable */
bool lse_row(const RowRef& r, int32_t V, double T, double* m_out, double* lnZ_out) {
    double m = -std::numeric_limits<double>::infinity();
    for (int32_t v = 0; v < V; ++v) {
        double x = r.at(v);
        if (std::isnan(x) || x == std::numeric_limits<double>::infinity()) return false;
        x /= T;
        if (x > m) m = x;
    }
    if (!(m > -std::numeric_limits<double>::infinity())) return false;
    double Z = 0.0;
    for (int32_t v = 0; v < V; ++v) Z += std::exp(r.at(v) / T - m);
    *m_out = m;
    *lnZ_out = std::log(Z);
    return true;
}

bool softmax_row(const RowRef& r, int32_t V, double T, double* prob) {
    double m = -std::numeric_limits<double>::infinity();
    for (int32_t v = 0; v < V; ++v) {
        double x = r.at(v);
        if (std::isnan(x) || x == std::numeric_limits<double>::infinity()) return false;
        x /= T;
        if (x > m) m = x;
    }
    if (!(m > -std::numeric_limits<double>::infinity())) return false;
    double Z = 0.0;
    for (int32_t v = 0; v < V; ++v) {
        prob[v] = std::exp(r.at(v) / T - m);
        Z += prob[v];
    }
    for (int32_t v = 0; v < V; ++v) prob[v] /= Z;
    return true;
}

double entropy_nats(const double* q, int32_t V) {
    double H = 0.0;
    for (int32_t v = 0; v < V; ++v)
        if (q[v] > 0.0) H -= q[v] * std::log(q[v]);
    return H;
}

/* lowest index of the maximum; -1 when the row holds NaN / +inf or only -inf */
int32_t argmax_row(const RowRef& r, int32_t V) {
    double best = -std::numeric_limits<double>::infinity();
    int32_t arg = -1;
    for (int32_t v = 0; v < V; ++v) {
        double x = r.at(v);
        if (std::isnan(x) || x == std::numeric_limits<double>::infinity()) return -1;
        if (x > best) {
            best = x;
            arg = v;
        }
    }
    return arg;
}

int32_t inverse_cdf(const double* w, int32_t V, double u, int32_t* near_boundary) {
    double W = 0.0;
    for (int32_t v = 0; v < V; ++v) W += w[v];
    if (near_boundary) *near_boundary = 0;
    if (!(W > 0.0)) return -1;
    const double tau = u * W;
    double cum = 0.0, lower = 0.0;
    int32_t chosen = -1, last_pos = -1;
    for (int32_t v = 0; v < V; ++v) {
        if (w[v] > 0.0) last_pos = v;
        double next = cum + w[v];
        if (next > tau) {
            chosen = v;
            lower = cum;
            cum = next;
            break;
        }
        cum = next;
    }
    if (chosen < 0) {
        chosen = last_pos;
        if (near_boundary) *near_boundary = 1;
        return chosen;
    }
    if (near_boundary) {
        /* upper boundary of the chosen token, and its lower boundary (= upper boundary of
         * the previous token with positive weight); the lower one only matters if a token
         * with positive weight precedes the chosen one.
         * bit 0: a boundary within 1e-6 of the threshold on the normalised CDF (1e-6 * W);
         * bit 1: within 1e-6 in the units of the weights themselves.  For weights that are probabilities
         * (W = 1) the two coincide; for a residual max(0, p - q) of small mass W the second is the wider
         * one: p and q are each known to about 1e-7 when the sums behind them are accumulated in fp32,
         * so their difference is known to about 1e-7 however small W is. */
        const double d_hi = std::fabs(cum - tau);
        const double d_lo = (lower > 0.0) ? std::fabs(tau - lower) : 1e300;
        const double d = std::min(d_hi, d_lo);
        *near_boundary = (d < 1e-6 * W ? 1 : 0) | (d < 1e-6 ? 2 : 0);
    }
    return chosen;
}

struct RowParams {
    int32_t gamma;
    double T;      /* temperature as given (0 => greedy) */
    int32_t status;
};

RowParams row_params(const oracle_batch* bt, int32_t b) {
    RowParams rp;
    rp.status = ORACLE_ROW_OK;
    rp.gamma = bt->gamma ? bt->gamma[b] : bt->gamma_max;
    float tf = bt->temperature ? bt->temperature[b] : bt->temperature_scalar;
    rp.T = static_cast<double>(tf);
    if (rp.gamma < 1 || rp.gamma > bt->gamma_max) rp.status |= ORACLE_ROW_BAD_GAMMA;
    if (!(rp.T >= 0.0) || std::isinf(rp.T)) rp.status |= ORACLE_ROW_BAD_TEMPERATURE;
    return rp;
}

inline RowRef draft_row(const oracle_batch* bt, int32_t b, int32_t i) {
    return RowRef{bt->draft, bt->dtype,
                  static_cast<int64_t>(b) * bt->draft_stride_row +
                      static_cast<int64_t>(i) * bt->draft_stride_pos};
}
inline RowRef target_row(const oracle_batch* bt, int32_t b, int32_t i) {
    return RowRef{bt->target, bt->dtype,
                  static_cast<int64_t>(b) * bt->target_stride_row +
                      static_cast<int64_t>(i) * bt->target_stride_pos};
}

/* ---- signals, one batch row (paper Sec. 4.2) ---- */
void signals_row(const oracle_batch* bt, int32_t b, double* H, double* C, double* feat,
                 int32_t* row_status) {
    const int32_t G = bt->gamma_max, V = bt->V;
    double* Hb = H ? H + static_cast<int64_t>(b) * G : nullptr;
    double* Cb = C ? C + static_cast<int64_t>(b) * G : nullptr;
    double* fb = feat ? feat + static_cast<int64_t>(b) * 4 : nullptr;
    if (Hb) std::fill(Hb, Hb + G, 0.0);
    if (Cb) std::fill(Cb, Cb + G, 0.0);
    if (fb) std::fill(fb, fb + 4, 0.0);

    RowParams rp = row_params(bt, b);
    if (rp.status) {
        if (row_status) row_status[b] |= rp.status;
        return;
    }
    const double Tsig = (rp.T == 0.0) ? 1.0 : rp.T;
    std::vector<double> q(V), Hi(rp.gamma), Ci(rp.gamma);
    for (int32_t i = 0; i < rp.gamma; ++i) {
        if (!softmax_row(draft_row(bt, b, i), V, Tsig, q.data())) {
            if (row_status) row_status[b] |= ORACLE_ROW_NONFINITE;
            return;
        }
        double h = entropy_nats(q.data(), V);
        if (bt->entropy_in_bits) h /= std::log(2.0);
        Hi[i] = h;
        Ci[i] = *std::max_element(q.begin(), q.end());
    }
    double Hsum = 0.0, Csum = 0.0, Hmax = Hi[0], Cmin = Ci[0];
    for (int32_t i = 0; i < rp.gamma; ++i) {
        Hsum += Hi[i];
        Csum += Ci[i];
        Hmax = std::max(Hmax, Hi[i]);
        Cmin = std::min(Cmin, Ci[i]);
        if (Hb) Hb[i] = Hi[i];
        if (Cb) Cb[i] = Ci[i];
    }
    if (fb) {
        fb[0] = Hsum / rp.gamma;
        fb[1] = Csum / rp.gamma;
        fb[2] = Hmax;
        fb[3] = Cmin;
    }
}

/* compression entries per row: what is left of n_in after the signals (and the gamma input) */
inline int32_t n_comp_of(const oracle_mlp* mlp) {
    return mlp->n_in - (mlp->feature_layout == 0 ? 3 : mlp->feature_layout == 1 ? 4 : 5);
}

/* ---- controller in the paper's own form (Sec. 4.3): one predictor f(x, gamma) -> a_hat with
 * x = [Hbar, cbar, Hmax, cmin, comp...] and the candidate gamma as the last input, evaluated once
 * per candidate; E = a_hat * gamma + 1 (Eq. 1); gamma* = argmax.  n_hidden = 0 is the linear
 * (Ridge) predictor: a_hat = W2 . [x, gamma] + b2. ---- */
void select_gamma_row_paper_form(const double* feat4, const float* comp, const oracle_mlp* mlp, double* scores,
                                 int32_t* gamma_next, int32_t* near) {
    const int32_t n_in = mlp->n_in;
    std::vector<double> x(n_in, 0.0);
    for (int32_t k = 0; k < 4; ++k) x[k] = feat4[k];
    for (int32_t k = 4; k < n_in - 1; ++k) x[k] = comp ? static_cast<double>(comp[k - 4]) : 0.0;
    int32_t best = 0;
    double best_e = 0.0, second_e = -std::numeric_limits<double>::infinity();
    for (int32_t j = 0; j < mlp->n_out; ++j) {
        x[n_in - 1] = static_cast<double>(mlp->gamma_choices[j]);
        double a_hat = static_cast<double>(mlp->b2[0]);
        if (mlp->n_hidden == 0) {
            for (int32_t f = 0; f < n_in; ++f) a_hat += static_cast<double>(mlp->W2[f]) * x[f];
        } else {
            for (int32_t k = 0; k < mlp->n_hidden; ++k) {
                double a = static_cast<double>(mlp->b1[k]);
                for (int32_t f = 0; f < n_in; ++f)
                    a += static_cast<double>(mlp->W1[static_cast<int64_t>(k) * n_in + f]) * x[f];
                if (a > 0.0) a_hat += static_cast<double>(mlp->W2[k]) * a;
            }
        }
        const double e = (mlp->score_transform == 0) ? a_hat * mlp->gamma_choices[j] + 1.0 : a_hat;
        if (scores) scores[j] = e;
        if (j == 0) {
            best_e = e;
        } else if (e > best_e) {
            second_e = best_e;
            best_e = e;
            best = j;
        } else if (e > second_e) {
            second_e = e;
        }
    }
    if (gamma_next) *gamma_next = mlp->gamma_choices[best];
    if (near) {
        bool tie = (mlp->n_out > 1) && (best_e - second_e) < 1e-5 * std::max(std::fabs(best_e), 1e-30);
        if (tie) *near |= ORACLE_NEAR_GAMMA;
    }
}

/* ---- controller, one row (paper Sec. 4.3, Eq. 1) ---- */
void select_gamma_row(const double* feat4, const float* comp, const oracle_mlp* mlp, double* scores,
                      int32_t* gamma_next, int32_t* near) {
    if (mlp->feature_layout == 2) {
        select_gamma_row_paper_form(feat4, comp, mlp, scores, gamma_next, near);
        return;
    }
    std::vector<double> x(mlp->n_in, 0.0);
    if (mlp->feature_layout == 0) {
        /* mean entropy, mean confidence, min confidence, two compression flags */
        x[0] = feat4[0];
        x[1] = feat4[1];
        x[2] = feat4[3];
        for (int32_t k = 3; k < mlp->n_in; ++k) x[k] = comp ? static_cast<double>(comp[k - 3]) : 0.0;
    } else {
        /* the paper's context vector [Hbar, cbar, Hmax, cmin, comp] */
        x[0] = feat4[0];
        x[1] = feat4[1];
        x[2] = feat4[2];
        x[3] = feat4[3];
        for (int32_t k = 4; k < mlp->n_in; ++k) x[k] = comp ? static_cast<double>(comp[k - 4]) : 0.0;
    }
    std::vector<double> h(mlp->n_hidden);
    for (int32_t k = 0; k < mlp->n_hidden; ++k) {
        double a = static_cast<double>(mlp->b1[k]);
        for (int32_t f = 0; f < mlp->n_in; ++f)
            a += static_cast<double>(mlp->W1[static_cast<int64_t>(k) * mlp->n_in + f]) * x[f];
        h[k] = a > 0.0 ? a : 0.0;
    }
    int32_t best = 0;
    double best_e = 0.0, second_e = -std::numeric_limits<double>::infinity();
    for (int32_t j = 0; j < mlp->n_out; ++j) {
        double o = static_cast<double>(mlp->b2[j]);
        for (int32_t k = 0; k < mlp->n_hidden; ++k)
            o += static_cast<double>(mlp->W2[static_cast<int64_t>(j) * mlp->n_hidden + k]) * h[k];
        double e = (mlp->score_transform == 0) ? o * mlp->gamma_choices[j] + 1.0 : o;
        if (scores) scores[j] = e;
        if (j == 0) {
            best_e = e;
        } else if (e > best_e) {
            second_e = best_e;
            best_e = e;
            best = j;
        } else if (e > second_e) {
            second_e = e;
        }
    }
    if (gamma_next) *gamma_next = mlp->gamma_choices[best];
    if (near) {
        bool tie = (mlp->n_out > 1) && (best_e - second_e) < 1e-5 * std::max(std::fabs(best_e), 1e-30);
        if (tie) *near |= ORACLE_NEAR_GAMMA;
    }
}

/* ---- verification, one row ---- */
void verify_row(const oracle_batch* bt, int32_t b, int32_t* n_accepted, int32_t* out_tokens,
                int32_t* row_status, int32_t* near) {
    const int32_t G = bt->gamma_max, V = bt->V;
    int32_t* ob = out_tokens + static_cast<int64_t>(b) * (G + 1);
    std::fill(ob, ob + G + 1, -1);
    n_accepted[b] = 0;

    RowParams rp = row_params(bt, b);
    if (rp.status) {
        if (row_status) row_status[b] |= rp.status;
        return;
    }
    const int32_t g = rp.gamma;
    const int32_t* xb = bt->draft_tokens + static_cast<int64_t>(b) * G;
    /* What flags a row, in this order (a flagged row emits nothing):
     *   a draft token outside [0, V)                       -> BAD_TOKEN;
     *   a non-finite draft row at any drafted position     -> NONFINITE, and nothing else is looked at;
     *   otherwise the positions are walked in order and the walk ends at the first position whose
     *   target row is non-finite (-> NONFINITE), whose draft token is out of range, or whose token
     *   is rejected.  Target rows behind that position are not part of the step: Sec. 3.1 emits the
     *   accepted prefix and one token at the first mismatch and discards whatever the target
     *   produced behind it, so those rows are neither read nor checked. */
    int32_t st = ORACLE_ROW_OK;
    for (int32_t i = 0; i < g; ++i)
        if (xb[i] < 0 || xb[i] >= V) st |= ORACLE_ROW_BAD_TOKEN;
    const double Tq = (rp.T == 0.0) ? 1.0 : rp.T;
    std::vector<double> mq(g), lzq(g);
    bool draft_bad = false;
    for (int32_t i = 0; i < g; ++i)
        if (!lse_row(draft_row(bt, b, i), V, Tq, &mq[i], &lzq[i])) draft_bad = true;
    if (draft_bad) {
        if (row_status) row_status[b] |= st | ORACLE_ROW_NONFINITE;
        return;
    }

    int32_t n = g, fresh = -1, nearbits = 0;

    if (rp.T == 0.0) {
        /* greedy rule of Sec. 3.1 */
        for (int32_t i = 0; i <= g; ++i) {
            const int32_t am = argmax_row(target_row(bt, b, i), V);
            if (am < 0) {
                st |= ORACLE_ROW_NONFINITE;
                break;
            }
            if (i < g && (xb[i] < 0 || xb[i] >= V)) break;
            if (i == g || xb[i] != am) {
                n = i;
                fresh = am;
                break;
            }
        }
        if (st) {
            if (row_status) row_status[b] |= st;
            return;
        }
    } else {
        const double T = rp.T;
        const float* ub = bt->uniforms + static_cast<int64_t>(b) * (G + 1) * 2;
        for (int32_t i = 0; i <= g; ++i) {
            double mp, lzp;
            if (!lse_row(target_row(bt, b, i), V, T, &mp, &lzp)) {
                st |= ORACLE_ROW_NONFINITE;
                break;
            }
            if (i == g) break; /* every drafted token accepted */
            if (xb[i] < 0 || xb[i] >= V) break;
            const double u = static_cast<double>(ub[2 * i + 0]);
            const double lnq = draft_row(bt, b, i).at(xb[i]) / T - mq[i] - lzq[i];
            const double lnp = target_row(bt, b, i).at(xb[i]) / T - mp - lzp;
            const double ratio = std::exp(lnp - lnq); /* p(x)/q(x); inf when q(x) = 0 < p(x) */
            if (std::fabs(u - ratio) < 1e-6) nearbits |= ORACLE_NEAR_ACCEPT;
            /* accept iff u*q(x) < p(x) */
            const bool accept = (std::log(u) + lnq) < lnp;
            if (!accept) {
                n = i;
                break;
            }
        }
        if (st) {
            if (row_status) row_status[b] |= st;
            return;
        }
        std::vector<double> p(V), w(V);
        softmax_row(target_row(bt, b, n), V, T, p.data());
        const double u2 = static_cast<double>(ub[2 * n + 1]);
        int32_t nb = 0;
        if (n < g) {
            std::vector<double> q(V);
            softmax_row(draft_row(bt, b, n), V, T, q.data());
            double Wres = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                w[v] = std::max(0.0, p[v] - q[v]);
                Wres += w[v];
            }
            fresh = inverse_cdf(w.data(), V, u2, &nb);
            if (fresh < 0) fresh = inverse_cdf(p.data(), V, u2, &nb); /* p == q numerically */
            /* A residual of total mass below 1e-5 (the probability that this rejection happens at all
             * under the rule of Sec. 2.1) is beyond what weights held in fp32 resolve: the draw is
             * exact here and the row carries a flag of its own. */
            if (Wres < 1e-5) nearbits |= ORACLE_NEAR_SMALL_RESIDUAL;
        } else {
            fresh = inverse_cdf(p.data(), V, u2, &nb);
        }
        if (nb & 1) nearbits |= ORACLE_NEAR_CDF;
        else if (nb & 2) nearbits |= ORACLE_NEAR_CDF_ABS;
    }

    n_accepted[b] = n;
    for (int32_t i = 0; i < n; ++i) ob[i] = xb[i];
    ob[n] = fresh;
    if (near) near[b] |= nearbits;
}

template <class F>
void for_rows(int32_t B, int32_t n_threads, F f) {
    n_threads = std::max(1, std::min(n_threads, B));
    if (n_threads == 1) {
        for (int32_t b = 0; b < B; ++b) f(b);
        return;
    }
    std::vector<std::thread> pool;
    for (int32_t t = 0; t < n_threads; ++t)
        pool.emplace_back([=]() {
            for (int32_t b = t; b < B; b += n_threads) f(b);
        });
    for (auto& th : pool) th.join();
}

bool batch_ok(const oracle_batch* bt, bool need_target) {
    if (!bt || bt->B < 0 || bt->gamma_max < 1 || bt->V < 1) return false;
    if (bt->dtype != ORACLE_DT_F32 && bt->dtype != ORACLE_DT_BF16) return false;
    if (bt->B > 0 && !bt->draft) return false;
    if (need_target && bt->B > 0 && (!bt->target || !bt->draft_tokens || !bt->uniforms)) return false;
    return true;
}

}  // namespace

extern "C" {

int oracle_softmax_row(const void* row, int32_t dtype, int32_t V, double T, double* prob) {
    return softmax_row(RowRef{row, dtype, 0}, V, T, prob) ? 0 : ORACLE_ROW_NONFINITE;
}

double oracle_entropy_nats(const double* prob, int32_t V) { return entropy_nats(prob, V); }

int32_t oracle_inverse_cdf(const double* w, int32_t V, double u, int32_t* near_boundary) {
    const int32_t tok = inverse_cdf(w, V, u, near_boundary);
    if (near_boundary) *near_boundary &= 1;
    return tok;
}

int32_t oracle_argmax_row(const void* row, int32_t dtype, int32_t V) {
    return argmax_row(RowRef{row, dtype, 0}, V);
}

int oracle_signals(const oracle_batch* bt, double* H, double* C, double* feat, int32_t* row_status) {
    if (!batch_ok(bt, false)) return 1;
    if (row_status) std::fill(row_status, row_status + bt->B, 0);
    for_rows(bt->B, bt->n_threads, [&](int32_t b) { signals_row(bt, b, H, C, feat, row_status); });
    return 0;
}

int oracle_select_gamma(int32_t B, const double* feat, const float* comp, const oracle_mlp* mlp,
                        double* scores, int32_t* gamma_next, int32_t* near) {
    if (B < 0 || !mlp || !feat || mlp->n_out < 1 || mlp->n_out > 8 || mlp->n_in < 4) return 1;
    if (mlp->n_hidden < (mlp->feature_layout == 2 ? 0 : 1)) return 1;
    if (mlp->feature_layout == 2 && mlp->n_in < 5) return 1;
    const int32_t n_comp = n_comp_of(mlp);
    for (int32_t b = 0; b < B; ++b)
        select_gamma_row(feat + static_cast<int64_t>(b) * 4,
                         comp ? comp + static_cast<int64_t>(b) * n_comp : nullptr, mlp,
                         scores ? scores + static_cast<int64_t>(b) * mlp->n_out : nullptr,
                         gamma_next ? gamma_next + b : nullptr, near ? near + b : nullptr);
    return 0;
}

int oracle_verify(const oracle_batch* bt, int32_t* n_accepted, int32_t* out_tokens,
                  int32_t* row_status, int32_t* near) {
    if (!batch_ok(bt, true) || !n_accepted || !out_tokens) return 1;
    if (row_status) std::fill(row_status, row_status + bt->B, 0);
    if (near) std::fill(near, near + bt->B, 0);
    for_rows(bt->B, bt->n_threads,
             [&](int32_t b) { verify_row(bt, b, n_accepted, out_tokens, row_status, near); });
    return 0;
}

/* Drafting (paper Sec. 3.1: the draft model proposes gamma tokens): position i of row b draws its
 * token from q_i = softmax(d[b,i] / T_b) by the same inverse-CDF convention as the verification
 * draws (vocabulary order, threshold u * sum); T_b = 0 takes the argmax (lowest index). */
int oracle_sample_draft(const oracle_batch* bt, const float* uniforms, int32_t* tokens,
                        int32_t* row_status, int32_t* near) {
    if (!batch_ok(bt, false) || !tokens || !uniforms) return 1;
    const int32_t G = bt->gamma_max, V = bt->V;
    if (row_status) std::fill(row_status, row_status + bt->B, 0);
    if (near) std::fill(near, near + bt->B, 0);
    for_rows(bt->B, bt->n_threads, [&](int32_t b) {
        int32_t* tb = tokens + static_cast<int64_t>(b) * G;
        std::fill(tb, tb + G, -1);
        const RowParams rp = row_params(bt, b);
        int32_t status = rp.status;
        std::vector<int32_t> tok(G, -1);
        std::vector<double> q(V);
        int32_t nearbits = 0;
        for (int32_t i = 0; !status && i < rp.gamma; ++i) {
            if (rp.T == 0.0) {
                const RowRef r = draft_row(bt, b, i);
                if (!softmax_row(r, V, 1.0, q.data())) { status |= ORACLE_ROW_NONFINITE; break; }
                tok[i] = argmax_row(r, V);
            } else {
                if (!softmax_row(draft_row(bt, b, i), V, rp.T, q.data())) { status |= ORACLE_ROW_NONFINITE; break; }
                int32_t nb = 0;
                tok[i] = inverse_cdf(q.data(), V, static_cast<double>(uniforms[static_cast<int64_t>(b) * G + i]), &nb);
                if (nb & 1) nearbits |= ORACLE_NEAR_CDF;
            }
        }
        if (!status) std::copy(tok.begin(), tok.end(), tb);
        if (row_status) row_status[b] = status;
        if (near) near[b] = nearbits;
    });
    return 0;
}

int oracle_step(const oracle_batch* bt, const float* comp, const oracle_mlp* mlp, double* H,
                double* C, double* feat, double* scores, int32_t* gamma_next,
                int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status, int32_t* near) {
    if (!batch_ok(bt, true) || !mlp || !feat || !n_accepted || !out_tokens || !row_status) return 1;
    std::fill(row_status, row_status + bt->B, 0);
    if (near) std::fill(near, near + bt->B, 0);
    const int32_t n_comp = n_comp_of(mlp);
    for_rows(bt->B, bt->n_threads, [&](int32_t b) {
        signals_row(bt, b, H, C, feat, row_status);
        verify_row(bt, b, n_accepted, out_tokens, row_status, near);
        double* sb = scores ? scores + static_cast<int64_t>(b) * mlp->n_out : nullptr;
        if (row_status[b]) {
            /* a flagged row takes no decision */
            if (sb) std::fill(sb, sb + mlp->n_out, 0.0);
            if (gamma_next) gamma_next[b] = 0;
            double* fb = feat + static_cast<int64_t>(b) * 4;
            std::fill(fb, fb + 4, 0.0);
            if (H) std::fill(H + static_cast<int64_t>(b) * bt->gamma_max,
                             H + static_cast<int64_t>(b + 1) * bt->gamma_max, 0.0);
            if (C) std::fill(C + static_cast<int64_t>(b) * bt->gamma_max,
                             C + static_cast<int64_t>(b + 1) * bt->gamma_max, 0.0);
            return;
        }
        select_gamma_row(feat + static_cast<int64_t>(b) * 4,
                         comp ? comp + static_cast<int64_t>(b) * n_comp : nullptr, mlp, sb,
                         gamma_next ? gamma_next + b : nullptr, near ? near + b : nullptr);
    });
    return 0;
}

}  // extern "C"
