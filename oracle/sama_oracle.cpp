// CPU checker for the SAMA meta-gradient step (arXiv 2310.05674).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
// statement of what the method computes; tests, the smoke check and the
// benchmark's CPU-baseline leg call it.  The CUDA library never does, and the
// two share no code.  Inputs are fp32 (the caller's storage type); every
// arithmetic step and every accumulation is in double.
//
// The method is an approximation followed by a finite difference, so there is
// no closed-form "true answer" to write down; the functions below take the
// paper's steps in the paper's order:
//   S1  Algorithmic adaptation, Eq. 4 with the Adam adaptation matrix of
//       Appendix C:          p = (du_adam/dg_base) * g_meta   (elementwise)
//   S2  Step size, Sec. 3.2: eps_fd = alpha / ||p||_2         (one global norm)
//   S3  Perturbation:        theta+- = theta +- eps_fd * p
//   S4  Base loss with per-sample weights (Sec. 4.1 reweighting objective):
//       L_base = (1/B) sum_i sigmoid(lambda_i) * CE(f(x_i; theta), y_i)
//   S5  Central difference, Eq. 5:
//       dL_meta/dlambda_i ~= -[dL_base(theta+)/dlambda_i
//                              - dL_base(theta-)/dlambda_i] / (2 eps_fd)
//
// Readings taken where Appendix C is garbled or silent (all checked by the
// CPU tests against brute-force differentiation of the Adam update):
//   * moments use beta1 for m and beta2 for the second moment (standard Adam);
//     the derivative is the exact one of the update;
//   * both "e" and "epsilon" in the denominators are Adam's epsilon;
//   * bias correction is on by default (the printed update has none; switch
//     bias_correction=0 reproduces the printed form);
//   * (m, s) are the state before the update that is differentiated;
//   * drop_eps_term=1 gives the paper's "epsilon << 1" approximation;
//   * identity=1 is SGD / SAMA-NA: the adaptation matrix is the identity.
//
// Pins (tests/test_oracle_pins.py): brute-force central differences of the
// Adam update in extended precision; the paper's printed numerator in its
// beta1 == beta2 special case; the RMS-normalised limit lr/sqrt(s); closed-form
// mixed second derivative on a linear-softmax model with O(alpha^2) error
// decay; brute-force nested differences on tiny MLPs; forward pass against a
// library matmul; antisymmetry, scaling and permutation invariants.
// The shared reweighting network of Sec. 4.1 (sama_oracle_reweight_grad, sama_oracle_fd_reweight) is pinned in
// tests/test_oracle_reweight_pins.py: extended-precision differences of the base objective in lambda_r,
// hand-computed special cases, nested differences on tiny MLPs.  Reading: the paper says "2-layer MLP" and
// gives neither width nor activations; ReLU hidden units and a sigmoid output are taken (as in the
// reweighting network the paper cites), the width is an argument.
// No function here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <vector>

extern "C" {

struct sama_oracle_adam {
    double lr, beta1, beta2, eps;
    int64_t step;
    int32_t bias_correction;
    int32_t drop_eps_term;
    int32_t identity;
};

// S1 -- Appendix C (Adam adaptation matrix), Eq. 4.
// u(g) = (lr/c1) * m' / (sqrt(s')/sqrt(c2) + eps),
//   m' = beta1 m + (1-beta1) g,  s' = beta2 s + (1-beta2) g^2,
//   c1 = 1-beta1^step, c2 = 1-beta2^step (1 without bias correction).
// du/dg = (lr/c1) * [(1-beta1) beta2 s - beta1 (1-beta2) m g
//                    + (1-beta1) eps sqrt(c2) r] / (sqrt(c2) r D^2),
//   r = sqrt(s'), D = r/sqrt(c2) + eps.
// At r = 0 (s = 0 and g = 0) the limit is (lr/c1)(1-beta1)/eps.
void sama_oracle_adapt(int64_t n, const float* m, const float* s, const float* g_base,
                       const float* g_meta, const sama_oracle_adam* h, double* p_out) {
    const double b1 = h->beta1, b2 = h->beta2, eps = h->eps;
    double c1 = 1.0, c2 = 1.0;
    if (h->bias_correction) {
        c1 = 1.0 - std::pow(b1, (double)h->step);
        c2 = 1.0 - std::pow(b2, (double)h->step);
    }
    const double rc2 = std::sqrt(c2);
    for (int64_t k = 0; k < n; ++k) {
        const double gm = (double)g_meta[k];
        if (h->identity) { p_out[k] = gm; continue; }
        const double mk = (double)m[k], sk = (double)s[k];
        const double g = g_base ? (double)g_base[k] : mk;
        const double s_new = b2 * sk + (1.0 - b2) * g * g;
        const double r = std::sqrt(s_new);
        const double D = r / rc2 + eps;
        double J;
        if (r > 0.0) {
            double num = (1.0 - b1) * b2 * sk - b1 * (1.0 - b2) * mk * g;
            if (!h->drop_eps_term) num += (1.0 - b1) * eps * rc2 * r;
            J = (h->lr / c1) * num / (rc2 * r * D * D);
        } else {
            J = h->drop_eps_term ? 0.0 : (h->lr / c1) * (1.0 - b1) / eps;
        }
        p_out[k] = J * gm;
    }
}

// S2 -- Sec. 3.2: squared L2 norm of the whole perturbation vector.
double sama_oracle_sumsq(int64_t n, const double* p) {
    double acc = 0.0;
    for (int64_t k = 0; k < n; ++k) acc += p[k] * p[k];
    return acc;
}

// S3 given S2's sum of squares -- Sec. 3.2: eps_fd = alpha/sqrt(sumsq),
// theta+- = theta +- eps_fd p on the n elements given (which may be a slice of
// the vector the sum was taken over).  Returns 1 (and theta+- = theta,
// eps_fd = 0) when the norm is 0 or not finite.
int sama_oracle_perturb_given_sumsq(int64_t n, const float* theta, const double* p, double sumsq, double alpha,
                                    double* theta_plus, double* theta_minus, double* eps_fd_out) {
    const double norm = std::sqrt(sumsq);
    const bool bad = !(norm > 0.0) || !std::isfinite(norm);
    const double eps_fd = bad ? 0.0 : alpha / norm;
    for (int64_t k = 0; k < n; ++k) {
        const double t = (double)theta[k];
        const double d = bad ? 0.0 : eps_fd * p[k];
        theta_plus[k] = t + d;
        theta_minus[k] = t - d;
    }
    *eps_fd_out = eps_fd;
    return bad ? 1 : 0;
}

// S2 + S3 -- Sec. 3.2 on a whole vector.
int sama_oracle_perturb(int64_t n, const float* theta, const double* p, double alpha,
                        double* theta_plus, double* theta_minus, double* eps_fd_out) {
    return sama_oracle_perturb_given_sumsq(n, theta, p, sama_oracle_sumsq(n, p), alpha, theta_plus, theta_minus,
                                           eps_fd_out);
}

// S4 -- per-sample cross-entropy of the base MLP at parameters theta.
// theta = W1, b1, W2, b2, ...; W_l is [d_l][d_{l-1}] row-major; ReLU between
// layers, last layer linear; loss_i = logsumexp(z_i) - z_i[y_i].
void sama_oracle_losses(int32_t n_layers, const int32_t* dims, const double* theta,
                        const float* X, const int32_t* y, int32_t B,
                        double* loss_out, double* logits_out) {
    int32_t widest = 0;
    for (int32_t l = 0; l <= n_layers; ++l) widest = dims[l] > widest ? dims[l] : widest;
    std::vector<double> h(widest), hn(widest);
    const int32_t C = dims[n_layers];
    for (int32_t i = 0; i < B; ++i) {
        for (int32_t k = 0; k < dims[0]; ++k) h[k] = (double)X[(int64_t)i * dims[0] + k];
        const double* W = theta;
        for (int32_t l = 0; l < n_layers; ++l) {
            const int32_t din = dims[l], dout = dims[l + 1];
            const double* b = W + (int64_t)din * dout;
            for (int32_t j = 0; j < dout; ++j) {
                double acc = b[j];
                const double* w = W + (int64_t)j * din;
                for (int32_t k = 0; k < din; ++k) acc += w[k] * h[k];
                hn[j] = (l + 1 < n_layers && acc < 0.0) ? 0.0 : acc;
            }
            h.swap(hn);
            W = b + dout;
        }
        double zmax = h[0];
        for (int32_t c = 1; c < C; ++c) zmax = h[c] > zmax ? h[c] : zmax;
        double se = 0.0;
        for (int32_t c = 0; c < C; ++c) se += std::exp(h[c] - zmax);
        loss_out[i] = std::log(se) + zmax - h[y[i]];
        if (logits_out)
            for (int32_t c = 0; c < C; ++c) logits_out[(int64_t)i * C + c] = h[c];
    }
}

// Direct gradient -- the first factor of Eq. 1, dL_meta/dtheta, for the meta objective of Sec. 4.1:
// L_meta(theta) = (1/B) sum_i CE(f(x_i; theta), y_i) on a clean batch.  Plain reverse-mode
// differentiation of the same MLP, layer by layer:
//   dz_L = (softmax(z_L) - onehot(y)) / B,
//   dW_l = dz_l h_{l-1}^T,  db_l = dz_l,  dh_{l-1} = W_l^T dz_l,  dz_{l-1} = dh_{l-1} * [z_{l-1} > 0].
// Returns L_meta; grad_out has the layout of theta.
double sama_oracle_meta_grad(int32_t n_layers, const int32_t* dims, const float* theta, const float* X,
                             const int32_t* y, int32_t B, double* grad_out) {
    int64_t n = 0;
    std::vector<int64_t> woff(n_layers), boff(n_layers);
    for (int32_t l = 0; l < n_layers; ++l) {
        woff[l] = n;
        n += (int64_t)dims[l] * dims[l + 1];
        boff[l] = n;
        n += dims[l + 1];
    }
    for (int64_t k = 0; k < n; ++k) grad_out[k] = 0.0;
    std::vector<std::vector<double>> h(n_layers + 1);  // h[l] = input of layer l (post-ReLU), h[L] = logits
    for (int32_t l = 0; l <= n_layers; ++l) h[l].resize(dims[l]);
    double loss = 0.0;
    const int32_t C = dims[n_layers];
    for (int32_t i = 0; i < B; ++i) {
        for (int32_t k = 0; k < dims[0]; ++k) h[0][k] = (double)X[(int64_t)i * dims[0] + k];
        for (int32_t l = 0; l < n_layers; ++l) {
            const int32_t din = dims[l], dout = dims[l + 1];
            for (int32_t j = 0; j < dout; ++j) {
                double acc = (double)theta[boff[l] + j];
                for (int32_t k = 0; k < din; ++k) acc += (double)theta[woff[l] + (int64_t)j * din + k] * h[l][k];
                const bool hidden = l + 1 < n_layers;
                h[l + 1][j] = (hidden && acc < 0.0) ? 0.0 : acc;
            }
        }
        double zmax = h[n_layers][0];
        for (int32_t c = 1; c < C; ++c) zmax = h[n_layers][c] > zmax ? h[n_layers][c] : zmax;
        double se = 0.0;
        for (int32_t c = 0; c < C; ++c) se += std::exp(h[n_layers][c] - zmax);
        loss += (std::log(se) + zmax - h[n_layers][y[i]]) / (double)B;
        std::vector<double> dz(C);
        for (int32_t c = 0; c < C; ++c)
            dz[c] = (std::exp(h[n_layers][c] - zmax) / se - (c == y[i] ? 1.0 : 0.0)) / (double)B;
        for (int32_t l = n_layers - 1; l >= 0; --l) {
            const int32_t din = dims[l], dout = dims[l + 1];
            std::vector<double> dh(din, 0.0);
            for (int32_t j = 0; j < dout; ++j) {
                grad_out[boff[l] + j] += dz[j];
                for (int32_t k = 0; k < din; ++k) {
                    grad_out[woff[l] + (int64_t)j * din + k] += dz[j] * h[l][k];
                    dh[k] += (double)theta[woff[l] + (int64_t)j * din + k] * dz[j];
                }
            }
            if (l > 0)  // h[l] is a ReLU output: the derivative passes where it is positive
                for (int32_t k = 0; k < din; ++k) dh[k] = h[l][k] > 0.0 ? dh[k] : 0.0;
            dz.swap(dh);
        }
    }
    return loss;
}

// S5 -- Eq. 5 for per-sample weight logits:
// dL_base/dlambda_i = sigmoid'(lambda_i) loss_i / B_norm, hence
// metagrad_i = -sigmoid'(lambda_i) (loss+_i - loss-_i) / (2 eps_fd B_norm).
// B_norm is the size of the whole base batch (the 1/|D| of the objective),
// which may exceed the number of samples evaluated here.
void sama_oracle_fd(int32_t count, const double* loss_plus, const double* loss_minus,
                    const float* lambda, double eps_fd, int32_t B_norm, double* metagrad_out) {
    for (int32_t i = 0; i < count; ++i) {
        if (!(eps_fd > 0.0)) { metagrad_out[i] = 0.0; continue; }
        const double sg = 1.0 / (1.0 + std::exp(-(double)lambda[i]));
        metagrad_out[i] = -sg * (1.0 - sg) * (loss_plus[i] - loss_minus[i]) / (2.0 * eps_fd * (double)B_norm);
    }
}

// Shared reweighting network -- the meta learner of Sec. 4.1, w(l; lambda_r): a 2-layer MLP on the
// scalar per-sample loss l with H hidden units and a sigmoid output,
//   a_j = v1_j l + c1_j,  h_j = max(0, a_j),  z = sum_j v2_j h_j + c2,  w = sigmoid(z),
// lambda_r = (v1[H], c1[H], v2[H], c2) in that order (3H + 1 numbers).  The base objective is
//   L_base(theta, lambda_r) = (1/B) sum_i w(l_i(theta); lambda_r) l_i(theta),
// so at fixed theta
//   dL_base/dlambda_r = (1/B) sum_i l_i w_i (1 - w_i) dz_i/dlambda_r,
//   dz/dc2 = 1,  dz/dv2_j = h_j,  dz/dc1_j = v2_j [a_j > 0],  dz/dv1_j = v2_j [a_j > 0] l.
// grad_out has 3H + 1 entries; weights_out (count entries, may be null) receives w_i.
void sama_oracle_reweight_grad(int32_t count, const double* loss, int32_t H, const float* lambda_r,
                               int32_t B_norm, double* grad_out, double* weights_out) {
    const float* v1 = lambda_r;
    const float* c1 = lambda_r + H;
    const float* v2 = lambda_r + 2 * (int64_t)H;
    const double c2 = (double)lambda_r[3 * (int64_t)H];
    for (int32_t k = 0; k < 3 * H + 1; ++k) grad_out[k] = 0.0;
    for (int32_t i = 0; i < count; ++i) {
        const double l = loss[i];
        double z = c2;
        for (int32_t j = 0; j < H; ++j) {
            const double a = (double)v1[j] * l + (double)c1[j];
            if (a > 0.0) z += (double)v2[j] * a;
        }
        const double w = 1.0 / (1.0 + std::exp(-z));
        if (weights_out) weights_out[i] = w;
        const double f = l * w * (1.0 - w) / (double)B_norm;
        for (int32_t j = 0; j < H; ++j) {
            const double a = (double)v1[j] * l + (double)c1[j];
            if (a > 0.0) {
                grad_out[j] += f * (double)v2[j] * l;          // v1_j
                grad_out[H + j] += f * (double)v2[j];          // c1_j
                grad_out[2 * (int64_t)H + j] += f * a;          // v2_j
            }
        }
        grad_out[3 * (int64_t)H] += f;                          // c2
    }
}

// Eq. 5 with the shared reweighting network as the meta learner:
//   metagrad = -[ dL_base(theta+)/dlambda_r - dL_base(theta-)/dlambda_r ] / (2 eps_fd),
// from the per-sample losses at theta+ and theta- (S4).  3H + 1 entries; zero when eps_fd is not positive.
void sama_oracle_fd_reweight(int32_t count, const double* loss_plus, const double* loss_minus, int32_t H,
                             const float* lambda_r, double eps_fd, int32_t B_norm, double* metagrad_out) {
    const int32_t dim = 3 * H + 1;
    std::vector<double> gp(dim), gm(dim);
    sama_oracle_reweight_grad(count, loss_plus, H, lambda_r, B_norm, gp.data(), nullptr);
    sama_oracle_reweight_grad(count, loss_minus, H, lambda_r, B_norm, gm.data(), nullptr);
    for (int32_t k = 0; k < dim; ++k)
        metagrad_out[k] = eps_fd > 0.0 ? -(gp[k] - gm[k]) / (2.0 * eps_fd) : 0.0;
}

// S1..S5 chained (the workflow of Fig. 2 with lambda = per-sample weights).
// Samples evaluated: rows [0, count) of X / y / lambda; B_norm as above.
// Outputs p, theta+-, (optional) per-sample losses, metagrad; returns the
// degenerate-norm flag of S2.
int sama_oracle_step(int32_t n_layers, const int32_t* dims, int64_t n,
                     const float* theta, const float* m, const float* s, const float* g_base,
                     const float* g_meta, const sama_oracle_adam* h, double alpha,
                     const float* X, const int32_t* y, const float* lambda,
                     int32_t count, int32_t B_norm,
                     double* p_out, double* theta_plus, double* theta_minus, double* eps_fd_out,
                     double* loss_plus_out, double* loss_minus_out, double* metagrad_out) {
    sama_oracle_adapt(n, m, s, g_base, g_meta, h, p_out);
    const int bad = sama_oracle_perturb(n, theta, p_out, alpha, theta_plus, theta_minus, eps_fd_out);
    std::vector<double> lp(count), lm(count);
    sama_oracle_losses(n_layers, dims, theta_plus, X, y, count, lp.data(), nullptr);
    sama_oracle_losses(n_layers, dims, theta_minus, X, y, count, lm.data(), nullptr);
    sama_oracle_fd(count, lp.data(), lm.data(), lambda, *eps_fd_out, B_norm, metagrad_out);
    for (int32_t i = 0; i < count; ++i) {
        if (loss_plus_out) loss_plus_out[i] = lp[i];
        if (loss_minus_out) loss_minus_out[i] = lm[i];
    }
    return bad;
}

}  // extern "C"
