// CPU oracle for the OD-SGD parameter-update pass.
//
// TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is
// checked against; the product never calls it.  It shares no code, header or
// constant with the CUDA path.  Plain scalar loops, single thread, host
// pointers only.
//
// Precision: the method is defined on fp32 state (weights, momentum,
// gradients), and the CUDA path must reproduce it bit for bit in its
// deterministic mode, so every statement below that contains one arithmetic
// operator is exactly one IEEE-754 binary32 round-to-nearest-even operation.
// Build with -ffp-contract=off (no fused multiply-add), no fast-math, no
// flush-to-zero.  An fp64 twin of each rule (suffix _f64) exists for the tests
// that bound the rounding error of the fp32 rules.
//
// What the rules are (paper notation: M workers, here n_workers; w_t global
// weights; g_m worker m's gradient; w_bak the worker's backup weights):
//
//  * global update, Algorithm 1 ("Update w_t with aggregated gradient" once
//    all M gradients have arrived).  The paper does not print the updater; it
//    is the stock momentum-SGD updater of the framework the paper used
//    (Section 3.3, "Local Updater"), with momentum and weight decay as listed
//    in Section 4:   gbar = (sum_m g_m) * (1/M);   d = gbar + wd * w;
//    v <- momentum * v - lr * d;   w <- w + v.   Workers are added in the order
//    m = 0, 1, ..., M-1.
//  * local update, Algorithm 2 (repeat-loop: "w_bak^t = w_t" followed by
//    "Update w_bak^t with g_m"), SGD flavour:  x_m = w_bak - local_lr * g_m,
//    where w_bak is the global weight vector *before* this iteration's global
//    update (the worker has not pulled the new one yet).
//  * SSGD step, Section 3.1: the server side of OD-SGD "keeps unchanged when
//    compared to SSGD", i.e. the same rule as the global update.
//  * ASGD step, Section 1 / 2.1: the server applies one worker's gradient as
//    soon as it arrives (no sum, no 1/M).
//  * DC-ASGD-c / DC-ASGD-a local updaters, Eq. 4, Eq. 5 and Eq. 6; local SGD with momentum
//    (Section 4.1's MNIST run); per-tensor multipliers; DC-ASGD at the server.
//
// Parity pins: every function here is pinned by tests/test_oracle_pins.py
// (hand-worked dyadic example, closed forms on a diagonal quadratic, exact
// rational re-evaluation, invariants, planted-mistake checks).

#include <cmath>
#include <cstddef>
#include <cstdint>

extern "C" {

// ---------------------------------------------------------------- Algorithm 1
// w, v: updated in place.  w_prev (may be null) receives the weights as they
// were before the update, i.e. the vector a worker would hold as w_bak.
int oracle_global_update(const float* const* grads, int n_workers, size_t n,
                         float* w, float* v, float* w_prev,
                         float lr, float momentum, float wd)
{
    if (n_workers < 1) return -1;
    const float inv_m = 1.0f / (float)n_workers;
    for (size_t i = 0; i < n; ++i) {
        float s = grads[0][i];
        for (int m = 1; m < n_workers; ++m) {
            s = s + grads[m][i];
        }
        const float gbar = s * inv_m;
        const float decay = wd * w[i];
        const float d = gbar + decay;
        const float keep = momentum * v[i];
        const float step = lr * d;
        const float v_new = keep - step;
        const float w_new = w[i] + v_new;
        if (w_prev) w_prev[i] = w[i];
        v[i] = v_new;
        w[i] = w_new;
    }
    return 0;
}

// SSGD server step: Section 3.1 states the parameter-server side is the same
// in SSGD and OD-SGD, so this is Algorithm 1's update without a backup copy.
int oracle_ssgd_step(const float* const* grads, int n_workers, size_t n,
                     float* w, float* v, float lr, float momentum, float wd)
{
    return oracle_global_update(grads, n_workers, n, w, v, nullptr, lr, momentum, wd);
}

// ---------------------------------------------------------------- Algorithm 2
// x = w_bak - local_lr * g   (x may alias w_bak: the paper updates w_bak in place)
int oracle_local_update(const float* w_bak, const float* g, size_t n, float* x, float local_lr)
{
    for (size_t i = 0; i < n; ++i) {
        const float step = local_lr * g[i];
        x[i] = w_bak[i] - step;
    }
    return 0;
}

// ---------------------------------------------------------------- ASGD
// One arriving gradient applied to the global state at once.
int oracle_asgd_step(const float* g, size_t n, float* w, float* v,
                     float lr, float momentum, float wd)
{
    for (size_t i = 0; i < n; ++i) {
        const float decay = wd * w[i];
        const float d = g[i] + decay;
        const float keep = momentum * v[i];
        const float step = lr * d;
        const float v_new = keep - step;
        v[i] = v_new;
        w[i] = w[i] + v_new;
    }
    return 0;
}

// ---------------------------------------------------------------- Eq. 4
// DC-ASGD-c used as the local updater.  Roles of the paper's symbols when the
// rule runs on a worker: w_{t+tau} is the vector being updated (w_bak, the
// freshly pulled global weights), w_t is the vector the gradient was computed
// on (x_prev, the weights the worker trained on this iteration), eta is the
// local learning rate and lambda the compensation coefficient.
//   x = w_bak - eta * (g + lambda * g * g * (w_bak - x_prev))
int oracle_local_update_dc_c(const float* w_bak, const float* g, const float* x_prev,
                             size_t n, float* x, float local_lr, float lambda)
{
    for (size_t i = 0; i < n; ++i) {
        const float diff = w_bak[i] - x_prev[i];
        const float gg = g[i] * g[i];
        const float lgg = lambda * gg;
        const float comp = lgg * diff;
        const float d = g[i] + comp;
        const float step = local_lr * d;
        x[i] = w_bak[i] - step;
    }
    return 0;
}

// ---------------------------------------------------------------- Eq. 5, Eq. 6
// DC-ASGD-a: lambda is divided by sqrt(MeanSquare + eps), MeanSquare being a
// running average of g*g with decay m (updated first, Eq. 6, then used, Eq. 5).
//   ms = m * ms + (1 - m) * g * g;
//   x  = w_bak - eta * (g + (lambda / sqrt(ms + eps)) * g * g * (w_bak - x_prev))
int oracle_local_update_dc_a(const float* w_bak, const float* g, const float* x_prev,
                             float* mean_square, size_t n, float* x,
                             float local_lr, float lambda, float m, float eps)
{
    const float one_minus_m = 1.0f - m;
    for (size_t i = 0; i < n; ++i) {
        const float gg = g[i] * g[i];
        const float a = m * mean_square[i];
        const float b = one_minus_m * gg;
        const float ms = a + b;
        mean_square[i] = ms;
        const float den = std::sqrt(ms + eps);
        const float lam = lambda / den;
        const float diff = w_bak[i] - x_prev[i];
        const float lgg = lam * gg;
        const float comp = lgg * diff;
        const float d = g[i] + comp;
        const float step = local_lr * d;
        x[i] = w_bak[i] - step;
    }
    return 0;
}

// ---------------------------------------------------------------- local SGD with momentum
// Section 3.3 lets the local updater be any existing SGD-based algorithm, and the MNIST run
// of Section 4.1 uses SGD with the same learning rate and momentum as the server.  That is
// the server's own rule applied by worker m to its backup weights with its own gradient and
// its own velocity u_m (one arena per worker):
//   d = g + wd_l * w_bak;   u <- momentum_l * u - local_lr * d;   x = w_bak + u
int oracle_local_update_momentum(const float* w_bak, const float* g, float* u, size_t n, float* x,
                                 float local_lr, float momentum, float wd)
{
    for (size_t i = 0; i < n; ++i) {
        const float decay = wd * w_bak[i];
        const float d = g[i] + decay;
        const float keep = momentum * u[i];
        const float step = local_lr * d;
        const float u_new = keep - step;
        u[i] = u_new;
        x[i] = w_bak[i] + u_new;
    }
    return 0;
}

// ---------------------------------------------------------------- per-tensor multipliers
// The stock updater of the framework the paper used scales the learning rate and the
// weight decay per parameter tensor (lr_mult, wd_mult; biases and batch-norm scales
// commonly get wd_mult = 0).  Tensor t owns elements [offsets[t], offsets[t+1]).
//   lr_t = lr * lr_mult[t];  wd_t = wd * wd_mult[t];  then Algorithm 1's update with lr_t, wd_t.
int oracle_global_update_mult(const float* const* grads, int n_workers, size_t n,
                              float* w, float* v, float* w_prev,
                              float lr, float momentum, float wd,
                              const size_t* offsets, size_t n_tensors,
                              const float* lr_mult, const float* wd_mult)
{
    if (n_workers < 1 || n_tensors < 1 || offsets[0] != 0 || offsets[n_tensors] != n) return -1;
    const float inv_m = 1.0f / (float)n_workers;
    for (size_t t = 0; t < n_tensors; ++t) {
        const float lr_t = lr * lr_mult[t];
        const float wd_t = wd * wd_mult[t];
        for (size_t i = offsets[t]; i < offsets[t + 1]; ++i) {
            float s = grads[0][i];
            for (int m = 1; m < n_workers; ++m) s = s + grads[m][i];
            const float gbar = s * inv_m;
            const float decay = wd_t * w[i];
            const float d = gbar + decay;
            const float keep = momentum * v[i];
            const float step = lr_t * d;
            const float v_new = keep - step;
            const float w_new = w[i] + v_new;
            if (w_prev) w_prev[i] = w[i];
            v[i] = v_new;
            w[i] = w_new;
        }
    }
    return 0;
}

// ---------------------------------------------------------------- DC-ASGD at the server
// The paper's fourth comparison algorithm (Section 4.1): Eq. 4 / Eq. 5 applied by the
// parameter server to each arriving gradient.  w is the current global vector (the
// paper's w_{t+tau}); w_bak_m is the copy worker m pulled before computing g (the
// paper's w_t).  After the step worker m pulls again, so its backup becomes the new w.
// No momentum and no weight decay appear in Eq. 4 / Eq. 5 (Section 4.1 sets momentum 0).
//   w <- w - eta * (g + lambda * g*g * (w - w_bak_m));   w_bak_m <- w
int oracle_dcasgd_step_c(const float* g, size_t n, float* w, float* w_bak_m, float lr, float lambda)
{
    for (size_t i = 0; i < n; ++i) {
        const float diff = w[i] - w_bak_m[i];
        const float gg = g[i] * g[i];
        const float lgg = lambda * gg;
        const float comp = lgg * diff;
        const float d = g[i] + comp;
        const float step = lr * d;
        const float w_new = w[i] - step;
        w[i] = w_new;
        w_bak_m[i] = w_new;
    }
    return 0;
}

// Eq. 6 then Eq. 5 at the server; mean_square is the server's single running average.
int oracle_dcasgd_step_a(const float* g, size_t n, float* w, float* w_bak_m, float* mean_square,
                         float lr, float lambda, float m, float eps)
{
    const float one_minus_m = 1.0f - m;
    for (size_t i = 0; i < n; ++i) {
        const float gg = g[i] * g[i];
        const float a = m * mean_square[i];
        const float b = one_minus_m * gg;
        const float ms = a + b;
        mean_square[i] = ms;
        const float den = std::sqrt(ms + eps);
        const float lam = lambda / den;
        const float diff = w[i] - w_bak_m[i];
        const float lgg = lam * gg;
        const float comp = lgg * diff;
        const float d = g[i] + comp;
        const float step = lr * d;
        const float w_new = w[i] - step;
        w[i] = w_new;
        w_bak_m[i] = w_new;
    }
    return 0;
}

// ---------------------------------------------------------------- fp64 twins
// Same rules, all arithmetic in binary64 on binary64 state.  Used only to
// bound the rounding error of the fp32 rules in the tests.
int oracle_global_update_f64(const double* const* grads, int n_workers, size_t n,
                             double* w, double* v, double* w_prev,
                             double lr, double momentum, double wd)
{
    if (n_workers < 1) return -1;
    for (size_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int m = 0; m < n_workers; ++m) s += grads[m][i];
        const double d = s / (double)n_workers + wd * w[i];
        const double v_new = momentum * v[i] - lr * d;
        if (w_prev) w_prev[i] = w[i];
        v[i] = v_new;
        w[i] = w[i] + v_new;
    }
    return 0;
}

int oracle_local_update_f64(const double* w_bak, const double* g, size_t n, double* x,
                            double local_lr)
{
    for (size_t i = 0; i < n; ++i) x[i] = w_bak[i] - local_lr * g[i];
    return 0;
}

int oracle_asgd_step_f64(const double* g, size_t n, double* w, double* v,
                         double lr, double momentum, double wd)
{
    for (size_t i = 0; i < n; ++i) {
        const double d = g[i] + wd * w[i];
        const double v_new = momentum * v[i] - lr * d;
        v[i] = v_new;
        w[i] = w[i] + v_new;
    }
    return 0;
}

}  // extern "C"
