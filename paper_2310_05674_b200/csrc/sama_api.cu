// Host side of the C ABI: argument validation, workspace, launch sequencing.
// Every step of the SAMA update runs in the kernels; nothing here computes on
// the CPU beyond the scalar constants of the Adam adaptation matrix.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "sama_internal.h"

using namespace sama;

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

inline int cuda_fail(sama_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    return SAMA_ERR_CUDA;
}
#define SAMA_CUDA(ctx, expr)                                   \
    do {                                                       \
        cudaError_t e__ = (expr);                              \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);  \
    } while (0)

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// true if [a, a+na) and [b, b+nb) share a byte
inline bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

}  // namespace

namespace sama {
int check_adam(const sama_adam_t* a, AdaptConsts* out) {
    if (!a) return SAMA_ERR_NULL;
    AdaptConsts c;
    std::memset(&c, 0, sizeof(c));
    c.identity = a->identity ? 1 : 0;
    c.drop_eps_term = a->drop_eps_term ? 1 : 0;
    if (!c.identity) {
        if (!(a->beta1 >= 0.f && a->beta1 < 1.f) || !(a->beta2 >= 0.f && a->beta2 < 1.f)) return SAMA_ERR_PARAM;
        if (!std::isfinite(a->lr) || !(a->lr > 0.f)) return SAMA_ERR_PARAM;
        if (!std::isfinite(a->eps) || !(a->eps >= 0.f)) return SAMA_ERR_PARAM;
        double c1 = 1.0, c2 = 1.0;
        if (a->bias_correction) {
            if (a->step < 1) return SAMA_ERR_PARAM;
            c1 = 1.0 - std::pow((double)a->beta1, (double)a->step);
            c2 = 1.0 - std::pow((double)a->beta2, (double)a->step);
            if (!(c1 > 0.0) || !(c2 > 0.0)) return SAMA_ERR_PARAM;
        }
        c.a = (float)((double)a->lr / c1);
        c.b1 = a->beta1;
        c.b2 = a->beta2;
        c.omb1 = (float)(1.0 - (double)a->beta1);
        c.omb2 = (float)(1.0 - (double)a->beta2);
        c.inv_rc2 = (float)(1.0 / std::sqrt(c2));
        c.eps = a->eps;
    }
    *out = c;
    return SAMA_OK;
}

int validate_adapt(int64_t max_n, int64_t n, const float* m, const float* s, const float* g_base,
                   const float* g_meta, const sama_adam_t* adam, float* p_out, double* sumsq_out,
                   AdaptConsts* c) {
    if (!adam || !g_meta || !p_out) return SAMA_ERR_NULL;
    const int rc = check_adam(adam, c);
    if (rc != SAMA_OK) return rc;
    if (!c->identity && (!m || !s)) return SAMA_ERR_NULL;
    if (n < 0 || n > max_n) return SAMA_ERR_SIZE;
    if (!aligned(m, 4) || !aligned(s, 4) || !aligned(g_base, 4) || !aligned(g_meta, 4) || !aligned(p_out, 4) ||
        !aligned(sumsq_out, 8))
        return SAMA_ERR_ALIGN;
    const size_t bytes = (size_t)n * 4;
    if (overlaps(p_out, bytes, m, bytes) || overlaps(p_out, bytes, s, bytes) ||
        overlaps(p_out, bytes, g_base, bytes) || overlaps(p_out, bytes, sumsq_out, 8))
        return SAMA_ERR_OVERLAP;
    if (p_out != g_meta && overlaps(p_out, bytes, g_meta, bytes)) return SAMA_ERR_OVERLAP;
    return SAMA_OK;
}

}  // namespace sama

namespace {

int check_mlp(const sama_mlp_t* mlp) {
    if (!mlp || !mlp->dims) return SAMA_ERR_NULL;
    if (mlp->n_layers < 1 || mlp->n_layers > kMaxLayers) return SAMA_ERR_SIZE;
    for (int l = 0; l <= mlp->n_layers; ++l)
        if (mlp->dims[l] < 1) return SAMA_ERR_SIZE;
    return SAMA_OK;
}

int validate_perturb(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* p_sumsq,
                     float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out,
                     bool outputs_optional = false) {
    if (!ctx || !theta || !p || (!outputs_optional && (!theta_plus || !theta_minus))) return SAMA_ERR_NULL;
    if (n < 0 || n > ctx->max_n) return SAMA_ERR_SIZE;
    if (!std::isfinite(alpha) || !(alpha > 0.f)) return SAMA_ERR_PARAM;
    if (!aligned(theta, 4) || !aligned(p, 4) || !aligned(theta_plus, 4) || !aligned(theta_minus, 4) ||
        !aligned(p_sumsq, 8) || !aligned(eps_fd_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t bytes = (size_t)n * 4;
    if (overlaps(theta_plus, bytes, theta_minus, bytes) || overlaps(theta_plus, bytes, theta, bytes) ||
        overlaps(theta_plus, bytes, p, bytes) || overlaps(theta_minus, bytes, p, bytes) ||
        overlaps(theta_plus, bytes, eps_fd_out, 4) || overlaps(theta_minus, bytes, eps_fd_out, 4) ||
        overlaps(theta_plus, bytes, p_sumsq, 8) || overlaps(theta_minus, bytes, p_sumsq, 8))
        return SAMA_ERR_OVERLAP;
    if (theta_minus != theta && overlaps(theta_minus, bytes, theta, bytes)) return SAMA_ERR_OVERLAP;
    return SAMA_OK;
}

int validate_fd(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta_plus, const float* theta_minus,
                const float* X, const int32_t* y, const float* lambda, int32_t B, const float* eps_fd,
                float* metagrad_out, float* loss_plus_out, float* loss_minus_out) {
    if (!ctx || !theta_plus || !theta_minus || !X || !y || !lambda || !metagrad_out) return SAMA_ERR_NULL;
    const int rc = check_mlp(mlp);
    if (rc != SAMA_OK) return rc;
    if (B < 1 || B > ctx->max_batch || ctx->max_classes == 0) return SAMA_ERR_SIZE;
    const int L = mlp->n_layers;
    for (int l = 1; l < L; ++l)
        if (mlp->dims[l] > ctx->max_width) return SAMA_ERR_SIZE;
    if (mlp->dims[L] > ctx->max_classes) return SAMA_ERR_SIZE;
    if (!aligned(theta_plus, 4) || !aligned(theta_minus, 4) || !aligned(X, 4) || !aligned(y, 4) ||
        !aligned(lambda, 4) || !aligned(eps_fd, 4) || !aligned(metagrad_out, 4) || !aligned(loss_plus_out, 4) ||
        !aligned(loss_minus_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t nb = (size_t)sama_mlp_param_count(mlp) * 4, bb = (size_t)B * 4;
    float* outs[3] = {metagrad_out, loss_plus_out, loss_minus_out};
    for (int i = 0; i < 3; ++i) {
        if (!outs[i]) continue;
        if (overlaps(outs[i], bb, theta_plus, nb) || overlaps(outs[i], bb, theta_minus, nb) ||
            overlaps(outs[i], bb, X, (size_t)B * mlp->dims[0] * 4) || overlaps(outs[i], bb, y, bb) ||
            overlaps(outs[i], bb, lambda, bb) || overlaps(outs[i], bb, eps_fd, 4))
            return SAMA_ERR_OVERLAP;
        for (int j = i + 1; j < 3; ++j)
            if (overlaps(outs[i], bb, outs[j], bb)) return SAMA_ERR_OVERLAP;
    }
    return SAMA_OK;
}

}  // namespace

namespace sama {
SplitLayout make_split_layout(const sama_mlp_t* mlp) {
    SplitLayout lay;
    std::memset(&lay, 0, sizeof(lay));
    lay.n_layers = mlp->n_layers;
    int64_t off = 0, soff = 0;
    for (int l = 0; l < mlp->n_layers; ++l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        lay.K[l] = din;
        lay.Kp[l] = (din + 31) & ~31;
        lay.w_off[l] = off;
        lay.w_cnt[l] = (int64_t)din * dout;
        lay.s_off[l] = soff;
        lay.N[l] = dout;
        off += (int64_t)din * dout + dout;
        soff += (int64_t)dout * lay.Kp[l];
    }
    lay.slab = soff;
    const int last = mlp->n_layers - 1;
    lay.head_layer = head_applicable(mlp->dims[last + 1]) ? last : -1;
    lay.head_cnt = lay.head_layer >= 0 ? lay.w_cnt[last] : 0;
    int64_t boff = lay.head_cnt;
    for (int l = 0; l < mlp->n_layers; ++l) {
        lay.b_off[l] = boff;
        boff += lay.N[l];
    }
    lay.small = (boff + 3) & ~(int64_t)3;
    return lay;
}

}  // namespace sama

namespace {

// Whether this model fits the operand-split workspace of the tensor-core path.
bool tc_fits(const sama_ctx* ctx, const sama_mlp_t* mlp, int32_t B) {
    auto r32 = [](int x) { return (size_t)((x + 31) & ~31); };
    const int L = mlp->n_layers;
    if (ctx->x_split_half == 0 || (size_t)B * r32(mlp->dims[0]) > ctx->x_split_half) return false;
    const SplitLayout lay = make_split_layout(mlp);
    if (2 * (size_t)lay.slab > ctx->w_split_half || (size_t)lay.small > ctx->pm_small_half) return false;
    for (int l = 0; l + 1 < L; ++l)
        if (2 * (size_t)B * r32(mlp->dims[l + 1]) > ctx->a_split_half) return false;
    return true;
}

// A single-layer model with a narrow output runs entirely in the fused head: no tensor-core product, no X split.
bool fused_head_only_model(const sama_mlp_t* mlp) {
    return mlp->n_layers == 1 && head_applicable(mlp->dims[1]);
}

// Layers of the tensor-core forward whose W operands the product kernel can form itself from theta and p
// (bit l set), given that the preconditions of the fused perturbation sweep hold (16-byte aligned theta and p,
// every weight block at a multiple of 4 with K % 4 == 0): every matrix-product layer with K >= 32 except a
// narrow last one, which takes the 16-wide tile.
uint32_t wfuse_mask(const sama_ctx* ctx, const sama_mlp_t* mlp) {
    if (ctx->gemm_mode != 3) return 0u;
    const bool fused_head = head_applicable(mlp->dims[mlp->n_layers]);
    const int L = fused_head ? mlp->n_layers - 1 : mlp->n_layers;
    uint32_t mask = 0u;
    for (int l = 0; l < L; ++l) {
        const bool narrow_last = (l + 1 == L) && mlp->dims[l + 1] <= 16;
        if (!narrow_last && mlp->dims[l] >= 32) mask |= 1u << l;
    }
    return mask;
}

// Forward pass of both branches on the tensor cores (3xTF32).  Operands are TF32 hi/lo pairs: X is split
// here, hidden activations by the epilogue that produces them, and the weights either by the fused
// perturbation sweep (w_presplit), or by the product kernel itself from theta and p (layers in `wfuse`, which
// implies w_presplit for the rest), or here, layer by layer.
int run_forward_tc(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta_plus, const float* theta_minus,
                   const float* X, int32_t B, bool w_presplit, bool x_presplit, bool fused_head, cudaStream_t st,
                   const float* theta0 = nullptr, const float* p = nullptr, uint32_t wfuse = 0u) {
    // with a fused head the last layer is not a matrix product here, and the layer before it
    // leaves fp32 activations (ReLU applied) in the context's activation buffer
    const int L = fused_head ? mlp->n_layers - 1 : mlp->n_layers;
    if (L == 0) return SAMA_OK;
    float* f32_out = fused_head ? ctx->act[0] : ctx->logits;
    const SplitLayout lay = make_split_layout(mlp);
    float* w_hi = ctx->w_split;
    float* w_lo = ctx->w_split + ctx->w_split_half;
    if (!x_presplit)
        SAMA_CUDA(ctx, launch_split_tf32(ctx, X, X, 1, B, mlp->dims[0], ctx->x_split,
                                         ctx->x_split + ctx->x_split_half, 0, st));
    for (int l = 0; l < L; ++l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        const bool last = (l + 1 == L);
        if (!w_presplit)
            SAMA_CUDA(ctx, launch_split_tf32(ctx, theta_plus + lay.w_off[l], theta_minus + lay.w_off[l], 2, dout, din,
                                             w_hi + lay.s_off[l], w_lo + lay.s_off[l], lay.slab, st));
        TcLayer t;
        if (l == 0) {
            t.a_hi = ctx->x_split;
            t.a_lo = ctx->x_split + ctx->x_split_half;
        } else {
            t.a_hi = ctx->a_split[(l - 1) & 1];
            t.a_lo = ctx->a_split[(l - 1) & 1] + ctx->a_split_half;
        }
        t.w_hi = w_hi + lay.s_off[l];
        t.w_lo = w_lo + lay.s_off[l];
        t.w_slab = lay.slab;
        if ((wfuse >> l) & 1u) {
            t.w_theta = theta0 + lay.w_off[l];
            t.w_p = p + lay.w_off[l];
            t.eps_fd = &ctx->scalars->eps_fd;
        }
        // biases: from the compact slab the fused perturbation sweep filled, else straight from theta+-
        t.bias[0] = w_presplit ? ctx->pm_small + lay.b_off[l] : theta_plus + lay.w_off[l] + lay.w_cnt[l];
        t.bias[1] = w_presplit ? ctx->pm_small + lay.small + lay.b_off[l] : theta_minus + lay.w_off[l] + lay.w_cnt[l];
        t.out_f32[0] = f32_out;
        t.out_f32[1] = f32_out + (int64_t)B * dout;
        t.out_hi = last ? nullptr : ctx->a_split[l & 1];
        t.out_lo = last ? nullptr : ctx->a_split[l & 1] + ctx->a_split_half;
        t.M = B;
        t.N = dout;
        t.K = din;
        t.ldc = dout;
        t.relu = (last && !fused_head) ? 0 : 1;
        t.last = last ? 1 : 0;
        t.shared_a = (l == 0) ? 1 : 0;
        t.layer = l;
        SAMA_CUDA(ctx, launch_gemm_tf32x3(ctx, t, st));
    }
    return SAMA_OK;
}

// The dual-branch forward and the finite difference, arguments already validated.
int run_fd(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta_plus, const float* theta_minus,
           const float* X, const int32_t* y, const float* lambda, int32_t B, const float* eps_fd,
           float* metagrad_out, float* loss_plus_out, float* loss_minus_out, cudaStream_t st,
           bool w_presplit = false, bool x_presplit = false, const float* theta0 = nullptr, const float* p = nullptr,
           uint32_t wfuse = 0u) {
    const int L = mlp->n_layers;
    const int C = mlp->dims[L];
    const bool fits = tc_fits(ctx, mlp, B);
    if (ctx->gemm_mode >= 2 && !fits) return SAMA_ERR_SIZE;
    const bool use_tc = ctx->gemm_mode != 1 && fits;
    ctx->last_forward_path = use_tc ? (wfuse ? 3 : 2) : 1;
    const bool fused_head = head_applicable(C);
    const float* eps = eps_fd ? eps_fd : &ctx->scalars->eps_fd;
    float* diff_out = ctx->rw_buf ? ctx->rw_buf + 4 * (size_t)ctx->max_batch : nullptr;
    const int n_gemm = fused_head ? L - 1 : L;  // layers computed as matrix products
    const float* in[2] = {X, X};                // fp32 input of the next stage
    int ld_in = mlp->dims[0];

    if (use_tc) {
        const int rc = run_forward_tc(ctx, mlp, theta_plus, theta_minus, X, B, w_presplit, x_presplit, fused_head, st,
                                      theta0, p, wfuse);
        if (rc != SAMA_OK) return rc;
        if (n_gemm > 0) {
            float* out = fused_head ? ctx->act[0] : ctx->logits;
            in[0] = out;
            in[1] = out + (int64_t)B * mlp->dims[n_gemm];
            ld_in = mlp->dims[n_gemm];
        }
    } else {
        int64_t off = 0;
        for (int l = 0; l < n_gemm; ++l) {
            const int din = mlp->dims[l], dout = mlp->dims[l + 1];
            const bool last = (l + 1 == L);
            float* out0 = last ? ctx->logits : ctx->act[l & 1];
            GemmArgs g;
            g.A[0] = in[0];
            g.A[1] = in[1];
            g.W[0] = theta_plus + off;
            g.W[1] = theta_minus + off;
            g.bias[0] = theta_plus + off + (int64_t)din * dout;
            g.bias[1] = theta_minus + off + (int64_t)din * dout;
            g.C[0] = out0;
            g.C[1] = out0 + (int64_t)B * dout;
            g.M = B;
            g.N = dout;
            g.K = din;
            g.lda = ld_in;
            g.ldw = din;
            g.ldc = dout;
            g.relu = last ? 0 : 1;
            g.layer = l;
            SAMA_CUDA(ctx, launch_gemm(ctx, g, st));
            in[0] = g.C[0];
            in[1] = g.C[1];
            ld_in = dout;
            off += (int64_t)din * dout + dout;
        }
    }
    if (fused_head) {
        int64_t off = 0;
        for (int l = 0; l + 1 < L; ++l) off += (int64_t)mlp->dims[l] * mlp->dims[l + 1] + mlp->dims[l + 1];
        const int K = mlp->dims[L - 1];
        // the head's fp32 weights and biases: from the compact slab after a fused perturbation sweep, else from theta+-
        const float* wp = theta_plus + off;
        const float* wm = theta_minus + off;
        const float* bp = wp + (int64_t)K * C;
        const float* bm = wm + (int64_t)K * C;
        if (use_tc && w_presplit) {
            const SplitLayout lay = make_split_layout(mlp);
            wp = ctx->pm_small;
            wm = ctx->pm_small + lay.small;
            bp = wp + lay.b_off[L - 1];
            bm = wm + lay.b_off[L - 1];
        }
        SAMA_CUDA(ctx, launch_head_ce_fd(ctx, in[0], in[1], ld_in, wp, wm, bp, bm, y,
                                         lambda, B, C, K, eps, metagrad_out, loss_plus_out, loss_minus_out, diff_out, st));
    } else {
        SAMA_CUDA(ctx, launch_ce_fd(ctx, in[0], in[1], C, y, lambda, B, C, eps, metagrad_out, loss_plus_out,
                                    loss_minus_out, diff_out, st));
    }
    return SAMA_OK;
}

}  // namespace

namespace sama {
thread_local int pdl_override = -1;
bool pdl_enabled() {
    static const bool on = []() { const char* e = std::getenv("SAMA_NO_PDL"); return !(e && e[0] == '1'); }();
    return on;
}
cudaError_t launch_gemm(sama_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
    return launch_gemm_ffma(ctx, g, st);
}
}  // namespace sama

extern "C" {

int64_t sama_mlp_param_count(const sama_mlp_t* mlp) {
    if (check_mlp(mlp) != SAMA_OK) return -1;
    int64_t n = 0;
    for (int l = 0; l < mlp->n_layers; ++l) n += (int64_t)mlp->dims[l] * mlp->dims[l + 1] + mlp->dims[l + 1];
    return n;
}

int sama_create(sama_ctx** out, int device, int64_t max_n, int32_t max_batch, const sama_mlp_t* mlp) {
    if (!out) return SAMA_ERR_NULL;
    *out = nullptr;
    if (max_n < 0 || max_batch < 0) return SAMA_ERR_SIZE;
    if (mlp) {
        const int rc = check_mlp(mlp);
        if (rc != SAMA_OK) return rc;
        if (max_batch < 1) return SAMA_ERR_SIZE;
    }
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return SAMA_ERR_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    sama_ctx* ctx = new (std::nothrow) sama_ctx();
    if (!ctx) return SAMA_ERR_NOMEM;
    std::memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->max_n = max_n;
    ctx->max_batch = max_batch;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return SAMA_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    if (const char* e = std::getenv("SAMA_NO_FUSED_SWEEP")) ctx->no_fused_sweep = (e[0] == '1');
    bool ok = cudaMalloc(&ctx->scalars, sizeof(DeviceScalars)) == cudaSuccess &&
              cudaMemset(ctx->scalars, 0, sizeof(DeviceScalars)) == cudaSuccess &&
              cudaMalloc(&ctx->partials, sizeof(double) * kMaxPartials) == cudaSuccess;
    if (ok && mlp) {
        const int L = mlp->n_layers;
        int width = 0;
        for (int l = 1; l < L; ++l) width = mlp->dims[l] > width ? mlp->dims[l] : width;
        ctx->max_width = width;
        ctx->max_classes = mlp->dims[L];
        if (width > 0) {
            const size_t bytes = sizeof(float) * 2 * (size_t)max_batch * width;
            ok = cudaMalloc(&ctx->act[0], bytes) == cudaSuccess && cudaMalloc(&ctx->act[1], bytes) == cudaSuccess;
        }
        ok = ok && cudaMalloc(&ctx->logits, sizeof(float) * 2 * (size_t)max_batch * ctx->max_classes) == cudaSuccess;
        // operand splits of the tensor-core path
        auto r32 = [](int x) { return (size_t)((x + 31) & ~31); };
        size_t amax = 0;
        for (int l = 0; l + 1 < L; ++l) {
            const size_t ae = r32(mlp->dims[l + 1]);
            amax = ae > amax ? ae : amax;
        }
        ctx->x_split_half = (size_t)max_batch * r32(mlp->dims[0]);
        ctx->w_split_half = 2 * (size_t)make_split_layout(mlp).slab;
        ctx->a_split_half = 2 * (size_t)max_batch * amax;
        ok = ok && cudaMalloc(&ctx->x_split, sizeof(float) * 2 * ctx->x_split_half) == cudaSuccess &&
             cudaMalloc(&ctx->w_split, sizeof(float) * 2 * ctx->w_split_half) == cudaSuccess;
        ctx->pm_small_half = (size_t)make_split_layout(mlp).small;
        ok = ok && cudaMalloc(&ctx->pm_small, sizeof(float) * 2 * ctx->pm_small_half) == cudaSuccess;
        ctx->tc_ws_floats = (size_t)ctx->sm_count * 128 * 256;
        ok = ok && cudaMalloc(&ctx->tc_ws, sizeof(float) * ctx->tc_ws_floats) == cudaSuccess &&
             cudaMalloc(&ctx->tc_flags, sizeof(int) * kTcFlags) == cudaSuccess &&
             cudaMemset(ctx->tc_flags, 0, sizeof(int) * kTcFlags) == cudaSuccess;
        ctx->mg_ws_floats = meta_grad_workspace_floats(mlp, max_batch);
        ok = ok && cudaMalloc(&ctx->mg_ws, sizeof(float) * ctx->mg_ws_floats) == cudaSuccess;
        ctx->mg_tc_floats = meta_grad_tc_floats(mlp, max_batch);
        ok = ok && cudaMalloc(&ctx->mg_tc, sizeof(float) * ctx->mg_tc_floats) == cudaSuccess;
        if (ok && amax > 0)
            ok = cudaMalloc(&ctx->a_split[0], sizeof(float) * 2 * ctx->a_split_half) == cudaSuccess &&
                 cudaMalloc(&ctx->a_split[1], sizeof(float) * 2 * ctx->a_split_half) == cudaSuccess;
        ok = ok && cudaMalloc(&ctx->rw_partials, sizeof(double) * (size_t)kMaxReweightBlocks *
                                                     (3 * kMaxReweightHidden + 1)) == cudaSuccess &&
             cudaMalloc(&ctx->rw_buf, sizeof(float) * 5 * (size_t)max_batch) == cudaSuccess &&
             cudaMemset(ctx->rw_buf, 0, sizeof(float) * 5 * (size_t)max_batch) == cudaSuccess;
        if (ok) {
            const cudaError_t e = tc_state_create(ctx);
            if (e != cudaSuccess) {
                ctx->last_cuda_error = (int)e;
                cudaGetLastError();
                sama_destroy(ctx);
                return SAMA_ERR_CUDA;
            }
        }
    }
    if (!ok || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        sama_destroy(ctx);
        return SAMA_ERR_NOMEM;
    }
    *out = ctx;
    return SAMA_OK;
}

int sama_destroy(sama_ctx* ctx) {
    if (!ctx) return SAMA_OK;
    DeviceGuard guard(ctx->device);
    cudaFree(ctx->scalars);
    cudaFree(ctx->partials);
    cudaFree(ctx->act[0]);
    cudaFree(ctx->act[1]);
    cudaFree(ctx->logits);
    cudaFree(ctx->x_split);
    cudaFree(ctx->w_split);
    cudaFree(ctx->a_split[0]);
    cudaFree(ctx->a_split[1]);
    cudaFree(ctx->tc_ws);
    cudaFree(ctx->tc_flags);
    cudaFree(ctx->mg_ws);
    cudaFree(ctx->mg_tc);
    cudaFree(ctx->stage);
    cudaFree(ctx->pm_small);
    cudaFree(ctx->pm_scratch);
    cudaFree(ctx->rw_partials);
    cudaFree(ctx->rw_buf);
    cudaFree(ctx->br_partials);
    tc_state_destroy(ctx);
    if (ctx->prof) {
        for (auto& r : ctx->prof->records) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
        delete ctx->prof;
    }
    delete ctx;
    return SAMA_OK;
}

int sama_adapt(sama_ctx* ctx, int64_t n, const float* m, const float* s, const float* g_base,
               const float* g_meta, const sama_adam_t* adam, float* p_out, double* sumsq_out, void* stream) {
    AdaptConsts c;
    if (!ctx) return SAMA_ERR_NULL;
    const int rc = validate_adapt(ctx->max_n, n, m, s, g_base, g_meta, adam, p_out, sumsq_out, &c);
    if (rc != SAMA_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    SAMA_CUDA(ctx, launch_adapt_sumsq(ctx, n, m, s, c.identity ? nullptr : g_base, g_meta, c, p_out, sumsq_out,
                                      (cudaStream_t)stream));
    return SAMA_OK;
}

int sama_perturb(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* p_sumsq,
                 float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out, void* stream) {
    const int rc = validate_perturb(ctx, n, theta, p, p_sumsq, alpha, theta_plus, theta_minus, eps_fd_out);
    if (rc != SAMA_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (!p_sumsq) {
        SAMA_CUDA(ctx, launch_sumsq(ctx, n, p, st));
        p_sumsq = &ctx->scalars->sumsq;
    }
    SAMA_CUDA(ctx, launch_perturb(ctx, n, theta, p, p_sumsq, alpha, theta_plus, theta_minus, eps_fd_out, st));
    return SAMA_OK;
}

int sama_fd_metagrad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta_plus, const float* theta_minus,
                     const float* X, const int32_t* y, const float* lambda, int32_t B, const float* eps_fd,
                     float* metagrad_out, float* loss_plus_out, float* loss_minus_out, void* stream) {
    const int rc = validate_fd(ctx, mlp, theta_plus, theta_minus, X, y, lambda, B, eps_fd, metagrad_out,
                               loss_plus_out, loss_minus_out);
    if (rc != SAMA_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    return run_fd(ctx, mlp, theta_plus, theta_minus, X, y, lambda, B, eps_fd, metagrad_out, loss_plus_out,
                  loss_minus_out, (cudaStream_t)stream);
}

int sama_step(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta, const float* m,
              const float* s, const float* g_base, const float* g_meta, const sama_adam_t* adam, float alpha,
              const float* X, const int32_t* y, const float* lambda, int32_t B,
              float* p_out, float* theta_plus, float* theta_minus, float* metagrad_out,
              float* loss_plus_out, float* loss_minus_out, void* stream) {
    if (!ctx) return SAMA_ERR_NULL;
    int rc = check_mlp(mlp);
    if (rc != SAMA_OK) return rc;
    if (n != sama_mlp_param_count(mlp)) return SAMA_ERR_SIZE;
    AdaptConsts c;
    rc = validate_adapt(ctx->max_n, n, m, s, g_base, g_meta, adam, p_out, nullptr, &c);
    if (rc != SAMA_OK) return rc;
    rc = validate_perturb(ctx, n, theta, p_out, nullptr, alpha, theta_plus, theta_minus, nullptr, true);
    if (rc != SAMA_OK) return rc;
    // (theta+- are optional here; the forward's own checks get stand-ins that overlap nothing)
    rc = validate_fd(ctx, mlp, theta_plus ? theta_plus : theta, theta_minus ? theta_minus : theta, X, y, lambda, B,
                     nullptr, metagrad_out, loss_plus_out, loss_minus_out);
    if (rc != SAMA_OK) return rc;
    // outputs of the early stages must not be inputs of the later ones
    const size_t nb = (size_t)n * 4, bb = (size_t)B * 4;
    const void* ins[6] = {m, s, g_base, X, lambda, y};
    const size_t inb[6] = {nb, nb, nb, (size_t)B * mlp->dims[0] * 4, bb, bb};
    for (int i = 0; i < 6; ++i)
        if (overlaps(theta_plus, nb, ins[i], inb[i]) || overlaps(theta_minus, nb, ins[i], inb[i]) ||
            (i >= 3 && overlaps(p_out, nb, ins[i], inb[i])))
            return SAMA_ERR_OVERLAP;
    if (overlaps(theta_plus, nb, g_meta, nb) || overlaps(theta_minus, nb, g_meta, nb) ||
        overlaps(p_out, nb, theta, nb))
        return SAMA_ERR_OVERLAP;
    float* outs[3] = {metagrad_out, loss_plus_out, loss_minus_out};
    for (int i = 0; i < 3; ++i)
        if (overlaps(outs[i], bb, p_out, nb) || overlaps(outs[i], bb, theta, nb) ||
            overlaps(outs[i], bb, g_meta, nb) || overlaps(outs[i], bb, m, nb) || overlaps(outs[i], bb, s, nb) ||
            overlaps(outs[i], bb, g_base, nb))
            return SAMA_ERR_OVERLAP;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // With the tensor-core forward, the perturbation sweep also emits the TF32 operand split of W+-.
    SplitLayout lay = make_split_layout(mlp);
    const bool fused = ctx->gemm_mode != 1 && tc_fits(ctx, mlp, B) &&
                       perturb_split_applicable(lay, theta, p_out, theta_plus, theta_minus);
    // ... except for the layers whose product kernel forms them itself from theta and p
    // (not when theta+ or theta- is written over theta, the in-place nudge: the products read theta after the sweep)
    const bool theta_kept = !overlaps(theta_plus, nb, theta, nb) && !overlaps(theta_minus, nb, theta, nb);
    const uint32_t wfuse = (fused && theta_kept) ? wfuse_mask(ctx, mlp) : 0u;
    lay.skip_w = wfuse;
    // ... and for a model small enough, adaptation and norm join it in one launch
    const bool one_launch = fused && aligned(g_meta, 16) && (c.identity || (aligned(m, 16) && aligned(s, 16))) &&
                            (c.identity || !g_base || aligned(g_base, 16)) && fused_sweep_applicable(ctx, n);
    if (!one_launch)
        SAMA_CUDA(ctx, launch_adapt_sumsq(ctx, n, m, s, c.identity ? nullptr : g_base, g_meta, c, p_out, nullptr, st));
    // ... and, where the batch allows vector access, the split of X as well (one launch fewer)
    XSplitJob xjob;
    std::memset(&xjob, 0, sizeof(xjob));
    const bool x_fused = fused && (mlp->dims[0] % 4 == 0) && aligned(X, 16) &&
                         !(fused_head_only_model(mlp));
    if (x_fused) {
        xjob.x = X;
        xjob.hi = ctx->x_split;
        xjob.lo = ctx->x_split + ctx->x_split_half;
        xjob.rows = B;
        xjob.cols = mlp->dims[0];
        xjob.ld_out = (mlp->dims[0] + 31) & ~31;
    }
    bool swept = false;
    if (one_launch) {
        const cudaError_t e = launch_fused_sweep(ctx, n, theta, m, s, c.identity ? nullptr : g_base, g_meta, c, alpha,
                                                 p_out, theta_plus, theta_minus, lay, ctx->w_split,
                                                 ctx->w_split + ctx->w_split_half, ctx->pm_small, xjob, st);
        if (e == cudaSuccess) {
            swept = true;
        } else {
            // a cooperative launch the device would not take (its blocks must all be resident): nothing has run;
            // remember that, and take the two launches from here on
            cudaGetLastError();
            ctx->fused_sweep_blocks = -1;
            SAMA_CUDA(ctx, launch_adapt_sumsq(ctx, n, m, s, c.identity ? nullptr : g_base, g_meta, c, p_out, nullptr, st));
        }
    }
    if (swept) {
    } else if (fused) {
        SAMA_CUDA(ctx, launch_perturb_split(ctx, n, theta, p_out, &ctx->scalars->sumsq, alpha, theta_plus,
                                            theta_minus, nullptr, lay, ctx->w_split,
                                            ctx->w_split + ctx->w_split_half, ctx->pm_small, xjob, st));
    } else {
        // this path's forward reads theta+- themselves: a caller that wants neither gets them in scratch
        if (!theta_plus || !theta_minus) {
            const size_t nn = ((size_t)n + 63) & ~(size_t)63;
            if (ctx->pm_scratch_floats < 2 * nn) {
                SAMA_CUDA(ctx, cudaStreamSynchronize(st));
                cudaFree(ctx->pm_scratch);
                ctx->pm_scratch = nullptr;
                ctx->pm_scratch_floats = 0;
                if (cudaMalloc(&ctx->pm_scratch, sizeof(float) * 2 * nn) != cudaSuccess) { cudaGetLastError(); return SAMA_ERR_NOMEM; }
                ctx->pm_scratch_floats = 2 * nn;
            }
            if (!theta_plus) theta_plus = ctx->pm_scratch;
            if (!theta_minus) theta_minus = ctx->pm_scratch + nn;
        }
        SAMA_CUDA(ctx, launch_perturb(ctx, n, theta, p_out, &ctx->scalars->sumsq, alpha, theta_plus, theta_minus,
                                      nullptr, st));
    }
    return run_fd(ctx, mlp, theta_plus, theta_minus, X, y, lambda, B, nullptr, metagrad_out, loss_plus_out,
                  loss_minus_out, st, fused, x_fused, theta, p_out, wfuse);
}

int sama_fd_metagrad_reweight(sama_ctx* ctx, int32_t B, const float* loss_plus, const float* loss_minus,
                              const float* loss_diff, int32_t hidden, const float* lambda_r, const float* eps_fd,
                              int32_t B_norm, float* metagrad_r_out, void* stream) {
    if (!ctx || !loss_minus || (!loss_plus && !loss_diff) || !lambda_r || !metagrad_r_out) return SAMA_ERR_NULL;
    if (!ctx->rw_partials || B < 1 || B > ctx->max_batch || B_norm < 1 || hidden < 1 || hidden > kMaxReweightHidden)
        return SAMA_ERR_SIZE;
    if (!aligned(loss_plus, 4) || !aligned(loss_minus, 4) || !aligned(loss_diff, 4) || !aligned(lambda_r, 4) ||
        !aligned(eps_fd, 4) || !aligned(metagrad_r_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t bb = (size_t)B * 4, lb = (size_t)(3 * hidden + 1) * 4;
    if (overlaps(metagrad_r_out, lb, loss_plus, bb) || overlaps(metagrad_r_out, lb, loss_minus, bb) ||
        overlaps(metagrad_r_out, lb, loss_diff, bb) ||
        overlaps(metagrad_r_out, lb, lambda_r, lb) || overlaps(metagrad_r_out, lb, eps_fd, 4))
        return SAMA_ERR_OVERLAP;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    SAMA_CUDA(ctx, launch_reweight_fd(ctx, loss_plus, loss_minus, loss_diff, B, B_norm, hidden, lambda_r,
                                      eps_fd ? eps_fd : &ctx->scalars->eps_fd, metagrad_r_out, (cudaStream_t)stream));
    return SAMA_OK;
}

int sama_step_reweight(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta, const float* m,
                       const float* s, const float* g_base, const float* g_meta, const sama_adam_t* adam,
                       float alpha, const float* X, const int32_t* y, int32_t B, int32_t hidden,
                       const float* lambda_r, float* p_out, float* theta_plus, float* theta_minus,
                       float* metagrad_r_out, float* loss_plus_out, float* loss_minus_out, void* stream) {
    if (!ctx || !lambda_r || !metagrad_r_out) return SAMA_ERR_NULL;
    if (!ctx->rw_buf || B < 1 || B > ctx->max_batch || hidden < 1 || hidden > kMaxReweightHidden) return SAMA_ERR_SIZE;
    if (!aligned(lambda_r, 4) || !aligned(metagrad_r_out, 4)) return SAMA_ERR_ALIGN;
    const size_t nb = (size_t)(n > 0 ? n : 0) * 4, lb = (size_t)(3 * hidden + 1) * 4;
    if (overlaps(metagrad_r_out, lb, p_out, nb) || overlaps(metagrad_r_out, lb, theta_plus, nb) ||
        overlaps(metagrad_r_out, lb, theta_minus, nb) || overlaps(metagrad_r_out, lb, lambda_r, lb) ||
        overlaps(metagrad_r_out, lb, loss_plus_out, (size_t)B * 4) || overlaps(metagrad_r_out, lb, loss_minus_out, (size_t)B * 4) ||
        overlaps(lambda_r, lb, p_out, nb) || overlaps(lambda_r, lb, theta_plus, nb) || overlaps(lambda_r, lb, theta_minus, nb))
        return SAMA_ERR_OVERLAP;
    // the forward pass and its per-sample losses are those of sama_step; the per-sample logits it wants are the
    // context's zeros and its per-sample meta gradient goes to scratch
    float* lp = loss_plus_out ? loss_plus_out : ctx->rw_buf;
    float* lm = loss_minus_out ? loss_minus_out : ctx->rw_buf + ctx->max_batch;
    const float* zeros = ctx->rw_buf + 2 * (size_t)ctx->max_batch;
    float* scratch = ctx->rw_buf + 3 * (size_t)ctx->max_batch;
    const int rc = sama_step(ctx, mlp, n, theta, m, s, g_base, g_meta, adam, alpha, X, y, zeros, B, p_out, theta_plus,
                             theta_minus, scratch, lp, lm, stream);
    if (rc != SAMA_OK) return rc;
    return sama_fd_metagrad_reweight(ctx, B, lp, lm, ctx->rw_buf + 4 * (size_t)ctx->max_batch, hidden, lambda_r, nullptr, B,
                                     metagrad_r_out, stream);
}

int sama_biasreg_direct_grad(sama_ctx* ctx, int32_t d, int32_t n_val, const float* Xv, const float* yv,
                             const float* w, float* g_meta_out, float* meta_loss_out, void* stream) {
    if (!ctx || !Xv || !yv || !w || !g_meta_out) return SAMA_ERR_NULL;
    if (d < 1 || n_val < 1 || d > 24 * 1024 || (int64_t)d > ctx->max_n) return SAMA_ERR_SIZE;
    if (!aligned(Xv, 4) || !aligned(yv, 4) || !aligned(w, 4) || !aligned(g_meta_out, 4) || !aligned(meta_loss_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t db = (size_t)d * 4;
    if (overlaps(g_meta_out, db, Xv, (size_t)n_val * d * 4) || overlaps(g_meta_out, db, yv, (size_t)n_val * 4) ||
        overlaps(g_meta_out, db, w, db) || overlaps(g_meta_out, db, meta_loss_out, 4))
        return SAMA_ERR_OVERLAP;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // the row chunks' partial gradients, then the residuals
    const size_t need = (size_t)biasreg_grid(ctx, n_val) * ((size_t)d + 1) + (size_t)n_val;
    if (ctx->br_partials_doubles < need) {
        SAMA_CUDA(ctx, cudaStreamSynchronize(st));
        cudaFree(ctx->br_partials);
        ctx->br_partials = nullptr;
        ctx->br_partials_doubles = 0;
        const size_t take = 2 * (size_t)ctx->sm_count * ((size_t)d + 1) + (size_t)n_val;
        if (cudaMalloc(&ctx->br_partials, sizeof(double) * take) != cudaSuccess) { cudaGetLastError(); return SAMA_ERR_NOMEM; }
        ctx->br_partials_doubles = take;
    }
    SAMA_CUDA(ctx, launch_biasreg_direct_grad(ctx, d, n_val, Xv, yv, w, g_meta_out, meta_loss_out, st));
    return SAMA_OK;
}

int sama_biasreg_fd_metagrad(sama_ctx* ctx, int64_t d, const float* w_plus, const float* w_minus,
                             const float* lambda, float beta, const float* eps_fd, float* metagrad_out,
                             void* stream) {
    if (!ctx || !w_plus || !w_minus || !lambda || !metagrad_out) return SAMA_ERR_NULL;
    if (d < 0 || d > ctx->max_n) return SAMA_ERR_SIZE;
    if (!std::isfinite(beta) || !(beta >= 0.f)) return SAMA_ERR_PARAM;
    if (!aligned(w_plus, 4) || !aligned(w_minus, 4) || !aligned(lambda, 4) || !aligned(eps_fd, 4) ||
        !aligned(metagrad_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t db = (size_t)d * 4;
    if (overlaps(metagrad_out, db, w_plus, db) || overlaps(metagrad_out, db, w_minus, db) ||
        overlaps(metagrad_out, db, lambda, db) || overlaps(metagrad_out, db, eps_fd, 4))
        return SAMA_ERR_OVERLAP;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    SAMA_CUDA(ctx, launch_biasreg_fd(ctx, d, w_plus, w_minus, lambda, beta, eps_fd ? eps_fd : &ctx->scalars->eps_fd,
                                     metagrad_out, (cudaStream_t)stream));
    return SAMA_OK;
}

int sama_biasreg_step(sama_ctx* ctx, int32_t d, int32_t n_val, const float* Xv, const float* yv, const float* w,
                      const float* lambda, float beta, const float* m, const float* s, const float* g_base,
                      const sama_adam_t* adam, float alpha, float* g_meta_out, float* p_out, float* w_plus,
                      float* w_minus, float* metagrad_out, void* stream) {
    if (!ctx || !lambda || !metagrad_out || !p_out || !w_plus || !w_minus || !adam) return SAMA_ERR_NULL;
    // the four stages validate their own arguments; what only the chain can get wrong is checked here
    const size_t db = (size_t)(d > 0 ? d : 0) * 4;
    if (overlaps(metagrad_out, db, p_out, db) || overlaps(metagrad_out, db, g_meta_out, db) ||
        overlaps(w_plus, db, g_meta_out, db) || overlaps(w_minus, db, g_meta_out, db) ||
        overlaps(p_out, db, lambda, db) || overlaps(w_plus, db, lambda, db) || overlaps(w_minus, db, lambda, db))
        return SAMA_ERR_OVERLAP;
    int rc = sama_biasreg_direct_grad(ctx, d, n_val, Xv, yv, w, g_meta_out, nullptr, stream);
    if (rc != SAMA_OK) return rc;
    rc = sama_adapt(ctx, d, m, s, g_base, g_meta_out, adam, p_out, nullptr, stream);
    if (rc != SAMA_OK) return rc;
    rc = sama_perturb(ctx, d, w, p_out, &ctx->scalars->sumsq, alpha, w_plus, w_minus, nullptr, stream);
    if (rc != SAMA_OK) return rc;
    return sama_biasreg_fd_metagrad(ctx, d, w_plus, w_minus, lambda, beta, nullptr, metagrad_out, stream);
}

int sama_meta_grad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X_meta,
                   const int32_t* y_meta, int32_t B, float* g_meta_out, float* loss_out, void* stream) {
    if (!ctx || !theta || !X_meta || !y_meta || !g_meta_out) return SAMA_ERR_NULL;
    const int rc = check_mlp(mlp);
    if (rc != SAMA_OK) return rc;
    if (B < 1 || B > ctx->max_batch || !ctx->mg_ws) return SAMA_ERR_SIZE;
    if (meta_grad_workspace_floats(mlp, B) > ctx->mg_ws_floats) return SAMA_ERR_SIZE;
    if (!aligned(theta, 4) || !aligned(X_meta, 4) || !aligned(y_meta, 4) || !aligned(g_meta_out, 4) ||
        !aligned(loss_out, 4))
        return SAMA_ERR_ALIGN;
    const size_t nb = (size_t)sama_mlp_param_count(mlp) * 4, bb = (size_t)B * 4;
    if (overlaps(g_meta_out, nb, theta, nb) || overlaps(g_meta_out, nb, X_meta, (size_t)B * mlp->dims[0] * 4) ||
        overlaps(g_meta_out, nb, y_meta, bb) || overlaps(g_meta_out, nb, loss_out, 4) ||
        overlaps(loss_out, 4, theta, nb) || overlaps(loss_out, 4, X_meta, (size_t)B * mlp->dims[0] * 4))
        return SAMA_ERR_OVERLAP;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    SAMA_CUDA(ctx, run_meta_grad(ctx, mlp, theta, X_meta, y_meta, B, g_meta_out, loss_out, (cudaStream_t)stream));
    return SAMA_OK;
}

int sama_step_host(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta_host, const float* m_host,
                   const float* s_host, const float* g_base_host, const float* g_meta_host,
                   const sama_adam_t* adam, float alpha, const float* X_host, const int32_t* y_host,
                   const float* lambda_host, int32_t B, float* metagrad_out_host, float* eps_fd_out_host,
                   float* theta_minus_out_host, void* stream) {
    if (!ctx || !theta_host || !g_meta_host || !X_host || !y_host || !lambda_host || !metagrad_out_host || !adam)
        return SAMA_ERR_NULL;
    int rc = check_mlp(mlp);
    if (rc != SAMA_OK) return rc;
    if (n != sama_mlp_param_count(mlp) || n > ctx->max_n || B < 1 || B > ctx->max_batch) return SAMA_ERR_SIZE;
    if (!adam->identity && (!m_host || !s_host)) return SAMA_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // staging layout (floats): theta m s g_base g_meta p theta- | X | lambda | metagrad | y
    const size_t nn = ((size_t)n + 63) & ~(size_t)63;
    const size_t xs = (((size_t)B * mlp->dims[0]) + 63) & ~(size_t)63;
    const size_t bs = ((size_t)B + 63) & ~(size_t)63;
    const size_t need = (7 * nn + xs + 3 * bs) * sizeof(float);
    if (ctx->stage_bytes < need) {
        SAMA_CUDA(ctx, cudaStreamSynchronize(st));
        cudaFree(ctx->stage);
        ctx->stage = nullptr;
        ctx->stage_bytes = 0;
        if (cudaMalloc(&ctx->stage, need) != cudaSuccess) { cudaGetLastError(); return SAMA_ERR_NOMEM; }
        ctx->stage_bytes = need;
    }
    float* d_theta = ctx->stage;
    float* d_m = d_theta + nn;
    float* d_s = d_m + nn;
    float* d_g = d_s + nn;
    float* d_gm = d_g + nn;
    float* d_p = d_gm + nn;
    float* d_tm = d_p + nn;
    float* d_X = d_tm + nn;
    float* d_lam = d_X + xs;
    float* d_mg = d_lam + bs;
    int32_t* d_y = reinterpret_cast<int32_t*>(d_mg + bs);
    const size_t nb = (size_t)n * 4;
    SAMA_CUDA(ctx, cudaMemcpyAsync(d_theta, theta_host, nb, cudaMemcpyHostToDevice, st));
    if (m_host) SAMA_CUDA(ctx, cudaMemcpyAsync(d_m, m_host, nb, cudaMemcpyHostToDevice, st));
    if (s_host) SAMA_CUDA(ctx, cudaMemcpyAsync(d_s, s_host, nb, cudaMemcpyHostToDevice, st));
    if (g_base_host) SAMA_CUDA(ctx, cudaMemcpyAsync(d_g, g_base_host, nb, cudaMemcpyHostToDevice, st));
    SAMA_CUDA(ctx, cudaMemcpyAsync(d_gm, g_meta_host, nb, cudaMemcpyHostToDevice, st));
    SAMA_CUDA(ctx, cudaMemcpyAsync(d_X, X_host, (size_t)B * mlp->dims[0] * 4, cudaMemcpyHostToDevice, st));
    SAMA_CUDA(ctx, cudaMemcpyAsync(d_y, y_host, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    SAMA_CUDA(ctx, cudaMemcpyAsync(d_lam, lambda_host, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    rc = sama_step(ctx, mlp, n, d_theta, m_host ? d_m : nullptr, s_host ? d_s : nullptr,
                   g_base_host ? d_g : nullptr, d_gm, adam, alpha, d_X, d_y, d_lam, B, d_p, nullptr,
                   theta_minus_out_host ? d_tm : nullptr, d_mg, nullptr, nullptr, stream);
    if (rc != SAMA_OK) return rc;
    SAMA_CUDA(ctx, cudaMemcpyAsync(metagrad_out_host, d_mg, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    if (eps_fd_out_host)
        SAMA_CUDA(ctx, cudaMemcpyAsync(eps_fd_out_host, &ctx->scalars->eps_fd, 4, cudaMemcpyDeviceToHost, st));
    if (theta_minus_out_host)
        SAMA_CUDA(ctx, cudaMemcpyAsync(theta_minus_out_host, d_tm, nb, cudaMemcpyDeviceToHost, st));
    SAMA_CUDA(ctx, cudaStreamSynchronize(st));
    return SAMA_OK;
}

double* sama_ctx_sumsq(sama_ctx* ctx) { return ctx ? &ctx->scalars->sumsq : nullptr; }
float* sama_ctx_loss_diff(sama_ctx* ctx) { return (ctx && ctx->rw_buf) ? ctx->rw_buf + 4 * (size_t)ctx->max_batch : nullptr; }
float* sama_ctx_eps_fd(sama_ctx* ctx) { return ctx ? &ctx->scalars->eps_fd : nullptr; }

int sama_device_status(sama_ctx* ctx, void* stream, int32_t* status_out) {
    if (!ctx || !status_out) return SAMA_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t v = 0;
    SAMA_CUDA(ctx, cudaMemcpyAsync(&v, &ctx->scalars->status, 4, cudaMemcpyDeviceToHost, st));
    SAMA_CUDA(ctx, cudaMemsetAsync(&ctx->scalars->status, 0, 4, st));
    SAMA_CUDA(ctx, cudaStreamSynchronize(st));
    *status_out = v;
    return SAMA_OK;
}

int sama_selftest_wait_expiry(sama_ctx* ctx, int64_t limit_cycles, int64_t* waited_cycles_out, void* stream) {
    if (!ctx) return SAMA_ERR_NULL;
    if (limit_cycles < 1 || limit_cycles > (int64_t)2000000000) return SAMA_ERR_PARAM;   // at most about a second
    if (!aligned(waited_cycles_out, 8)) return SAMA_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    SAMA_CUDA(ctx, launch_wait_expiry(ctx, (long long)limit_cycles, reinterpret_cast<long long*>(waited_cycles_out),
                                      (cudaStream_t)stream));
    return SAMA_OK;
}

int sama_last_cuda_error(sama_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int sama_set_gemm_mode(sama_ctx* ctx, int mode) {
    if (!ctx) return SAMA_ERR_NULL;
    if (mode < 0 || mode > 3) return SAMA_ERR_PARAM;
    ctx->gemm_mode = mode;
    return SAMA_OK;
}

int64_t sama_launch_count(sama_ctx* ctx) { return ctx ? ctx->launches : 0; }

int sama_last_forward_path(sama_ctx* ctx) { return ctx ? ctx->last_forward_path : 0; }

int sama_profile_enable(sama_ctx* ctx, int32_t on) {
    if (!ctx) return SAMA_ERR_NULL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    if (!ctx->prof) {
        ctx->prof = new (std::nothrow) Profiler();
        if (!ctx->prof) return SAMA_ERR_NOMEM;
    }
    for (auto& r : ctx->prof->records) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    ctx->prof->records.clear();
    ctx->prof->on = (on != 0);
    ctx->prof->grouped = (on == 2);
    return SAMA_OK;
}

int sama_profile_collect(sama_ctx* ctx, sama_kernel_time_t* out, int32_t capacity, int32_t* count_out) {
    if (!ctx || !count_out || (capacity > 0 && !out)) return SAMA_ERR_NULL;
    *count_out = 0;
    if (!ctx->prof) return SAMA_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SAMA_ERR_CUDA;
    int32_t k = 0;
    for (auto& r : ctx->prof->records) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(r.stop);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.start, r.stop);
        cudaEventDestroy(r.start);
        cudaEventDestroy(r.stop);
        if (e != cudaSuccess) { ctx->prof->records.clear(); return cuda_fail(ctx, e); }
        if (k < capacity) { out[k].kind = r.kind; out[k].layer = r.layer; out[k].ms = ms; out[k].launches = r.launches; ++k; }
    }
    ctx->prof->records.clear();
    *count_out = k;
    return SAMA_OK;
}

const char* sama_status_string(int status) {
    switch (status) {
        case SAMA_OK: return "ok";
        case SAMA_ERR_NULL: return "a required pointer is NULL";
        case SAMA_ERR_ALIGN: return "a pointer is not aligned to its element type";
        case SAMA_ERR_SIZE: return "a size is negative, inconsistent or beyond the context's limits";
        case SAMA_ERR_PARAM: return "a scalar parameter is out of range or not finite";
        case SAMA_ERR_OVERLAP: return "buffers overlap in a way that is not allowed";
        case SAMA_ERR_CUDA: return "a CUDA runtime call failed";
        case SAMA_ERR_NOMEM: return "workspace allocation failed";
        case SAMA_ERR_UNSUPPORTED: return "not supported by this build";
        default: return "unknown status";
    }
}

}  // extern "C"
