// Direct gradient dL_meta/dtheta (the first factor of Eq. 1): mean cross-entropy of the base MLP on a
// clean batch, differentiated by hand.  This is the vector g_meta that the adaptation step (Eq. 4)
// consumes; computing it here makes the meta-gradient step self-contained on the device.
//
//   forward   h_l = relu(h_{l-1} W_l^T + b_l)            (activations kept, fp32)
//   dz_L      = (softmax(z_L) - onehot(y)) / B
//   dW_l      = dz_l^T h_{l-1},   db_l = column sums of dz_l
//   dz_{l-1}  = (dz_l W_l) * [h_{l-1} > 0]
//
// All four products are one fp32 FMA kernel with arbitrary operand strides, so that the contraction
// can run over the features (forward), over the outputs (dz W) or over the batch (dz^T h) without
// transposed copies.  Reductions have a fixed order: results are reproducible bit for bit.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int TB = 64;   // tile edge (M and N)
constexpr int TK = 16;   // k-block
constexpr int TPAD = 4;

struct StridedGemm {
    const float* A;   // element (m, k) at A[m * a_sm + k * a_sk]
    const float* B;   // element (n, k) at B[n * b_sn + k * b_sk]
    float* C;         // [M][ldc]
    const float* bias;  // [N] or null
    const float* mask;  // [M][ldm] or null: C is zeroed where mask <= 0
    int64_t a_sm, a_sk, b_sn, b_sk;
    int M, N, K, ldc, ldm, relu;
};

__global__ void __launch_bounds__(256)
gemm_strided_kernel(StridedGemm g) {
    pdl_trigger();
    pdl_wait();
    __shared__ __align__(16) float As[2][TK][TB + TPAD];
    __shared__ __align__(16) float Bs[2][TK][TB + TPAD];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * TB, n0 = blockIdx.x * TB;
    const bool a_kfast = (g.a_sk == 1), b_kfast = (g.b_sk == 1);
    float ra[4], rb[4];

    // Each thread stages 4 elements of each tile; consecutive threads walk the unit-stride direction.
    auto fetch = [&](const float* base, int64_t s_row, int64_t s_k, int row0, int rows, int k0, bool kfast, float* r) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int idx = tid + q * 256;
            const int row = kfast ? idx / TK : idx % TB;
            const int k = kfast ? idx % TK : idx / TB;
            const int gr = row0 + row, gk = k0 + k;
            r[q] = (gr < rows && gk < g.K) ? base[gr * s_row + gk * s_k] : 0.f;
        }
    };
    auto stash = [&](float (*S)[TB + TPAD], bool kfast, const float* r) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int idx = tid + q * 256;
            const int row = kfast ? idx / TK : idx % TB;
            const int k = kfast ? idx % TK : idx / TB;
            S[k][row] = r[q];
        }
    };

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    const int ktiles = (g.K + TK - 1) / TK;
    fetch(g.A, g.a_sm, g.a_sk, m0, g.M, 0, a_kfast, ra);
    fetch(g.B, g.b_sn, g.b_sk, n0, g.N, 0, b_kfast, rb);
    stash(As[0], a_kfast, ra);
    stash(Bs[0], b_kfast, rb);
    __syncthreads();
    for (int t = 0; t < ktiles; ++t) {
        const int buf = t & 1;
        if (t + 1 < ktiles) {
            fetch(g.A, g.a_sm, g.a_sk, m0, g.M, (t + 1) * TK, a_kfast, ra);
            fetch(g.B, g.b_sn, g.b_sk, n0, g.N, (t + 1) * TK, b_kfast, rb);
        }
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        if (t + 1 < ktiles) {
            stash(As[buf ^ 1], a_kfast, ra);
            stash(Bs[buf ^ 1], b_kfast, rb);
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= g.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= g.N) continue;
            float v = acc[i][j] + (g.bias ? g.bias[n] : 0.f);
            if (g.relu && v < 0.f) v = 0.f;
            if (g.mask && !(g.mask[(int64_t)m * g.ldm + n] > 0.f)) v = 0.f;
            g.C[(int64_t)m * g.ldc + n] = v;
        }
    }
}

// dz = (softmax(z) - onehot(y)) / B in place, per-sample loss to `loss`.  One warp per sample.
__global__ void __launch_bounds__(128)
softmax_grad_kernel(float* __restrict__ z, const int32_t* __restrict__ y, int B, int C, float* __restrict__ loss,
                    DeviceScalars* sc) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (i >= B) return;
    float* row = z + (int64_t)i * C;
    float mx = -INFINITY;
    for (int c = lane; c < C; c += 32) mx = fmaxf(mx, row[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = 0.f;
    for (int c = lane; c < C; c += 32) se += expf(row[c] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const int label = y[i];
    const bool ok = label >= 0 && label < C;
    if (!ok && lane == 0) atomicOr(&sc->status, (int)SAMA_DEV_BAD_LABEL);
    if (lane == 0) loss[i] = ok ? logf(se) + mx - row[label] : 0.f;
    __syncwarp();
    const float inv = 1.0f / se, invB = 1.0f / (float)B;
    for (int c = lane; c < C; c += 32) {
        const float p = expf(row[c] - mx) * inv;
        row[c] = ok ? (p - (c == label ? 1.f : 0.f)) * invB : 0.f;  // a bad label contributes nothing
    }
}

// out[j] = sum_i dz[i][j].  A block takes 32 columns; each of its 32 warps adds a contiguous share of the
// rows in row order (sixteen loads in flight), and the warps' sums are added in warp order: a fixed order, and
// enough rows in flight that the sweep is not a chain of B dependent loads per column.
constexpr int kColsumWarps = 32;
__global__ void __launch_bounds__(32 * kColsumWarps)
colsum_kernel(const float* __restrict__ dz, int B, int N, float* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    __shared__ float part[kColsumWarps][32];
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + lane;
    const int per = (B + kColsumWarps - 1) / kColsumWarps;
    const int i0 = grp * per, i1 = min(B, i0 + per);
    float s = 0.f;
    if (j < N) {
        const float* col = dz + j;
        int i = i0;
        for (; i + 15 < i1; i += 16) {
            float v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = col[(int64_t)(i + k) * N];
#pragma unroll
            for (int k = 0; k < 16; ++k) s += v[k];
        }
        for (; i < i1; ++i) s += col[(int64_t)i * N];
    }
    part[grp][lane] = s;
    __syncthreads();
    if (grp == 0 && j < N) {
        float t = 0.f;
#pragma unroll
        for (int k = 0; k < kColsumWarps; ++k) t += part[k][lane];
        out[j] = t;
    }
}

// *out = (1/B) sum_i loss[i], one block, fixed order.
__global__ void __launch_bounds__(256)
mean_kernel(const float* __restrict__ loss, int B, float* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    __shared__ double part[256];
    double s = 0.0;
    for (int i = threadIdx.x; i < B; i += 256) s += (double)loss[i];
    part[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int k = 0; k < 256; ++k) t += part[k];
        *out = (float)(t / (double)B);
    }
}

cudaError_t run_gemm(sama_ctx* ctx, const StridedGemm& g, int layer, cudaStream_t st) {
    dim3 grid((g.N + TB - 1) / TB, (g.M + TB - 1) / TB, 1);
    KernelScope scope(ctx, SAMA_K_META_GEMM, layer, st);
    return launch_dependent(gemm_strided_kernel, grid, dim3(256), 0, st, g);
}

}  // namespace

// Workspace layout (floats): activations h_1 .. h_{L-1} and logits, each [B][d_l]; two dz buffers
// [B][widest]; per-sample losses [B].
size_t meta_grad_workspace_floats(const sama_mlp_t* mlp, int64_t B) {
    size_t acts = 0, widest = 0;
    for (int l = 1; l <= mlp->n_layers; ++l) {
        acts += (size_t)mlp->dims[l];
        widest = (size_t)mlp->dims[l] > widest ? (size_t)mlp->dims[l] : widest;
    }
    for (int l = 0; l < mlp->n_layers; ++l) widest = (size_t)mlp->dims[l] > widest ? (size_t)mlp->dims[l] : widest;
    return (size_t)B * (acts + 2 * widest + 1);
}

namespace {

inline size_t r32(size_t x) { return (x + 31) & ~(size_t)31; }

// Operand buffers of the tensor-core path (floats; each region holds hi then lo).
struct TcPlan {
    size_t dzs;    // dz split            [B][r32(widest)]
    size_t wt;     // W_l^T split          [d_{l-1}][r32(d_l)], largest layer
    size_t tz;     // dz^T split           [widest][r32(B)]
    size_t th;     // h^T split            [widest][r32(B)]
    size_t total;
    size_t half_dzs, half_wt, half_t;
};
TcPlan tc_plan(const sama_mlp_t* mlp, int64_t B) {
    size_t widest = 0, wt = 0;
    for (int l = 0; l <= mlp->n_layers; ++l) widest = (size_t)mlp->dims[l] > widest ? (size_t)mlp->dims[l] : widest;
    for (int l = 0; l < mlp->n_layers; ++l) {
        const size_t e = (size_t)mlp->dims[l] * r32(mlp->dims[l + 1]);
        wt = e > wt ? e : wt;
    }
    TcPlan p;
    p.half_dzs = (size_t)B * r32(widest);
    p.half_wt = wt;
    p.half_t = widest * r32((size_t)B);
    p.dzs = 0;
    p.wt = p.dzs + 2 * p.half_dzs;
    p.tz = p.wt + 2 * p.half_wt;
    p.th = p.tz + 2 * p.half_t;
    p.total = p.th + 2 * p.half_t;
    return p;
}

}  // namespace

size_t meta_grad_tc_floats(const sama_mlp_t* mlp, int64_t B) { return tc_plan(mlp, B).total; }

// Same computation with every matrix product on the tensor cores (three TF32 products per fp32 product,
// as in the forward pass of the step): operands are split, and transposed where the contraction runs
// over the batch or the outputs, by small HBM-bound kernels.
static cudaError_t run_meta_grad_tc(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X,
                                    const int32_t* y, int32_t B, float* g_out, float* loss_out, cudaStream_t st) {
    const int L = mlp->n_layers;
    const SplitLayout lay = make_split_layout(mlp);
    const TcPlan plan = tc_plan(mlp, B);
    // On large models the small kernels of this chain (splits, transposes, column sums) are launched without
    // dependent-launch overlap: launched early they let the next persistent matrix product become resident
    // behind them, and its CTAs (which hold most of an SM's registers and shared memory) then starve the small
    // kernel's remaining waves.  Measured: 4096-4096-4096-1000, B = 2048: 2.86 ms with the overlap everywhere,
    // 2.4-2.6 ms with it on the matrix products only; the smaller workloads (whose small kernels fit in one
    // wave) are 3-20 % faster with the overlap everywhere.
    size_t widest_dim = 0;
    for (int l = 0; l <= L; ++l) widest_dim = (size_t)mlp->dims[l] > widest_dim ? (size_t)mlp->dims[l] : widest_dim;
    PdlScope overlap((size_t)B * widest_dim >= ((size_t)6 << 20) ? 0 : -1);
    size_t widest = 0;
    for (int l = 0; l <= L; ++l) widest = (size_t)mlp->dims[l] > widest ? (size_t)mlp->dims[l] : widest;
    // fp32 workspace: kept activations, dz ping-pong, losses (same carving as the FMA path)
    float* cur = ctx->mg_ws;
    const float* h[kMaxLayers + 1];
    float* hbuf[kMaxLayers + 1];
    h[0] = X;
    for (int l = 1; l <= L; ++l) {
        hbuf[l] = cur;
        h[l] = cur;
        cur += (size_t)B * mlp->dims[l];
    }
    float* dzb[2] = {cur, cur + (size_t)B * widest};
    float* losses = cur + 2 * (size_t)B * widest;
    float* tc = ctx->mg_tc;
    float* w_hi = ctx->w_split;
    float* w_lo = ctx->w_split + ctx->w_split_half;
    cudaError_t e;
    // forward: operands of theta and X, then one single-branch product per layer that keeps fp32 and
    // writes the next operand
    if ((e = launch_split_tf32(ctx, X, X, 1, B, mlp->dims[0], ctx->x_split, ctx->x_split + ctx->x_split_half, 0, st)) !=
        cudaSuccess)
        return e;
    for (int l = 0; l < L; ++l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        const bool last = (l + 1 == L);
        if ((e = launch_split_tf32(ctx, theta + lay.w_off[l], theta + lay.w_off[l], 1, dout, din, w_hi + lay.s_off[l],
                                   w_lo + lay.s_off[l], lay.slab, st)) != cudaSuccess)
            return e;
        TcLayer t;
        t.a_hi = l == 0 ? ctx->x_split : ctx->a_split[(l - 1) & 1];
        t.a_lo = l == 0 ? ctx->x_split + ctx->x_split_half : ctx->a_split[(l - 1) & 1] + ctx->a_split_half;
        t.w_hi = w_hi + lay.s_off[l];
        t.w_lo = w_lo + lay.s_off[l];
        t.w_slab = (int64_t)dout * lay.Kp[l];
        t.bias[0] = t.bias[1] = theta + lay.w_off[l] + lay.w_cnt[l];
        t.out_f32[0] = t.out_f32[1] = hbuf[l + 1];
        t.out_hi = last ? nullptr : ctx->a_split[l & 1];
        t.out_lo = last ? nullptr : ctx->a_split[l & 1] + ctx->a_split_half;
        t.M = B; t.N = dout; t.K = din; t.ldc = dout;
        t.relu = last ? 0 : 1; t.last = last ? 1 : 0; t.shared_a = 1; t.layer = l;
        t.branches = 1; t.both = last ? 0 : 1;
        if ((e = launch_gemm_tf32x3(ctx, t, st)) != cudaSuccess) return e;
    }
    const int C = mlp->dims[L];
    {
        KernelScope scope(ctx, SAMA_K_META_AUX, -1, st);
        if ((e = launch_dependent(softmax_grad_kernel, dim3((B + 3) / 4), dim3(128), 0, st, hbuf[L], y, (int)B, C,
                                  losses, ctx->scalars)) != cudaSuccess)
            return e;
    }
    if (loss_out) {
        KernelScope scope(ctx, SAMA_K_META_AUX, -1, st);
        if ((e = launch_dependent(mean_kernel, dim3(1), dim3(256), 0, st, (const float*)losses, (int)B, loss_out)) !=
            cudaSuccess)
            return e;
    }
    const float* dz = hbuf[L];
    const int Bp = (int)r32((size_t)B);
    for (int l = L - 1; l >= 0; --l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        // dW[dout][din] = dz^T h_{l}: both operands transposed so that the batch is the contraction index
        if ((e = launch_split_transpose_tf32(ctx, dz, B, dout, tc + plan.tz, tc + plan.tz + plan.half_t, st)) != cudaSuccess)
            return e;
        if ((e = launch_split_transpose_tf32(ctx, h[l], B, din, tc + plan.th, tc + plan.th + plan.half_t, st)) != cudaSuccess)
            return e;
        TcLayer tw;
        tw.a_hi = tc + plan.tz; tw.a_lo = tc + plan.tz + plan.half_t;
        tw.w_hi = tc + plan.th; tw.w_lo = tc + plan.th + plan.half_t;
        tw.w_slab = (int64_t)din * Bp;
        tw.bias[0] = tw.bias[1] = nullptr;
        tw.out_f32[0] = tw.out_f32[1] = g_out + lay.w_off[l];
        tw.out_hi = tw.out_lo = nullptr;
        tw.M = dout; tw.N = din; tw.K = B; tw.ldc = din;
        tw.relu = 0; tw.last = 1; tw.shared_a = 1; tw.layer = l; tw.branches = 1;
        if ((e = launch_gemm_tf32x3(ctx, tw, st)) != cudaSuccess) return e;
        {
            KernelScope scope(ctx, SAMA_K_META_AUX, l, st);
            if ((e = launch_dependent(colsum_kernel, dim3((dout + 31) / 32), dim3(32 * kColsumWarps), 0, st, dz, (int)B, dout,
                                      g_out + lay.w_off[l] + lay.w_cnt[l])) != cudaSuccess)
                return e;
        }
        if (l > 0) {
            // dz_{l-1}[B][din] = (dz W_l) masked by h_l > 0: W_l transposed so that its outputs are the contraction index
            if ((e = launch_split_tf32(ctx, dz, dz, 1, B, dout, tc + plan.dzs, tc + plan.dzs + plan.half_dzs, 0, st)) !=
                cudaSuccess)
                return e;
            if ((e = launch_split_transpose_tf32(ctx, theta + lay.w_off[l], dout, din, tc + plan.wt,
                                                 tc + plan.wt + plan.half_wt, st)) != cudaSuccess)
                return e;
            TcLayer th_;
            th_.a_hi = tc + plan.dzs; th_.a_lo = tc + plan.dzs + plan.half_dzs;
            th_.w_hi = tc + plan.wt; th_.w_lo = tc + plan.wt + plan.half_wt;
            th_.w_slab = (int64_t)din * (int64_t)r32((size_t)dout);
            th_.bias[0] = th_.bias[1] = nullptr;
            float* out = dzb[l & 1];
            th_.out_f32[0] = th_.out_f32[1] = out;
            th_.out_hi = th_.out_lo = nullptr;
            th_.M = B; th_.N = din; th_.K = dout; th_.ldc = din;
            th_.relu = 0; th_.last = 1; th_.shared_a = 1; th_.layer = l; th_.branches = 1;
            th_.mask = h[l]; th_.ldm = din;
            if ((e = launch_gemm_tf32x3(ctx, th_, st)) != cudaSuccess) return e;
            dz = out;
        }
    }
    return cudaSuccess;
}

static cudaError_t run_meta_grad_fma(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X,
                                     const int32_t* y, int32_t B, float* g_out, float* loss_out, cudaStream_t st) {
    const int L = mlp->n_layers;
    size_t widest = 0;
    for (int l = 0; l <= L; ++l) widest = (size_t)mlp->dims[l] > widest ? (size_t)mlp->dims[l] : widest;
    // carve the workspace
    float* ws = ctx->mg_ws;
    const float* h[kMaxLayers + 1];
    h[0] = X;
    float* cur = ws;
    float* hbuf[kMaxLayers + 1];
    for (int l = 1; l <= L; ++l) {
        hbuf[l] = cur;
        h[l] = cur;
        cur += (size_t)B * mlp->dims[l];
    }
    float* dzb[2] = {cur, cur + (size_t)B * widest};
    float* losses = cur + 2 * (size_t)B * widest;
    int64_t woff[kMaxLayers], boff[kMaxLayers];
    int64_t off = 0;
    for (int l = 0; l < L; ++l) {
        woff[l] = off;
        boff[l] = off + (int64_t)mlp->dims[l] * mlp->dims[l + 1];
        off = boff[l] + mlp->dims[l + 1];
    }
    cudaError_t e;
    // forward
    for (int l = 0; l < L; ++l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        StridedGemm g;
        g.A = h[l]; g.a_sm = din; g.a_sk = 1;
        g.B = theta + woff[l]; g.b_sn = din; g.b_sk = 1;
        g.C = hbuf[l + 1]; g.ldc = dout;
        g.bias = theta + boff[l];
        g.mask = nullptr; g.ldm = 0;
        g.M = B; g.N = dout; g.K = din;
        g.relu = (l + 1 < L) ? 1 : 0;
        if ((e = run_gemm(ctx, g, l, st)) != cudaSuccess) return e;
    }
    // dz_L in place over the logits
    const int C = mlp->dims[L];
    {
        KernelScope scope(ctx, SAMA_K_META_AUX, -1, st);
        if ((e = launch_dependent(softmax_grad_kernel, dim3((B + 3) / 4), dim3(128), 0, st, hbuf[L], y, (int)B, C,
                                  losses, ctx->scalars)) != cudaSuccess)
            return e;
    }
    if (loss_out) {
        KernelScope scope(ctx, SAMA_K_META_AUX, -1, st);
        if ((e = launch_dependent(mean_kernel, dim3(1), dim3(256), 0, st, (const float*)losses, (int)B, loss_out)) !=
            cudaSuccess)
            return e;
    }
    // backward
    const float* dz = hbuf[L];
    for (int l = L - 1; l >= 0; --l) {
        const int din = mlp->dims[l], dout = mlp->dims[l + 1];
        StridedGemm gw;  // dW[dout][din] = sum_i dz[i][dout] h_{l}[i][din]
        gw.A = dz; gw.a_sm = 1; gw.a_sk = dout;
        gw.B = h[l]; gw.b_sn = 1; gw.b_sk = din;
        gw.C = g_out + woff[l]; gw.ldc = din;
        gw.bias = nullptr; gw.mask = nullptr; gw.ldm = 0;
        gw.M = dout; gw.N = din; gw.K = B; gw.relu = 0;
        if ((e = run_gemm(ctx, gw, l, st)) != cudaSuccess) return e;
        {
            KernelScope scope(ctx, SAMA_K_META_AUX, l, st);
            if ((e = launch_dependent(colsum_kernel, dim3((dout + 31) / 32), dim3(32 * kColsumWarps), 0, st, dz, (int)B, dout,
                                      g_out + boff[l])) != cudaSuccess)
                return e;
        }
        if (l > 0) {
            StridedGemm gh;  // dh[B][din] = dz[B][dout] W[dout][din], masked by h_l > 0
            gh.A = dz; gh.a_sm = dout; gh.a_sk = 1;
            gh.B = theta + woff[l]; gh.b_sn = 1; gh.b_sk = din;
            float* out = dzb[l & 1];
            gh.C = out; gh.ldc = din;
            gh.bias = nullptr;
            gh.mask = h[l]; gh.ldm = din;
            gh.M = B; gh.N = din; gh.K = dout; gh.relu = 0;
            if ((e = run_gemm(ctx, gh, l, st)) != cudaSuccess) return e;
            dz = out;
        }
    }
    return cudaSuccess;
}

// Tensor cores unless the context is in fp32-FMA mode or the model does not fit the operand workspaces.
cudaError_t run_meta_grad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X, const int32_t* y,
                          int32_t B, float* g_out, float* loss_out, cudaStream_t st) {
    const int L = mlp->n_layers;
    bool fits = ctx->gemm_mode != 1 && ctx->mg_tc && tc_plan(mlp, B).total <= ctx->mg_tc_floats &&
                ctx->x_split_half >= (size_t)B * r32(mlp->dims[0]) &&
                (size_t)make_split_layout(mlp).slab <= ctx->w_split_half;
    for (int l = 0; l + 1 < L && fits; ++l) fits = 2 * (size_t)B * r32(mlp->dims[l + 1]) <= ctx->a_split_half * 2;
    if (fits) return run_meta_grad_tc(ctx, mlp, theta, X, y, B, g_out, loss_out, st);
    return run_meta_grad_fma(ctx, mlp, theta, X, y, B, g_out, loss_out, st);
}

}  // namespace sama
