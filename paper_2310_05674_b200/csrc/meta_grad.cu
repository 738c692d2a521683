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

// out[j] = sum_i dz[i][j], rows added in order; one thread per column.
__global__ void __launch_bounds__(256)
colsum_kernel(const float* __restrict__ dz, int B, int N, float* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= N) return;
    float s = 0.f;
    for (int i = 0; i < B; ++i) s += dz[(int64_t)i * N + j];
    out[j] = s;
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

cudaError_t run_meta_grad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X, const int32_t* y,
                          int32_t B, float* g_out, float* loss_out, cudaStream_t st) {
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
            if ((e = launch_dependent(colsum_kernel, dim3((dout + 255) / 256), dim3(256), 0, st, dz, (int)B, dout,
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

}  // namespace sama
