// SAMA on the biased-regression problem of Appendix E:
//   L_meta(w)         = || X' w - y' ||^2
//   L_base(w, lambda) = || X w - y ||^2 + beta || w - lambda ||^2
// Two kernels, both specific to this objective; adaptation, norm and perturbation are the library's own.
//
//   direct gradient (Eq. 1):  g_meta = dL_meta/dw = 2 X'^T (X' w - y')
//   central difference (Eq. 5) of g_lambda(w) = dL_base/dlambda = -2 beta (w - lambda):
//                             metagrad = -[g_lambda(w+) - g_lambda(w-)] / (2 eps_fd)
//
// The direct gradient reads X' once from HBM: a block takes a contiguous run of rows, eight at a time; each warp
// forms one residual r_i = x_i . w - y_i, then all threads add r_i x_i into the block's partial gradient in
// shared memory (the rows come back from L1 / L2).  A second small kernel adds the blocks' partials column by
// column in block order.  Accumulation is double throughout; nothing depends on scheduling.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kThreads = 256;
constexpr int kRows = kThreads / 32;  // rows in flight per block = warps

// VEC: d % 4 == 0 and 16-byte aligned X', w: 16-byte loads, four times as many bytes in flight per thread.
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
biasreg_partials_kernel(int d, int n_val, const float* __restrict__ Xv, const float* __restrict__ yv,
                        const float* __restrict__ w, double* __restrict__ partials) {
    extern __shared__ double g_s[];        // [d] partial gradient, then [kRows] residuals
    double* r_s = g_s + d;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c = threadIdx.x; c < d; c += kThreads) g_s[c] = 0.0;
    // this block's rows: a contiguous run, the same for every launch of this shape
    const int per = (n_val + gridDim.x - 1) / gridDim.x;
    const int row0 = blockIdx.x * per, row1 = min(n_val, row0 + per);
    double sq = 0.0;                        // sum of r_i^2 over this warp's rows (lane 0)
    __syncthreads();
    for (int base = row0; base < row1; base += kRows) {
        const int i = base + warp;
        double r = 0.0;
        if (i < row1) {
            const float* x = Xv + (int64_t)i * d;
            double r0 = 0.0, r1 = 0.0, r2 = 0.0, r3 = 0.0;   // four independent chains
            if (VEC) {
                const float4* x4 = reinterpret_cast<const float4*>(x);
                const float4* w4 = reinterpret_cast<const float4*>(w);
                const int q = d >> 2;
                int c = lane;
                for (; c + 96 < q; c += 128) {
                    const float4 a0 = __ldg(x4 + c), a1 = __ldg(x4 + c + 32), a2 = __ldg(x4 + c + 64), a3 = __ldg(x4 + c + 96);
                    const float4 b0 = __ldg(w4 + c), b1 = __ldg(w4 + c + 32), b2 = __ldg(w4 + c + 64), b3 = __ldg(w4 + c + 96);
                    r0 = fma((double)a0.x, (double)b0.x, r0); r0 = fma((double)a0.y, (double)b0.y, r0);
                    r0 = fma((double)a0.z, (double)b0.z, r0); r0 = fma((double)a0.w, (double)b0.w, r0);
                    r1 = fma((double)a1.x, (double)b1.x, r1); r1 = fma((double)a1.y, (double)b1.y, r1);
                    r1 = fma((double)a1.z, (double)b1.z, r1); r1 = fma((double)a1.w, (double)b1.w, r1);
                    r2 = fma((double)a2.x, (double)b2.x, r2); r2 = fma((double)a2.y, (double)b2.y, r2);
                    r2 = fma((double)a2.z, (double)b2.z, r2); r2 = fma((double)a2.w, (double)b2.w, r2);
                    r3 = fma((double)a3.x, (double)b3.x, r3); r3 = fma((double)a3.y, (double)b3.y, r3);
                    r3 = fma((double)a3.z, (double)b3.z, r3); r3 = fma((double)a3.w, (double)b3.w, r3);
                }
                for (; c < q; c += 32) {
                    const float4 a0 = __ldg(x4 + c), b0 = __ldg(w4 + c);
                    r0 = fma((double)a0.x, (double)b0.x, r0); r0 = fma((double)a0.y, (double)b0.y, r0);
                    r0 = fma((double)a0.z, (double)b0.z, r0); r0 = fma((double)a0.w, (double)b0.w, r0);
                }
            } else {
                int c = lane;
                for (; c + 96 < d; c += 128) {
                    r0 = fma((double)x[c], (double)w[c], r0);
                    r1 = fma((double)x[c + 32], (double)w[c + 32], r1);
                    r2 = fma((double)x[c + 64], (double)w[c + 64], r2);
                    r3 = fma((double)x[c + 96], (double)w[c + 96], r3);
                }
                for (; c < d; c += 32) r0 = fma((double)x[c], (double)w[c], r0);
            }
            r = (r0 + r1) + (r2 + r3);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
            r -= (double)yv[i];
            if (lane == 0) sq += r * r;
        }
        if (lane == 0) r_s[warp] = (i < row1) ? r : 0.0;   // a row past the end contributes nothing
        __syncthreads();
        if (VEC) {
            const int q = d >> 2;
            for (int c = threadIdx.x; c < q; c += kThreads) {
                float4 xv[kRows];
#pragma unroll
                for (int k = 0; k < kRows; ++k)
                    xv[k] = (base + k < row1) ? __ldg(reinterpret_cast<const float4*>(Xv + (int64_t)(base + k) * d) + c)
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
                double a0 = g_s[4 * c], a1 = g_s[4 * c + 1], a2 = g_s[4 * c + 2], a3 = g_s[4 * c + 3];
#pragma unroll
                for (int k = 0; k < kRows; ++k) {
                    a0 = fma((double)xv[k].x, r_s[k], a0); a1 = fma((double)xv[k].y, r_s[k], a1);
                    a2 = fma((double)xv[k].z, r_s[k], a2); a3 = fma((double)xv[k].w, r_s[k], a3);
                }
                g_s[4 * c] = a0; g_s[4 * c + 1] = a1; g_s[4 * c + 2] = a2; g_s[4 * c + 3] = a3;
            }
        } else {
            for (int c = threadIdx.x; c < d; c += kThreads) {
                float xv[kRows];
#pragma unroll
                for (int k = 0; k < kRows; ++k) xv[k] = (base + k < row1) ? Xv[(int64_t)(base + k) * d + c] : 0.f;
                double a = g_s[c];
#pragma unroll
                for (int k = 0; k < kRows; ++k) a = fma((double)xv[k], r_s[k], a);
                g_s[c] = a;
            }
        }
        __syncthreads();
    }
    double* mine = partials + (size_t)blockIdx.x * (d + 1);
    for (int c = threadIdx.x; c < d; c += kThreads) mine[c] = g_s[c];
    // the block's share of the meta loss: warps in order
    if (lane == 0) r_s[warp] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int k = 0; k < kRows; ++k) t += r_s[k];
        mine[d] = t;
    }
}

// Column c of the result = 2 x (sum over blocks, in block order, of their partials); column d is the meta loss.
__global__ void __launch_bounds__(128)
biasreg_reduce_kernel(int d, int blocks, const double* __restrict__ partials, float* __restrict__ g_out,
                      float* __restrict__ loss_out) {
    pdl_trigger();
    pdl_wait();
    const int c = blockIdx.x * 128 + threadIdx.x;
    if (c > d) return;
    double t = 0.0;
#pragma unroll 8
    for (int b = 0; b < blocks; ++b) t += __ldcg(partials + (size_t)b * (d + 1) + c);
    if (c < d) g_out[c] = (float)(2.0 * t);
    else if (loss_out) *loss_out = (float)t;
}

__global__ void __launch_bounds__(kThreads)
biasreg_fd_kernel(int64_t d, const float* __restrict__ w_plus, const float* __restrict__ w_minus,
                  const float* __restrict__ lambda, float beta, const float* __restrict__ eps_fd,
                  float* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    // double: w+- - lambda is then exact, so the only rounding the quotient amplifies is that of w+- themselves
    const double eps = (double)*eps_fd;
    const double inv = eps > 0.0 ? 1.0 / (2.0 * eps) : 0.0;
    const double b2 = 2.0 * (double)beta;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t k = (int64_t)blockIdx.x * kThreads + threadIdx.x; k < d; k += stride) {
        const double lam = (double)lambda[k];
        const double gp = -b2 * ((double)w_plus[k] - lam);    // dL_base/dlambda at w+
        const double gm = -b2 * ((double)w_minus[k] - lam);   // ... at w-
        out[k] = (float)(-(gp - gm) * inv);
    }
}

}  // namespace

int biasreg_grid(const sama_ctx* ctx, int n_val) {
    int g = (n_val + kRows - 1) / kRows;
    if (g > 2 * ctx->sm_count) g = 2 * ctx->sm_count;
    return g < 1 ? 1 : g;
}

cudaError_t launch_biasreg_direct_grad(sama_ctx* ctx, int d, int n_val, const float* Xv, const float* yv,
                                       const float* w, float* g_out, float* loss_out, cudaStream_t st) {
    const size_t smem = sizeof(double) * ((size_t)d + kRows);
    const bool vec = (d % 4 == 0) && ((reinterpret_cast<uintptr_t>(Xv) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(w) & 15u) == 0);
    if (smem > 48 * 1024) {
        const cudaError_t e = vec ? cudaFuncSetAttribute(biasreg_partials_kernel<true>,
                                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                  : cudaFuncSetAttribute(biasreg_partials_kernel<false>,
                                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int grid = biasreg_grid(ctx, n_val);
    {
        KernelScope scope(ctx, SAMA_K_BIASREG_GRAD, -1, st);
        if (vec) biasreg_partials_kernel<true><<<grid, kThreads, smem, st>>>(d, n_val, Xv, yv, w, ctx->br_partials);
        else biasreg_partials_kernel<false><<<grid, kThreads, smem, st>>>(d, n_val, Xv, yv, w, ctx->br_partials);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    KernelScope scope(ctx, SAMA_K_BIASREG_GRAD, -1, st);
    return launch_dependent(biasreg_reduce_kernel, dim3((d + 1 + 127) / 128), dim3(128), 0, st, d, grid,
                            (const double*)ctx->br_partials, g_out, loss_out);
}

cudaError_t launch_biasreg_fd(sama_ctx* ctx, int64_t d, const float* w_plus, const float* w_minus,
                              const float* lambda, float beta, const float* eps_fd, float* out, cudaStream_t st) {
    int64_t blocks = (d + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    KernelScope scope(ctx, SAMA_K_BIASREG_FD, -1, st);
    return launch_dependent(biasreg_fd_kernel, dim3((unsigned)blocks), dim3(kThreads), 0, st, d, w_plus, w_minus, lambda,
                            beta, eps_fd, out);
}

}  // namespace sama
