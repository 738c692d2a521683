// SAMA on the biased-regression problem of Appendix E:
//   L_meta(w)         = || X' w - y' ||^2
//   L_base(w, lambda) = || X w - y ||^2 + beta || w - lambda ||^2
// Two kernels, both specific to this objective; adaptation, norm and perturbation are the library's own.
//
//   direct gradient (Eq. 1):  g_meta = dL_meta/dw = 2 X'^T (X' w - y')
//   central difference (Eq. 5) of g_lambda(w) = dL_base/dlambda = -2 beta (w - lambda):
//                             metagrad = -[g_lambda(w+) - g_lambda(w-)] / (2 eps_fd)
//
// The direct gradient is two sweeps over X', each at streaming rate, instead of one that keeps a block's partial
// gradient in shared memory (that form needs two block-wide phases per handful of rows and is latency-bound):
//   1. residuals: one warp per row forms r_i = x_i . w - y_i (every load of a row segment in flight at once; the
//      sum kept as pairs of floats that carry a double's precision) and stores it in double;
//   2. column sums: a block takes a strip of 1024 columns (one float4 per thread) and a chunk of rows, reads the
//      strip of each row (4 KB, contiguous; the chunks run from the last rows backwards, so that what the first
//      sweep left in L2 is read from there), and adds
//      r_i x_i into four double accumulators per thread; the chunk's partial goes to global memory.
// A third small kernel adds the chunks' partials column by column in chunk order.  Accumulation carries a
// double's precision throughout; nothing depends on scheduling.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// VEC: d % 4 == 0 and 16-byte aligned X', w: 16-byte loads, kSeg of them per lane in flight before the first is
// used (a row is a chain of dependent steps for its warp, so the loads in flight per lane set the pace).
constexpr int kSeg = 8;

// One more term x w of a dot product kept as an unevaluated sum s + e of two floats: the product is exact as
// ph + pl (fused multiply-add), s + ph is exact as t + (rounding error) by Knuth's two-sum, and the small parts
// gather in e.  The result carries about 2^-45 of the sum of |x w|, like a double accumulator, without the
// float-to-double conversions (two per term), which this device issues slowly: measured 37 -> 29 us for the
// sweep below at d = 4096, n' = 8192, with results equal to the double form's to 12 digits.
// (Intrinsics, so that no multiply is contracted into a neighbouring add.)
__device__ __forceinline__ void dot_step(float& s, float& e, float x, float w) {
    const float ph = __fmul_rn(x, w);
    const float pl = __fmaf_rn(x, w, -ph);
    const float t = __fadd_rn(s, ph);
    const float z = __fsub_rn(t, s);
    const float err = __fadd_rn(__fsub_rn(s, __fsub_rn(t, z)), __fsub_rn(ph, z));
    e = __fadd_rn(e, __fadd_rn(err, pl));
    s = t;
}
__device__ __forceinline__ void dot_step4(float& s, float& e, float4 x, float4 w) {
    dot_step(s, e, x.x, w.x);
    dot_step(s, e, x.y, w.y);
    dot_step(s, e, x.z, w.z);
    dot_step(s, e, x.w, w.w);
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads, 4)
biasreg_residual_kernel(int d, int n_val, const float* __restrict__ Xv, const float* __restrict__ yv,
                        const float* __restrict__ w, double* __restrict__ res) {
    const int lane = threadIdx.x & 31;
    const int warp = blockIdx.x * kWarps + (threadIdx.x >> 5), n_warps = gridDim.x * kWarps;
    for (int i = warp; i < n_val; i += n_warps) {
        const float* x = Xv + (int64_t)i * d;
        double r;
        if (VEC) {
            const float4* x4 = reinterpret_cast<const float4*>(x);
            const float4* w4 = reinterpret_cast<const float4*>(w);
            const int q = d >> 2;
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;   // four independent chains
            for (int c0 = 0; c0 < q; c0 += 32 * kSeg) {
                float4 a[kSeg];
#pragma unroll
                for (int k = 0; k < kSeg; ++k) {
                    const int c = c0 + lane + 32 * k;
                    a[k] = c < q ? __ldg(x4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int k = 0; k < kSeg; k += 4) {
                    float4 b[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int c = c0 + lane + 32 * (k + j);
                        b[j] = c < q ? __ldg(w4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);   // w: 4 d bytes, from L1
                    }
                    dot_step4(s0, e0, a[k], b[0]);
                    dot_step4(s1, e1, a[k + 1], b[1]);
                    dot_step4(s2, e2, a[k + 2], b[2]);
                    dot_step4(s3, e3, a[k + 3], b[3]);
                }
            }
            r = (((double)s0 + (double)e0) + ((double)s1 + (double)e1)) + (((double)s2 + (double)e2) + ((double)s3 + (double)e3));
        } else {
            double r0 = 0.0, r1 = 0.0, r2 = 0.0, r3 = 0.0;
            int c = lane;
            for (; c + 96 < d; c += 128) {
                r0 = fma((double)x[c], (double)w[c], r0);
                r1 = fma((double)x[c + 32], (double)w[c + 32], r1);
                r2 = fma((double)x[c + 64], (double)w[c + 64], r2);
                r3 = fma((double)x[c + 96], (double)w[c + 96], r3);
            }
            for (; c < d; c += 32) r0 = fma((double)x[c], (double)w[c], r0);
            r = (r0 + r1) + (r2 + r3);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
        if (lane == 0) res[i] = r - (double)yv[i];
    }
}

// Block (strip, chunk): partial[chunk][c] = sum over the chunk's rows, in row order, of r_i x_ic for the strip's
// columns; the strip-0 block also leaves the chunk's sum of r_i^2 in column d (the meta loss).
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
biasreg_colsum_kernel(int d, int n_val, int rows_per_chunk, const float* __restrict__ Xv,
                      const double* __restrict__ res, double* __restrict__ partials) {
    pdl_trigger();
    pdl_wait();
    // the first sweep touched the last rows last: chunks are taken from the end, while those rows are still in L2
    const int chunk = (int)gridDim.y - 1 - (int)blockIdx.y;
    const int row0 = chunk * rows_per_chunk, row1 = min(n_val, row0 + rows_per_chunk);
    double* mine = partials + (size_t)chunk * (d + 1);
    if (VEC) {
        const int c4 = blockIdx.x * kThreads + threadIdx.x;   // this thread's float4 of every row
        if (c4 < (d >> 2)) {
            const float4* col = reinterpret_cast<const float4*>(Xv) + c4;
            const int64_t q = d >> 2;
            double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
            int i = row0;
            for (; i + 7 < row1; i += 8) {
                float4 x[8];
                double r[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) x[k] = __ldg(col + (int64_t)(i + k) * q);
#pragma unroll
                for (int k = 0; k < 8; ++k) r[k] = __ldg(res + i + k);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    a0 = fma((double)x[k].x, r[k], a0); a1 = fma((double)x[k].y, r[k], a1);
                    a2 = fma((double)x[k].z, r[k], a2); a3 = fma((double)x[k].w, r[k], a3);
                }
            }
            for (; i < row1; ++i) {
                const float4 x = __ldg(col + (int64_t)i * q);
                const double r = __ldg(res + i);
                a0 = fma((double)x.x, r, a0); a1 = fma((double)x.y, r, a1);
                a2 = fma((double)x.z, r, a2); a3 = fma((double)x.w, r, a3);
            }
            mine[4 * c4] = a0; mine[4 * c4 + 1] = a1; mine[4 * c4 + 2] = a2; mine[4 * c4 + 3] = a3;
        }
    } else {
        const int c = blockIdx.x * kThreads + threadIdx.x;
        if (c < d) {
            double a = 0.0;
            for (int i = row0; i < row1; ++i) a = fma((double)Xv[(int64_t)i * d + c], __ldg(res + i), a);
            mine[c] = a;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double t = 0.0;
        for (int i = row0; i < row1; ++i) { const double r = __ldg(res + i); t = fma(r, r, t); }
        mine[d] = t;
    }
}

// Column c of the result = 2 x (sum over the row chunks of their partials); column d is the meta loss.  A block
// takes 32 columns; each of its eight warps adds a contiguous eighth of the chunks, in chunk order, and the eight
// sums are added in warp order: a fixed order, whatever the scheduling.
__global__ void __launch_bounds__(kThreads)
biasreg_reduce_kernel(int d, int blocks, const double* __restrict__ partials, float* __restrict__ g_out,
                      float* __restrict__ loss_out) {
    pdl_trigger();
    pdl_wait();
    __shared__ double part[kWarps][32];
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    const int per = (blocks + kWarps - 1) / kWarps;
    const int b0 = grp * per, b1 = min(blocks, b0 + per);
    double t = 0.0;
    if (c <= d) {
#pragma unroll 8
        for (int b = b0; b < b1; ++b) t += __ldcg(partials + (size_t)b * (d + 1) + c);
    }
    part[grp][lane] = t;
    __syncthreads();
    if (grp == 0 && c <= d) {
        double sum = 0.0;
#pragma unroll
        for (int k = 0; k < kWarps; ++k) sum += part[k][lane];
        if (c < d) g_out[c] = (float)(2.0 * sum);
        else if (loss_out) *loss_out = (float)sum;
    }
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

// Row chunks of the second sweep: at least 32 rows each and no more chunks than twice the SM count (the
// partials buffer is sized for that many).
int biasreg_grid(const sama_ctx* ctx, int n_val) {
    const int cap = 2 * ctx->sm_count;
    int rows = (n_val + cap - 1) / cap;
    if (rows < 32) rows = 32;
    const int g = (n_val + rows - 1) / rows;
    return g < 1 ? 1 : g;
}

// `partials` holds biasreg_grid() x (d + 1) doubles followed by n_val doubles of residuals.
cudaError_t launch_biasreg_direct_grad(sama_ctx* ctx, int d, int n_val, const float* Xv, const float* yv,
                                       const float* w, float* g_out, float* loss_out, cudaStream_t st) {
    const bool vec = (d % 4 == 0) && ((reinterpret_cast<uintptr_t>(Xv) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(w) & 15u) == 0);
    const int chunks = biasreg_grid(ctx, n_val);
    const int rows_per_chunk = (n_val + chunks - 1) / chunks;
    double* partials = ctx->br_partials;
    double* res = partials + (size_t)chunks * ((size_t)d + 1);
    {
        int grid = (n_val + kWarps - 1) / kWarps;
        if (grid > 4 * ctx->sm_count) grid = 4 * ctx->sm_count;   // one resident wave; warps stride over the rows
        if (grid < 1) grid = 1;
        KernelScope scope(ctx, SAMA_K_BIASREG_GRAD, -1, st);
        if (vec) biasreg_residual_kernel<true><<<grid, kThreads, 0, st>>>(d, n_val, Xv, yv, w, res);
        else biasreg_residual_kernel<false><<<grid, kThreads, 0, st>>>(d, n_val, Xv, yv, w, res);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    {
        const int strips = vec ? ((d >> 2) + kThreads - 1) / kThreads : (d + kThreads - 1) / kThreads;
        KernelScope scope(ctx, SAMA_K_BIASREG_GRAD, -1, st);
        const dim3 grid(strips < 1 ? 1 : strips, chunks);
        const cudaError_t e =
            vec ? launch_dependent(biasreg_colsum_kernel<true>, grid, dim3(kThreads), 0, st, d, n_val, rows_per_chunk, Xv,
                                   (const double*)res, partials)
                : launch_dependent(biasreg_colsum_kernel<false>, grid, dim3(kThreads), 0, st, d, n_val, rows_per_chunk, Xv,
                                   (const double*)res, partials);
        if (e != cudaSuccess) return e;
    }
    KernelScope scope(ctx, SAMA_K_BIASREG_GRAD, -1, st);
    return launch_dependent(biasreg_reduce_kernel, dim3((d + 1 + 31) / 32), dim3(kThreads), 0, st, d, chunks,
                            (const double*)partials, g_out, loss_out);
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
