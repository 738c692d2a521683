// Elementwise stages of the SAMA step: HBM-streaming kernels.
//
//   adapt_sumsq : p = (du_adam/dg) * g_meta (Eq. 4, Appendix C) fused with
//                 sum p^2 (Sec. 3.2) -- one sweep, 20 B/element (16 without g_base)
//   sumsq       : sum p^2 alone, for a perturbation that did not come from adapt
//   perturb     : eps_fd = alpha/||p||; theta+- = theta +- eps_fd p (Sec. 3.2)
//                 -- one sweep, 16 B/element
//
// All three are persistent grid-stride kernels sized to the SM count, move
// 16-byte vectors, issue every load of an iteration before the first use and
// mark read-once inputs as streaming.  The norm is accumulated in double per
// thread, reduced by warp shuffles and shared memory to one partial per
// block, and the last block to arrive adds the partials in a fixed order, so
// the result does not depend on scheduling.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 2;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

// One element of Eq. 4 with the Adam matrix of Appendix C, in the split form
//   J = a [ (1-b1)/D  -  m' (1-b2) g / (sqrt(c2) r D^2) ],   r = sqrt(s'),  D = r/sqrt(c2) + eps,
// whose second term vanishes at r = 0.
__device__ __forceinline__ float adapt_one(float m, float s, float g, float gm, const AdaptConsts& c) {
    if (c.identity) return gm;
    const float m_new = fmaf(c.b1, m, c.omb1 * g);
    const float s_new = fmaf(c.b2, s, c.omb2 * g * g);
    const float r = sqrtf(s_new);
    const float D = fmaf(r, c.inv_rc2, c.eps);
    const float invD = 1.0f / D;
    float t = c.omb1 * invD;
    if (r > 0.0f) t -= ((m_new * g) / r) * (c.omb2 * c.inv_rc2) * invD * invD;
    if (c.drop_eps_term) t -= c.omb1 * c.eps * invD * invD;
    return c.a * t * gm;
}

__device__ __forceinline__ float4 adapt_four(float4 vm, float4 vs, float4 vg, float4 vq, const AdaptConsts& c) {
    float4 o;
    o.x = adapt_one(vm.x, vs.x, vg.x, vq.x, c);
    o.y = adapt_one(vm.y, vs.y, vg.y, vq.y, c);
    o.z = adapt_one(vm.z, vs.z, vg.z, vq.z, c);
    o.w = adapt_one(vm.w, vs.w, vg.w, vq.w, c);
    return o;
}

__device__ __forceinline__ double sq4(float4 o) {
    return (double)o.x * o.x + (double)o.y * o.y + (double)o.z * o.z + (double)o.w * o.w;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; valid in thread 0.  Fixed order.
__device__ __forceinline__ double block_sum(double v, double* smem) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) t += smem[w];
    }
    return t;
}

// Publishes this block's partial; the last block to arrive adds all partials
// in index order and writes the total.
__device__ __forceinline__ void finish_sum(double acc, double* partials, DeviceScalars* sc, double* sumsq_out) {
    __shared__ double smem[kThreads / 32];
    __shared__ bool is_last;
    const double total = block_sum(acc, smem);
    if (threadIdx.x == 0) {
        partials[blockIdx.x] = total;
        __threadfence();
        const unsigned prev = atomicAdd(&sc->counter, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double v = 0.0;
    for (unsigned i = threadIdx.x; i < gridDim.x; i += kThreads) v += __ldcg(partials + i);
    const double sum = block_sum(v, smem);
    if (threadIdx.x == 0) {
        sc->sumsq = sum;
        if (sumsq_out) *sumsq_out = sum;
        sc->counter = 0u;
    }
}

template <bool HAS_G>
__global__ void __launch_bounds__(kThreads)
adapt_sumsq_vec4(int64_t n, const float* __restrict__ m, const float* __restrict__ s,
                 const float* __restrict__ g, const float* gm, float* p, AdaptConsts c,
                 double* partials, DeviceScalars* sc, double* sumsq_out) {
    const int64_t items = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const float4* m4 = reinterpret_cast<const float4*>(m);
    const float4* s4 = reinterpret_cast<const float4*>(s);
    const float4* g4 = reinterpret_cast<const float4*>(g);
    const float4* gm4 = reinterpret_cast<const float4*>(gm);
    float4* p4 = reinterpret_cast<float4*>(p);
    double acc = 0.0;

    for (; i + stride * (kUnroll - 1) < items; i += stride * kUnroll) {
        float4 vm[kUnroll], vs[kUnroll], vg[kUnroll], vq[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t j = i + stride * u;
            if (!c.identity) {
                vm[u] = ld_stream(m4 + j);
                vs[u] = ld_stream(s4 + j);
                if (HAS_G) vg[u] = ld_stream(g4 + j);
            } else {
                vm[u] = vs[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            vq[u] = ld_stream(gm4 + j);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (!HAS_G) vg[u] = vm[u];
            const float4 o = adapt_four(vm[u], vs[u], vg[u], vq[u], c);
            p4[i + stride * u] = o;
            acc += sq4(o);
        }
    }
    for (; i < items; i += stride) {
        float4 vm = make_float4(0.f, 0.f, 0.f, 0.f), vs = vm, vg = vm;
        if (!c.identity) {
            vm = ld_stream(m4 + i);
            vs = ld_stream(s4 + i);
            vg = HAS_G ? ld_stream(g4 + i) : vm;
        }
        const float4 o = adapt_four(vm, vs, vg, ld_stream(gm4 + i), c);
        p4[i] = o;
        acc += sq4(o);
    }
    // ragged tail (n % 4 elements)
    if (blockIdx.x == 0) {
        const int64_t k = (items << 2) + threadIdx.x;
        if (k < n) {
            float vm = 0.f, vs = 0.f, vg = 0.f;
            if (!c.identity) { vm = m[k]; vs = s[k]; vg = HAS_G ? g[k] : vm; }
            const float o = adapt_one(vm, vs, vg, gm[k], c);
            p[k] = o;
            acc += (double)o * o;
        }
    }
    finish_sum(acc, partials, sc, sumsq_out);
}

// Any alignment.
template <bool HAS_G>
__global__ void __launch_bounds__(kThreads)
adapt_sumsq_scalar(int64_t n, const float* m, const float* s, const float* g, const float* gm, float* p,
                   AdaptConsts c, double* partials, DeviceScalars* sc, double* sumsq_out) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    double acc = 0.0;
    for (int64_t k = (int64_t)blockIdx.x * kThreads + threadIdx.x; k < n; k += stride) {
        float vm = 0.f, vs = 0.f, vg = 0.f;
        if (!c.identity) { vm = m[k]; vs = s[k]; vg = HAS_G ? g[k] : vm; }
        const float o = adapt_one(vm, vs, vg, gm[k], c);
        p[k] = o;
        acc += (double)o * o;
    }
    finish_sum(acc, partials, sc, sumsq_out);
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
sumsq_kernel(int64_t n, const float* __restrict__ p, double* partials, DeviceScalars* sc) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    double acc = 0.0;
    if (VEC) {
        const int64_t items = n >> 2;
        const float4* p4 = reinterpret_cast<const float4*>(p);
        for (; i < items; i += stride) acc += sq4(p4[i]);
        if (blockIdx.x == 0) {
            const int64_t k = (items << 2) + threadIdx.x;
            if (k < n) acc += (double)p[k] * p[k];
        }
    } else {
        for (; i < n; i += stride) acc += (double)p[i] * p[i];
    }
    finish_sum(acc, partials, sc, nullptr);
}

// eps_fd = alpha / sqrt(sumsq); 0 with `bad` set when the norm is 0 or not finite.
__device__ __forceinline__ float step_size(double sumsq, float alpha, bool& bad) {
    const double norm = sqrt(sumsq);
    bad = !(norm > 0.0) || isinf(norm);
    return bad ? 0.0f : (float)((double)alpha / norm);
}

// eps == 0 marks the degenerate norm: theta+- = theta even where p is not finite.
__device__ __forceinline__ void plus_minus(float eps, float4 vt, float4 vp, float4& a, float4& b) {
    if (eps == 0.0f) { a = vt; b = vt; return; }
    a.x = fmaf(eps, vp.x, vt.x); b.x = fmaf(-eps, vp.x, vt.x);
    a.y = fmaf(eps, vp.y, vt.y); b.y = fmaf(-eps, vp.y, vt.y);
    a.z = fmaf(eps, vp.z, vt.z); b.z = fmaf(-eps, vp.z, vt.z);
    a.w = fmaf(eps, vp.w, vt.w); b.w = fmaf(-eps, vp.w, vt.w);
}

template <bool VEC>
__global__ void __launch_bounds__(kThreads)
perturb_kernel(int64_t n, const float* theta, const float* __restrict__ p, const double* __restrict__ sumsq,
               float alpha, float* theta_plus, float* theta_minus, DeviceScalars* sc, float* eps_fd_out) {
    bool bad;
    const float eps = step_size(*sumsq, alpha, bad);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        sc->eps_fd = eps;
        if (eps_fd_out) *eps_fd_out = eps;
        if (bad) atomicOr(&sc->status, (int)SAMA_DEV_DEGENERATE_NORM);
    }
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (VEC) {
        const int64_t items = n >> 2;
        const float4* t4 = reinterpret_cast<const float4*>(theta);
        const float4* p4 = reinterpret_cast<const float4*>(p);
        float4* tp4 = reinterpret_cast<float4*>(theta_plus);
        float4* tm4 = reinterpret_cast<float4*>(theta_minus);
        for (; i + stride * (kUnroll - 1) < items; i += stride * kUnroll) {
            float4 vt[kUnroll], vp[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                vt[u] = ld_stream(t4 + i + stride * u);
                vp[u] = ld_stream(p4 + i + stride * u);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                float4 a, b;
                plus_minus(eps, vt[u], vp[u], a, b);
                tp4[i + stride * u] = a;
                tm4[i + stride * u] = b;
            }
        }
        for (; i < items; i += stride) {
            float4 a, b;
            plus_minus(eps, ld_stream(t4 + i), ld_stream(p4 + i), a, b);
            tp4[i] = a;
            tm4[i] = b;
        }
        if (blockIdx.x == 0) {
            const int64_t k = (items << 2) + threadIdx.x;
            if (k < n) {
                const float t = theta[k], q = p[k];
                theta_plus[k] = eps == 0.0f ? t : fmaf(eps, q, t);
                theta_minus[k] = eps == 0.0f ? t : fmaf(-eps, q, t);
            }
        }
    } else {
        for (; i < n; i += stride) {
            const float t = theta[i], q = p[i];
            theta_plus[i] = eps == 0.0f ? t : fmaf(eps, q, t);
            theta_minus[i] = eps == 0.0f ? t : fmaf(-eps, q, t);
        }
    }
}

__device__ __forceinline__ float tf32_round(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}
__device__ __forceinline__ void tf32_split(float4 x, float4& h, float4& l) {
    h.x = tf32_round(x.x); l.x = tf32_round(x.x - h.x);
    h.y = tf32_round(x.y); l.y = tf32_round(x.y - h.y);
    h.z = tf32_round(x.z); l.z = tf32_round(x.z - h.z);
    h.w = tf32_round(x.w); l.w = tf32_round(x.w - h.w);
}

// perturb (Sec. 3.2) fused with the operand preparation of the tensor-core
// forward pass: besides theta+ and theta-, every weight element is written as
// TF32 hi / lo into the row-padded split buffers of both branches, so the
// forward pass needs no further sweep over the parameters.  32 B/element.
// Preconditions (checked on the host): 16-byte aligned pointers, every weight
// block starts at a multiple of 4 and has K % 4 == 0 and fewer than 2^31 elements.
__global__ void __launch_bounds__(kThreads)
perturb_split_kernel(int64_t n, const float* theta, const float* __restrict__ p, const double* __restrict__ sumsq,
                     float alpha, float* theta_plus, float* theta_minus, DeviceScalars* sc, float* eps_fd_out,
                     SplitLayout lay, float* __restrict__ hi, float* __restrict__ lo, XSplitJob xjob) {
    pdl_trigger();
    // The batch does not depend on the adaptation: its operand split runs before the wait, i.e. while
    // the previous kernel may still be draining.
    if (xjob.rows > 0) {
        const int q = xjob.ld_out >> 2;
        const int64_t total = xjob.rows * q, xstride = (int64_t)gridDim.x * kThreads;
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += xstride) {
            const int64_t r = i / q;
            const int c = (int)(i - r * q) << 2;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f), h, l;
            if (c < xjob.cols) x = __ldg(reinterpret_cast<const float4*>(xjob.x + r * xjob.cols + c));
            tf32_split(x, h, l);
            *reinterpret_cast<float4*>(xjob.hi + r * xjob.ld_out + c) = h;
            *reinterpret_cast<float4*>(xjob.lo + r * xjob.ld_out + c) = l;
        }
    }
    pdl_wait();  // p and the sum of squares come from the adaptation kernel just before
    bool bad;
    const float eps = step_size(*sumsq, alpha, bad);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        sc->eps_fd = eps;
        if (eps_fd_out) *eps_fd_out = eps;
        if (bad) atomicOr(&sc->status, (int)SAMA_DEV_DEGENERATE_NORM);
    }
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    const int64_t items = n >> 2;
    const float4* t4 = reinterpret_cast<const float4*>(theta);
    const float4* p4 = reinterpret_cast<const float4*>(p);
    float4* tp4 = reinterpret_cast<float4*>(theta_plus);
    float4* tm4 = reinterpret_cast<float4*>(theta_minus);

    auto emit = [&](int64_t i, float4 vt, float4 vp) {
        float4 a, b;
        plus_minus(eps, vt, vp, a, b);
        // theta+- themselves are not read again by the forward (only their biases and a narrow head are):
        // streaming stores keep them from displacing the hi / lo operands, which the next kernel reads, in L2
        __stcs(tp4 + i, a);
        __stcs(tm4 + i, b);
        const int64_t e = i << 2;
        int l = -1;
#pragma unroll 1
        for (int k = 0; k < lay.n_layers; ++k)
            if (e >= lay.w_off[k] && e < lay.w_off[k] + lay.w_cnt[k]) { l = k; break; }
        if (l < 0) return;  // a bias
        const uint32_t rel = (uint32_t)(e - lay.w_off[l]);
        const uint32_t K = (uint32_t)lay.K[l], Kp = (uint32_t)lay.Kp[l];
        const uint32_t row = rel / K, col = rel - row * K;
        const int64_t dst = lay.s_off[l] + (int64_t)row * Kp + col;
        float4 h, q;
        tf32_split(a, h, q);
        *reinterpret_cast<float4*>(hi + dst) = h;
        *reinterpret_cast<float4*>(lo + dst) = q;
        tf32_split(b, h, q);
        *reinterpret_cast<float4*>(hi + lay.slab + dst) = h;
        *reinterpret_cast<float4*>(lo + lay.slab + dst) = q;
        if (Kp != K && col + 4 == K) {  // this thread closes the row: zero its padding
            const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t c = 4; c < Kp - K + 4; c += 4) {
                *reinterpret_cast<float4*>(hi + dst + c) = z;
                *reinterpret_cast<float4*>(lo + dst + c) = z;
                *reinterpret_cast<float4*>(hi + lay.slab + dst + c) = z;
                *reinterpret_cast<float4*>(lo + lay.slab + dst + c) = z;
            }
        }
    };

    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    for (; i + stride < items; i += stride * 2) {
        const float4 vt0 = ld_stream(t4 + i), vp0 = ld_stream(p4 + i);
        const float4 vt1 = ld_stream(t4 + i + stride), vp1 = ld_stream(p4 + i + stride);
        emit(i, vt0, vp0);
        emit(i + stride, vt1, vp1);
    }
    for (; i < items; i += stride) emit(i, ld_stream(t4 + i), ld_stream(p4 + i));
    if (blockIdx.x == 0) {  // n % 4 trailing elements: never weights under the preconditions
        const int64_t k = (items << 2) + threadIdx.x;
        if (k < n) {
            const float t = theta[k], q = p[k];
            theta_plus[k] = eps == 0.0f ? t : fmaf(eps, q, t);
            theta_minus[k] = eps == 0.0f ? t : fmaf(-eps, q, t);
        }
    }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int stream_grid(const sama_ctx* ctx, int64_t work_items, int per_thread) {
    int64_t blocks = (work_items + (int64_t)kThreads * per_thread - 1) / ((int64_t)kThreads * per_thread);
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks > kMaxPartials) blocks = kMaxPartials;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

cudaError_t launch_adapt_sumsq(sama_ctx* ctx, int64_t n, const float* m, const float* s, const float* g_base,
                               const float* g_meta, const AdaptConsts& c, float* p_out, double* sumsq_out,
                               cudaStream_t st) {
    const bool vec = aligned16(m) && aligned16(s) && aligned16(g_meta) && aligned16(p_out) &&
                     (g_base == nullptr || aligned16(g_base));
    KernelScope scope(ctx, SAMA_K_ADAPT, -1, st);
    if (vec) {
        const int grid = stream_grid(ctx, n >> 2, kUnroll);
        if (g_base)
            adapt_sumsq_vec4<true><<<grid, kThreads, 0, st>>>(n, m, s, g_base, g_meta, p_out, c, ctx->partials,
                                                              ctx->scalars, sumsq_out);
        else
            adapt_sumsq_vec4<false><<<grid, kThreads, 0, st>>>(n, m, s, nullptr, g_meta, p_out, c, ctx->partials,
                                                               ctx->scalars, sumsq_out);
    } else {
        const int grid = stream_grid(ctx, n, 4);
        if (g_base)
            adapt_sumsq_scalar<true><<<grid, kThreads, 0, st>>>(n, m, s, g_base, g_meta, p_out, c, ctx->partials,
                                                                ctx->scalars, sumsq_out);
        else
            adapt_sumsq_scalar<false><<<grid, kThreads, 0, st>>>(n, m, s, nullptr, g_meta, p_out, c,
                                                                 ctx->partials, ctx->scalars, sumsq_out);
    }
    return cudaGetLastError();
}

cudaError_t launch_sumsq(sama_ctx* ctx, int64_t n, const float* p, cudaStream_t st) {
    KernelScope scope(ctx, SAMA_K_SUMSQ, -1, st);
    if (aligned16(p))
        sumsq_kernel<true><<<stream_grid(ctx, n >> 2, 4), kThreads, 0, st>>>(n, p, ctx->partials, ctx->scalars);
    else
        sumsq_kernel<false><<<stream_grid(ctx, n, 8), kThreads, 0, st>>>(n, p, ctx->partials, ctx->scalars);
    return cudaGetLastError();
}

cudaError_t launch_perturb(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* sumsq,
                           float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out,
                           cudaStream_t st) {
    const bool vec = aligned16(theta) && aligned16(p) && aligned16(theta_plus) && aligned16(theta_minus);
    KernelScope scope(ctx, SAMA_K_PERTURB, -1, st);
    if (vec)
        perturb_kernel<true><<<stream_grid(ctx, n >> 2, kUnroll), kThreads, 0, st>>>(
            n, theta, p, sumsq, alpha, theta_plus, theta_minus, ctx->scalars, eps_fd_out);
    else
        perturb_kernel<false><<<stream_grid(ctx, n, 4), kThreads, 0, st>>>(
            n, theta, p, sumsq, alpha, theta_plus, theta_minus, ctx->scalars, eps_fd_out);
    return cudaGetLastError();
}

bool perturb_split_applicable(const SplitLayout& lay, const float* theta, const float* p, const float* theta_plus,
                              const float* theta_minus) {
    if (!aligned16(theta) || !aligned16(p) || !aligned16(theta_plus) || !aligned16(theta_minus)) return false;
    for (int l = 0; l < lay.n_layers; ++l)
        if ((lay.w_off[l] & 3) || (lay.K[l] & 3) || lay.w_cnt[l] >= ((int64_t)1 << 31)) return false;
    return true;
}

cudaError_t launch_perturb_split(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* sumsq,
                                 float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out,
                                 const SplitLayout& lay, float* hi, float* lo, const XSplitJob& xjob, cudaStream_t st) {
    KernelScope scope(ctx, SAMA_K_PERTURB_SPLIT, -1, st);
    return launch_dependent(perturb_split_kernel, dim3(stream_grid(ctx, n >> 2, kUnroll)), dim3(kThreads), 0, st, n,
                            theta, p, sumsq, alpha, theta_plus, theta_minus, ctx->scalars, eps_fd_out, lay, hi, lo, xjob);
}

}  // namespace sama
