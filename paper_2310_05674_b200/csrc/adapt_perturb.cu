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
// whose second term vanishes at r = 0.  The approximation printed last in Appendix C (drop_eps_term)
// removes a (1-b1) eps / D^2 from the bracket; at r = 0 that leaves exactly nothing (the value the
// approximate form tends to along g = 0, and the mean of its two one-sided limits along s = 0), which is
// written out as 0 rather than left to the rounding of two equal terms.
__device__ __forceinline__ float adapt_one(float m, float s, float g, float gm, const AdaptConsts& c) {
    if (c.identity) return gm;
    const float m_new = fmaf(c.b1, m, c.omb1 * g);
    const float s_new = fmaf(c.b2, s, c.omb2 * g * g);
    const float r = sqrtf(s_new);
    const float D = fmaf(r, c.inv_rc2, c.eps);
    const float invD = 1.0f / D;
    float t = c.omb1 * invD;
    if (r > 0.0f) {
        t -= ((m_new * g) / r) * (c.omb2 * c.inv_rc2) * invD * invD;
        if (c.drop_eps_term) t -= c.omb1 * c.eps * invD * invD;
    } else if (c.drop_eps_term) {
        t = 0.0f;
    }
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

// One 16-byte group of the fused perturbation + operand split: theta+- (each stored only if wanted), then, by
// the region of the flat vector the group lies in, TF32 hi / lo of both branches into the row-padded operand
// slabs (a weight), or fp32 into the compact slab (a bias; a weight of the narrow last layer the fused head
// multiplies itself).
struct SplitDst {
    float* theta_plus;
    float* theta_minus;
    float* hi;
    float* lo;
    float* small;
};
// Whether the group of four elements starting at e is a weight of a layer the sweep writes no operands for (so
// that, when theta+- are not stored either, the group need not even be read).
__device__ __forceinline__ bool skipped_weight(const SplitLayout& lay, int64_t e) {
#pragma unroll 1
    for (int k = 0; k < lay.n_layers; ++k)
        if (e >= lay.w_off[k] && e < lay.w_off[k] + lay.w_cnt[k]) return ((lay.skip_w >> k) & 1u) != 0;
    return false;
}
__device__ __forceinline__ void emit_split(const SplitLayout& lay, const SplitDst& o, float eps, int64_t i, float4 vt,
                                           float4 vp) {
    float4 a, b;
    plus_minus(eps, vt, vp, a, b);
    // theta+- themselves are not read again by the forward: streaming stores keep them from displacing the
    // hi / lo operands, which the next kernel reads, in L2
    if (o.theta_plus) __stcs(reinterpret_cast<float4*>(o.theta_plus) + i, a);
    if (o.theta_minus) __stcs(reinterpret_cast<float4*>(o.theta_minus) + i, b);
    float* small_m = o.small + lay.small;   // the minus branch's slab
    const int64_t e = i << 2;
    int l = -1;
#pragma unroll 1
    for (int k = 0; k < lay.n_layers; ++k)
        if (e >= lay.w_off[k] && e < lay.w_off[k] + lay.w_cnt[k] + lay.N[k]) { l = k; break; }
    if (l < 0) return;
    const int64_t rel64 = e - lay.w_off[l];
    if (rel64 >= lay.w_cnt[l]) {  // a bias: fp32, compact
        const int64_t dst = lay.b_off[l] + (rel64 - lay.w_cnt[l]);
        *reinterpret_cast<float4*>(o.small + dst) = a;
        *reinterpret_cast<float4*>(small_m + dst) = b;
        return;
    }
    if (l == lay.head_layer) {    // the fused head's weights: fp32, compact; it takes no split operands
        *reinterpret_cast<float4*>(o.small + rel64) = a;
        *reinterpret_cast<float4*>(small_m + rel64) = b;
        return;
    }
    if ((lay.skip_w >> l) & 1u) return;   // the product kernel forms this layer's operands itself
    const uint32_t rel = (uint32_t)rel64;
    const uint32_t K = (uint32_t)lay.K[l], Kp = (uint32_t)lay.Kp[l];
    const uint32_t row = rel / K, col = rel - row * K;
    const int64_t dst = lay.s_off[l] + (int64_t)row * Kp + col;
    float4 h, q;
    tf32_split(a, h, q);
    *reinterpret_cast<float4*>(o.hi + dst) = h;
    *reinterpret_cast<float4*>(o.lo + dst) = q;
    tf32_split(b, h, q);
    *reinterpret_cast<float4*>(o.hi + lay.slab + dst) = h;
    *reinterpret_cast<float4*>(o.lo + lay.slab + dst) = q;
    if (Kp != K && col + 4 == K) {  // this thread closes the row: zero its padding
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t c = 4; c < Kp - K + 4; c += 4) {
            *reinterpret_cast<float4*>(o.hi + dst + c) = z;
            *reinterpret_cast<float4*>(o.lo + dst + c) = z;
            *reinterpret_cast<float4*>(o.hi + lay.slab + dst + c) = z;
            *reinterpret_cast<float4*>(o.lo + lay.slab + dst + c) = z;
        }
    }
}
// The n % 4 trailing elements: under the preconditions of the fused sweep, the end of the last layer's bias.
__device__ __forceinline__ void emit_split_tail(const SplitLayout& lay, const SplitDst& o, float eps, int64_t k, float t,
                                                float q) {
    const float a = eps == 0.0f ? t : fmaf(eps, q, t), b = eps == 0.0f ? t : fmaf(-eps, q, t);
    if (o.theta_plus) o.theta_plus[k] = a;
    if (o.theta_minus) o.theta_minus[k] = b;
    const int last = lay.n_layers - 1;
    const int64_t j = k - lay.w_off[last] - lay.w_cnt[last];
    if (j >= 0 && j < lay.N[last]) {
        o.small[lay.b_off[last] + j] = a;
        o.small[lay.small + lay.b_off[last] + j] = b;
    }
}

// perturb (Sec. 3.2) fused with the operand preparation of the tensor-core
// forward pass: besides theta+ and theta- (each optional: a caller that wants
// neither saves their 8 B/element), every weight element is written as
// TF32 hi / lo into the row-padded split buffers of both branches, and the few
// values the forward pass reads in fp32 (biases, the weights of a narrow last
// layer that the fused head multiplies itself) go to a compact slab per
// branch, so the forward pass needs no further sweep over the parameters and
// never reads theta+-.  8 B/element read, 32 written for the operands, 8 for theta+-.
// Preconditions (checked on the host): 16-byte aligned pointers, every weight
// block starts at a multiple of 4 and has K % 4 == 0 and fewer than 2^31 elements.
__global__ void __launch_bounds__(kThreads)
perturb_split_kernel(int64_t n, const float* theta, const float* __restrict__ p, const double* __restrict__ sumsq,
                     float alpha, float* theta_plus, float* theta_minus, DeviceScalars* sc, float* eps_fd_out,
                     SplitLayout lay, float* __restrict__ hi, float* __restrict__ lo, float* __restrict__ small,
                     XSplitJob xjob) {
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

    const SplitDst dst{theta_plus, theta_minus, hi, lo, small};
    auto emit = [&](int64_t i, float4 vt, float4 vp) { emit_split(lay, dst, eps, i, vt, vp); };

    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (!theta_plus && !theta_minus && lay.skip_w != 0u) {
        // nothing is stored for the skipped layers' weights: only the other groups are read at all
        for (; i < items; i += stride)
            if (!skipped_weight(lay, i << 2)) emit(i, ld_stream(t4 + i), ld_stream(p4 + i));
        i = items;
    }
    for (; i + stride < items; i += stride * 2) {
        const float4 vt0 = ld_stream(t4 + i), vp0 = ld_stream(p4 + i);
        const float4 vt1 = ld_stream(t4 + i + stride), vp1 = ld_stream(p4 + i + stride);
        emit(i, vt0, vp0);
        emit(i + stride, vt1, vp1);
    }
    for (; i < items; i += stride) emit(i, ld_stream(t4 + i), ld_stream(p4 + i));
    if (blockIdx.x == 0) {  // n % 4 trailing elements: under the preconditions, the end of the last layer's bias
        const int64_t k = (items << 2) + threadIdx.x;
        if (k < n) emit_split_tail(lay, dst, eps, k, theta[k], p[k]);
    }
}

// adaptation + norm + perturbation + operand split in one launch (Eq. 4, Appendix C, Sec. 3.2), for parameter
// vectors small enough that every block keeps its share of p in shared memory across the norm: launched
// cooperatively (all blocks resident), a thread takes up to kFusedVec groups of four elements, writes p (it is an
// output) and its block's partial sum of squares, waits at a grid-wide barrier, adds the partials in index
// order (every block does, so all get the same bits), and goes on to the perturbation of the same elements.
// Against two launches this saves a launch, a ramp and a tail, and the re-read of p.  The barrier's wait is
// bounded: if it runs out the block raises SAMA_DEV_TIMEOUT and returns without perturbing.
constexpr int kFusedVec = 8;
constexpr long long kBarrierCycles = 4000000000LL;  // ~2 s

constexpr int kFusedSmem = kFusedVec * kThreads * 16;  // a block's share of p

template <bool HAS_G>
__global__ void __launch_bounds__(kThreads, 4)
fused_sweep_kernel(int64_t n, const float* theta, const float* __restrict__ m, const float* __restrict__ s,
                   const float* __restrict__ g, const float* gm, float* p, AdaptConsts c, float alpha,
                   float* theta_plus, float* theta_minus, double* partials, DeviceScalars* sc, SplitLayout lay,
                   float* __restrict__ hi, float* __restrict__ lo, float* __restrict__ small, XSplitJob xjob) {
    extern __shared__ float4 p_s[];   // [kFusedVec][kThreads]
    __shared__ double smem[kThreads / 32];
    __shared__ int gave_up;
    // the batch's operand split depends on nothing before it
    if (xjob.rows > 0) {
        const int q = xjob.ld_out >> 2;
        const int64_t total = xjob.rows * q, xstride = (int64_t)gridDim.x * kThreads;
        for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += xstride) {
            const int64_t r = i / q;
            const int col = (int)(i - r * q) << 2;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f), h, l;
            if (col < xjob.cols) x = __ldg(reinterpret_cast<const float4*>(xjob.x + r * xjob.cols + col));
            tf32_split(x, h, l);
            *reinterpret_cast<float4*>(xjob.hi + r * xjob.ld_out + col) = h;
            *reinterpret_cast<float4*>(xjob.lo + r * xjob.ld_out + col) = l;
        }
    }
    const int64_t items = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    const int64_t i0 = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const float4* m4 = reinterpret_cast<const float4*>(m);
    const float4* s4 = reinterpret_cast<const float4*>(s);
    const float4* g4 = reinterpret_cast<const float4*>(g);
    const float4* gm4 = reinterpret_cast<const float4*>(gm);
    const float4* t4 = reinterpret_cast<const float4*>(theta);
    float4* p4 = reinterpret_cast<float4*>(p);
    double acc = 0.0;
    // ---- first half: p and the block's share of sum p^2
#pragma unroll 4
    for (int v = 0; v < kFusedVec; ++v) {
        const int64_t i = i0 + stride * v;
        if (i < items) {
            float4 vm = make_float4(0.f, 0.f, 0.f, 0.f), vs = vm, vg = vm;
            if (!c.identity) {
                vm = ld_stream(m4 + i);
                vs = ld_stream(s4 + i);
                vg = HAS_G ? ld_stream(g4 + i) : vm;
            }
            const float4 o = adapt_four(vm, vs, vg, ld_stream(gm4 + i), c);
            p_s[v * kThreads + threadIdx.x] = o;
            p4[i] = o;
            acc += sq4(o);
        }
    }
    float tail_p = 0.f;
    const int64_t tail_k = (items << 2) + threadIdx.x;
    const bool has_tail = blockIdx.x == 0 && tail_k < n;
    if (has_tail) {
        float vm = 0.f, vs = 0.f, vg = 0.f;
        if (!c.identity) { vm = m[tail_k]; vs = s[tail_k]; vg = HAS_G ? g[tail_k] : vm; }
        tail_p = adapt_one(vm, vs, vg, gm[tail_k], c);
        p[tail_k] = tail_p;
        acc += (double)tail_p * tail_p;
    }
    const double mine = block_sum(acc, smem);
    // ---- grid barrier: publish, arrive, wait (bounded) for everybody
    if (threadIdx.x == 0) {
        partials[blockIdx.x] = mine;
        __threadfence();
        atomicAdd(&sc->counter, 1u);
        int bad = 0;
        const long long t0 = clock64();
        while (*reinterpret_cast<volatile unsigned int*>(&sc->counter) < gridDim.x) {
            if (clock64() - t0 > kBarrierCycles) { bad = 1; break; }
        }
        if (bad) atomicOr(&sc->status, (int)SAMA_DEV_TIMEOUT);
        gave_up = bad;
        __threadfence();
        // the last block to leave puts both counters back (everybody is past the wait by then)
        if (!bad && atomicAdd(&sc->departed, 1u) == gridDim.x - 1) {
            sc->counter = 0u;
            sc->departed = 0u;
        }
    }
    __syncthreads();
    if (gave_up) return;
    // ---- second half: the norm (same order in every block), then the perturbation of the same elements
    double v = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += kThreads) v += __ldcg(partials + b);
    const double part = block_sum(v, smem);
    __shared__ double total_s;
    if (threadIdx.x == 0) total_s = part;
    __syncthreads();
    const double sumsq = total_s;
    bool bad;
    const float eps = step_size(sumsq, alpha, bad);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        sc->sumsq = sumsq;
        sc->eps_fd = eps;
        if (bad) atomicOr(&sc->status, (int)SAMA_DEV_DEGENERATE_NORM);
    }
    const SplitDst dst{theta_plus, theta_minus, hi, lo, small};
    const bool sparse = !theta_plus && !theta_minus && lay.skip_w != 0u;  // most groups have nothing to store
#pragma unroll 2
    for (int vv = 0; vv < kFusedVec; ++vv) {
        const int64_t i = i0 + stride * vv;
        if (i < items && !(sparse && skipped_weight(lay, i << 2)))
            emit_split(lay, dst, eps, i, ld_stream(t4 + i), p_s[vv * kThreads + threadIdx.x]);
    }
    if (has_tail) emit_split_tail(lay, dst, eps, tail_k, theta[tail_k], tail_p);
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

bool fused_sweep_applicable(sama_ctx* ctx, int64_t n) {
    if (ctx->no_fused_sweep) return false;
    if (ctx->fused_sweep_blocks == 0) {
        int a = 0, b = 0;
        const bool ok = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, fused_sweep_kernel<true>, kThreads, kFusedSmem) == cudaSuccess &&
                        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, fused_sweep_kernel<false>, kThreads, kFusedSmem) == cudaSuccess;
        int coop = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device);
        const int per_sm = a < b ? a : b;
        ctx->fused_sweep_blocks = (ok && coop && per_sm >= 1) ? per_sm : -1;
        cudaGetLastError();
    }
    if (ctx->fused_sweep_blocks < 1) return false;
    int64_t grid = (int64_t)ctx->sm_count * ctx->fused_sweep_blocks;
    if (grid > kMaxPartials) grid = kMaxPartials;
    return (n >> 2) <= grid * kThreads * kFusedVec;
}

cudaError_t launch_fused_sweep(sama_ctx* ctx, int64_t n, const float* theta, const float* m, const float* s,
                               const float* g_base, const float* g_meta, const AdaptConsts& c, float alpha, float* p_out,
                               float* theta_plus, float* theta_minus, const SplitLayout& lay, float* hi, float* lo,
                               float* small, const XSplitJob& xjob, cudaStream_t st) {
    int64_t cap = (int64_t)ctx->sm_count * ctx->fused_sweep_blocks;
    if (cap > kMaxPartials) cap = kMaxPartials;
    // every block the device can hold at once: the sweep is latency-bound on small vectors, and more threads
    // mean more loads in flight (a thread then takes fewer than kFusedVec groups)
    int64_t grid = cap;
    const int64_t useful = ((n >> 2) + kThreads - 1) / kThreads;
    if (grid > useful) grid = useful < 1 ? 1 : useful;
    // all blocks must be resident at the barrier: a cooperative launch fails instead of deadlocking if they cannot be
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kFusedSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    KernelScope scope(ctx, SAMA_K_FUSED_SWEEP, -1, st);
    if (g_base)
        return cudaLaunchKernelEx(&cfg, fused_sweep_kernel<true>, n, theta, m, s, g_base, g_meta, p_out, c, alpha, theta_plus,
                                  theta_minus, ctx->partials, ctx->scalars, lay, hi, lo, small, xjob);
    return cudaLaunchKernelEx(&cfg, fused_sweep_kernel<false>, n, theta, m, s, (const float*)nullptr, g_meta, p_out, c, alpha,
                              theta_plus, theta_minus, ctx->partials, ctx->scalars, lay, hi, lo, small, xjob);
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
                                 const SplitLayout& lay, float* hi, float* lo, float* small, const XSplitJob& xjob,
                                 cudaStream_t st) {
    KernelScope scope(ctx, SAMA_K_PERTURB_SPLIT, -1, st);
    return launch_dependent(perturb_split_kernel, dim3(stream_grid(ctx, n >> 2, kUnroll)), dim3(kThreads), 0, st, n,
                            theta, p, sumsq, alpha, theta_plus, theta_minus, ctx->scalars, eps_fd_out, lay, hi, lo, small,
                            xjob);
}

}  // namespace sama
