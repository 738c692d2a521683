// Fused narrow classifier head + cross-entropy + central difference (Eq. 5).
//
// When the last layer has few outputs (C <= 16: the 10- and 4-class workloads)
// a tiled matrix product wastes almost all of its tile, and the logits would
// make a round trip through HBM only to be read once.  Here WPS warps (4 or 2 for
// small batches, so that the dependent-load chain is short and the grid still
// fills the machine; 1 for large batches) own one sample for BOTH branches:
// their threads split the contraction index, each thread accumulates the C
// partial dot products of z+ and z- in registers, warp shuffles and one pass
// through shared memory add them up in a fixed order, and one thread finishes
//   loss+- = logsumexp(z+-) - z+-[y],  metagrad = -sigmoid'(lambda) (loss+ - loss-) / (2 eps_fd B).
// Inputs are the fp32 hidden activations of both branches (or X itself for a
// single-layer model) and the last layer's weights and biases taken directly
// from theta+ and theta-.  All arithmetic is fp32 FMA.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kWarps = 8;

template <int CT, bool VEC, int WPS>
__global__ void __launch_bounds__(kWarps * 32)
head_ce_fd_kernel(const float* __restrict__ hp, const float* __restrict__ hm, int ldh,
                  const float* __restrict__ wp, const float* __restrict__ wm,
                  const float* __restrict__ bp, const float* __restrict__ bm,
                  const int32_t* __restrict__ y, const float* __restrict__ lambda, int B, int C, int K,
                  const float* __restrict__ eps_fd, float* __restrict__ metagrad,
                  float* __restrict__ loss_plus, float* __restrict__ loss_minus, float* __restrict__ loss_diff,
                  DeviceScalars* sc) {
    pdl_trigger();
    pdl_wait();
    constexpr int SPB = kWarps / WPS;  // samples per block
    __shared__ float part[kWarps][2 * CT];
    __shared__ float tot[SPB][2 * CT];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = warp / WPS, sub = warp % WPS;
    const int i = blockIdx.x * SPB + grp;
    const bool valid = i < B;
    const int row = valid ? i : 0;
    const int Kv = valid ? K : 0;  // a group past the end does no work but still reaches the barriers
    const float* xp = hp + (int64_t)row * ldh;
    const float* xm = hm + (int64_t)row * ldh;
    float ap[CT], am[CT];
#pragma unroll
    for (int c = 0; c < CT; ++c) ap[c] = am[c] = 0.f;

    if (VEC) {
        for (int k = (sub * 32 + lane) * 4; k < Kv; k += WPS * 128) {
            const float4 vp = *reinterpret_cast<const float4*>(xp + k);
            const float4 vm = *reinterpret_cast<const float4*>(xm + k);
#pragma unroll
            for (int c = 0; c < CT; ++c) {
                if (c < C) {
                    const float4 a = __ldg(reinterpret_cast<const float4*>(wp + (int64_t)c * K + k));
                    const float4 b = __ldg(reinterpret_cast<const float4*>(wm + (int64_t)c * K + k));
                    ap[c] = fmaf(vp.x, a.x, ap[c]); ap[c] = fmaf(vp.y, a.y, ap[c]);
                    ap[c] = fmaf(vp.z, a.z, ap[c]); ap[c] = fmaf(vp.w, a.w, ap[c]);
                    am[c] = fmaf(vm.x, b.x, am[c]); am[c] = fmaf(vm.y, b.y, am[c]);
                    am[c] = fmaf(vm.z, b.z, am[c]); am[c] = fmaf(vm.w, b.w, am[c]);
                }
            }
        }
    } else {
        for (int k = sub * 32 + lane; k < Kv; k += WPS * 32) {
            const float vp = xp[k], vm = xm[k];
#pragma unroll
            for (int c = 0; c < CT; ++c) {
                if (c < C) {
                    ap[c] = fmaf(vp, __ldg(wp + (int64_t)c * K + k), ap[c]);
                    am[c] = fmaf(vm, __ldg(wm + (int64_t)c * K + k), am[c]);
                }
            }
        }
    }
#pragma unroll
    for (int c = 0; c < CT; ++c) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ap[c] += __shfl_xor_sync(0xffffffffu, ap[c], o);
            am[c] += __shfl_xor_sync(0xffffffffu, am[c], o);
        }
        if (lane == 0) {
            part[warp][c] = ap[c];
            part[warp][CT + c] = am[c];
        }
    }
    __syncthreads();
    if (sub == 0 && lane < 2 * CT) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < WPS; ++w) t += part[grp * WPS + w][lane];
        tot[grp][lane] = t;
    }
    __syncthreads();
    if (sub != 0 || lane != 0 || !valid) return;

    const int label = y[i];
    const bool ok = (label >= 0 && label < C);
    if (!ok) atomicOr(&sc->status, (int)SAMA_DEV_BAD_LABEL);
    float mp = -INFINITY, mm = -INFINITY, zyp = 0.f, zym = 0.f;
#pragma unroll
    for (int c = 0; c < CT; ++c) {
        if (c < C) {
            ap[c] = tot[grp][c] + bp[c];
            am[c] = tot[grp][CT + c] + bm[c];
            mp = fmaxf(mp, ap[c]);
            mm = fmaxf(mm, am[c]);
            if (c == label) { zyp = ap[c]; zym = am[c]; }
        }
    }
    float sp = 0.f, sm = 0.f;
#pragma unroll
    for (int c = 0; c < CT; ++c) {
        if (c < C) {
            sp += expf(ap[c] - mp);
            sm += expf(am[c] - mm);
        }
    }
    const float lse_p = logf(sp) + mp, lse_m = logf(sm) + mm;
    if (loss_plus) loss_plus[i] = lse_p - zyp;
    if (loss_minus) loss_minus[i] = lse_m - zym;
    const float eps = *eps_fd;
    const float d = (lse_p - lse_m) - (zyp - zym);
    if (loss_diff) loss_diff[i] = ok ? d : 0.f;   // loss+ - loss- without the rounding of the two losses to fp32
    float out = 0.f;
    if (ok && eps > 0.f) {
        const float sg = 1.0f / (1.0f + expf(-lambda[i]));
        out = -(sg * (1.0f - sg)) * d / (2.0f * eps * (float)B);
    }
    metagrad[i] = out;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

bool head_applicable(int C) { return C >= 1 && C <= 16; }

cudaError_t launch_head_ce_fd(sama_ctx* ctx, const float* h_plus, const float* h_minus, int ldh,
                              const float* w_plus, const float* w_minus, const float* b_plus, const float* b_minus,
                              const int32_t* y, const float* lambda, int B, int C, int K, const float* eps_fd,
                              float* metagrad, float* loss_plus, float* loss_minus, float* loss_diff,
                              cudaStream_t st) {
    const bool vec = (K % 4 == 0) && (ldh % 4 == 0) && aligned16(h_plus) && aligned16(h_minus) &&
                     aligned16(w_plus) && aligned16(w_minus);
    // a whole block per sample while that still gives every SM a few blocks; a warp per sample beyond
    // warps per sample: more of them shorten each thread's chain of dependent loads, fewer give each block
    // more samples to reuse the head's weights from L1 (measured: 4 is best up to B = 8 #SM, 2 up to 32 #SM)
    const int64_t sms = ctx->sm_count;
    const int wps = (int64_t)B <= 8 * sms ? 4 : ((int64_t)B <= 32 * sms ? 2 : 1);
    const int spb = kWarps / wps;
    const int grid = (B + spb - 1) / spb;
    KernelScope scope(ctx, SAMA_K_HEAD, -1, st);
    cudaError_t err = cudaSuccess;
#define SAMA_HEAD2(CT, V, W)                                                                                       \
    err = launch_dependent(head_ce_fd_kernel<CT, V, W>, dim3(grid), dim3(kWarps * 32), 0, st, h_plus, h_minus, ldh, \
                           w_plus, w_minus, b_plus, b_minus, y, lambda, B, C, K, eps_fd, metagrad, loss_plus,      \
                           loss_minus, loss_diff, ctx->scalars)
#define SAMA_HEAD(CT, V) do { if (wps == 4) SAMA_HEAD2(CT, V, 4); else if (wps == 2) SAMA_HEAD2(CT, V, 2); else SAMA_HEAD2(CT, V, 1); } while (0)
    if (C <= 4) { if (vec) SAMA_HEAD(4, true); else SAMA_HEAD(4, false); }
    else if (C <= 10) { if (vec) SAMA_HEAD(10, true); else SAMA_HEAD(10, false); }
    else { if (vec) SAMA_HEAD(16, true); else SAMA_HEAD(16, false); }
#undef SAMA_HEAD
#undef SAMA_HEAD2
    return err;
}

}  // namespace sama
