// Cross-entropy of both branches and the central difference of Eq. 5.
//
// One warp per sample: lanes stride over the C logits of z+ and z-, a
// max / sum-exp pair per branch is reduced by shuffles, and lane 0 forms
//   loss+- = logsumexp(z+-) - z+-[y]
//   d      = (lse+ - lse-) - (z+[y] - z-[y])          (difference taken in one thread)
//   metagrad = -sigmoid'(lambda) d / (2 eps_fd B).
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kWarpsPerBlock = 4;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float logsumexp_row(const float* __restrict__ z, int C, int lane) {
    float mx = -INFINITY;
    for (int c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
    mx = warp_max(mx);
    float se = 0.f;
    for (int c = lane; c < C; c += 32) se += expf(z[c] - mx);
    se = warp_sum(se);
    return logf(se) + mx;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
ce_fd_kernel(const float* __restrict__ zp, const float* __restrict__ zm, int ldz, const int32_t* __restrict__ y,
             const float* __restrict__ lambda, int B, int C, const float* __restrict__ eps_fd,
             float* __restrict__ metagrad, float* __restrict__ loss_plus, float* __restrict__ loss_minus,
             float* __restrict__ loss_diff, DeviceScalars* sc) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (i >= B) return;
    const float* rp = zp + (int64_t)i * ldz;
    const float* rm = zm + (int64_t)i * ldz;
    const float lse_p = logsumexp_row(rp, C, lane);
    const float lse_m = logsumexp_row(rm, C, lane);
    if (lane != 0) return;
    const int label = y[i];
    const bool ok = (label >= 0 && label < C);
    if (!ok) atomicOr(&sc->status, (int)SAMA_DEV_BAD_LABEL);
    const float zyp = ok ? rp[label] : 0.f, zym = ok ? rm[label] : 0.f;
    if (loss_plus) loss_plus[i] = lse_p - zyp;
    if (loss_minus) loss_minus[i] = lse_m - zym;
    const float eps = *eps_fd;
    const float d = (lse_p - lse_m) - (zyp - zym);
    // loss+ - loss- as formed here, i.e. without the rounding of the two losses to fp32 (which is of the order
    // of the difference itself when the perturbation is small)
    if (loss_diff) loss_diff[i] = ok ? d : 0.f;
    float out = 0.f;
    if (ok && eps > 0.f) {
        const float sg = 1.0f / (1.0f + expf(-lambda[i]));
        out = -(sg * (1.0f - sg)) * d / (2.0f * eps * (float)B);
    }
    metagrad[i] = out;
}

}  // namespace

cudaError_t launch_ce_fd(sama_ctx* ctx, const float* z_plus, const float* z_minus, int ldz, const int32_t* y,
                         const float* lambda, int B, int C, const float* eps_fd, float* metagrad,
                         float* loss_plus, float* loss_minus, float* loss_diff, cudaStream_t st) {
    const int grid = (B + kWarpsPerBlock - 1) / kWarpsPerBlock;
    KernelScope scope(ctx, SAMA_K_CE_FD, -1, st);
    return launch_dependent(ce_fd_kernel, dim3(grid), dim3(kWarpsPerBlock * 32), 0, st, z_plus, z_minus, ldz, y, lambda,
                            B, C, eps_fd, metagrad, loss_plus, loss_minus, loss_diff, ctx->scalars);
}

}  // namespace sama
