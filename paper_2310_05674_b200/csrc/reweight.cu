// Eq. 5 with a shared reweighting network as the meta learner (Sec. 4.1).
//
// The meta learner w(l; lambda_r) is a 2-layer MLP on the scalar per-sample loss:
//   a_j = v1_j l + c1_j,  h_j = max(0, a_j),  z = sum_j v2_j h_j + c2,  w = sigmoid(z),
// lambda_r = (v1[H], c1[H], v2[H], c2).  With L_base = (1/B) sum_i w(l_i) l_i, at fixed theta
//   dL_base/dlambda_r = (1/B) sum_i l_i w_i (1 - w_i) dz_i/dlambda_r,
// and the meta gradient is the central difference of that vector between theta+ and theta-,
//   metagrad_r = -[dL_base(theta+)/dlambda_r - dL_base(theta-)/dlambda_r] / (2 eps_fd).
// Input: the per-sample losses of both branches and, where available, their difference as the forward pass's
// last kernel formed it (the two fp32 losses each carry a rounding of the order of their difference).
//
// One warp per sample (grid-stride): the lanes split the hidden units, a shuffle reduction gives z for each
// branch, and every lane adds the per-sample DIFFERENCE of the two branches' terms for its own units to
// accumulators in registers.  Warps are added up through shared memory in warp order, blocks through a
// workspace in block order by the last block to arrive: no atomics on data, bitwise reproducible.  The
// arithmetic is double throughout (a few Mflop): the only rounding that matters is that of the fp32 losses.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int kWarps = 4;
constexpr int kUnitsPerLane = kMaxReweightHidden / 32;

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kWarps * 32)
reweight_fd_kernel(const float* __restrict__ loss_plus, const float* __restrict__ loss_minus,
                   const float* __restrict__ loss_diff, int B, int B_norm,
                   int H, const float* __restrict__ lambda_r, const float* __restrict__ eps_fd,
                   float* __restrict__ out, double* partials, DeviceScalars* sc) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int dim = 3 * H + 1;
    // this lane's hidden units: lane, lane + 32, ...
    double v1[kUnitsPerLane], c1[kUnitsPerLane], v2[kUnitsPerLane];
    double g_v1[kUnitsPerLane], g_c1[kUnitsPerLane], g_v2[kUnitsPerLane], g_c2 = 0.0;
#pragma unroll
    for (int u = 0; u < kUnitsPerLane; ++u) {
        const int j = lane + 32 * u;
        const bool in = j < H;
        v1[u] = in ? (double)lambda_r[j] : 0.0;
        c1[u] = in ? (double)lambda_r[H + j] : 0.0;
        v2[u] = in ? (double)lambda_r[2 * H + j] : 0.0;
        g_v1[u] = g_c1[u] = g_v2[u] = 0.0;
    }
    const double c2 = (double)lambda_r[3 * H];
    for (int i = blockIdx.x * kWarps + warp; i < B; i += gridDim.x * kWarps) {
        // with the difference given, loss+ is rebuilt from it: the fp32 rounding of loss+ itself is of the order
        // of loss+ - loss- for a small perturbation
        const double lm = (double)loss_minus[i];
        const double lp = loss_diff ? lm + (double)loss_diff[i] : (double)loss_plus[i];
        double zp = 0.0, zm = 0.0;
#pragma unroll
        for (int u = 0; u < kUnitsPerLane; ++u) {
            const double ap = fma(v1[u], lp, c1[u]), am = fma(v1[u], lm, c1[u]);
            if (ap > 0.0) zp = fma(v2[u], ap, zp);
            if (am > 0.0) zm = fma(v2[u], am, zm);
        }
        zp = warp_sum_d(zp) + c2;
        zm = warp_sum_d(zm) + c2;
        const double wp = 1.0 / (1.0 + exp(-zp)), wm = 1.0 / (1.0 + exp(-zm));
        const double fp = lp * wp * (1.0 - wp), fm = lm * wm * (1.0 - wm);
#pragma unroll
        for (int u = 0; u < kUnitsPerLane; ++u) {
            const double ap = fma(v1[u], lp, c1[u]), am = fma(v1[u], lm, c1[u]);
            const double tp = ap > 0.0 ? fp * v2[u] : 0.0, tm = am > 0.0 ? fm * v2[u] : 0.0;
            g_v1[u] += tp * lp - tm * lm;
            g_c1[u] += tp - tm;
            g_v2[u] += (ap > 0.0 ? fp * ap : 0.0) - (am > 0.0 ? fm * am : 0.0);
        }
        g_c2 += fp - fm;   // the same value in every lane
    }
    // warps -> block, in warp order
    __shared__ double acc[kWarps][3 * kMaxReweightHidden + 1];
    __shared__ bool is_last;
#pragma unroll
    for (int u = 0; u < kUnitsPerLane; ++u) {
        const int j = lane + 32 * u;
        if (j < H) {
            acc[warp][j] = g_v1[u];
            acc[warp][H + j] = g_c1[u];
            acc[warp][2 * H + j] = g_v2[u];
        }
    }
    if (lane == 0) acc[warp][3 * H] = g_c2;
    __syncthreads();
    for (int k = threadIdx.x; k < dim; k += kWarps * 32) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += acc[w][k];
        partials[(size_t)blockIdx.x * dim + k] = t;
    }
    // blocks -> total, in block order, by the last block to arrive
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(&sc->counter, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const double eps = (double)*eps_fd;
    const double scale = eps > 0.0 ? -1.0 / (2.0 * eps * (double)B_norm) : 0.0;
    for (int k = threadIdx.x; k < dim; k += kWarps * 32) {
        double t = 0.0;
        for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(partials + (size_t)b * dim + k);
        out[k] = (float)(t * scale);
    }
    if (threadIdx.x == 0) sc->counter = 0u;
}

}  // namespace

int reweight_grid(const sama_ctx* ctx, int B) {
    int g = (B + kWarps - 1) / kWarps;
    if (g > 2 * ctx->sm_count) g = 2 * ctx->sm_count;
    if (g > kMaxReweightBlocks) g = kMaxReweightBlocks;
    return g < 1 ? 1 : g;
}

cudaError_t launch_reweight_fd(sama_ctx* ctx, const float* loss_plus, const float* loss_minus,
                               const float* loss_diff, int B, int B_norm, int H, const float* lambda_r,
                               const float* eps_fd, float* out, cudaStream_t st) {
    KernelScope scope(ctx, SAMA_K_REWEIGHT_FD, -1, st);
    return launch_dependent(reweight_fd_kernel, dim3(reweight_grid(ctx, B)), dim3(kWarps * 32), 0, st, loss_plus,
                            loss_minus, loss_diff, B, B_norm, H, lambda_r, eps_fd, out, ctx->rw_partials, ctx->scalars);
}

}  // namespace sama
