// Dual-branch layer of the perturbed forward pass (Eq. 5) on the fp32 FMA
// pipe:   C[b] = act(A[b] W[b]^T + bias[b]),  b = 0 (theta+), 1 (theta-).
//
// A is [M][K] (batch x d_in), W is [N][K] (d_out x d_in), both row-major, so
// both operands are contiguous along the contraction index.  Tiles are
// staged through shared memory transposed to [k][row] with register
// prefetch of the next k-block (double buffering); each thread owns a
// TM x TN block of the output split into 4-wide groups so that shared-memory
// reads are 16-byte and conflict-free.  Both branches run in one launch
// (grid.z = 2) so that they see identical tile order and reduction order.
// Any M, N, K and any 4-byte alignment are accepted: out-of-range rows and
// k-indices read as zero, and unaligned operands take scalar loads.
#include "sama_internal.h"

namespace sama {

namespace {

constexpr int BK = 16;
constexpr int PAD = 4;

template <int BM, int BN, int TM, int TN, bool VEC>
__global__ void __launch_bounds__((BM / TM) * (BN / TN), 2)
gemm_ffma_kernel(GemmArgs g) {
    constexpr int NT = (BM / TM) * (BN / TN);
    constexpr int GM = TM / 4, GN = TN / 4;       // 4-wide groups per thread
    constexpr int SM_ = BM / GM, SN_ = BN / GN;   // distance between a thread's groups
    constexpr int QA = BM * BK / 4 / NT, QB = BN * BK / 4 / NT;
    static_assert(QA >= 1 && QB >= 1 && TM % 4 == 0 && TN % 4 == 0, "tile shape");

    __shared__ __align__(16) float As[2][BK][BM + PAD];
    __shared__ __align__(16) float Bs[2][BK][BN + PAD];

    const int br = blockIdx.z;
    const float* __restrict__ A = br ? g.A[1] : g.A[0];
    const float* __restrict__ W = br ? g.W[1] : g.W[0];
    const int M = g.M, N = g.N, K = g.K;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x;
    const int tx = tid % (BN / TN), ty = tid / (BN / TN);

    float4 ra[QA], rb[QB];

    auto fetch = [&](const float* __restrict__ base, int ld, int row0, int rows, int k0, int q) -> float4 {
        const int idx = tid + q * NT;
        const int row = row0 + idx / (BK / 4);
        const int k = k0 + (idx % (BK / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < rows) {
            const float* src = base + (int64_t)row * ld + k;
            if (VEC) {
                if (k < K) v = *reinterpret_cast<const float4*>(src);
            } else {
                if (k + 0 < K) v.x = src[0];
                if (k + 1 < K) v.y = src[1];
                if (k + 2 < K) v.z = src[2];
                if (k + 3 < K) v.w = src[3];
            }
        }
        return v;
    };
    auto load_tiles = [&](int k0) {
#pragma unroll
        for (int q = 0; q < QA; ++q) ra[q] = fetch(A, g.lda, m0, M, k0, q);
#pragma unroll
        for (int q = 0; q < QB; ++q) rb[q] = fetch(W, g.ldw, n0, N, k0, q);
    };
    auto store_tiles = [&](int buf) {
#pragma unroll
        for (int q = 0; q < QA; ++q) {
            const int idx = tid + q * NT, row = idx / (BK / 4), kq = (idx % (BK / 4)) * 4;
            As[buf][kq + 0][row] = ra[q].x;
            As[buf][kq + 1][row] = ra[q].y;
            As[buf][kq + 2][row] = ra[q].z;
            As[buf][kq + 3][row] = ra[q].w;
        }
#pragma unroll
        for (int q = 0; q < QB; ++q) {
            const int idx = tid + q * NT, row = idx / (BK / 4), kq = (idx % (BK / 4)) * 4;
            Bs[buf][kq + 0][row] = rb[q].x;
            Bs[buf][kq + 1][row] = rb[q].y;
            Bs[buf][kq + 2][row] = rb[q].z;
            Bs[buf][kq + 3][row] = rb[q].w;
        }
    };

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    const int ktiles = (K + BK - 1) / BK;
    load_tiles(0);
    store_tiles(0);
    __syncthreads();

    for (int t = 0; t < ktiles; ++t) {
        const int buf = t & 1;
        if (t + 1 < ktiles) load_tiles((t + 1) * BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[TM], b[TN];
#pragma unroll
            for (int gi = 0; gi < GM; ++gi) {
                const float4 v = *reinterpret_cast<const float4*>(&As[buf][kk][gi * SM_ + ty * 4]);
                a[gi * 4 + 0] = v.x; a[gi * 4 + 1] = v.y; a[gi * 4 + 2] = v.z; a[gi * 4 + 3] = v.w;
            }
#pragma unroll
            for (int gj = 0; gj < GN; ++gj) {
                const float4 v = *reinterpret_cast<const float4*>(&Bs[buf][kk][gj * SN_ + tx * 4]);
                b[gj * 4 + 0] = v.x; b[gj * 4 + 1] = v.y; b[gj * 4 + 2] = v.z; b[gj * 4 + 3] = v.w;
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (t + 1 < ktiles) {
            store_tiles(buf ^ 1);
            __syncthreads();
        }
    }

    // epilogue: bias, ReLU, store
    const float* __restrict__ bias = br ? g.bias[1] : g.bias[0];
    float* __restrict__ C = br ? g.C[1] : g.C[0];
    const bool vec_out = ((g.ldc & 3) == 0) && ((reinterpret_cast<uintptr_t>(C) & 15u) == 0);
#pragma unroll
    for (int gj = 0; gj < GN; ++gj) {
        const int n = n0 + gj * SN_ + tx * 4;
        float bv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) bv[j] = (bias != nullptr && n + j < N) ? bias[n + j] : 0.f;
#pragma unroll
        for (int gi = 0; gi < GM; ++gi) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + gi * SM_ + ty * 4 + i;
                if (m >= M) continue;
                float o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float v = acc[gi * 4 + i][gj * 4 + j] + bv[j];
                    o[j] = (g.relu && v < 0.f) ? 0.f : v;
                }
                float* dst = C + (int64_t)m * g.ldc + n;
                if (vec_out && n + 3 < N) {
                    *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (n + j < N) dst[j] = o[j];
                }
            }
        }
    }
}

template <int BM, int BN, int TM, int TN>
cudaError_t launch_variant(const GemmArgs& g, bool vec, cudaStream_t st) {
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, 2);
    constexpr int NT = (BM / TM) * (BN / TN);
    if (vec)
        gemm_ffma_kernel<BM, BN, TM, TN, true><<<grid, NT, 0, st>>>(g);
    else
        gemm_ffma_kernel<BM, BN, TM, TN, false><<<grid, NT, 0, st>>>(g);
    return cudaGetLastError();
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

cudaError_t launch_gemm_ffma(sama_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
    const bool vec = aligned16(g.A[0]) && aligned16(g.A[1]) && aligned16(g.W[0]) && aligned16(g.W[1]) &&
                     (g.lda % 4 == 0) && (g.ldw % 4 == 0) && (g.K % 4 == 0);
    auto ctas = [&](int bm, int bn) {
        return (int64_t)((g.M + bm - 1) / bm) * ((g.N + bn - 1) / bn) * 2;
    };
    KernelScope scope(ctx, SAMA_K_GEMM_FFMA, g.layer, st);
    // Largest tile that still gives every SM work; small problems take small tiles.
    if (ctas(128, 128) >= ctx->sm_count) return launch_variant<128, 128, 8, 8>(g, vec, st);
    if (ctas(64, 64) >= ctx->sm_count) return launch_variant<64, 64, 4, 4>(g, vec, st);
    return launch_variant<32, 32, 4, 4>(g, vec, st);
}

}  // namespace sama
