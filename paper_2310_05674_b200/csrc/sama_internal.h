// Internal declarations shared by the translation units of libsama.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "sama.h"

namespace sama {

constexpr int kMaxLayers = 16;
constexpr int kMaxPartials = 4096;  // upper bound on the grid of the reduction kernels
constexpr int kTcFlags = 1024;      // arrival counters of the tensor-core kernel's shared tail tiles
constexpr int kMaxReweightHidden = 256;  // widest hidden layer of the shared reweighting network
constexpr int kMaxReweightBlocks = 512;  // upper bound on the grid of its reduction

// Device scalars owned by a context.
struct DeviceScalars {
    double sumsq;          // sum p^2 of the last adapt
    float eps_fd;          // alpha / ||p|| of the last perturb
    int32_t status;        // OR of SAMA_DEV_* bits
    unsigned int counter;  // arrival counter of the last-block-done reductions and of the fused sweep's grid barrier (returns to 0)
    unsigned int departed; // blocks that have left the fused sweep's grid barrier (returns to 0)
};

// Host-precomputed constants of the Adam adaptation matrix (Appendix C).
struct AdaptConsts {
    float a;        // lr / c1
    float b1, b2;   // beta1, beta2
    float omb1;     // 1 - beta1
    float omb2;     // 1 - beta2
    float inv_rc2;  // 1 / sqrt(c2)
    float eps;      // Adam's epsilon
    int drop_eps_term;
    int identity;
};

// Where each layer's weight matrix lives in the flat parameter vector and in one
// branch slab of the TF32 hi/lo split buffers (rows padded to a multiple of 32).
struct SplitLayout {
    int n_layers;
    int32_t K[kMaxLayers], Kp[kMaxLayers];
    int64_t w_off[kMaxLayers];  // offset of W_l in theta
    int64_t w_cnt[kMaxLayers];  // d_l * d_{l-1}
    int64_t s_off[kMaxLayers];  // offset of layer l inside a slab
    int64_t slab;               // floats per slab = sum_l d_l * Kp_l
    // What the forward pass reads in fp32 besides the split operands, kept compact per branch ("small slab"):
    // the weights of a narrow last layer that the fused head kernel multiplies itself (first, so that every
    // block starts at a multiple of 4), then every layer's bias.
    int32_t N[kMaxLayers];      // d_l (length of layer l's bias)
    int64_t b_off[kMaxLayers];  // offset of layer l's bias inside a small slab
    int head_layer;             // index of the layer whose fp32 weights are kept (the fused head's), or -1
    int64_t head_cnt;           // its weight count (at offset 0 of the small slab), else 0
    int64_t small;              // floats per small slab
    // Bit l set: the forward forms layer l's W operands itself from theta and p, so the sweep writes none for it.
    uint32_t skip_w;
};

// The batch X as an extra job of the fused perturbation sweep: its TF32 hi/lo split, rows padded to ld_out.
// rows == 0 means "no X job".  Requires cols % 4 == 0 and a 16-byte aligned X.
struct XSplitJob {
    const float* x;
    float* hi;
    float* lo;
    int64_t rows;
    int cols, ld_out;
};

struct ProfRecord {
    int kind, layer, launches;
    cudaEvent_t start, stop;
};
struct Profiler {
    bool on = false;
    bool grouped = false;  // consecutive launches of one kind share a record (one event pair around the run)
    std::vector<ProfRecord> records;
};

}  // namespace sama

struct sama_ctx {
    int device;
    int sm_count;
    int64_t max_n;
    int32_t max_batch;
    int32_t max_width;    // widest hidden layer the forward workspace covers, 0 if none
    int32_t max_classes;  // largest d_L covered, 0 if the context has no forward workspace
    int gemm_mode;        // 0 auto, 1 ffma, 2 3xTF32, 3 3xTF32 with W+- formed in the product kernel's operand stage
    int last_cuda_error;
    int fused_sweep_blocks;  // co-resident blocks per SM of the fused sweep kernel on this device (0: not yet asked, -1: unavailable)
    int no_fused_sweep;      // SAMA_NO_FUSED_SWEEP=1 (experiment switch, read at sama_create)
    int last_forward_path;  // how the last forward pass multiplied matrices: 0 none yet, 1 fp32 FMA, 2 tensor cores
    void* tc_state;       // host: state of the tensor-core path (switches, unit counts, tensor-map cache), or null
    int64_t launches;
    sama::DeviceScalars* scalars;  // device
    double* partials;              // device [kMaxPartials]
    float* act[2];                 // device: ping-pong activations, each [2][max_batch][max_width]
    float* logits;                 // device [2][max_batch][max_classes]
    // TF32 hi/lo operand splits of the tensor-core path, each buffer holds hi then lo
    float* x_split;                // device [2][max_batch][round32(d_0)]
    float* w_split;                // device [hi, lo][2 branches][slab]: every layer's W, rows padded to 32
    float* a_split[2];             // device, ping-pong: [2][2][max_batch][round32(max hidden)]
    size_t x_split_half, w_split_half, a_split_half;  // floats per hi (or lo) part; 0 = path unavailable
    float* pm_small;               // device [2 branches][pm_small_half]: fp32 biases and fused-head weights of theta+ / theta-
    size_t pm_small_half;
    float* pm_scratch;             // device [2][n]: theta+ / theta- when the caller wants neither and the forward needs them (allocated on first use)
    size_t pm_scratch_floats;
    float* tc_ws;                  // device: partial tiles of the tensor-core path's K-split (one 128 x 256 tile per SM)
    int* tc_flags;                 // device [kTcFlags], zero between launches
    size_t tc_ws_floats;
    float* mg_ws;                  // device: workspace of the direct gradient (activations, dz, losses)
    size_t mg_ws_floats;
    float* mg_tc;                  // device: TF32 operand buffers of the direct gradient's tensor-core path
    size_t mg_tc_floats;
    double* rw_partials;           // device [kMaxReweightBlocks][3 kMaxReweightHidden + 1]: block partials of the reweighting-network gradient
    float* rw_buf;                 // device [5][max_batch]: losses of both branches, zero logits, scratch meta gradient (sama_step_reweight);
                                   // [4]: loss+ - loss- of the last forward pass, as formed inside its last kernel
    double* br_partials;           // device: block partials of the biased-regression direct gradient (allocated on first use)
    size_t br_partials_doubles;
    float* stage;                  // device: staging of the host entry point (allocated on first use)
    size_t stage_bytes;
    sama::Profiler* prof;          // host
};

namespace sama {

// Counts a launch and, while profiling is on, brackets it with two events on its stream.
struct KernelScope {
    sama_ctx* ctx;
    cudaStream_t st;
    cudaEvent_t stop = nullptr;
    KernelScope(sama_ctx* c, int kind, int layer, cudaStream_t s) : ctx(c), st(s) {
        ctx->launches += 1;
        if (ctx->prof && ctx->prof->on) {
            std::vector<ProfRecord>& recs = ctx->prof->records;
            if (ctx->prof->grouped && !recs.empty() && recs.back().kind == kind) {
                // same kind as the launch before: no event in between (it would serialise the two launches and
                // undo their dependent-launch overlap); the record's stop event is recorded again after this one
                recs.back().launches += 1;
                recs.back().layer = -1;
                stop = recs.back().stop;
                return;
            }
            ProfRecord r{kind, layer, 1, nullptr, nullptr};
            if (cudaEventCreate(&r.start) == cudaSuccess && cudaEventCreate(&r.stop) == cudaSuccess) {
                cudaEventRecord(r.start, st);
                stop = r.stop;
                recs.push_back(r);
            }
        }
    }
    ~KernelScope() {
        if (stop) cudaEventRecord(stop, st);
    }
};

// sama_api.cu : host-side checks of the adaptation's arguments (no launch)
int check_adam(const sama_adam_t* a, AdaptConsts* out);
int validate_adapt(int64_t max_n, int64_t n, const float* m, const float* s, const float* g_base,
                   const float* g_meta, const sama_adam_t* adam, float* p_out, double* sumsq_out, AdaptConsts* c);

// Programmatic dependent launch: a kernel launched this way may start (and run its prologue) while
// the previous kernel on the stream is still finishing; it must execute pdl_wait() before it touches
// anything the previous kernels wrote or still read.  pdl_wait() is a no-op under a plain launch.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
bool pdl_enabled();
extern thread_local int pdl_override;  // -1: follow pdl_enabled(); 0 / 1: force off / on for the launches that follow
struct PdlScope {  // sets pdl_override for the lifetime of the object
    int old;
    explicit PdlScope(int v) : old(pdl_override) { pdl_override = v; }
    ~PdlScope() { pdl_override = old; }
    PdlScope(const PdlScope&) = delete;
    PdlScope& operator=(const PdlScope&) = delete;
};
template <typename... KArgs, typename... Args>
cudaError_t launch_clustered(int cluster_x, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                             cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (cluster_x > 1) {  // thread-block cluster of cluster_x CTAs along x
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster_x;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl_override >= 0 ? pdl_override != 0 : pdl_enabled()) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             Args&&... args) {
    return launch_clustered(1, kernel, grid, block, smem, st, static_cast<Args&&>(args)...);
}

// adapt_perturb.cu
cudaError_t launch_adapt_sumsq(sama_ctx* ctx, int64_t n, const float* m, const float* s, const float* g_base,
                               const float* g_meta, const AdaptConsts& c, float* p_out, double* sumsq_out,
                               cudaStream_t st);
cudaError_t launch_sumsq(sama_ctx* ctx, int64_t n, const float* p, cudaStream_t st);
cudaError_t launch_perturb(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* sumsq,
                           float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out, cudaStream_t st);
// perturb that also writes the TF32 hi/lo split of every weight matrix of theta+ and theta- (same sweep)
// adaptation + norm + perturbation + operand split in ONE cooperative launch, for models small enough that p
// stays in registers between the two halves (a grid-wide barrier with a bounded wait separates them)
bool fused_sweep_applicable(sama_ctx* ctx, int64_t n);
cudaError_t launch_fused_sweep(sama_ctx* ctx, int64_t n, const float* theta, const float* m, const float* s,
                               const float* g_base, const float* g_meta, const AdaptConsts& c, float alpha, float* p_out,
                               float* theta_plus, float* theta_minus, const SplitLayout& lay, float* hi, float* lo,
                               float* small, const XSplitJob& xjob, cudaStream_t st);
bool perturb_split_applicable(const SplitLayout& lay, const float* theta, const float* p, const float* theta_plus,
                              const float* theta_minus);
cudaError_t launch_perturb_split(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* sumsq,
                                 float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out,
                                 const SplitLayout& lay, float* hi, float* lo, float* small, const XSplitJob& xjob,
                                 cudaStream_t st);

// One layer of both branches: C[b] = act(A[b] * W[b]^T + bias[b]) for b in {0, 1}
struct GemmArgs {
    const float* A[2];     // [M][lda]
    const float* W[2];     // [N][ldw]
    const float* bias[2];  // [N]
    float* C[2];           // [M][ldc]
    int M, N, K;
    int lda, ldw, ldc;
    int relu;
    int layer;
};
// gemm_ffma.cu
cudaError_t launch_gemm_ffma(sama_ctx* ctx, const GemmArgs& g, cudaStream_t st);
// sama_api.cu : picks the matrix-product path of one layer
cudaError_t launch_gemm(sama_ctx* ctx, const GemmArgs& g, cudaStream_t st);

// gemm_tf32x3.cu : tensor-core path (3xTF32)
struct TcLayer {
    const float* a_hi;     // [shared_a ? 1 : 2][M][round32(K)]
    const float* a_lo;
    const float* w_hi;     // [2][N][round32(K)], branch b at w_hi + b * w_slab
    const float* w_lo;
    int64_t w_slab;
    const float* bias[2];  // [N]
    float* out_f32[2];     // last layer: [M][ldc]
    float* out_hi;         // hidden layers: [2][M][round32(N)]
    float* out_lo;
    int M, N, K, ldc;
    int relu, last, shared_a, layer;
    int branches = 2;            // 1: only branch 0 (the direct gradient)
    int both = 0;                // hidden layer that also stores fp32 to out_f32
    const float* mask = nullptr; // [M][ldm]: zero the result where mask <= 0
    int ldm = 0;
    // When w_theta is given, w_hi / w_lo are ignored: the kernel forms the operands of theta +- eps_fd p itself
    // from this layer's weights inside theta and p ([N][K] fp32; 16-byte aligned, K % 4 == 0, K >= 32).
    const float* w_theta = nullptr;
    const float* w_p = nullptr;
    const float* eps_fd = nullptr;  // device
};
// hi/lo of the TRANSPOSE of a dense fp32 matrix [rows][cols]: out [cols][round32(rows)], zero padded
cudaError_t launch_split_transpose_tf32(sama_ctx* ctx, const float* src, int64_t rows, int cols, float* hi, float* lo,
                                        cudaStream_t st);
cudaError_t launch_split_tf32(sama_ctx* ctx, const float* src0, const float* src1, int branches, int64_t rows,
                              int cols, float* hi, float* lo, int64_t slab, cudaStream_t st);
cudaError_t launch_gemm_tf32x3(sama_ctx* ctx, const TcLayer& L, cudaStream_t st);
cudaError_t launch_wait_expiry(sama_ctx* ctx, long long limit_cycles, long long* waited_cycles, cudaStream_t st);
cudaError_t tc_state_create(sama_ctx* ctx);  // with ctx->device current and ctx->sm_count set
void tc_state_destroy(sama_ctx* ctx);

// ce_fd.cu
cudaError_t launch_ce_fd(sama_ctx* ctx, const float* z_plus, const float* z_minus, int ldz, const int32_t* y,
                         const float* lambda, int B, int C, const float* eps_fd, float* metagrad,
                         float* loss_plus, float* loss_minus, float* loss_diff, cudaStream_t st);

// head_ce_fd.cu : narrow last layer (C <= 16) + cross-entropy + central difference in one kernel
bool head_applicable(int C);
cudaError_t launch_head_ce_fd(sama_ctx* ctx, const float* h_plus, const float* h_minus, int ldh,
                              const float* w_plus, const float* w_minus, const float* b_plus, const float* b_minus,
                              const int32_t* y, const float* lambda, int B, int C, int K, const float* eps_fd,
                              float* metagrad, float* loss_plus, float* loss_minus, float* loss_diff,
                              cudaStream_t st);

// reweight.cu : Eq. 5 with the shared reweighting network of Sec. 4.1
cudaError_t launch_reweight_fd(sama_ctx* ctx, const float* loss_plus, const float* loss_minus,
                               const float* loss_diff, int B, int B_norm, int H, const float* lambda_r,
                               const float* eps_fd, float* out, cudaStream_t st);

// biasreg.cu : the biased-regression objective of Appendix E
int biasreg_grid(const sama_ctx* ctx, int n_val);
cudaError_t launch_biasreg_direct_grad(sama_ctx* ctx, int d, int n_val, const float* Xv, const float* yv,
                                       const float* w, float* g_out, float* loss_out, cudaStream_t st);
cudaError_t launch_biasreg_fd(sama_ctx* ctx, int64_t d, const float* w_plus, const float* w_minus,
                              const float* lambda, float beta, const float* eps_fd, float* out, cudaStream_t st);

// meta_grad.cu : direct gradient dL_meta/dtheta (Eq. 1)
size_t meta_grad_workspace_floats(const sama_mlp_t* mlp, int64_t B);
size_t meta_grad_tc_floats(const sama_mlp_t* mlp, int64_t B);
SplitLayout make_split_layout(const sama_mlp_t* mlp);  // sama_api.cu
cudaError_t run_meta_grad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X, const int32_t* y,
                          int32_t B, float* g_out, float* loss_out, cudaStream_t st);

}  // namespace sama
