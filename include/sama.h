/*
 * sama.h -- C ABI of the B200 (sm_100a) SAMA meta-gradient library.
 *
 * SAMA ("Making Scalable Meta Learning Practical", arXiv 2310.05674) computes
 * the meta gradient without second-order products:
 *
 *   p        = (du/dg_base) * g_meta             Eq. 4; Adam matrix: Appendix C
 *   eps_fd   = alpha / ||p||_2                   Sec. 3.2
 *   theta+-  = theta +- eps_fd * p               Sec. 3.2
 *   dL_meta/dlambda ~= -[dL_base(theta+)/dlambda - dL_base(theta-)/dlambda] / (2 eps_fd)   Eq. 5
 *
 * Here lambda are per-sample weight logits of a data-reweighting objective
 * (Sec. 4.1):  L_base = (1/B) sum_i sigmoid(lambda_i) * CE(f(x_i; theta), y_i),
 * f an MLP, so Eq. 5 needs only per-sample losses at theta+ and theta-.
 *
 * Conventions
 *   - Every array pointer is a DEVICE pointer owned by the caller unless the
 *     argument is documented as "host".  The library never frees, reallocates
 *     or keeps caller memory.  Structs (sama_adam_t, sama_mlp_t and the dims
 *     array) are HOST memory, read during the call only.
 *   - Arrays are fp32, contiguous.  Pointers need 4-byte alignment; 16-byte
 *     alignment selects the vectorised kernels (same results).
 *   - The flat parameter vector is W1, b1, W2, b2, ..., W_l stored
 *     [d_l][d_{l-1}] row-major; the batch X is [B][d_0] row-major; labels are
 *     int32 in [0, d_L).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *     work is enqueued on it; no call synchronises unless it says so.
 *   - Return value: SAMA_OK or a negative sama_status.  Argument errors are
 *     detected on the host before anything is launched.  Conditions that only
 *     the device can see (zero / non-finite ||p||, label out of range, an
 *     internal wait that ran out) set bits in a device status word that
 *     sama_device_status() reads; the kernels then write defined values
 *     (theta+- = theta, metagrad = 0) instead of faulting.
 *   - A context serialises nothing: calls that use the same context on
 *     different streams at the same time race on its workspace.
 */
#ifndef SAMA_H
#define SAMA_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum sama_status {
    SAMA_OK = 0,
    SAMA_ERR_NULL = -1,    /* a required pointer is NULL */
    SAMA_ERR_ALIGN = -2,   /* a pointer is not aligned to its element type */
    SAMA_ERR_SIZE = -3,    /* n < 0, n != parameter count of the MLP, B < 1, sizes beyond the context's limits */
    SAMA_ERR_PARAM = -4,   /* step < 1 with bias correction, beta outside [0,1), non-finite or non-positive lr/eps/alpha */
    SAMA_ERR_OVERLAP = -5, /* buffers overlap in a way that is not allowed */
    SAMA_ERR_CUDA = -6,    /* a CUDA runtime call failed; see sama_last_cuda_error() */
    SAMA_ERR_NOMEM = -7,   /* workspace allocation failed */
    SAMA_ERR_UNSUPPORTED = -8
} sama_status;

/* Bits of the device status word. */
enum {
    SAMA_DEV_DEGENERATE_NORM = 1, /* ||p|| was 0 or not finite: eps_fd = 0, theta+- = theta, metagrad = 0 */
    SAMA_DEV_BAD_LABEL = 2,       /* a label outside [0, d_L): that sample's metagrad is 0 */
    SAMA_DEV_TIMEOUT = 4          /* a bounded wait inside a kernel expired; outputs of that call are invalid, and the
                                     context's arrival counters may be left non-zero: destroy and recreate it */
};

/* Base optimiser state that the adaptation differentiates (Appendix C).
 * The update is u = (lr/c1) m' / (sqrt(s')/sqrt(c2) + eps) with
 * m' = beta1 m + (1-beta1) g, s' = beta2 s + (1-beta2) g^2 and
 * c1 = 1-beta1^step, c2 = 1-beta2^step.  (m, s) are the moments BEFORE this
 * update; `step` >= 1 is the index of the update. */
typedef struct sama_adam_t {
    float lr, beta1, beta2, eps;
    int64_t step;
    int32_t bias_correction; /* 1: as above.  0: c1 = c2 = 1, the form printed in Appendix C */
    int32_t drop_eps_term;   /* 0: exact derivative.  1: Appendix C's last line (eps-term of the numerator dropped) */
    int32_t identity;        /* 1: du/dg = I (SGD base optimiser, Sec. 3.2; the SAMA-NA variant of Sec. 4.1) */
} sama_adam_t;

/* Base model: fully connected, ReLU between layers, last layer linear.
 * dims (host) has n_layers + 1 entries d_0 .. d_L. */
typedef struct sama_mlp_t {
    int32_t n_layers;
    const int32_t* dims;
} sama_mlp_t;

typedef struct sama_ctx sama_ctx;

/* Creates a context on `device` with workspace for flat vectors up to max_n
 * elements and, if `mlp` is given, for forward passes of that model (or any
 * model whose widest layer and class count are not larger) on batches up to
 * max_batch.  Allocates device memory; synchronises.  mlp may be NULL
 * (adapt/perturb only). */
int sama_create(sama_ctx** out, int device, int64_t max_n, int32_t max_batch, const sama_mlp_t* mlp);

/* Frees the workspace.  The caller must have synchronised the streams used. */
int sama_destroy(sama_ctx* ctx);

/* Eq. 4 + Appendix C, fused with the squared norm of Sec. 3.2:
 *   p_out[k] = J_k * g_meta[k],  J_k = du/dg at element k,  and  sum_k p_out[k]^2.
 * m, s, g_meta: [n].  g_base: [n] or NULL (then g := m, the optimiser's own
 * running estimate of the gradient).  p_out: [n]; may be the same pointer as
 * g_meta (in place).  sumsq_out: one double on the device, or NULL; the sum
 * is also left in the context (sama_ctx_sumsq).  The sum is accumulated in
 * double in a fixed order: repeated calls give bit-identical results.
 * n = 0 is allowed (sum = 0). */
int sama_adapt(sama_ctx* ctx, int64_t n, const float* m, const float* s, const float* g_base,
               const float* g_meta, const sama_adam_t* adam, float* p_out, double* sumsq_out, void* stream);

/* sama_adapt without a context and without any allocation.  (The paper has no
 * counterpart: this entry point exists for the deployment reason below.)
 *
 * sama_create allocates the reduction's scratch with cudaMalloc.  Callers that
 * may not allocate -- code living under a framework whose caching allocator
 * owns the device and forbids raw cudaMalloc, a plug-in loaded after a serving
 * engine has sized and frozen its memory pools, initialisation paths where a
 * synchronising allocation is not permitted -- use this instead: the scratch
 * (one partial per block, an arrival counter; 33,024 bytes) is a static device
 * array that every GPU loading the library holds until the process exits.
 *
 * Same arguments and results as sama_adapt, on the CURRENT device, except:
 *   - sumsq_out (one double on the device) is required: there is no context
 *     to leave the sum in;
 *   - n may not exceed SAMA_NOALLOC_MAX_N; larger n returns SAMA_ERR_SIZE
 *     before anything is launched (use sama_adapt with a context);
 *   - the first call on each device resolves the array's device address
 *     (cudaGetSymbolAddress) and reads the SM count; make that first call
 *     outside any stream capture;
 *   - every call on a device shares the one array.  It is cleared on the
 *     stream at the start of each call, so calls issued one after another on
 *     one stream are safe; calls that can overlap on the GPU (different
 *     streams, no ordering) race on it and give wrong sums.
 *   - the resolved address is remembered for the life of the process; after a
 *     cudaDeviceReset on that device it is stale, and this entry point must
 *     not be called again in that process.
 * Calls cudaGetDevice, cudaGetSymbolAddress / cudaDeviceGetAttribute (first
 * call only), cudaMemsetAsync and one kernel launch; never cudaMalloc or
 * cudaFree. */
#define SAMA_NOALLOC_MAX_N ((int64_t)1 << 30)
int sama_adapt_noalloc(int64_t n, const float* m, const float* s, const float* g_base, const float* g_meta,
                       const sama_adam_t* adam, float* p_out, double* sumsq_out, void* stream);

/* Sec. 3.2: eps_fd = alpha / sqrt(sumsq);  theta_plus = theta + eps_fd p,
 * theta_minus = theta - eps_fd p, written in one sweep.
 * p_sumsq: device double holding sum p^2 (e.g. sama_adapt's), or NULL to have
 * it computed here from p (one extra read of p).  theta_minus may be the same
 * pointer as theta: that is the base-parameter nudge theta <- theta - eps_fd p
 * the paper applies at each meta update (Sec. 3.2).  eps_fd_out: one float on
 * the device, or NULL; eps_fd is also left in the context (sama_ctx_eps_fd).
 * If the norm is 0 or not finite: eps_fd = 0, theta+- = theta,
 * SAMA_DEV_DEGENERATE_NORM is set. */
int sama_perturb(sama_ctx* ctx, int64_t n, const float* theta, const float* p, const double* p_sumsq,
                 float alpha, float* theta_plus, float* theta_minus, float* eps_fd_out, void* stream);

/* Eq. 5 for per-sample weight logits.  Runs the MLP on X at theta_plus and at
 * theta_minus (both branches in the same launches), then
 *   metagrad[i] = -sigmoid'(lambda_i) (loss+_i - loss-_i) / (2 eps_fd B),
 *   loss_i = logsumexp(z_i) - z_i[y_i].
 * theta_plus, theta_minus: [n_params(mlp)].  X: [B][d_0].  y: int32 [B].
 * lambda: [B].  eps_fd: one float on the device (NULL: the context's, as left
 * by the last sama_perturb).  metagrad_out: [B].  loss_plus_out,
 * loss_minus_out: [B] or NULL.  All matrix products are carried out in
 * arithmetic that is faithful to fp32 (the difference of the two branches is
 * ~1e-3 of the losses, so reduced-precision products are not usable). */
int sama_fd_metagrad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta_plus, const float* theta_minus,
                     const float* X, const int32_t* y, const float* lambda, int32_t B, const float* eps_fd,
                     float* metagrad_out, float* loss_plus_out, float* loss_minus_out, void* stream);

/* The whole meta-gradient step of Fig. 2 with lambda = per-sample weights:
 * sama_adapt -> sama_perturb -> sama_fd_metagrad on one stream, no host
 * synchronisation in between.  n must equal the parameter count of mlp.
 * Outputs: p_out [n] (may alias g_meta), theta_plus [n], theta_minus [n] (may
 * alias theta), metagrad_out [B]; loss_*_out optional.  theta_plus and / or
 * theta_minus may be NULL when the caller has no use for them: the tensor-core
 * forward reads its own operand copies, so a NULL output is then never written
 * to memory at all (4 B/element less traffic each); on the fp32 FMA path the
 * context keeps it in scratch allocated on first use (cudaMalloc; synchronises). */
int sama_step(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta, const float* m,
              const float* s, const float* g_base, const float* g_meta, const sama_adam_t* adam, float alpha,
              const float* X, const int32_t* y, const float* lambda, int32_t B,
              float* p_out, float* theta_plus, float* theta_minus, float* metagrad_out,
              float* loss_plus_out, float* loss_minus_out, void* stream);

/* Direct gradient, the first factor of Eq. 1: g_meta = dL_meta/dtheta for the meta objective of
 * Sec. 4.1, L_meta(theta) = (1/B) sum_i CE(f(x_i; theta), y_i) on a clean batch, by reverse
 * differentiation of the same MLP (fp32).  Its output is the `g_meta` input of sama_adapt / sama_step.
 * theta: [n_params(mlp)].  X_meta: [B][d_0].  y_meta: int32 [B].  g_meta_out: [n_params(mlp)], must not
 * overlap the inputs.  loss_out: one float on the device (the mean loss), or NULL.  A label outside
 * [0, d_L) sets SAMA_DEV_BAD_LABEL and that sample contributes nothing.  Needs a context created
 * with an mlp whose layer widths are not smaller, B <= max_batch.  Results are reproducible bit for bit. */
int sama_meta_grad(sama_ctx* ctx, const sama_mlp_t* mlp, const float* theta, const float* X_meta,
                   const int32_t* y_meta, int32_t B, float* g_meta_out, float* loss_out, void* stream);

/* Eq. 5 when the meta learner is a shared reweighting network w(l; lambda_r) (Sec. 4.1) instead of
 * per-sample logits:  L_base = (1/B) sum_i w(l_i(theta); lambda_r) l_i(theta),  w a 2-layer MLP on the
 * scalar loss,  a_j = v1_j l + c1_j,  z = sum_j v2_j max(0, a_j) + c2,  w = sigmoid(z).
 * lambda_r: [3 hidden + 1] = v1[hidden], c1[hidden], v2[hidden], c2; 1 <= hidden <= 256.  (The paper says
 * "2-layer MLP" only; ReLU hidden units and a sigmoid output are this library's reading.)
 * loss_plus, loss_minus: [B] per-sample losses at theta+ and theta- (the loss outputs of sama_step or
 * sama_fd_metagrad).  loss_diff: [B] loss_plus - loss_minus as the forward pass formed it (sama_ctx_loss_diff), or
 * NULL.  Give it whenever it is available: each fp32 loss carries a rounding of about 1e-7 of its size, which
 * for a small perturbation (alpha = 1e-2) is several 1e-3 of the difference; with loss_diff, loss_plus is
 * rebuilt as loss_minus + loss_diff and may be NULL.  eps_fd: one float on the device (NULL: the context's).
 * B_norm: the 1/B of the objective (pass B).  metagrad_r_out: [3 hidden + 1],
 *   metagrad_r = -[dL_base(theta+)/dlambda_r - dL_base(theta-)/dlambda_r] / (2 eps_fd),
 * all zero when eps_fd is 0.  This is the vector a data-parallel run would all-reduce once per meta step
 * (Sec. 3.3).  Accumulated in double in a fixed order: bitwise reproducible.  Needs a context created
 * with an mlp (for its workspace); B <= max_batch. */
int sama_fd_metagrad_reweight(sama_ctx* ctx, int32_t B, const float* loss_plus, const float* loss_minus,
                              const float* loss_diff, int32_t hidden, const float* lambda_r, const float* eps_fd,
                              int32_t B_norm, float* metagrad_r_out, void* stream);

/* The step of Fig. 2 with the shared reweighting network as the meta learner: sama_adapt -> sama_perturb
 * -> dual forward pass -> sama_fd_metagrad_reweight, one stream, no host synchronisation.  Arguments as
 * sama_step, with (hidden, lambda_r, metagrad_r_out) in place of (lambda, metagrad_out). */
int sama_step_reweight(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta, const float* m,
                       const float* s, const float* g_base, const float* g_meta, const sama_adam_t* adam,
                       float alpha, const float* X, const int32_t* y, int32_t B, int32_t hidden,
                       const float* lambda_r, float* p_out, float* theta_plus, float* theta_minus,
                       float* metagrad_r_out, float* loss_plus_out, float* loss_minus_out, void* stream);

/* SAMA on the biased-regression problem of Appendix E,
 *   L_meta(w) = ||X' w - y'||^2,   L_base(w, lambda) = ||X w - y||^2 + beta ||w - lambda||^2,
 * whose meta parameter lambda has the dimension d of w.
 *
 * sama_biasreg_direct_grad: the direct gradient of Eq. 1, g_meta = dL_meta/dw = 2 X'^T (X' w - y').
 * Xv: [n_val][d] row-major, yv: [n_val], w: [d], g_meta_out: [d] (must not overlap the inputs),
 * meta_loss_out: one float on the device (L_meta(w)) or NULL.  Accumulated in double in a fixed order.
 * Allocates a workspace inside the context on the first call and when d grows (cudaMalloc; synchronises).
 *
 * sama_biasreg_fd_metagrad: Eq. 5 for this objective.  With g_lambda(w) = dL_base/dlambda = -2 beta (w - lambda),
 *   metagrad = -[g_lambda(w_plus) - g_lambda(w_minus)] / (2 eps_fd)      (all [d]; 0 when eps_fd is 0).
 * eps_fd: one float on the device (NULL: the context's, as left by sama_perturb).
 *
 * sama_biasreg_step: direct gradient -> sama_adapt -> sama_perturb -> sama_biasreg_fd_metagrad on one stream.
 * An SGD base optimiser is adam->identity = 1 (m, s, g_base may then be NULL).  Outputs g_meta_out, p_out,
 * w_plus, w_minus, metagrad_out: [d] each, pairwise distinct (p_out may alias g_meta_out). */
int sama_biasreg_direct_grad(sama_ctx* ctx, int32_t d, int32_t n_val, const float* Xv, const float* yv,
                             const float* w, float* g_meta_out, float* meta_loss_out, void* stream);
int sama_biasreg_fd_metagrad(sama_ctx* ctx, int64_t d, const float* w_plus, const float* w_minus,
                             const float* lambda, float beta, const float* eps_fd, float* metagrad_out,
                             void* stream);
int sama_biasreg_step(sama_ctx* ctx, int32_t d, int32_t n_val, const float* Xv, const float* yv, const float* w,
                      const float* lambda, float beta, const float* m, const float* s, const float* g_base,
                      const sama_adam_t* adam, float alpha, float* g_meta_out, float* p_out, float* w_plus,
                      float* w_minus, float* metagrad_out, void* stream);

/* sama_step (Fig. 2) for callers whose data lives in HOST memory: every
 * pointer below is a host pointer (pinned memory makes the copies
 * asynchronous).  Copies the inputs to staging buffers owned by the context
 * (allocated on the first call, grown when needed), runs the step, copies
 * metagrad (and eps_fd) back and synchronises `stream` before returning.
 * theta_minus_out_host may be NULL; if given it receives theta - eps_fd p.
 * Needs a context created with an mlp. */
int sama_step_host(sama_ctx* ctx, const sama_mlp_t* mlp, int64_t n, const float* theta_host, const float* m_host,
                   const float* s_host, const float* g_base_host, const float* g_meta_host,
                   const sama_adam_t* adam, float alpha, const float* X_host, const int32_t* y_host,
                   const float* lambda_host, int32_t B, float* metagrad_out_host, float* eps_fd_out_host,
                   float* theta_minus_out_host, void* stream);

/* Device addresses of the context's scalar slots of Sec. 3.2 (sum p^2 and
 * eps_fd), valid until sama_destroy. */
double* sama_ctx_sumsq(sama_ctx* ctx);
float* sama_ctx_eps_fd(sama_ctx* ctx);

/* Device address of the context's [max_batch] buffer that every forward pass through this context
 * (sama_fd_metagrad, sama_step, ...) fills with loss+_i - loss-_i, formed inside its last kernel before
 * either loss is rounded to fp32.  NULL for a context created without an mlp.  Valid until sama_destroy. */
float* sama_ctx_loss_diff(sama_ctx* ctx);

/* Synchronises `stream`, returns the OR of the device status bits raised since
 * the last call in *status_out and clears them. */
int sama_device_status(sama_ctx* ctx, void* stream, int32_t* status_out);

/* Self-test of the bounded waits.  Every wait inside the tensor-core kernels (on a copy, on a peer CTA, on an
 * arrival counter) gives up after a cycle limit, raises SAMA_DEV_TIMEOUT and lets the kernel return.  This
 * launches one warp that waits, with that same routine, on a barrier nothing ever arrives on, for at most
 * limit_cycles (1 .. 2e9) SM clock cycles.  Afterwards sama_device_status reports SAMA_DEV_TIMEOUT, the context
 * and the device remain usable, and *waited_cycles_out (one int64 on the device, or NULL) holds how long the
 * wait lasted.  Nothing faults, traps or spins without bound. */
int sama_selftest_wait_expiry(sama_ctx* ctx, int64_t limit_cycles, int64_t* waited_cycles_out, void* stream);

/* cudaError_t value of the last failed runtime call on this context (0 if none). */
int sama_last_cuda_error(sama_ctx* ctx);

/* Parameter count sum_l (d_{l-1} d_l + d_l), or -1 for an invalid description. */
int64_t sama_mlp_param_count(const sama_mlp_t* mlp);

/* Static text for a sama_status value. */
const char* sama_status_string(int status);

/* Selects how the forward pass of Eq. 5 multiplies matrices: 0 = automatic
 * (the tensor cores where the model fits their workspaces), 1 = fp32 FMA on
 * the CUDA cores, 2 = tensor cores with each fp32 operand split into two
 * TF32 terms and three products per block (error comparable to fp32),
 * 3 = as 2, and in sama_step the product kernel itself forms the weights of
 * both branches, theta +- eps_fd p (Sec. 3.2), in its operand stage from theta
 * and p: the perturbed weights then never exist in device memory and the
 * perturbation sweep writes no operand copy (layers with d_in >= 32, inputs
 * 16-byte aligned; other layers and the other entry points behave as in 2).
 * Modes 2 and 3 return SAMA_ERR_SIZE from the forward when the model does
 * not fit the workspaces.  Returns SAMA_ERR_PARAM for an unknown mode. */
int sama_set_gemm_mode(sama_ctx* ctx, int mode);

/* How the last forward pass run through this context (sama_fd_metagrad, sama_step, sama_step_host)
 * multiplied matrices: 0 = none yet, 1 = fp32 FMA on the CUDA cores, 2 = tensor cores (3xTF32), 3 = tensor
 * cores with the perturbed weights formed in the operand stage (mode 3 of sama_set_gemm_mode).  In
 * automatic mode a model that does not fit the operand workspace sized at sama_create takes path 1,
 * which is several times slower; this query makes that visible. */
int sama_last_forward_path(sama_ctx* ctx);

/* Number of kernels the library has launched through this context. */
int64_t sama_launch_count(sama_ctx* ctx);

/* Per-kernel timing.  While enabled, the library records a pair of CUDA events
 * around every kernel it launches through this context, on the stream the
 * kernel is launched on.  The kinds name the stages of the step: adaptation +
 * norm (Eq. 4, Sec. 3.2), norm alone, perturbation (Sec. 3.2), one layer of
 * the dual-branch forward pass, cross-entropy + central difference (Eq. 5). */
enum {
    SAMA_K_ADAPT = 0,
    SAMA_K_SUMSQ = 1,
    SAMA_K_PERTURB = 2,
    SAMA_K_GEMM_FFMA = 3,
    SAMA_K_CE_FD = 4,
    SAMA_K_SPLIT = 5,
    SAMA_K_GEMM_TF32X3 = 6,
    SAMA_K_HEAD = 7, /* narrow last layer fused with cross-entropy + central difference */
    SAMA_K_PERTURB_SPLIT = 8, /* perturbation that also writes the tensor-core operands of W+ and W- */
    SAMA_K_META_GEMM = 9,     /* matrix products of the direct gradient (forward, dz W, dz^T h) */
    SAMA_K_META_AUX = 10,     /* softmax gradient, bias sums, mean loss of the direct gradient */
    SAMA_K_REWEIGHT_FD = 11,  /* central difference of the shared reweighting network's gradient (Eq. 5, Sec. 4.1) */
    SAMA_K_BIASREG_GRAD = 12, /* direct gradient of the biased-regression meta objective (Appendix E) */
    SAMA_K_BIASREG_FD = 13,   /* central difference for the biased-regression base objective */
    SAMA_K_FUSED_SWEEP = 14   /* adaptation + norm + perturbation + operand split in one launch (small models) */
};
typedef struct sama_kernel_time_t {
    int32_t kind;     /* SAMA_K_* */
    int32_t layer;    /* layer index for the forward kernels, else -1 */
    float ms;         /* device time between the two events */
    int32_t launches; /* launches between the two events: 1, or the length of a run in grouped mode */
} sama_kernel_time_t;

/* on == 1: start recording, one event pair per launch (discarding earlier records).  on == 2: grouped --
 * consecutive launches of the same kind (the layers of one forward pass) share one event pair, so no event
 * sits between them and they overlap as they do in an untimed step (programmatic dependent launch).
 * on == 0: stop and discard. */
int sama_profile_enable(sama_ctx* ctx, int32_t on);

/* Waits for the recorded events, writes up to `capacity` records (launch
 * order) to the host array `out`, stores the number of records taken in
 * *count_out and clears them.  Recording stays enabled. */
int sama_profile_collect(sama_ctx* ctx, sama_kernel_time_t* out, int32_t capacity, int32_t* count_out);

#ifdef __cplusplus
}
#endif
#endif /* SAMA_H */
