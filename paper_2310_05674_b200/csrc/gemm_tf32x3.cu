// Dual-branch layer of the perturbed forward pass (Eq. 5) on the 5th-generation
// tensor cores, in arithmetic that stays faithful to fp32.
//
// Each fp32 operand x is carried as two TF32 numbers, hi = tf32(x) and
// lo = tf32(x - hi), so that hi + lo holds x to about 2^-22 relative.  A product
// A W^T is then three tensor-core products accumulated in fp32 in tensor
// memory:  Ahi Wlo^T + Alo Whi^T + Ahi Whi^T  (the lo*lo term, 2^-22 relative, is
// dropped).  The finite difference of Eq. 5 divides the difference of two
// forward passes by 2 eps_fd, which amplifies rounding by 1/eps_fd; plain TF32
// (2^-11) would drown the signal, which is why the split is needed.
//
// Structure of gemm_tf32x3_kernel (persistent: a CTA, or a CTA pair, walks several 128 x BN, or
// 256 x 256, output tiles of both branches; 2 + 4 or 2 + 8 warps):
//   warp 0    : TMA producer.  Per k-block of 32 floats it loads four tiles
//               (A hi/lo: 128 x 32, W hi/lo: BN x 32) with cp.async.bulk.tensor
//               into 128-byte-swizzled shared memory and signals a "full"
//               mbarrier with the byte count.  No multicast.
//   warp 1    : allocates tensor memory (two accumulators), then one lane issues,
//               per k-block, 4 k-steps of tcgen05.mma kind::tf32 (K = 8) from
//               shared-memory descriptors -- three products per k-step, or two
//               wider ones on single-CTA tiles (see CONCAT) -- and commits to the
//               stage's "empty" mbarrier; every few k-blocks it commits the chunk's
//               accumulator and moves to the other one.  The pipeline keeps running
//               across tile boundaries.
//   warps 2.. : epilogue.  Each warp reads its 32 lanes of a finished chunk with
//               tcgen05.ld and adds it to a running fp32 sum in registers (the
//               tensor core's own accumulation rounds toward zero, see kChunkKb);
//               after a tile's last chunk it adds the bias, applies ReLU, and stores
//               fp32 results and / or the next layer's hi/lo operands through a
//               shared-memory transpose, while the next tile is being multiplied.
//   warps 2 + EPI .. (XF > 0 only): operand transform.  The weights of the two branches are theta +- eps_fd p
//               (Sec. 3.2).  Instead of reading them as a pre-split copy, the producer then loads the tile of
//               theta into the W hi slot and the tile of p into the W lo slot, and these warps replace them in
//               place by hi / lo of fma(+-eps_fd, p, theta) before the products read them: the perturbed
//               weights never exist in global memory.
// A layer with fewer tiles than SMs gives each tile to a cluster of 2 or 4 CTAs that split the
// contraction and exchange partial sums (see ksplit).
// Operands are K-major in global memory ([rows][K], K padded to a multiple of
// 32 with zeros), which is what both TMA and the K-major UMMA descriptor want.
// Every mbarrier wait is bounded: if one expires the CTA raises
// SAMA_DEV_TIMEOUT in the device status word, stops issuing work, waits (again
// bounded) for the copies it has in flight, frees its tensor memory and exits.
#include <cuda.h>

#include <cstdlib>
#include <new>

#include "sama_internal.h"

namespace sama {

namespace {

constexpr int BM = 128;       // rows of the output tile = TMEM lanes
constexpr int BKF = 32;       // floats per k-block = one 128-byte swizzle row
constexpr int UMMA_K = 8;     // K of one kind::tf32 instruction
// The tensor core adds each product into its fp32 accumulator with round-toward-zero, so a long
// contraction kept in tensor memory drifts towards zero by about 2^-24 per instruction (measured:
// 6e-5 relative at K = 4096).  The contraction is therefore cut into chunks of kChunkKb k-blocks that
// alternate between two accumulators in tensor memory; the epilogue warps add each finished chunk
// into fp32 registers (round-to-nearest) while the next chunk is being multiplied.
constexpr int kChunkKb = 4;
// epi = 4 or 8 epilogue warps, xf = 0 or 2 operand-transform warps
__host__ __device__ constexpr int threads_for(int epi, int xf = 0) { return 64 + 32 * epi + 32 * xf; }
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s at 2 GHz

// `wrows` = rows of W one CTA stages per k-block: BN, or BN / 2 when a CTA pair shares the W tile.
__host__ __device__ constexpr int stage_bytes(int wrows) { return 2 * BM * BKF * 4 + 2 * wrows * BKF * 4; }
__host__ __device__ constexpr int stages_for(int wrows) {
    return (200 * 1024) / stage_bytes(wrows) > 5 ? 5 : (200 * 1024) / stage_bytes(wrows);
}
constexpr int kXf = 2;  // operand-transform warps of the kernels that form W from theta and p
constexpr int kStoreStageBytes = 32 * 32 * 4;  // per epilogue warp: a 32 x 32 fp32 block on its way to row-contiguous stores
__host__ __device__ constexpr int smem_bytes(int wrows) {
    return stages_for(wrows) * stage_bytes(wrows) + 1024 + 256 + 8 * kStoreStageBytes;
}

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within kWaitCycles, or if another role of the CTA
// has given up meanwhile (`abort`, looked at only once the first try has failed).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile uint32_t* abort = nullptr,
                                          long long limit = kWaitCycles) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try(bar, parity)) return true;
        if (abort && *abort) return false;
        if (clock64() - t0 > limit) return false;
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}

// CTA-pair (cta_group::2) forms.  Shared-memory addresses of a cluster carry the CTA rank in bit 24:
// clearing it names the same offset in the even ("leader") CTA of the pair.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;
// try_wait whose success also makes another CTA's earlier writes (released at cluster scope) visible
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on a barrier on which another CTA of the cluster arrives with release.cluster.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, const volatile uint32_t* abort) {
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_cluster(bar, parity)) return true;
        if (abort && *abort) return false;
        if (clock64() - t0 > kWaitCycles) return false;
    }
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// The shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Execution barrier only: used where no memory ordering is needed (the exit of a pair).
__device__ __forceinline__ void cluster_sync_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
// Load into THIS CTA's shared memory; completion bytes are signalled on the leader's mbarrier.  No multicast.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// One instruction drives both SMs: D (256 x N, 128 rows in each CTA's tensor memory) += A (each CTA's 128 rows)
// x B^T (N rows, half of them staged by each CTA).
__device__ __forceinline__ void umma_tf32_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the barrier at this offset in both CTAs of the pair once the products issued so far are done.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
        ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier is signalled when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Two 16-column reads in flight, one wait.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr + 16u));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrival on a barrier that may live in the other CTA of the pair (shared::cluster address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes
// with the 128-byte swizzle: start address / 16 in bits [0,14), leading byte
// offset (unused for swizzled K-major, 1) in [16,30), stride between groups of
// 8 rows (1024 bytes) / 16 in [32,46), descriptor version 1 in [46,48), layout
// type 2 (128-byte swizzle) in [61,64).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// Instruction descriptor: D = fp32 (1 at bit 4), A and B = TF32 (2 at bits 7 and
// 10), both K-major (bits 15, 16 clear), N/8 at bit 17, M/16 at bit 24.
__host__ __device__ constexpr uint32_t make_idesc(int n, int m = BM) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ float to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// Round-to-nearest (ties away from zero) to TF32 with integer arithmetic: same result as cvt.rna.tf32.f32 on
// finite values, at the full integer rate (the conversion instruction issues at a fraction of it, which shows
// in the epilogue, where eight warps convert a whole tile).
// NaN and infinity (exponent field all ones) pass through unchanged: the add could otherwise carry a NaN's
// mantissa into the sign bit and turn it into a zero.
__device__ __forceinline__ float round_tf32(float x) {
    const uint32_t u = __float_as_uint(x);
    const uint32_t r = (u + 0x1000u) & 0xFFFFE000u;
    return __uint_as_float((u & 0x7F800000u) == 0x7F800000u ? u : r);
}
// Bias, then ReLU as a select that keeps NaN (max(NaN, 0) would return 0 and hide a non-finite input):
// floor_v is 0 for ReLU and -infinity (never below) otherwise.
__device__ __forceinline__ float bias_act(float x, float b, float floor_v) {
    const float v = x + b;
    return v < floor_v ? 0.f : v;
}

struct TcArgs {
    const float* bias[2];  // [N] fp32 (slices of theta+ / theta-), may be unaligned
    float* out_f32[2];     // fp32 output (logits, or activations feeding a fused head): [M][ldc]
    float* out_hi;         // hidden layers: next operand hi, [2][M][ld_next]
    float* out_lo;
    int M, N, num_kb;
    int ldc, ld_next;      // ld_next = N rounded up to 32 (zero-filled tail)
    int relu, last, shared_a;
    int both;              // hidden layer that also stores its fp32 result (kept for a backward pass)
    const float* mask;     // [M][ldm] or null: results are zeroed where mask <= 0
    int ldm;
    int tiles_m, tiles_n, group_n;
    int branches;          // 1 or 2; a work item is (branch, tile)
    int ksplit;            // single-CTA tiles only: CTAs of a cluster that share one tile's contraction (1, 2 or 4)
    float4* ws;            // ksplit > 1: partial tiles, [item][ksplit][128 x BN floats]
    // Pair tiles only: when the tiles do not fill the last round, every unit first takes `full_rounds` whole
    // tiles, then the `tail_tiles` remaining ones are each shared by two units (half of the k-blocks each).
    int full_rounds, tail_tiles;
    int* flags;            // arrival counters of the shared tail tiles [tail tile][2 halves][2 CTAs], zero between launches
    uint32_t tx_bytes;     // bytes the four copies of one k-block deliver (XF > 0: the two copies of A)
    uint32_t w_tx_bytes;   // XF > 0: bytes of the theta and p tiles one CTA receives per k-block
    const float* eps_fd;   // XF > 0: the finite-difference step (device); branch 0 takes +eps_fd, branch 1 -eps_fd
    int32_t* status;
};

// Stores one 32 x 32 block of a tile that a warp has laid out in shared memory (`stg`: 32 rows of eight
// 16-byte chunks, chunk c of row r at position c ^ (r & 7)).  Eight lanes cover one row's 32 columns, so an
// instruction writes four full 128-byte segments.  Adds the bias, applies ReLU and the mask, and writes fp32
// and / or the next layer's hi / lo operands.
__device__ __forceinline__ void store_block(const TcArgs& args, const float4* stg, int br, int m_base, int n_base,
                                         int valid_cols, int lane) {
    const int c4 = lane & 7;
    if (4 * c4 >= valid_cols) return;  // (the 16-wide tile fills only half of the block)
    const int n = n_base + 4 * c4;
    const int N = args.N;
    const int r0 = lane >> 3;          // this lane's rows of the block: r0, r0 + 4, ..., r0 + 28
    const int rows = min(32, args.M - m_base);
    const float* bias = br ? args.bias[1] : args.bias[0];
    float* outf = br ? args.out_f32[1] : args.out_f32[0];
    const bool want_f32 = args.last || args.both;
    const bool want_split = !args.last && n < args.ld_next;
    const bool relu = args.relu != 0;
    const bool full = n + 3 < N;       // all four columns exist
    const bool vec_f32 = full && (args.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(outf) & 15u) == 0;
    float b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = (bias != nullptr && n + j < N) ? bias[n + j] : 0.f;
    // everything that depends on the row advances by a fixed stride (4 rows) per iteration
    const int64_t row0 = (int64_t)m_base + r0;
    const float* mk = args.mask ? args.mask + row0 * args.ldm + n : nullptr;
    float* dst = outf + row0 * args.ldc + n;
    float* dh = args.out_hi + ((int64_t)br * args.M + row0) * args.ld_next + n;
    float* dl = args.out_lo + ((int64_t)br * args.M + row0) * args.ld_next + n;
    const int64_t mk_step = 4 * (int64_t)args.ldm, dst_step = 4 * (int64_t)args.ldc, split_step = 4 * (int64_t)args.ld_next;
    // chunk position of this lane's columns in rows r0 + 8 j and in rows r0 + 4 + 8 j
    const float4* src_even = stg + r0 * 8 + (c4 ^ r0);
    const float4* src_odd = stg + (r0 + 4) * 8 + (c4 ^ (r0 + 4));
    // all eight rows are fetched first (rows beyond M hold stale data that is never stored), so that the
    // eight independent chains of arithmetic and stores can overlap
    float4 t[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) t[i] = ((i & 1) ? src_odd : src_even)[(i >> 1) * 64];
    const float floor_v = relu ? 0.f : -INFINITY;  // values below floor_v become 0: ReLU, or nothing
    if (full && rows == 32 && mk == nullptr && (vec_f32 || !want_f32)) {
        // interior block: no per-row or per-column conditions (branches cost more here than the arithmetic)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float v0 = bias_act(t[i].x, b[0], floor_v), v1 = bias_act(t[i].y, b[1], floor_v);
            const float v2 = bias_act(t[i].z, b[2], floor_v), v3 = bias_act(t[i].w, b[3], floor_v);
            if (want_f32) *reinterpret_cast<float4*>(dst + i * dst_step) = make_float4(v0, v1, v2, v3);
            if (want_split) {
                const float h0 = round_tf32(v0), h1 = round_tf32(v1), h2 = round_tf32(v2), h3 = round_tf32(v3);
                *reinterpret_cast<float4*>(dh + i * split_step) = make_float4(h0, h1, h2, h3);
                *reinterpret_cast<float4*>(dl + i * split_step) =
                    make_float4(round_tf32(v0 - h0), round_tf32(v1 - h1), round_tf32(v2 - h2), round_tf32(v3 - h3));
            }
        }
        return;
    }
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
        const int rl = r0 + 4 * i;
        if (rl < rows) {
            const float4 ti = ((i & 1) ? src_odd : src_even)[(i >> 1) * 64];
            float v[4] = {bias_act(ti.x, b[0], floor_v), bias_act(ti.y, b[1], floor_v), bias_act(ti.z, b[2], floor_v),
                          bias_act(ti.w, b[3], floor_v)};
            if (mk) {  // backward pass: the derivative passes only where the forward activation was positive
                const float* mrow = mk + i * mk_step;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (n + j < N && !(mrow[j] > 0.f)) v[j] = 0.f;
            }
            if (want_f32) {
                float* drow = dst + i * dst_step;
                if (vec_f32) {
                    *reinterpret_cast<float4*>(drow) = make_float4(v[0], v[1], v[2], v[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (n + j < N) drow[j] = v[j];
                }
            }
            if (want_split) {
                // columns in [N, ld_next) are the next layer's zero padding along K
                float hi[4], lo[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float x = (full || n + j < N) ? v[j] : 0.f;
                    hi[j] = round_tf32(x);
                    lo[j] = round_tf32(x - hi[j]);
                }
                *reinterpret_cast<float4*>(dh + i * split_step) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<float4*>(dl + i * split_step) = make_float4(lo[0], lo[1], lo[2], lo[3]);
            }
        }
    }
}

// Persistent kernel: CTA (or CTA pair) u of U works on tiles u, u + U, u + 2U, ... of the layer; the copy
// pipeline and the two accumulators keep running across tiles, so the stores of one tile overlap the
// products of the next.
// Layers with fewer tiles than SMs can instead give one tile to a cluster of `ksplit` CTAs, each taking a
// share of the k-blocks; the CTAs then exchange partial sums through a small L2-resident workspace (ordered
// by cluster-scope mbarriers) so that each adds up, in rank order, and stores an equal share of the columns.
// PAIR = true: two CTAs of a cluster work on one 256 x BN tile.  Each stages its own 128 rows of A and half of
// the W tile; the leader CTA issues cta_group::2 products that read both CTAs' shared memory and write both
// CTAs' tensor memory.  Per CTA and flop that is fewer operand bytes than two independent 128 x BN tiles.
// XF > 0: map_w_hi covers this layer's weights inside theta and map_w_lo the same block of p ([N][K] fp32, one
// slab); XF warps form the operands of theta +- eps_fd p in shared memory.
template <int BN, bool PAIR, int EPI, int XF>
__global__ void __launch_bounds__(threads_for(EPI, XF), 1)
gemm_tf32x3_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                   const __grid_constant__ CUtensorMap map_w_hi, const __grid_constant__ CUtensorMap map_w_lo,
                   const __grid_constant__ TcArgs args) {
    constexpr int WROWS = PAIR ? BN / 2 : BN;  // rows of W this CTA stages
    constexpr int STAGES = stages_for(WROWS);
    constexpr int A_BYTES = BM * BKF * 4, W_BYTES = WROWS * BKF * 4;
    constexpr int STAGE = stage_bytes(WROWS);
    // Single-CTA tiles of 64 or 128 columns issue two products per k-step instead of three: W hi and W lo
    // sit back to back in shared memory, so A hi x [W hi; W lo]^T is one instruction of twice the width
    // (A hi is fetched once, and fewer, larger instructions keep the tensor pipe fuller), and A lo x W hi^T
    // joins the small terms in the second half of the accumulator.  The epilogue adds the two halves.
    constexpr bool CONCAT = !PAIR && BN >= 64;
    constexpr uint32_t ACC_COLS = CONCAT ? 2 * BN : (BN < 32 ? 32 : BN);   // one accumulator
    constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;       // two, alternating by chunk
    constexpr int CPW = BN / (EPI / 4);                // accumulator columns per epilogue thread
    constexpr int ACC_REGS = CPW < 32 ? 32 : CPW;
    static_assert(CPW <= 128, "at most 128 accumulator columns per epilogue thread");
    constexpr uint32_t IDESC = make_idesc(BN, PAIR ? 2 * BM : BM);
    constexpr uint32_t IDESC_CAT = make_idesc(CONCAT ? 2 * BN : BN, BM);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // tiles need 1024-byte alignment
    const uint32_t bars = base + STAGES * STAGE;                   // full[STAGES], empty[STAGES], accumulators, tmem slot
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto acc_full_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };        // chunk in accumulator b is complete
    auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };   // accumulator b has been read out
    const uint32_t part_bar = bars + 8u * (2 * STAGES + 4);   // K-split: the other CTAs' partial sums have been written
    const uint32_t tmem_slot = bars + 8u * (2 * STAGES + 5);
    const uint32_t abort_slot = tmem_slot + 4;
    // XF > 0: theta and p tiles of stage s have landed in this CTA; the W operands of stage s are in place (the
    // leader's barrier, for a pair)
    auto wfull_bar = [&](int s) { return bars + 8u * (2 * STAGES + 7 + s); };
    auto ready_bar = [&](int s) { return bars + 8u * (3 * STAGES + 7 + s); };
    static_assert(8 * (4 * stages_for(PAIR ? BN / 2 : BN) + 7) <= 256, "barriers fit in front of the store staging");
    volatile uint32_t* abort_flag =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (abort_slot - smem_u32(smem_raw)));
    volatile uint32_t* tmem_ptr_slot =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ks = PAIR ? 1 : args.ksplit;
    const uint32_t crank = cluster_ctarank();             // 0 without a cluster
    const uint32_t rank = PAIR ? crank : 0u;              // 0 = leader of the pair
    const int kpart = PAIR ? 0 : (int)crank;              // which share of the contraction
    const int csize = PAIR ? 2 : ks;
    const int unit = (int)blockIdx.x / csize;
    const int n_units = (int)gridDim.x / csize;
    const int tiles_per_branch = args.tiles_m * args.tiles_n;
    const int n_items = tiles_per_branch * args.branches;
    // this CTA's k-blocks (the host makes every share non-empty)
    const int kb_per_part = (args.num_kb + ks - 1) / ks;
    const int kb_begin = kpart * kb_per_part;
    const int num_kb = min(kb_per_part, args.num_kb - kb_begin);
    // The step-th piece of work of this unit: a tile and a range of its k-blocks.  tpart >= 0: a tail tile
    // shared with another pair, of which this is half `tpart`.
    auto next_work = [&](int step, int& item, int& kb0, int& nkb, int& tpart) -> bool {
        tpart = -1;
        if (PAIR && args.tail_tiles > 0) {
            if (step < args.full_rounds) { item = unit + step * n_units; kb0 = 0; nkb = args.num_kb; return true; }
            if (step == args.full_rounds && unit < 2 * args.tail_tiles) {
                item = args.full_rounds * n_units + (unit >> 1);
                tpart = unit & 1;
                const int half = (args.num_kb + 1) / 2;
                kb0 = tpart * half;
                nkb = tpart ? args.num_kb - half : half;
                return true;
            }
            return false;
        }
        item = unit + step * n_units;
        kb0 = kb_begin;
        nkb = num_kb;
        return item < n_items;
    };
    // Work item -> branch and tile origin.  Tile order inside a branch: items that run together cover all
    // M-tiles of a group of `group_n` N-tiles, so one wave re-uses a bounded set of W tiles and every A tile
    // from L2 instead of sweeping all of W.
    auto locate = [&](int item, int& br, int& m0, int& n0) {
        br = item / tiles_per_branch;
        const int tile_id = item - br * tiles_per_branch;
        const int per_group = args.group_n * args.tiles_m;
        const int group = tile_id / per_group, rem = tile_id - group * per_group;
        const int first_n = group * args.group_n;
        const int gsz = min(args.group_n, args.tiles_n - first_n);
        const int tile_n = first_n + rem % gsz;
        const int tile_m = rem / gsz;
        m0 = tile_m * (PAIR ? 2 * BM : BM) + (int)rank * BM;
        n0 = tile_n * BN;
    };

    if (threadIdx.x == 32) {  // descriptor fetches off the first copies' critical path
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a_hi) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a_lo) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w_hi) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w_lo) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            if (XF > 0) {
                mbar_init(wfull_bar(s), 1);
                mbar_init(ready_bar(s), XF * (PAIR ? 2 : 1));  // one arrival per transform warp (of both CTAs of a pair)
            }
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full_bar(b), 1);
            mbar_init(acc_empty_bar(b), EPI * (PAIR ? 2 : 1));  // one arrival per epilogue warp (of both CTAs of a pair)
        }
        mbar_init(part_bar, EPI * (ks > 1 ? ks - 1 : 1));       // one arrival per epilogue warp of every other CTA
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // epilogue warps that have finished the exchange of a shared tail tile
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) tmem_alloc_pair(tmem_slot, TMEM_COLS); else tmem_alloc(tmem_slot, TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR || ks > 1) cluster_sync();  // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_slot;
    // everything above (barriers, tensor memory) overlapped the previous kernel's tail; its outputs
    // (our operands) are only touched from here on
    pdl_trigger();
    pdl_wait();

    auto raise_timeout = [&]() {
        *abort_flag = 1;
        atomicOr(args.status, (int)SAMA_DEV_TIMEOUT);
    };

    if (warp == 0) {
        // ---------------------------------------------------------- TMA producer
        if (lane == 0) {
            int issued = 0;  // k-blocks copied so far, over all of this CTA's tiles
            int s = 0;
            uint32_t empty_parity = 1;  // parity of the phase that frees stage s for its next round
            bool ok = true;
            for (int step = 0; ok; ++step) {
                int item, kb0, nkb, tpart;
                if (!next_work(step, item, kb0, nkb, tpart)) break;
                int br, m0, n0;
                locate(item, br, m0, n0);
                const int nw0 = n0 + (int)rank * WROWS;  // first W row this CTA stages
                const int za = args.shared_a ? 0 : br;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (issued >= STAGES && !mbar_wait(empty_bar(s), empty_parity, abort_flag)) { raise_timeout(); ok = false; break; }
                    const uint32_t st = base + s * STAGE;
                    const int kx = (kb0 + kb) * BKF;
                    if (XF > 0) {
                        // theta into the W hi slot, p into the W lo slot: this CTA's own barrier, for its transform warps
                        mbar_expect_tx(wfull_bar(s), args.w_tx_bytes);
                        tma_load_3d(st + 2 * A_BYTES, &map_w_hi, wfull_bar(s), kx, nw0, 0);
                        tma_load_3d(st + 2 * A_BYTES + W_BYTES, &map_w_lo, wfull_bar(s), kx, nw0, 0);
                    }
                    if (PAIR) {
                        // both CTAs' copies complete on the leader's barrier, which the leader arms for all of them
                        const uint32_t lbar = full_bar(s) & kPeerBitMask;
                        if (rank == 0) mbar_expect_tx(full_bar(s), args.tx_bytes);
                        tma_load_3d_pair(st, &map_a_hi, lbar, kx, m0, za);
                        tma_load_3d_pair(st + A_BYTES, &map_a_lo, lbar, kx, m0, za);
                        if (XF == 0) {
                            tma_load_3d_pair(st + 2 * A_BYTES, &map_w_hi, lbar, kx, nw0, br);
                            tma_load_3d_pair(st + 2 * A_BYTES + W_BYTES, &map_w_lo, lbar, kx, nw0, br);
                        }
                    } else {
                        mbar_expect_tx(full_bar(s), args.tx_bytes);
                        tma_load_3d(st, &map_a_hi, full_bar(s), kx, m0, za);
                        tma_load_3d(st + A_BYTES, &map_a_lo, full_bar(s), kx, m0, za);
                        if (XF == 0) {
                            tma_load_3d(st + 2 * A_BYTES, &map_w_hi, full_bar(s), kx, n0, br);
                            tma_load_3d(st + 2 * A_BYTES + W_BYTES, &map_w_lo, full_bar(s), kx, n0, br);
                        }
                    }
                    ++issued;
                    if (++s == STAGES) { s = 0; empty_parity ^= 1u; }
                }
            }
            if (*abort_flag) {
                // let the copies already issued land before the CTA's shared memory goes away
                for (int i = (issued > STAGES ? issued - STAGES : 0); i < issued; ++i) {
                    if (rank == 0) mbar_wait(full_bar(i % STAGES), (i / STAGES) & 1);
                    if (XF > 0) mbar_wait(wfull_bar(i % STAGES), (i / STAGES) & 1);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (the leader's, for a pair)
        if (lane == 0 && rank == 0) {
            bool ok = true;
            int s = 0, chunk = 0;  // chunk counts over all of this CTA's tiles: accumulator = chunk & 1
            uint32_t full_parity = 0;
            for (int step = 0; ok; ++step) {
                int item, kb0, nkb, tpart;
                if (!next_work(step, item, kb0, nkb, tpart)) break;
                int in_chunk = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    const int buf = chunk & 1;
                    const bool chunk_first = in_chunk == 0;
                    if (chunk_first && chunk >= 2) {
                        // the epilogue warps have drained this accumulator's previous chunk
                        if (!mbar_wait(acc_empty_bar(buf), ((chunk >> 1) - 1) & 1, abort_flag)) { raise_timeout(); ok = false; break; }
                    }
                    if (!mbar_wait(full_bar(s), full_parity, abort_flag)) { raise_timeout(); ok = false; break; }
                    if (XF > 0) {  // the W operands of this stage have been formed (in both CTAs of a pair)
                        const bool got = PAIR ? mbar_wait_cluster(ready_bar(s), full_parity, abort_flag)
                                              : mbar_wait(ready_bar(s), full_parity, abort_flag);
                        if (!got) { raise_timeout(); ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t st = base + s * STAGE;
                    const uint32_t acc = tmem_base + (uint32_t)buf * ACC_COLS;
                    const uint64_t a_hi = make_desc(st), a_lo = make_desc(st + A_BYTES);
                    const uint64_t w_hi = make_desc(st + 2 * A_BYTES), w_lo = make_desc(st + 2 * A_BYTES + W_BYTES);
#pragma unroll
                    for (int k = 0; k < BKF / UMMA_K; ++k) {
                        const uint64_t adv = (uint64_t)((k * UMMA_K * 4) >> 4);  // 32 bytes per k-step inside the swizzled row
                        const uint32_t keep = (chunk_first && k == 0) ? 0u : 1u;  // a chunk starts from zero
                        if (PAIR) {
                            umma_tf32_pair(acc, a_hi + adv, w_lo + adv, IDESC, keep);
                            umma_tf32_pair(acc, a_lo + adv, w_hi + adv, IDESC, 1);
                            umma_tf32_pair(acc, a_hi + adv, w_hi + adv, IDESC, 1);
                        } else if (CONCAT) {
                            umma_tf32(acc, a_hi + adv, w_hi + adv, IDESC_CAT, keep);   // [A hi W hi^T | A hi W lo^T]
                            umma_tf32(acc + BN, a_lo + adv, w_hi + adv, IDESC, 1);      // the other small term
                        } else {
                            umma_tf32(acc, a_hi + adv, w_lo + adv, IDESC, keep);
                            umma_tf32(acc, a_lo + adv, w_hi + adv, IDESC, 1);
                            umma_tf32(acc, a_hi + adv, w_hi + adv, IDESC, 1);
                        }
                    }
                    // frees the stage (in both CTAs of a pair) once these products have read it
                    if (PAIR) umma_commit_pair(empty_bar(s)); else umma_commit(empty_bar(s));
                    if (in_chunk == kChunkKb - 1 || kb == nkb - 1) {
                        if (PAIR) umma_commit_pair(acc_full_bar(buf)); else umma_commit(acc_full_bar(buf));
                        in_chunk = 0;
                        ++chunk;
                    } else {
                        ++in_chunk;
                    }
                    if (++s == STAGES) { s = 0; full_parity ^= 1u; }
                }
            }
        }
    } else if (XF > 0 && warp >= 2 + EPI) {
        // ------------------------------------------------- operand transform: W hi / lo of theta +- eps_fd p
        // Both buffers of a stage carry the same 128-byte swizzle at the same alignment, so the element at byte
        // offset o of the theta tile meets its p at offset o of the p tile, and hi / lo go back to the same places:
        // the transform is elementwise over the raw bytes and never needs the row / column of an element.
        constexpr int NT = XF > 0 ? 32 * XF : 32;
        constexpr int CHUNKS = W_BYTES / 16;      // 16-byte groups per buffer
        constexpr int PER = CHUNKS / NT;
        constexpr int BATCH = PER < 4 ? PER : 4;
        static_assert(CHUNKS % NT == 0 && PER % BATCH == 0, "the transform threads share a buffer evenly");
        const int t = (int)threadIdx.x - 32 * (2 + EPI);
        const float eps = *args.eps_fd;
        // eps == 0 marks the degenerate norm: the weights are theta itself even where p is not finite, so p's
        // factor is forced to zero by reading p as zero (0 * NaN would not do)
        const bool degenerate = eps == 0.f;
        // hi = tf32(w) with round-to-nearest on the integer pipe (two operations; a conversion instruction
        // issues at a fraction of that rate).  The add can carry a NaN's mantissa into the sign bit and so turn
        // it into a zero; the fused multiply-add by zero puts it back (0 * w is NaN exactly when w is not finite,
        // and then so must the operand be).  lo = tf32(w - hi) needs no such care: it multiplies the same
        // operands as a hi that is already NaN.
        auto split = [](float w, float& hi, float& lo) {
            const float h = __uint_as_float((__float_as_uint(w) + 0x1000u) & 0xFFFFE000u);
            hi = fmaf(0.f, w, h);
            lo = __uint_as_float((__float_as_uint(w - hi) + 0x1000u) & 0xFFFFE000u);
        };
        int s = 0;
        uint32_t parity = 0;
        bool ok = true;
        for (int step = 0; ok; ++step) {
            int item, kb0, nkb, tpart;
            if (!next_work(step, item, kb0, nkb, tpart)) break;
            const float e = (item / tiles_per_branch) ? -eps : eps;
            for (int kb = 0; kb < nkb; ++kb) {
                ok = mbar_wait(wfull_bar(s), parity, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) raise_timeout(); break; }
                float4* th = reinterpret_cast<float4*>(smem_raw + (base + s * STAGE + 2 * A_BYTES - smem_u32(smem_raw))) + t;
                float4* pp = th + CHUNKS;
                // software pipeline: the next batch's loads are issued before this batch's stores (the two never
                // touch the same 16 bytes, which the compiler cannot know)
                float4 vt[BATCH], vp[BATCH];
#pragma unroll
                for (int j = 0; j < BATCH; ++j) {
                    vt[j] = th[j * NT];
                    vp[j] = pp[j * NT];
                }
#pragma unroll 1
                for (int j0 = 0; j0 < PER; j0 += BATCH) {
                    float4 h[BATCH], l[BATCH];
#pragma unroll
                    for (int j = 0; j < BATCH; ++j) {
                        const float4 q = degenerate ? make_float4(0.f, 0.f, 0.f, 0.f) : vp[j];
                        split(fmaf(e, q.x, vt[j].x), h[j].x, l[j].x);
                        split(fmaf(e, q.y, vt[j].y), h[j].y, l[j].y);
                        split(fmaf(e, q.z, vt[j].z), h[j].z, l[j].z);
                        split(fmaf(e, q.w, vt[j].w), h[j].w, l[j].w);
                    }
                    if (j0 + BATCH < PER) {
#pragma unroll
                        for (int j = 0; j < BATCH; ++j) {
                            vt[j] = th[(j0 + BATCH + j) * NT];
                            vp[j] = pp[(j0 + BATCH + j) * NT];
                        }
                    }
#pragma unroll
                    for (int j = 0; j < BATCH; ++j) {
                        th[(j0 + j) * NT] = h[j];
                        pp[(j0 + j) * NT] = l[j];
                    }
                }
                // these writes, made through the generic proxy, must be visible to the tensor core's reads
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_cluster(ready_bar(s) & kPeerBitMask); else mbar_arrive(ready_bar(s));
                }
                if (++s == STAGES) { s = 0; parity ^= 1u; }
            }
        }
    } else {
        // -------------------------------------------------------------- epilogue
        const int q = warp & 3;            // a warp may only touch TMEM lanes [32 q, 32 q + 32)
        const int col0 = ((warp - 2) >> 2) * CPW;  // with eight epilogue warps, two share a lane quarter and split the columns
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)col0;
        int total_chunks = 0;
        for (int step = 0;; ++step) {
            int item, kb0, nkb, tpart;
            if (!next_work(step, item, kb0, nkb, tpart)) break;
            total_chunks += (nkb + kChunkKb - 1) / kChunkKb;
        }
        int chunk = 0;  // counts over all of this CTA's tiles, like the issuer's
        bool ok = true;
        for (int step = 0; ok; ++step) {
            int item, kb0, nkb, tpart;
            if (!next_work(step, item, kb0, nkb, tpart)) break;
            const int n_chunks = (nkb + kChunkKb - 1) / kChunkKb;
            int br, m0, n0;
            locate(item, br, m0, n0);
            float acc[ACC_REGS];
#pragma unroll
            for (int j = 0; j < ACC_REGS; ++j) acc[j] = 0.f;
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c, ++chunk) {
                const int buf = chunk & 1;
                if (lane == 0) {
                    // the chunk is complete when its barrier flips, or never if a producer gave up
                    const long long t0 = clock64();
                    while (!mbar_try(acc_full_bar(buf), (chunk >> 1) & 1)) {
                        if (*abort_flag) { ok = false; break; }
                        if (clock64() - t0 > 2 * kWaitCycles) { raise_timeout(); ok = false; break; }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                tc_fence_after();
                const uint32_t src = lane_addr + (uint32_t)buf * ACC_COLS;
#pragma unroll
                for (int cc = 0; cc < ACC_REGS; cc += 32) {
                    float v[32];
                    if (CONCAT) {            // the small terms first
                        tmem_ld32(src + BN + cc, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[cc + j] += v[j];
                    }
                    tmem_ld32(src + cc, v);   // all lanes take part (sync.aligned)
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[cc + j] += v[j];
                }
                // this warp's reads are done: hand the accumulator back to the MMA issuer
                tc_fence_before();
                __syncwarp();
                // (not for the last two chunks: nobody waits for them, and no arrival on the peer's barrier may
                // still be on its way when that CTA exits)
                if (lane == 0 && chunk + 2 < total_chunks) {
                    if (PAIR) mbar_arrive_cluster(acc_empty_bar(buf) & kPeerBitMask); else mbar_arrive(acc_empty_bar(buf));
                }
            }
            if (!ok) break;
            if (ks > 1) {
                // K-split: thread t of every CTA of the cluster holds partial sums of the same rows and columns.
                // The tile's columns are dealt out in ks equal shares; for every 32-column block that another
                // CTA owns, this thread leaves its partial sums in its own slab of the workspace, then the
                // owner adds the slabs in rank order and stores its share (so all CTAs store, not just one).
                // Layout of a slab: [epilogue warp][float4 index][lane]: a warp's accesses are contiguous.
                const int share = BN / ks;  // >= 32 columns
                const uint32_t stage_u32 = bars + 256u;  // the warps' store-staging blocks, 4 KB each
                const int wi = warp - 2;
                if (EPI == 8 && ks == 2) {
                    // Two CTAs: a warp's columns all belong to one of them (CPW = BN / 2), so in each CTA four
                    // warps send and four receive.  The partials go straight into the receiving CTA's staging
                    // blocks through distributed shared memory (the receiver's own block and that of its
                    // sending neighbour, which is idle): no round trip through L2, no device-scope fences.
                    const bool sender = (wi >> 2) != kpart;
                    if (sender) {
                        const uint32_t remote = map_to_rank(stage_u32, (uint32_t)(kpart ^ 1));
#pragma unroll
                        for (int k = 0; k < CPW / 4; ++k) {
                            const int slot = k < 8 ? wi : (wi ^ 4);
                            st_cluster_f4(remote + (uint32_t)slot * kStoreStageBytes + (uint32_t)(((k & 7) * 32 + lane) * 16),
                                          acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive_cluster(map_to_rank(part_bar, (uint32_t)(kpart ^ 1)));
                        const long long t0 = clock64();
                        while (!mbar_try_cluster(part_bar, 0)) {   // one tile per cluster: first phase
                            if (*abort_flag) { ok = false; break; }
                            if (clock64() - t0 > 2 * kWaitCycles) { raise_timeout(); ok = false; break; }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (!sender) {
                        const float4* blocks = reinterpret_cast<const float4*>(smem_raw + (stage_u32 - smem_u32(smem_raw)));
#pragma unroll
                        for (int k = 0; k < CPW / 4; ++k) {
                            const int slot = k < 8 ? wi : (wi ^ 4);
                            const float4 t = blocks[slot * 256 + (k & 7) * 32 + lane];
                            acc[4 * k] += t.x; acc[4 * k + 1] += t.y; acc[4 * k + 2] += t.z; acc[4 * k + 3] += t.w;
                        }
                    }
                } else {
                float4* slabs = args.ws + (size_t)item * ks * (BM * BN / 4) + (wi * (CPW / 4)) * 32 + lane;
                float4* mine = slabs + (size_t)kpart * (BM * BN / 4);
#pragma unroll
                for (int g = 0; g < CPW / 32; ++g) {
                    if ((col0 + 32 * g) / share == kpart) continue;
#pragma unroll
                    for (int k = 8 * g; k < 8 * g + 8; ++k)
                        __stcg(mine + k * 32, make_float4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]));
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    for (int p = 0; p < ks; ++p)
                        if (p != kpart) mbar_arrive_cluster(map_to_rank(part_bar, (uint32_t)p));
                    const long long t0 = clock64();
                    while (!mbar_try(part_bar, 0)) {   // one tile per cluster: first phase
                        if (*abort_flag) { ok = false; break; }
                        if (clock64() - t0 > 2 * kWaitCycles) { raise_timeout(); ok = false; break; }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                __threadfence();
#pragma unroll
                for (int g = 0; g < CPW / 32; ++g) {
                    if ((col0 + 32 * g) / share != kpart) continue;
                    for (int p = 0; p < ks; ++p) {
                        if (p == kpart) continue;
                        const float4* theirs = slabs + (size_t)p * (BM * BN / 4);
#pragma unroll
                        for (int k = 8 * g; k < 8 * g + 8; ++k) {
                            const float4 t = __ldcg(theirs + k * 32);
                            acc[4 * k] += t.x; acc[4 * k + 1] += t.y; acc[4 * k + 2] += t.z; acc[4 * k + 3] += t.w;
                        }
                    }
                }
                }
            }
            if (PAIR && tpart >= 0) {
                // A tail tile shared with another pair (a separate cluster): each CTA leaves the column half it
                // does not own in the workspace, counts its arrival in global memory, waits (bounded) for the
                // CTA of the same pair rank in the other pair, and adds that CTA's partial sums to its own half.
                // Every pair of the launch is resident and this is its last tile, so the wait cannot cycle.
                const int t = item - args.full_rounds * n_units;
                const int wi = warp - 2;
                const int other = tpart ^ 1;
                float4* slabs = args.ws + ((size_t)t * 4 + rank) * (BM * BN / 4) + (wi * (CPW / 4)) * 32 + lane;
                float4* mine = slabs + (size_t)tpart * 2 * (BM * BN / 4);
                const bool sender = (col0 / (BN / 2)) != tpart;   // (CPW = BN / 2: a warp's columns lie in one half)
                if (sender) {
#pragma unroll
                    for (int k = 0; k < CPW / 4; ++k)
                        __stcg(mine + k * 32, make_float4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]));
                }
                __threadfence();
                __syncwarp();
                int* my_flag = args.flags + ((t * 2 + tpart) * 2 + (int)rank);
                if (lane == 0) {
                    atomicAdd(args.flags + ((t * 2 + other) * 2 + (int)rank), 1);
                    const long long t0 = clock64();
                    while (*reinterpret_cast<volatile int*>(my_flag) < EPI) {
                        if (*abort_flag) { ok = false; break; }
                        if (clock64() - t0 > 2 * kWaitCycles) { raise_timeout(); ok = false; break; }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                __threadfence();
                if (!sender) {
                    const float4* theirs = slabs + (size_t)other * 2 * (BM * BN / 4);
#pragma unroll
                    for (int k = 0; k < CPW / 4; ++k) {
                        const float4 v = __ldcg(theirs + k * 32);
                        acc[4 * k] += v.x; acc[4 * k + 1] += v.y; acc[4 * k + 2] += v.z; acc[4 * k + 3] += v.w;
                    }
                }
                // the last of this CTA's epilogue warps to get here puts the counter back to zero
                if (lane == 0 && atomicAdd(const_cast<uint32_t*>(abort_flag + 1), 1u) == (uint32_t)(EPI - 1)) *my_flag = 0;
            }
            // The tile's sum is in registers; the products of the next tile already run while it is stored.
            // A thread holds one row; to store whole 128-byte row segments the warp passes each 32 x 32 block
            // through shared memory (16-byte chunks XOR-swizzled by row: no bank conflicts either way).
            float4* stg = reinterpret_cast<float4*>(smem_raw + (bars + 256u - smem_u32(smem_raw))) + (warp - 2) * 256;
#pragma unroll
            for (int g = 0; g < ACC_REGS / 32; ++g) {
                if (ks > 1 && (col0 + 32 * g) / (BN / ks) != kpart) continue;  // another CTA of the cluster stores this block
                if (PAIR && tpart >= 0 && (col0 + 32 * g) / (BN / 2) != tpart) continue;  // the other pair stores it
                __syncwarp();
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    stg[lane * 8 + (k ^ (lane & 7))] =
                        make_float4(acc[32 * g + 4 * k], acc[32 * g + 4 * k + 1], acc[32 * g + 4 * k + 2], acc[32 * g + 4 * k + 3]);
                __syncwarp();
                store_block(args, stg, br, m0 + q * 32, n0 + col0 + 32 * g, CPW - 32 * g, lane);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    // A pair leaves together: the leader's products use the peer's shared and tensor memory.  (K-split CTAs
    // may leave on their own: the only remote access is the arrival that the first CTA has waited for.)
    if (PAIR) cluster_sync_relaxed();
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// The bounded wait on its own: one warp initialises a barrier on which nothing ever arrives and waits on it with
// the product kernels' wait routine and a caller-chosen limit.  The wait runs out, the status word gets
// SAMA_DEV_TIMEOUT, the kernel returns normally.  (How a test exercises the expiry path: no fault, no trap, no
// unbounded spin.)
__global__ void __launch_bounds__(32)
wait_expiry_kernel(long long limit_cycles, int32_t* status, long long* waited_cycles) {
    __shared__ alignas(8) unsigned long long bar_storage;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool completed = mbar_wait(bar, 0, nullptr, limit_cycles);
        if (!completed) atomicOr(status, (int)SAMA_DEV_TIMEOUT);
        if (waited_cycles) *waited_cycles = clock64() - t0;
    }
}

// Splits rows of a dense fp32 matrix [rows][cols] into TF32 hi / lo with the row
// length padded to ld_out (zeros).  grid.z selects the branch (source pointer
// and output slab).
struct SplitArgs {
    const float* src[2];
    int64_t rows, cols, slab;
    int ld_out;
    float* hi;
    float* lo;
};

template <bool VEC>
__global__ void __launch_bounds__(256)
split_tf32_kernel(SplitArgs a) {
    pdl_trigger();
    pdl_wait();
    const int br = blockIdx.z;
    const float* __restrict__ src = br ? a.src[1] : a.src[0];
    float* __restrict__ hi = a.hi + (int64_t)br * a.slab;
    float* __restrict__ lo = a.lo + (int64_t)br * a.slab;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        // cols % 4 == 0 and src 16-byte aligned: one float4 of a row per thread
        const int q = a.ld_out >> 2;
        const int64_t total = a.rows * q;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
            const int64_t r = i / q;
            const int c = (int)(i - r * q) << 2;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c < a.cols) x = __ldg(reinterpret_cast<const float4*>(src + r * a.cols + c));
            float4 h, l;
            h.x = to_tf32(x.x); l.x = to_tf32(x.x - h.x);
            h.y = to_tf32(x.y); l.y = to_tf32(x.y - h.y);
            h.z = to_tf32(x.z); l.z = to_tf32(x.z - h.z);
            h.w = to_tf32(x.w); l.w = to_tf32(x.w - h.w);
            *reinterpret_cast<float4*>(hi + r * a.ld_out + c) = h;
            *reinterpret_cast<float4*>(lo + r * a.ld_out + c) = l;
        }
    } else {
        const int64_t total = a.rows * a.ld_out;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
            const int64_t r = i / a.ld_out;
            const int c = (int)(i - r * a.ld_out);
            const float x = c < a.cols ? src[r * a.cols + c] : 0.f;
            const float h = to_tf32(x);
            hi[i] = h;
            lo[i] = to_tf32(x - h);
        }
    }
}

// hi / lo of the transpose: src [rows][cols] -> out [cols][ld_out], ld_out = rows rounded up to 32, zero padded.
// 32 x 32 tiles through shared memory so that both the read and the writes are coalesced.
__global__ void __launch_bounds__(256)
split_transpose_tf32_kernel(const float* __restrict__ src, int64_t rows, int cols, int ld_out,
                            float* __restrict__ hi, float* __restrict__ lo) {
    pdl_trigger();
    pdl_wait();
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
    const int64_t r0 = (int64_t)blockIdx.y * 32;
    const int c0 = blockIdx.x * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t r = r0 + ty + 8 * i;
        const int c = c0 + tx;
        tile[ty + 8 * i][tx] = (r < rows && c < cols) ? src[r * cols + c] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 8 * i;       // output row
        const int64_t r = r0 + tx;           // output column (< ld_out: the grid covers ld_out / 32 tiles)
        if (c < cols) {
            const float x = tile[tx][ty + 8 * i];
            const float h = to_tf32(x);
            hi[(int64_t)c * ld_out + r] = h;
            lo[(int64_t)c * ld_out + r] = to_tf32(x - h);
        }
    }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 3-D map over [slabs][rows][ld] fp32 with a box of 32 floats x box_rows rows, 128-byte swizzle, zero fill.
bool make_map(CUtensorMap* map, const float* base, int ld, int64_t rows, int slabs, int box_rows, int64_t slab) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)ld, (cuuint64_t)rows, (cuuint64_t)slabs};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)slab * 4};
    cuuint32_t box[3] = {(cuuint32_t)BKF, (cuuint32_t)box_rows, 1};  // caller keeps box_rows <= rows
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per-context state of the tensor-core path, set up once by tc_state_create on the context's device:
// experiment switches (environment variables read once), how many CTA pairs the cluster scheduler can keep
// resident, and a cache of encoded tensor maps, so that a warm launch path neither reads the environment nor
// calls into the driver.
struct TcMapKey {
    const void* base;
    int64_t rows, slab;
    int ld, slabs, box_rows;
    bool operator==(const TcMapKey& o) const {
        return base == o.base && rows == o.rows && slab == o.slab && ld == o.ld && slabs == o.slabs &&
               box_rows == o.box_rows;
    }
};
struct TcState {
    int tile = 0;          // SAMA_TC_TILE: 64 / 128 force a single-CTA tile width, 256 the CTA pair
    bool no_pair = false;  // SAMA_TC_PAIR=0
    bool no_ksplit = false;  // SAMA_TC_KSPLIT=1
    bool no_tail = false;  // SAMA_TC_TAIL=0
    int group = 0;         // SAMA_TC_GROUP
    int pair_units = 0;    // co-resident CTA pairs of the 256 x 256 kernel on this device
    static constexpr int kCache = 64;
    TcMapKey keys[kCache];
    CUtensorMap maps[kCache];
    int n_cached = 0, next_victim = 0;
};
inline TcState* tc_state(sama_ctx* ctx) { return static_cast<TcState*>(ctx->tc_state); }

// The map for `key`, encoded on first use.  nullptr if the driver refuses the encoding.
const CUtensorMap* cached_map(TcState* st, const float* base, int ld, int64_t rows, int slabs, int box_rows,
                              int64_t slab) {
    const TcMapKey key{base, rows, slab, ld, slabs, box_rows};
    for (int i = 0; i < st->n_cached; ++i)
        if (st->keys[i] == key) return &st->maps[i];
    int slot;
    if (st->n_cached < TcState::kCache) {
        slot = st->n_cached++;
    } else {
        slot = st->next_victim;
        st->next_victim = (st->next_victim + 1) % TcState::kCache;
    }
    if (!make_map(&st->maps[slot], base, ld, rows, slabs, box_rows, slab)) {
        st->n_cached = 0;  // the slot may hold half an encoding: start over
        return nullptr;
    }
    st->keys[slot] = key;
    return &st->maps[slot];
}

template <int BN, bool PAIR, int EPI, int XF>
cudaError_t tc_prepare_kernel() {
    return cudaFuncSetAttribute(gemm_tf32x3_kernel<BN, PAIR, EPI, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                smem_bytes(PAIR ? BN / 2 : BN));
}

// Launches the persistent kernel on min(work items, co-resident CTAs or CTA pairs) units.
template <int BN, bool PAIR, int EPI, int XF>
cudaError_t launch_tc(const CUtensorMap* const maps[4], const TcArgs& a, int items, int max_units, bool tail_ok,
                      cudaStream_t st, size_t ws_floats = 0, int tail_flags = 0) {
    const int ks = PAIR ? 1 : a.ksplit;
    constexpr int kSmem = smem_bytes(PAIR ? BN / 2 : BN);
    if (max_units < 1) return cudaErrorLaunchOutOfResources;
    if (ks > 1)  // one tile per cluster of ks CTAs
        return launch_clustered(ks, gemm_tf32x3_kernel<BN, PAIR, EPI, XF>, dim3(items * ks), dim3(threads_for(EPI, XF)),
                                (size_t)kSmem, st, *maps[0], *maps[1], *maps[2], *maps[3], a);
    const int units = items < max_units ? items : max_units;
    TcArgs b = a;
    b.full_rounds = 0;
    b.tail_tiles = 0;
    if (PAIR && items > max_units) {
        // tiles that do not fill the last round are each shared by two pairs when that takes no more pairs
        // than there are (and the contraction is long enough to be worth an exchange)
        const int rounds = items / max_units, tail = items % max_units;
        if (tail_ok && tail > 0 && 2 * tail <= max_units && a.num_kb >= 16 && a.flags && tail * 4 <= tail_flags &&
            (size_t)tail * 4 * BM * BN <= ws_floats) {
            b.full_rounds = rounds;
            b.tail_tiles = tail;
        }
    }
    return launch_clustered(PAIR ? 2 : 1, gemm_tf32x3_kernel<BN, PAIR, EPI, XF>, dim3(units * (PAIR ? 2 : 1)),
                            dim3(threads_for(EPI, XF)), (size_t)kSmem, st, *maps[0], *maps[1], *maps[2], *maps[3], b);
}

inline int round_up32(int x) { return (x + 31) & ~31; }

}  // namespace

cudaError_t launch_split_tf32(sama_ctx* ctx, const float* src0, const float* src1, int branches, int64_t rows,
                              int cols, float* hi, float* lo, int64_t slab, cudaStream_t st) {
    SplitArgs a;
    a.src[0] = src0;
    a.src[1] = src1;
    a.rows = rows;
    a.cols = cols;
    a.slab = slab;
    a.ld_out = round_up32(cols);
    a.hi = hi;
    a.lo = lo;
    const bool vec = (cols % 4 == 0) && ((reinterpret_cast<uintptr_t>(src0) & 15u) == 0) &&
                     ((reinterpret_cast<uintptr_t>(src1) & 15u) == 0);
    const int64_t total = rows * a.ld_out / (vec ? 4 : 1);
    int64_t blocks = (total + 256 * 2 - 1) / (256 * 2);
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    KernelScope scope(ctx, SAMA_K_SPLIT, -1, st);
    const dim3 grid((unsigned)blocks, 1, branches);
    return vec ? launch_dependent(split_tf32_kernel<true>, grid, dim3(256), 0, st, a)
               : launch_dependent(split_tf32_kernel<false>, grid, dim3(256), 0, st, a);
}

cudaError_t launch_wait_expiry(sama_ctx* ctx, long long limit_cycles, long long* waited_cycles, cudaStream_t st) {
    wait_expiry_kernel<<<1, 32, 0, st>>>(limit_cycles, &ctx->scalars->status, waited_cycles);
    return cudaGetLastError();
}

cudaError_t launch_split_transpose_tf32(sama_ctx* ctx, const float* src, int64_t rows, int cols, float* hi, float* lo,
                                        cudaStream_t st) {
    const int ld_out = round_up32((int)rows);
    dim3 grid((cols + 31) / 32, ld_out / 32, 1);
    KernelScope scope(ctx, SAMA_K_SPLIT, -1, st);
    return launch_dependent(split_transpose_tf32_kernel, grid, dim3(256), 0, st, src, rows, cols, ld_out, hi, lo);
}

// Set-up of the tensor-core path for a context (called by sama_create with the context's device current):
// reads the experiment switches, opts every kernel instantiation into its shared-memory size on this
// device, and asks how many CTA pairs can be resident.
cudaError_t tc_state_create(sama_ctx* ctx) {
    TcState* st = new (std::nothrow) TcState();
    if (!st) return cudaErrorMemoryAllocation;
    ctx->tc_state = st;
    if (const char* e = std::getenv("SAMA_TC_TILE")) st->tile = std::atoi(e);
    if (const char* e = std::getenv("SAMA_TC_PAIR")) st->no_pair = std::atoi(e) == 0;
    if (const char* e = std::getenv("SAMA_TC_KSPLIT")) st->no_ksplit = std::atoi(e) == 1;
    if (const char* e = std::getenv("SAMA_TC_TAIL")) st->no_tail = e[0] == '0';
    if (const char* e = std::getenv("SAMA_TC_GROUP")) st->group = std::atoi(e);
    cudaError_t e;
    if ((e = tc_prepare_kernel<256, true, 8, 0>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<128, false, 8, 0>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<64, false, 8, 0>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<16, false, 4, 0>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<256, true, 8, kXf>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<128, false, 8, kXf>()) != cudaSuccess) return e;
    if ((e = tc_prepare_kernel<64, false, 8, kXf>()) != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (ctx->sm_count / 2));
    cfg.blockDim = dim3(threads_for(8, kXf));
    cfg.dynamicSmemBytes = smem_bytes(128);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if ((e = cudaOccupancyMaxActiveClusters(&clusters, gemm_tf32x3_kernel<256, true, 8, kXf>, &cfg)) != cudaSuccess) return e;
    st->pair_units = clusters < ctx->sm_count / 2 ? clusters : ctx->sm_count / 2;
    return cudaSuccess;
}

void tc_state_destroy(sama_ctx* ctx) {
    delete tc_state(ctx);
    ctx->tc_state = nullptr;
}

// One layer on the tensor cores.  a_hi/a_lo: [shared_a ? 1 : 2][M][Kp]; w_hi/w_lo: [2][N][Kp]; Kp = K rounded
// up to 32.  Hidden layers write the next operands (out_hi/out_lo, [2][M][round_up32(N)]); the last layer
// writes fp32 logits.
cudaError_t launch_gemm_tf32x3(sama_ctx* ctx, const TcLayer& L, cudaStream_t st) {
    TcState* ts = tc_state(ctx);
    if (!ts) return cudaErrorInvalidValue;
    const int Kp = round_up32(L.K);
    const int nbr = L.branches == 1 ? 1 : 2;  // the direct gradient runs a single branch
    const int num_kb = Kp / BKF;
    // Tile shape.  A narrow last layer takes the 16-wide tile (hidden layers never do: their tiles must also
    // write the zero padding up to round_up32(N)).  Otherwise the candidates are single-CTA tiles of 128 x 64
    // and 128 x 128 and the CTA pair's 256 x 256; the one with the lowest estimate of
    //   rounds x (k-blocks x time per k-block + time to store a tile),  rounds = ceil(tiles / co-resident units)
    // is taken (a pair kernel whose last round is shared by two pairs per tile counts that round as half).
    // Times per k-block (microseconds, measured on the three workloads): wider tiles do more
    // work per staged operand byte, narrower ones fill the machine when the layer has few tiles.
    const bool narrow_last = L.last && L.N <= 16;
    int bn = 64, ksplit = 1;
    bool pair = false;
    if (narrow_last) {
        bn = 16;
    } else {
        struct Cand { int bn; bool pair; double t_kb, t_tile; };
        const Cand cands[3] = {{64, false, 0.55, 3.0}, {128, false, 0.72, 4.0}, {256, true, 1.12, 6.0}};
        const bool pair_ok = L.M > BM && L.N >= 256 && ts->pair_units > 0;
        const bool no_pair = ts->no_pair;
        double best = 0.0;
        for (const Cand& c : cands) {
            if (c.bn == 128 && L.N <= 64) continue;
            if (c.pair && (!pair_ok || no_pair)) continue;
            const int64_t tm = c.pair ? (L.M + 2 * BM - 1) / (2 * BM) : (L.M + BM - 1) / BM;
            const int64_t items = tm * ((L.N + c.bn - 1) / c.bn) * nbr;
            const int64_t units = c.pair ? ts->pair_units : ctx->sm_count;
            double rounds = (double)((items + units - 1) / units);
            if (c.pair && !ts->no_tail && items > units && items % units > 0 && 2 * (items % units) <= units &&
                num_kb >= 16)
                rounds = (double)(items / units) + 0.55;
            const double cost = rounds * (num_kb * c.t_kb + c.t_tile);
            if (best == 0.0 || cost < best) { best = cost; bn = c.bn; pair = c.pair; ksplit = 1; }
            // a layer with few tiles: a cluster of 2 or 4 CTAs shares each tile's contraction (one wave,
            // at least two k-blocks per CTA, about 4 us for the exchange; each CTA stores 1 / ks of the tile)
            for (int ks = 2; ks <= 4 && !c.pair && ctx->tc_ws; ks *= 2) {
                if (items * ks > units || num_kb < 2 * ks || c.bn / ks < 32 ||
                    (size_t)items * ks * BM * c.bn > ctx->tc_ws_floats)
                    break;
                const double cost_ks = ((num_kb + ks - 1) / ks) * c.t_kb + c.t_tile / ks + 4.0;
                if (cost_ks < best) { best = cost_ks; bn = c.bn; pair = false; ksplit = ks; }
            }
        }
        if (ts->no_ksplit) ksplit = 1;
        // overrides for experiments (SAMA_TC_TILE): 64 / 128 force a single-CTA width, 256 the pair
        const int ov = ts->tile;
        if (ov == 64 || ov == 128) { bn = ov; pair = false; ksplit = 1; }
        if (ov == 256 && pair_ok && !no_pair) { bn = 256; pair = true; ksplit = 1; }
    }
    const int a_slabs = (L.shared_a || nbr == 1) ? 1 : 2;
    // a box never exceeds the tensor's extent; rows of the shared-memory tile that no copy fills only
    // feed output rows / columns that the epilogue does not store
    const int wrows = pair ? bn / 2 : bn;
    const int a_box = L.M < BM ? L.M : BM, w_box = L.N < wrows ? L.N : wrows;
    const int64_t a_slab = (int64_t)L.M * Kp;
    // W operands: the pre-split copy, or (w_theta given) this layer's block of theta and of p themselves, rows
    // of K floats, from which the kernel forms them; columns beyond K read as zero
    const bool xf = L.w_theta != nullptr;
    if (xf && (narrow_last || !L.w_p || !L.eps_fd || L.K < BKF || (L.K & 3) || nbr != 2)) return cudaErrorInvalidValue;
    const CUtensorMap* maps[4] = {cached_map(ts, L.a_hi, Kp, L.M, a_slabs, a_box, a_slab),
                                  cached_map(ts, L.a_lo, Kp, L.M, a_slabs, a_box, a_slab),
                                  xf ? cached_map(ts, L.w_theta, L.K, L.N, 1, w_box, (int64_t)L.N * L.K)
                                     : cached_map(ts, L.w_hi, Kp, L.N, nbr, w_box, L.w_slab),
                                  xf ? cached_map(ts, L.w_p, L.K, L.N, 1, w_box, (int64_t)L.N * L.K)
                                     : cached_map(ts, L.w_lo, Kp, L.N, nbr, w_box, L.w_slab)};
    if (!maps[0] || !maps[1] || !maps[2] || !maps[3]) return cudaErrorInvalidValue;
    TcArgs a;
    a.bias[0] = L.bias[0];
    a.bias[1] = L.bias[1];
    a.out_f32[0] = L.out_f32[0];
    a.out_f32[1] = L.out_f32[1];
    a.out_hi = L.out_hi;
    a.out_lo = L.out_lo;
    a.M = L.M;
    a.N = L.N;
    a.num_kb = num_kb;
    a.ldc = L.ldc;
    a.ld_next = round_up32(L.N);
    a.relu = L.relu;
    a.last = L.last;
    a.shared_a = L.shared_a;
    a.both = L.both;
    a.mask = L.mask;
    a.ldm = L.ldm;
    // a pair's barrier counts both CTAs' copies
    a.tx_bytes = (uint32_t)(2 * a_box * BKF * 4 + (xf ? 0 : 2 * w_box * BKF * 4)) * (pair ? 2u : 1u);
    a.w_tx_bytes = (uint32_t)(2 * w_box * BKF * 4);
    a.eps_fd = L.eps_fd;
    a.status = &ctx->scalars->status;
    a.tiles_m = pair ? (L.M + 2 * BM - 1) / (2 * BM) : (L.M + BM - 1) / BM;
    a.tiles_n = (L.N + bn - 1) / bn;
    a.branches = nbr;
    a.ksplit = pair ? 1 : ksplit;
    a.ws = reinterpret_cast<float4*>(ctx->tc_ws);
    a.flags = ctx->tc_flags;
    a.full_rounds = 0;
    a.tail_tiles = 0;
    // about one wave of CTAs per group: group_n N-tiles x all M-tiles
    a.group_n = ctx->sm_count / a.tiles_m;
    if (a.group_n < 1) a.group_n = 1;
    if (a.group_n > a.tiles_n) a.group_n = a.tiles_n;
    if (ts->group >= 1 && ts->group <= a.tiles_n) a.group_n = ts->group;
    const int items = a.tiles_m * a.tiles_n * nbr;
    const int sms = ctx->sm_count;
    KernelScope scope(ctx, SAMA_K_GEMM_TF32X3, L.layer, st);
    // The matrix products keep the dependent-launch overlap even inside a chain that switched it off for
    // its small kernels (the direct gradient, see run_meta_grad_tc).
    PdlScope pdl(pdl_enabled() ? 1 : 0);
    // eight epilogue warps (two per lane quarter, each taking half of the columns) except on the 16-wide tile
    if (xf) {
        if (pair)
            return launch_tc<256, true, 8, kXf>(maps, a, items, ts->pair_units, !ts->no_tail, st, ctx->tc_ws_floats,
                                                ctx->tc_flags ? kTcFlags : 0);
        if (bn == 64) return launch_tc<64, false, 8, kXf>(maps, a, items, sms, false, st);
        return launch_tc<128, false, 8, kXf>(maps, a, items, sms, false, st);
    }
    if (pair)
        return launch_tc<256, true, 8, 0>(maps, a, items, ts->pair_units, !ts->no_tail, st, ctx->tc_ws_floats,
                                          ctx->tc_flags ? kTcFlags : 0);
    if (bn == 16) return launch_tc<16, false, 4, 0>(maps, a, items, sms, false, st);
    if (bn == 64) return launch_tc<64, false, 8, 0>(maps, a, items, sms, false, st);
    return launch_tc<128, false, 8, 0>(maps, a, items, sms, false, st);
}

}  // namespace sama
