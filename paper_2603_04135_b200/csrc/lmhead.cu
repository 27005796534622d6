// Fused LM-head + GRPO loss: the logits z = hidden W^T are produced tile by tile by the 5th-generation
// tensor cores (tcgen05.mma, accumulators in tensor memory) and consumed on the spot — the row-wise
// log-sum-exp and the sampled token's logit are folded in as each 128 x 256 tile leaves TMEM, so the
// [T x V] logits never exist in HBM (Eq. 1's pi_theta(o_t | ...) is a log-softmax of exactly these).
//
// One persistent CTA per SM owns 128 tokens at a time and sweeps the whole vocabulary:
//   warp 0      TMA producer: 64-wide K slabs of hidden (128 rows) and of W (256 rows), 128B-swizzled,
//               into a 4-stage shared-memory ring (no multicast)
//   warp 1      one elected thread issues tcgen05.mma (M=128, N=256, K=16 x 4 per slab) into one of two
//               256-column TMEM accumulators; tcgen05.commit releases smem stages / publishes the tile
//   warps 2-5   epilogue: each thread owns one token row; tcgen05.ld 32 columns at a time, online
//               (max, sum 2^x) in the base-2 domain, picks up z[y]; after the last vocabulary tile the
//               binary64 scalar stage of the loss sweep (same code) writes the row's terms
// While the epilogue drains accumulator b, the MMA warp already fills accumulator 1-b.
// Every wait is bounded; on a timeout the CTA records DPPO_STATUS_TIMEOUT, leaves its loops, frees its
// tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {

constexpr int kBM = 128;                 // tokens per tile (TMEM lanes)
constexpr int kBN = 256;                 // vocabulary entries per tile (TMEM columns of one accumulator)
constexpr int kBK = 64;                  // K slab: 64 bf16 = one 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kStageBytesA = kBM * kBK * 2;                  // 16 KB
constexpr int kStageBytesB = kBN * kBK * 2;                  // 32 KB
constexpr int kStageBytes = kStageBytesA + kStageBytesB;
constexpr int kLmThreads = 192;
constexpr int kTmemCols = 512;
constexpr unsigned long long kLmWaitLimitNs = 2000000000ull;

struct LmShared {
    unsigned long long full[kStages];    // TMA bytes have landed in stage s
    unsigned long long empty[kStages];   // the MMAs reading stage s are done
    unsigned long long acc_full[2];      // accumulator b holds a finished tile
    unsigned long long acc_empty[2];     // the epilogue has drained accumulator b (4 warps arrive)
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ uint32_t lm_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long lm_global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait; also leaves when another role has raised the abort flag.
__device__ __forceinline__ bool lm_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const unsigned long long t0 = lm_global_ns();
    for (;;) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
        if (*abort_flag) return false;
        if (lm_global_ns() - t0 > kLmWaitLimitNs) { *abort_flag = 1; return false; }
    }
}

// Bounded wait that ignores the abort flag (used on the way out).
__device__ __forceinline__ bool lm_wait_plain(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    const unsigned long long t0 = lm_global_ns();
    for (;;) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
        if (lm_global_ns() - t0 > limit_ns) return false;
    }
}

__device__ __forceinline__ void lm_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ float lm_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor of a K-major, 128B-swizzled tile whose rows are 128 bytes apart:
// start address >> 4, leading byte offset 1 (unused for swizzled K-major), stride byte offset 1024 >> 4
// (8-row swizzle atoms), descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t lm_smem_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// Instruction descriptor of kind::f16: D = f32, A = B = bf16, both K-major, N = 256, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

struct LmArgs {
    LossArgs loss;          // side inputs, outputs, scalars (logits / dlogits unused)
    int H;
    int n_mtiles, n_ntiles, n_ksteps;
};

__global__ void __launch_bounds__(kLmThreads, 1)
lmhead_fwd_kernel(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_w,
                  const LmArgs g) {
    extern __shared__ unsigned char lm_raw[];
    __shared__ LmShared sh;
    const uint32_t tiles = (lm_smem_u32(lm_raw) + 1023u) & ~1023u;      // 1024-byte aligned ring (swizzle atoms)
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const LossArgs& a = g.loss;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    const int n_mtiles = (int)min((long long)g.n_mtiles, (T + kBM - 1) / kBM);
    volatile int* abort_flag = &sh.abort;

    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.empty[s])));
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.acc_full[b])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" :: "r"(lm_smem_u32(&sh.acc_empty[b])));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                                     // tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(lm_smem_u32(&sh.tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;                                             // slab counter over the whole CTA lifetime
            for (int m = blockIdx.x; m < n_mtiles && !*abort_flag; m += gridDim.x) {
                for (int n = 0; n < g.n_ntiles && !*abort_flag; ++n) {
                    for (int k = 0; k < g.n_ksteps; ++k, ++it) {
                        const uint32_t s = it % kStages, use = it / kStages;
                        if (use > 0 && !lm_wait(lm_smem_u32(&sh.empty[s]), (use - 1) & 1, abort_flag)) break;
                        const uint32_t bar = lm_smem_u32(&sh.full[s]);
                        const uint32_t dst_a = tiles + s * kStageBytes, dst_b = dst_a + kStageBytesA;
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"((uint32_t)kStageBytes) : "memory");
                        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                                     :: "r"(dst_a), "l"(&map_hidden), "r"(bar), "r"(k * kBK), "r"(m * kBM) : "memory");
                        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                                     :: "r"(dst_b), "l"(&map_w), "r"(bar), "r"(k * kBK), "r"(n * kBN) : "memory");
                    }
                }
            }
            if (*abort_flag) {
                // leaving early: give this thread's own copies in flight a bounded chance to land before
                // the CTA (and its shared memory) goes away
                const uint32_t pending = it < (uint32_t)kStages ? it : (uint32_t)kStages;
                for (uint32_t j = 0; j < pending; ++j) {
                    const uint32_t i2 = it - 1 - j;
                    lm_wait_plain(lm_smem_u32(&sh.full[i2 % kStages]), (i2 / kStages) & 1, 200000000ull);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tile = 0;
            for (int m = blockIdx.x; m < n_mtiles && !*abort_flag; m += gridDim.x) {
                for (int n = 0; n < g.n_ntiles && !*abort_flag; ++n, ++tile) {
                    const uint32_t b = tile & 1, use_b = tile >> 1;
                    if (use_b > 0 && !lm_wait(lm_smem_u32(&sh.acc_empty[b]), (use_b - 1) & 1, abort_flag)) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d_tmem = tmem_base + b * kBN;
                    bool ok = true;
                    for (int k = 0; k < g.n_ksteps; ++k, ++it) {
                        const uint32_t s = it % kStages, use = it / kStages;
                        if (!lm_wait(lm_smem_u32(&sh.full[s]), use & 1, abort_flag)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t sa = tiles + s * kStageBytes, sb = sa + kStageBytesA;
                        const uint64_t da = lm_smem_desc(sa), db = lm_smem_desc(sb);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk) {          // 16 K elements = 32 bytes inside the swizzle row
                            const uint32_t accumulate = (k > 0 || kk > 0) ? 1u : 0u;
                            asm volatile("{\n\t.reg .pred p;\n\t"
                                         "setp.ne.b32 p, %4, 0;\n\t"
                                         "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                         :: "r"(d_tmem), "l"(da + (uint64_t)(kk * 2)), "l"(db + (uint64_t)(kk * 2)),
                                            "r"(kIdesc), "r"(accumulate) : "memory");
                        }
                        // frees this smem stage once the MMAs issued so far have read it
                        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                     :: "r"(lm_smem_u32(&sh.empty[s])) : "memory");
                    }
                    if (!ok) break;
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 :: "r"(lm_smem_u32(&sh.acc_full[b])) : "memory");
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                                          // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        const float c = a.scale2;
        uint32_t tile = 0;
        for (int m = blockIdx.x; m < n_mtiles; m += gridDim.x) {
            const long long t = (long long)m * kBM + row;
            const bool live = t < T;
            RowInputs in;
            in.state = 0; in.y = -1;
            if (live) row_gather(a, t, in, false);
            const int y = (live && in.state == 0) ? in.y : -1;
            float m2 = -INFINITY, s = 0.0f, zy = 0.0f;
            bool ok = true;
            for (int n = 0; n < g.n_ntiles; ++n, ++tile) {
                const uint32_t b = tile & 1, use_b = tile >> 1;
                // warp-uniform outcome: the tcgen05.ld below must be executed by all 32 lanes together
                if (!__all_sync(0xffffffffu, lm_wait(lm_smem_u32(&sh.acc_full[b]), use_b & 1, abort_flag))) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * kBN;
#pragma unroll 1
                for (int ch = 0; ch < kBN / 32; ++ch) {
                    uint32_t v[32];
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                                 : "r"(taddr + (uint32_t)(ch * 32)) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int col0 = n * kBN + ch * 32;
                    const int valid = a.V - col0;                        // columns of this chunk inside the vocabulary
                    float cm = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float x = __uint_as_float(v[j]);
                        if (j == y - col0) zy = x;
                        x = (j < valid) ? x * c : -INFINITY;
                        v[j] = __float_as_uint(x);
                        cm = fmaxf(cm, x);
                    }
                    if (cm > m2) { s *= lm_ex2(m2 - cm); m2 = cm; }
                    float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        acc0 += lm_ex2(__uint_as_float(v[j]) - m2);
                        acc1 += lm_ex2(__uint_as_float(v[j + 1]) - m2);
                    }
                    s += acc0 + acc1;
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) lm_arrive(lm_smem_u32(&sh.acc_empty[b]));
            }
            if (!ok) break;
            if (live) {
                in.zy = (double)zy / a.temperature;
                row_finish(a, t, in, m2, s, true);
            }
        }
    }

    // ---- common exit: nobody touches tensor memory any more, then the allocating warp frees it
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && sh.abort) set_status(a.status, DPPO_STATUS_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [rows x H] bf16 row-major; boxes of 64 columns x box_rows rows, 128B swizzle, zero fill out of bounds.
static int make_map(CUtensorMap* map, const void* base, long long rows, int H, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled failed with %d", (int)r);
    return DPPO_OK;
}

}  // namespace dppo

extern "C" size_t dppo_lmhead_workspace_bytes(const dppo_lmhead_params* p) {
    if (!p) return 0;
    return dppo_grpo_loss_workspace_bytes(&p->loss);
}

extern "C" int dppo_lmhead_grpo_loss(const dppo_lmhead_params* p, const void* hidden, const void* W,
                                     const int32_t* target, const float* logp_old, const float* logp_ref,
                                     const int32_t* cu_seqlens, const int32_t* n_tokens_dev, const float* adv,
                                     const float* w, const int32_t* seg_map, void* dhidden, void* dW,
                                     float* logp_out, float* lse_out, float* loss_out, void* workspace,
                                     size_t workspace_bytes, int32_t* status, void* stream) {
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL params");
    const dppo_loss_params& lp = p->loss;
    if (lp.T_max < 0 || lp.V < 1 || lp.S_max < 0 || p->H < 1)
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: T_max=%lld V=%d S_max=%d H=%d", (long long)lp.T_max, lp.V, lp.S_max, p->H);
    if (p->H % kBK != 0) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: H=%d must be a multiple of %d", p->H, kBK);
    if (lp.dtype != DPPO_BF16) return fail(DPPO_ERR_UNSUPPORTED, "lmhead: hidden and W must be bf16");
    if (!(lp.temperature > 0.0) || !(lp.eps_lo >= 0.0) || !(lp.eps_hi >= 0.0) || !(lp.beta == lp.beta))
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: temperature must be > 0, eps >= 0, beta a number");
    if (lp.T_max >= ((int64_t)1 << 31) - kBM) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: T_max too large");
    if (dhidden || dW) return fail(DPPO_ERR_UNSUPPORTED, "lmhead: the backward (dhidden, dW) is not built yet; pass NULL for both");
    if (!loss_out) return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL loss_out");
    if (lp.T_max > 0) {
        if (!hidden || !W || !target || !logp_old || !logp_ref || !cu_seqlens || !adv || !w)
            return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL array");
        if (lp.S_max < 1) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: tokens but no sequences (S_max=0)");
        if (((uintptr_t)hidden & 15) || ((uintptr_t)W & 15)) return fail(DPPO_ERR_MISALIGNED, "lmhead: hidden / W not 16-byte aligned");
    }
    const size_t need = dppo_lmhead_workspace_bytes(p);
    if (!workspace || workspace_bytes < need)
        return fail(DPPO_ERR_WORKSPACE_TOO_SMALL, "lmhead: workspace %zu < %zu bytes", workspace_bytes, need);
    if ((uintptr_t)workspace & 15) return fail(DPPO_ERR_MISALIGNED, "lmhead: workspace not 16-byte aligned");

    LmArgs g;
    LossArgs& a = g.loss;
    a.logits = nullptr; a.dlogits = nullptr;
    a.target = target; a.logp_old = logp_old; a.logp_ref = logp_ref;
    a.cu_seqlens = cu_seqlens; a.n_tokens_dev = n_tokens_dev; a.adv = adv; a.w = w; a.seg_map = seg_map;
    a.logp_out = logp_out; a.lse_out = lse_out; a.terms = (RowTerms*)workspace; a.status = status;
    a.T_max = lp.T_max; a.row_bytes = 0; a.V = lp.V; a.S_max = lp.S_max; a.bf16 = 1;
    a.eps_lo = lp.eps_lo; a.eps_hi = lp.eps_hi; a.beta = lp.beta; a.temperature = lp.temperature;
    a.scale2 = (float)(1.4426950408889634 / lp.temperature);
    g.H = p->H;
    g.n_mtiles = (int)((lp.T_max + kBM - 1) / kBM);
    g.n_ntiles = (lp.V + kBN - 1) / kBN;
    g.n_ksteps = p->H / kBK;
    cudaStream_t s = (cudaStream_t)stream;
    if (lp.T_max > 0) {
        alignas(64) CUtensorMap map_h, map_w;
        int rc = make_map(&map_h, hidden, lp.T_max, p->H, kBM);
        if (rc != DPPO_OK) return rc;
        rc = make_map(&map_w, W, lp.V, p->H, kBN);
        if (rc != DPPO_OK) return rc;
        const size_t dyn = (size_t)kStages * kStageBytes + 1024;
        cudaError_t e = cudaFuncSetAttribute(lmhead_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
        if (e != cudaSuccess) return cuda_fail(e, "lmhead: shared memory attribute");
        const int grid = g.n_mtiles < sm_count() ? g.n_mtiles : sm_count();
        lmhead_fwd_kernel<<<grid, kLmThreads, dyn, s>>>(map_h, map_w, g);
        DPPO_CHECK_LAUNCH("lmhead forward launch");
    }
    return launch_loss_reduce(a, loss_out, s);
}
