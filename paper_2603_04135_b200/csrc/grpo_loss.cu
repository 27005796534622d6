// Fused GRPO loss sweep over the logits (Eq. 1 with the rescaling weights of Eq. 18) and dlogits.
//
// Per token row: one streaming pass for (max, sum exp) -> lse, a scalar stage (one thread, binary64)
// for logp, the ratios, the clipped surrogate, the KL estimator and g = dloss/dlogp, then a second
// pass that writes dlogits = g (onehot - softmax)/temperature.  Row terms go to the workspace and a
// fixed-order binary64 reduction produces the five loss scalars, so results are bit-reproducible.
//
// This file holds the general kernel: any V, f32 or bf16, one CTA per row with both passes reading
// global memory (the second pass hits L2 for rows that still sit there).
#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {

// ---- kernel choice for variant 0 (from sweeps on B200 over rows of 2 KB to 594 KB, both dtypes) -------------
// Every row that fits goes to the shared-memory kernel, split over the smallest cluster whose slices stay at a size
// that keeps enough CTAs per SM in flight: the whole row in one CTA up to 44 KB (five CTAs per SM), two CTAs up to
// 55 KB slices (four per SM), else four or eight CTAs with slices up to 76 KB (three per SM).  Measured at rows of
// 32 / 64 / 128 KB: 6.7 / 6.5 / 6.4 TB/s with 1 / 2 / 4 CTAs against 2.8 / 3.5 / 3.7 TB/s for the general kernel
// and 2.6 / 4.4 / 6.4 with four CTAs throughout.  Below about 8 KB per row the grid's launch rate (one CTA per row,
// about 250 rows per microsecond) is the limit: rows of up to 8 KB go to the warp-per-row kernel (2 KB rows: 3.5-3.7
// TB/s against 1.0).
constexpr size_t kSliceMax1 = 44 * 1024;
constexpr size_t kSliceMax2 = 55 * 1024;
constexpr size_t kSliceMax48 = 76 * 1024;
constexpr int kClusterThreads = 256;                // bf16 slices above 28 KB (24 KB rows: 6.3 TB/s with 128 threads, 5.5
                                                    // with 256; 32 KB rows: 6.2 against 6.3), f32 slices above 64 KB
constexpr int kClusterThreadsSmall = 128;           // shorter slices (f32 has half the arithmetic per byte)

constexpr size_t kStreamMinRowBytes = 128 * 1024;   // forward-only calls: rows from this length on go to the streaming kernel
constexpr int kWarpRowMaxVecBf16 = 512;             // rows of up to 8 KB in either dtype (8 KB bf16 rows: 4.35 TB/s against
constexpr int kWarpRowMaxVecF32 = 512;              // 3.3 TB/s in one CTA of the shared-memory kernel)

static int auto_cluster_size(int nvec) {
    const size_t limit[4] = {kSliceMax1, kSliceMax2, kSliceMax48, kSliceMax48};
    for (int i = 0, C = 1; i < 4; ++i, C *= 2)
        if ((size_t)((nvec + C - 1) / C) * 16 <= limit[i]) return C;
    return 0;                                       // longer rows: the general kernel
}

// ---- general kernel --------------------------------------------------------------------------------
constexpr int kRowThreads = 512;
LossArgs loss_args_from_params(const dppo_loss_params* p);
int run_rows(LossArgs a, int variant, cudaStream_t s, bool launch, dppo_loss_kernel_choice* choice);

template <bool kBf16>
__global__ void __launch_bounds__(kRowThreads) grpo_loss_rows_kernel(const LossArgs a) {
    using E = Elems<kBf16>;
    constexpr int VW = E::kPerVec;
    __shared__ float s_ref[kRowThreads / 32], s_sum[kRowThreads / 32];
    __shared__ RowScalars s_row;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    const int nvec = a.V / VW;
    const float c = a.scale2;

    for (long long t = blockIdx.x; t < T; t += gridDim.x) {
        const char* row = a.logits + t * a.row_bytes;
        const uint4* rowv = reinterpret_cast<const uint4*>(row);

        // pass 1: running raw maximum m, reference r = m c, sum of 2^(z c - r).  While a thread has seen nothing
        // but -inf (a masked start of the vocabulary) its reference is still -inf: the offset added to z c is then
        // 0, not -r = +inf, so that those elements add 2^(-inf) = 0 (and not the NaN of -inf + inf) and s is a
        // clean 0 when the first finite maximum arrives.
        float m = -INFINITY, r = -INFINITY, nr = 0.0f, s = 0.0f;
        for (int i = tid; i < nvec; i += kRowThreads) {
            float f[VW];
            E::unpack(rowv[i], f);
            float mx = f[0];
#pragma unroll
            for (int e = 1; e < VW; ++e) mx = fmaxf(mx, f[e]);
            if (mx > m) {
                const float r_new = mx * c;
                s *= exp2f(r - r_new);                       // s is 0 while r is still -inf
                m = mx; r = r_new; nr = -r_new;
            }
#pragma unroll
            for (int e = 0; e < VW; ++e) s += exp2f(fmaf(f[e], c, nr));
        }
        for (int v = nvec * VW + tid; v < a.V; v += kRowThreads) {      // ragged tail
            const float z = E::load1(row, v);
            if (z > m) {
                const float r_new = z * c;
                s *= exp2f(r - r_new);
                m = z; r = r_new; nr = -r_new;
            }
            s += exp2f(fmaf(z, c, nr));
        }
        // combine (r, s) pairs: warp, then block
        float R = warp_max(r);
        s = (r == -INFINITY) ? 0.0f : s * exp2f(r - R);
        s = warp_sum(s);
        if (lane == 0) { s_ref[warp] = R; s_sum[warp] = s; }
        __syncthreads();
        if (warp == 0) {
            float rr = lane < kRowThreads / 32 ? s_ref[lane] : -INFINITY;
            float ss = lane < kRowThreads / 32 ? s_sum[lane] : 0.0f;
            const float RR = warp_max(rr);
            ss = (rr == -INFINITY) ? 0.0f : ss * exp2f(rr - RR);
            ss = warp_sum(ss);
            if (lane == 0) s_row = row_scalar_stage(a, t, RR, ss);
        }
        __syncthreads();
        const RowScalars rs = s_row;

        // pass 2: dlogits = g/tau * (onehot - 2^(z c - lse2))
        if (a.dlogits) {
            char* drow = a.dlogits + t * a.row_bytes;
            uint4* drowv = reinterpret_cast<uint4*>(drow);
            const float g = rs.valid ? rs.g_over_tau : 0.0f;
            const int y = rs.valid ? a.target[t] : -1;
            for (int i = tid; i < nvec; i += kRowThreads) {
                float f[VW];
                E::unpack(rowv[i], f);
#pragma unroll
                for (int e = 0; e < VW; ++e) {
                    const float p = exp2f(fmaf(f[e], c, -rs.lse2_hi) - rs.lse2_lo);
                    f[e] = -g * p;
                }
                const int off = y - i * VW;
                if (off >= 0 && off < VW) {
#pragma unroll
                    for (int e = 0; e < VW; ++e) if (e == off) f[e] += g;
                }
                drowv[i] = E::pack(f);
            }
            for (int v = nvec * VW + tid; v < a.V; v += kRowThreads) {
                const float p = exp2f(fmaf(E::load1(row, v), c, -rs.lse2_hi) - rs.lse2_lo);
                E::store1(drow, v, -g * p + (v == y ? g : 0.0f));
            }
        }
        __syncthreads();                                     // s_row / s_ref are reused by the next row
    }
}

// ---- final reduction: fixed order, binary64 ------------------------------------------------------
// Two launches.  The first cuts the rows into kReduceBlocks contiguous ranges, one block each (one
// block alone is held to a single SM's load bandwidth); the second adds the per-block partial sums.
// Ranges, strides and both trees depend on T only, so the result is the same on every run.
constexpr int kReduceThreads = 256;

__device__ __forceinline__ void block_tree_sum4(double (&sh)[4][kReduceThreads], double (&acc)[4], int n) {
#pragma unroll
    for (int k = 0; k < 4; ++k) sh[k][threadIdx.x] = acc[k];
    __syncthreads();
    for (int half = n / 2; half > 0; half >>= 1) {
        if ((int)threadIdx.x < half) {
#pragma unroll
            for (int k = 0; k < 4; ++k) sh[k][threadIdx.x] += sh[k][threadIdx.x + half];
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kReduceThreads)
loss_partial_kernel(const RowTerms* __restrict__ terms, long long T_max, const int32_t* __restrict__ n_tokens_dev,
                    RowTerms* __restrict__ partials) {
    __shared__ double sh[4][kReduceThreads];
    const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
    const long long per = (T + kReduceBlocks - 1) / kReduceBlocks;
    const long long lo = min(T, per * blockIdx.x), hi = min(T, lo + per);
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (long long t = lo + threadIdx.x; t < hi; t += kReduceThreads) {
        const RowTerms x = terms[t];
        acc[0] += x.loss; acc[1] += x.pg; acc[2] += x.kl; acc[3] += x.clipped;
    }
    block_tree_sum4(sh, acc, kReduceThreads);
    if (threadIdx.x == 0) {
        RowTerms r; r.loss = sh[0][0]; r.pg = sh[1][0]; r.kl = sh[2][0]; r.clipped = sh[3][0];
        partials[blockIdx.x] = r;
    }
}

__global__ void __launch_bounds__(kReduceThreads)
loss_final_kernel(const RowTerms* __restrict__ partials, long long T_max, const int32_t* __restrict__ n_tokens_dev,
                  float* __restrict__ loss_out) {
    static_assert(kReduceBlocks <= kReduceThreads && (kReduceBlocks & (kReduceBlocks - 1)) == 0, "one partial per thread");
    __shared__ double sh[4][kReduceThreads];
    const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    if (threadIdx.x < kReduceBlocks) {
        const RowTerms x = partials[threadIdx.x];
        acc[0] = x.loss; acc[1] = x.pg; acc[2] = x.kl; acc[3] = x.clipped;
    }
    block_tree_sum4(sh, acc, kReduceThreads);
    if (threadIdx.x == 0) {
        loss_out[0] = (float)sh[0][0];
        loss_out[1] = (float)sh[1][0];
        loss_out[2] = (float)sh[2][0];
        loss_out[3] = T > 0 ? (float)(sh[3][0] / (double)T) : 0.0f;
        loss_out[4] = (float)T;
    }
}

// One warp per sequence: lanes stride over the tokens, binary64, fixed-order tree.
__global__ void __launch_bounds__(256)
sequence_log_ratio_kernel(const float* __restrict__ logp, const float* __restrict__ logp_old,
                          const int32_t* __restrict__ cu, int S, float* __restrict__ out) {
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (s >= S) return;
    const int a = cu[s], b = cu[s + 1];
    double acc = 0.0;
    for (int t = a + lane; t < b; t += 32) acc += (double)logp[t] - (double)logp_old[t];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[s] = b > a ? (float)(acc / (double)(b - a)) : 0.0f;
}

int launch_rows_general(const LossArgs& a, cudaStream_t s) {
    const long long blocks = a.T_max < (long long)sm_count() * 4 ? a.T_max : (long long)sm_count() * 4;
    if (a.bf16) grpo_loss_rows_kernel<true><<<(unsigned)blocks, kRowThreads, 0, s>>>(a);
    else        grpo_loss_rows_kernel<false><<<(unsigned)blocks, kRowThreads, 0, s>>>(a);
    DPPO_CHECK_LAUNCH("grpo_loss rows launch");
    return DPPO_OK;
}

int launch_loss_reduce(const LossArgs& a, float* loss_out, cudaStream_t s) {
    RowTerms* partials = loss_partials(a.terms, a.T_max);
    loss_partial_kernel<<<kReduceBlocks, kReduceThreads, 0, s>>>(a.terms, a.T_max, a.n_tokens_dev, partials);
    DPPO_CHECK_LAUNCH("grpo_loss partial sums launch");
    loss_final_kernel<<<1, kReduceThreads, 0, s>>>(partials, a.T_max, a.n_tokens_dev, loss_out);
    DPPO_CHECK_LAUNCH("grpo_loss reduce launch");
    return DPPO_OK;
}

// The shape-dependent part of the kernel arguments (pointers are filled in by the caller).
LossArgs loss_args_from_params(const dppo_loss_params* p) {
    LossArgs a = {};
    const size_t esize = p->dtype == DPPO_BF16 ? 2 : 4;
    a.T_max = p->T_max; a.row_bytes = (long long)p->row_stride * (long long)esize;
    a.V = p->V; a.S_max = p->S_max; a.bf16 = p->dtype == DPPO_BF16 ? 1 : 0;
    a.eps_lo = p->eps_lo; a.eps_hi = p->eps_hi; a.beta = p->beta; a.temperature = p->temperature;
    a.scale2 = (float)(1.4426950408889634 / p->temperature);
    a.seq_log_ratio = p->seq_log_ratio; a.no_length_norm = p->no_length_norm;
    a.wait_limit_ns = kDefaultWaitLimitNs; a.test_extra_tx = 0;
    return a;
}

// Picks the row kernel for `variant` and launches it (launch = true) or only runs the checks a launch would make.
// variant: 0 picks the kernel from the shape; 1 forces the general kernel; 2 the warp-per-row kernel; 3 the
// streaming kernel (forward-only calls); 4 the tile kernel; C*10000 + threads forces the shared-memory kernel with C CTAs per row (a tuning aid; unsupported shapes are an
// error); kSelfTestVariant + one of those runs the self-test of the bounded waits (shared-memory, streaming and tile kernels).
// choice (nullable) receives what was taken; fell_back = 1 when the device refused the kernel the shape asked for
// and the general kernel took over.
constexpr int kSelfTestVariant = 1000000;

// Rows the tile kernel is chosen for: dense rows (no ragged tail of less than a vector, 16-byte aligned) of up to
// 16 KB.  With dlogits, measured on the call a training step makes: bf16 rows of 2 to 16 KB 5.6-5.7 TB/s (the
// warp-per-row kernel 3.5-4.5, one CTA per row of the shared-memory kernel 4.2-5.0), 1 KB rows 4.7 (2.2), f32 rows
// of 2 to 16 KB 6.2-6.5 (3.8-5.2).  Rows of 16 to 32 KB leave a stage partly empty (one row per tile) and stay with
// the shared-memory kernel (bf16 rows of 20 KB: 4.0 against 5.4; of 32 KB, which fill a stage: 5.7 against 6.2-6.4).
// Forward only: 4.0-4.1 TB/s on bf16 rows of 2 to 16 KB against 2.1-3.3, 4.4-4.8 on f32 rows against 2.2-4.6.
static bool tile_kernel_takes(const LossArgs& a) {
    const int per_vec = a.bf16 ? 8 : 4;
    if (a.V < per_vec || a.V % per_vec != 0 || a.row_bytes % 16 != 0) return false;
    if ((((uintptr_t)a.logits) | ((uintptr_t)a.dlogits)) & 15) return false;
    return a.row_bytes <= 16384;
}

int run_rows(LossArgs a, int variant, cudaStream_t s, bool launch, dppo_loss_kernel_choice* choice) {
    dppo_loss_kernel_choice ch = {DPPO_KERNEL_GENERAL, 1, kRowThreads, 0};
    const bool self_test = variant >= kSelfTestVariant;
    if (self_test) {
        variant -= kSelfTestVariant;
        a.wait_limit_ns = kSelfTestWaitLimitNs;
        a.test_extra_tx = 8;
    }
    int rc;
    if (variant == 1) {
        rc = launch ? launch_rows_general(a, s) : DPPO_OK;
    } else if (variant == 2) {
        ch.kernel = DPPO_KERNEL_WARP; ch.threads = 32;
        rc = launch_rows_warp(a, s, launch);
    } else if (variant == 3) {
        ch.kernel = DPPO_KERNEL_STREAM; ch.threads = 512;
        rc = launch_rows_stream(a, s, launch);
    } else if (variant == 4) {
        ch.kernel = DPPO_KERNEL_TILE; ch.threads = 512;
        rc = launch_rows_tile(a, s, launch);
    } else if (variant >= 10000) {
        ch.kernel = DPPO_KERNEL_SHARED; ch.ctas_per_row = variant / 10000; ch.threads = variant % 10000;
        rc = launch_rows_cluster(a, ch.ctas_per_row, ch.threads, s, launch);
    } else if (variant == 0) {
        rc = DPPO_ERR_UNSUPPORTED;
        const int nvec = a.V >> (a.bf16 ? 3 : 2);
        const int C = auto_cluster_size(nvec);
        bool refused = false;
        if (a.dlogits == nullptr && (size_t)nvec * 16 >= kStreamMinRowBytes) {
            // forward-only call on a long row: stream it (5.7 against 4.6 TB/s at 297 KB bf16 rows, 6.7 against 4.1 at
            // 594 KB f32 rows; the shared-memory kernel stays ahead below about 128 KB: 4.6 against 3.7 at 64 KB)
            ch.kernel = DPPO_KERNEL_STREAM; ch.threads = 512;
            rc = launch_rows_stream(a, s, launch);
            refused = rc == DPPO_ERR_UNSUPPORTED;
        } else if (tile_kernel_takes(a)) {
            ch.kernel = DPPO_KERNEL_TILE; ch.threads = 512;
            rc = launch_rows_tile(a, s, launch);
            refused = rc == DPPO_ERR_UNSUPPORTED;
        } else if (nvec <= (a.bf16 ? kWarpRowMaxVecBf16 : kWarpRowMaxVecF32)) {
            ch.kernel = DPPO_KERNEL_WARP; ch.threads = 32;
            rc = launch_rows_warp(a, s, launch);
            refused = rc == DPPO_ERR_UNSUPPORTED;
        } else if (C > 0) {
            const size_t slice = (size_t)((nvec + C - 1) / C) * 16;
            // 256 threads for bf16 slices above 28 KB and f32 slices above 64 KB, else 128
            const int threads = slice > (a.bf16 ? 28u : 64u) * 1024 ? kClusterThreads : kClusterThreadsSmall;
            ch.kernel = DPPO_KERNEL_SHARED; ch.ctas_per_row = C; ch.threads = threads;
            rc = launch_rows_cluster(a, C, threads, s, launch);
            refused = rc == DPPO_ERR_UNSUPPORTED;
        }
        if (rc == DPPO_ERR_UNSUPPORTED) {                  // too long for eight slices, or refused by this device
            ch.kernel = DPPO_KERNEL_GENERAL; ch.ctas_per_row = 1; ch.threads = kRowThreads; ch.fell_back = refused ? 1 : 0;
            rc = launch ? launch_rows_general(a, s) : DPPO_OK;
        }
    } else {
        rc = fail(DPPO_ERR_INVALID_ARG, "grpo_loss: variant %d", variant);
    }
    if (rc == DPPO_OK && self_test && ch.kernel != DPPO_KERNEL_SHARED && ch.kernel != DPPO_KERNEL_STREAM && ch.kernel != DPPO_KERNEL_TILE)
        return fail(DPPO_ERR_UNSUPPORTED, "grpo_loss: the wait self-test runs on the shared-memory, streaming and tile kernels only");
    if (choice) *choice = ch;
    return rc;
}

}  // namespace dppo

extern "C" size_t dppo_grpo_loss_workspace_bytes(const dppo_loss_params* p) {
    if (!p || p->T_max < 0) return 0;
    return dppo::loss_terms_bytes(p->T_max);
}

extern "C" int dppo_grpo_loss_fwd_bwd(const dppo_loss_params* p, const void* logits, const int32_t* target,
                                      const float* logp_old, const float* logp_ref,
                                      const int32_t* cu_seqlens, const int32_t* n_tokens_dev,
                                      const float* adv, const float* w, const int32_t* seg_map,
                                      void* dlogits, float* logp_out, float* lse_out, float* loss_out,
                                      void* workspace, size_t workspace_bytes, int32_t* status,
                                      void* stream) {
    dppo::NvtxRange nvtx_range("dppo_grpo_loss_fwd_bwd");
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: NULL params");
    if (p->T_max < 0 || p->V < 1 || p->S_max < 0)
        return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: T_max=%lld V=%d S_max=%d", (long long)p->T_max, p->V, p->S_max);
    if (p->dtype != DPPO_F32 && p->dtype != DPPO_BF16) return fail(DPPO_ERR_UNSUPPORTED, "grpo_loss: dtype %d", p->dtype);
    if (p->row_stride < p->V) return fail(DPPO_ERR_BAD_SHAPE, "grpo_loss: row_stride %lld < V %d", (long long)p->row_stride, p->V);
    if (!(p->temperature > 0.0) || !(p->eps_lo >= 0.0) || !(p->eps_hi >= 0.0) || !(p->beta == p->beta))
        return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: temperature must be > 0, eps >= 0, beta a number");
    if (p->no_length_norm != 0 && p->no_length_norm != 1) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: no_length_norm %d", p->no_length_norm);
    if (p->seq_log_ratio && p->no_length_norm) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: the sequence-level ratio needs the 1/|o| normalisation");
    if (p->variant < 0) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: variant %d", p->variant);
    if (p->T_max >= ((int64_t)1 << 31)) return fail(DPPO_ERR_BAD_SHAPE, "grpo_loss: T_max must be below 2^31");
    if (!loss_out) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: NULL loss_out");
    const size_t esize = p->dtype == DPPO_BF16 ? 2 : 4;
    if (p->T_max > 0) {
        if (!logits || !target || !logp_old || !logp_ref || !cu_seqlens || !adv || !w)
            return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: NULL array");
        if (p->S_max < 1) return fail(DPPO_ERR_BAD_SHAPE, "grpo_loss: tokens but no sequences (S_max=0)");
        if (((uintptr_t)logits & 15) || ((uintptr_t)dlogits & 15) || ((size_t)p->row_stride * esize) % 16 != 0)
            return fail(DPPO_ERR_MISALIGNED, "grpo_loss: logits/dlogits base and row stride must be multiples of 16 bytes");
    }
    const size_t need = dppo_grpo_loss_workspace_bytes(p);
    if (!workspace || workspace_bytes < need)
        return fail(DPPO_ERR_WORKSPACE_TOO_SMALL, "grpo_loss: workspace %zu < %zu bytes", workspace_bytes, need);
    if ((uintptr_t)workspace & 15) return fail(DPPO_ERR_MISALIGNED, "grpo_loss: workspace not 16-byte aligned");

    LossArgs a = loss_args_from_params(p);
    a.logits = (const char*)logits; a.dlogits = (char*)dlogits;
    a.target = target; a.logp_old = logp_old; a.logp_ref = logp_ref;
    a.cu_seqlens = cu_seqlens; a.n_tokens_dev = n_tokens_dev; a.adv = adv; a.w = w; a.seg_map = seg_map;
    a.logp_out = logp_out; a.lse_out = lse_out; a.terms = (RowTerms*)workspace; a.status = status;
    cudaStream_t s = (cudaStream_t)stream;
    if (p->T_max > 0) {
        const int rc = run_rows(a, p->variant, s, true, nullptr);
        if (rc != DPPO_OK) return rc;
    }
    return launch_loss_reduce(a, loss_out, s);
}

extern "C" int dppo_grpo_loss_kernel_choice(const dppo_loss_params* p, int forward_only, dppo_loss_kernel_choice* out) {
    using namespace dppo;
    if (!p || !out) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss_kernel_choice: NULL argument");
    if (p->V < 1 || p->T_max < 0 || (p->dtype != DPPO_F32 && p->dtype != DPPO_BF16) || p->variant < 0 || !(p->temperature > 0.0))
        return fail(DPPO_ERR_INVALID_ARG, "grpo_loss_kernel_choice: V=%d T_max=%lld dtype=%d variant=%d", p->V,
                    (long long)p->T_max, p->dtype, p->variant);
    LossArgs a = loss_args_from_params(p);
    a.dlogits = forward_only ? nullptr : (char*)16;          // only tested against NULL on this path: nothing is launched
    return run_rows(a, p->variant, nullptr, false, out);
}

extern "C" int dppo_sequence_log_ratio(const float* logp, const float* logp_old, const int32_t* cu_seqlens, int S_max,
                                       float* out, int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_sequence_log_ratio");
    (void)status;
    if (S_max < 0) return dppo::fail(DPPO_ERR_INVALID_ARG, "sequence_log_ratio: S_max=%d", S_max);
    if (S_max == 0) return DPPO_OK;
    if (!logp || !logp_old || !cu_seqlens || !out) return dppo::fail(DPPO_ERR_INVALID_ARG, "sequence_log_ratio: NULL array");
    dppo::sequence_log_ratio_kernel<<<(S_max + 7) / 8, 256, 0, (cudaStream_t)stream>>>(logp, logp_old, cu_seqlens, S_max, out);
    DPPO_CHECK_LAUNCH("sequence_log_ratio launch");
    return DPPO_OK;
}
