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

// ---- 16-byte vectors ------------------------------------------------------------------------------
template <bool kBf16> struct Elems;
template <> struct Elems<true> {
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&f)[8]) {
        f[0] = __uint_as_float(q.x << 16); f[1] = __uint_as_float(q.x & 0xffff0000u);
        f[2] = __uint_as_float(q.y << 16); f[3] = __uint_as_float(q.y & 0xffff0000u);
        f[4] = __uint_as_float(q.z << 16); f[5] = __uint_as_float(q.z & 0xffff0000u);
        f[6] = __uint_as_float(q.w << 16); f[7] = __uint_as_float(q.w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[8]) {
        uint4 q;
        __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
        __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]), d = __floats2bfloat162_rn(f[6], f[7]);
        q.x = *reinterpret_cast<uint32_t*>(&a); q.y = *reinterpret_cast<uint32_t*>(&b);
        q.z = *reinterpret_cast<uint32_t*>(&c); q.w = *reinterpret_cast<uint32_t*>(&d);
        return q;
    }
    static __device__ __forceinline__ float load1(const void* row, int v) {
        return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(row)[v]);
    }
    static __device__ __forceinline__ void store1(void* row, int v, float x) {
        reinterpret_cast<__nv_bfloat16*>(row)[v] = __float2bfloat16_rn(x);
    }
};
template <> struct Elems<false> {
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&f)[4]) {
        f[0] = __uint_as_float(q.x); f[1] = __uint_as_float(q.y);
        f[2] = __uint_as_float(q.z); f[3] = __uint_as_float(q.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&f)[4]) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
    static __device__ __forceinline__ float load1(const void* row, int v) {
        return reinterpret_cast<const float*>(row)[v];
    }
    static __device__ __forceinline__ void store1(void* row, int v, float x) {
        reinterpret_cast<float*>(row)[v] = x;
    }
};

// ---- scalar stage (one thread per row) -----------------------------------------------------------
// ref2/sum2: the row's sum of 2^(z c) is sum2 * 2^ref2 with c = log2(e)/temperature as used in pass 1.
__device__ RowScalars row_scalar_stage(const LossArgs& a, long long t, float ref2, float sum2) {
    RowScalars out;
    const double lse2 = (double)ref2 + log2((double)sum2);           // base-2 log-sum-exp of z c
    const double lse = lse2 * 0.6931471805599453;                    // natural log-sum-exp of z / temperature
    out.lse2_hi = (float)lse2;
    out.lse2_lo = (float)(lse2 - (double)out.lse2_hi);
    out.g_over_tau = 0.0f;
    out.valid = false;
    const int y = a.target[t];
    RowTerms terms = {0.0, 0.0, 0.0, 0.0};
    float logp_f = 0.0f;
    // sequence of this token: the last s with cu_seqlens[s] <= t
    int lo = 0, hi = a.S_max;                                        // invariant: cu[lo] <= t (checked below)
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)a.cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    const long long seg_lo = a.cu_seqlens[lo], seg_hi = a.cu_seqlens[lo + 1];
    if (a.S_max < 1 || t < seg_lo || t >= seg_hi) {
        set_status(a.status, DPPO_STATUS_BAD_SEGMENTS);
    } else if (y < 0 || y >= a.V) {
        set_status(a.status, DPPO_STATUS_BAD_TARGET);
    } else {
        const int idx = a.seg_map ? a.seg_map[lo] : lo;
        const double A = (double)a.adv[idx];
        const double W = (double)a.w[idx] / (double)(seg_hi - seg_lo);
        const double zy = (double)(a.bf16 ? Elems<true>::load1(a.logits + t * a.row_bytes, y)
                                          : Elems<false>::load1(a.logits + t * a.row_bytes, y)) / a.temperature;
        const double logp = zy - lse;
        const double rho = exp(logp - (double)a.logp_old[t]);
        const double d = (double)a.logp_ref[t] - logp;
        const double rho_hat = exp(d);
        const double kl = rho_hat - d - 1.0;
        const double s1 = rho * A;
        const double s2 = fmin(fmax(rho, 1.0 - a.eps_lo), 1.0 + a.eps_hi) * A;
        const bool clipped = s2 < s1;
        const double surr = clipped ? s2 : s1;
        const double dj = (clipped ? 0.0 : A * rho) + a.beta * (rho_hat - 1.0);
        terms.loss = -W * (surr - a.beta * kl);
        terms.pg = -W * surr;
        terms.kl = W * kl;
        terms.clipped = clipped ? 1.0 : 0.0;
        out.g_over_tau = (float)(-W * dj / a.temperature);
        out.valid = true;
        logp_f = (float)logp;
    }
    a.terms[t] = terms;
    if (a.logp_out) a.logp_out[t] = logp_f;
    if (a.lse_out) a.lse_out[t] = (float)lse;
    return out;
}

// ---- general kernel --------------------------------------------------------------------------------
constexpr int kRowThreads = 512;

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

        // pass 1: running raw maximum m, reference r = m c, sum of 2^(z c - r)
        float m = -INFINITY, r = -INFINITY, s = 0.0f;
        for (int i = tid; i < nvec; i += kRowThreads) {
            float f[VW];
            E::unpack(rowv[i], f);
            float mx = f[0];
#pragma unroll
            for (int e = 1; e < VW; ++e) mx = fmaxf(mx, f[e]);
            if (mx > m) {
                const float r_new = mx * c;
                s *= exp2f(r - r_new);                       // 0 when r is still -inf
                m = mx; r = r_new;
            }
#pragma unroll
            for (int e = 0; e < VW; ++e) s += exp2f(fmaf(f[e], c, -r));
        }
        for (int v = nvec * VW + tid; v < a.V; v += kRowThreads) {      // ragged tail
            const float z = E::load1(row, v);
            if (z > m) {
                const float r_new = z * c;
                s *= exp2f(r - r_new);
                m = z; r = r_new;
            }
            s += exp2f(fmaf(z, c, -r));
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
constexpr int kReduceThreads = 1024;

__global__ void __launch_bounds__(kReduceThreads)
loss_reduce_kernel(const RowTerms* __restrict__ terms, long long T_max, const int32_t* __restrict__ n_tokens_dev,
                   float* __restrict__ loss_out) {
    __shared__ double sh[4][kReduceThreads];
    const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (long long t = threadIdx.x; t < T; t += kReduceThreads) {
        const RowTerms x = terms[t];
        acc[0] += x.loss; acc[1] += x.pg; acc[2] += x.kl; acc[3] += x.clipped;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) sh[k][threadIdx.x] = acc[k];
    __syncthreads();
    for (int half = kReduceThreads / 2; half > 0; half >>= 1) {
        if (threadIdx.x < half) {
#pragma unroll
            for (int k = 0; k < 4; ++k) sh[k][threadIdx.x] += sh[k][threadIdx.x + half];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        loss_out[0] = (float)sh[0][0];
        loss_out[1] = (float)sh[1][0];
        loss_out[2] = (float)sh[2][0];
        loss_out[3] = T > 0 ? (float)(sh[3][0] / (double)T) : 0.0f;
        loss_out[4] = (float)T;
    }
}

int launch_rows_general(const LossArgs& a, cudaStream_t s) {
    const long long blocks = a.T_max < (long long)sm_count() * 4 ? a.T_max : (long long)sm_count() * 4;
    if (a.bf16) grpo_loss_rows_kernel<true><<<(unsigned)blocks, kRowThreads, 0, s>>>(a);
    else        grpo_loss_rows_kernel<false><<<(unsigned)blocks, kRowThreads, 0, s>>>(a);
    DPPO_CHECK_LAUNCH("grpo_loss rows launch");
    return DPPO_OK;
}

int launch_loss_reduce(const LossArgs& a, float* loss_out, cudaStream_t s) {
    loss_reduce_kernel<<<1, kReduceThreads, 0, s>>>(a.terms, a.T_max, a.n_tokens_dev, loss_out);
    DPPO_CHECK_LAUNCH("grpo_loss reduce launch");
    return DPPO_OK;
}

}  // namespace dppo

extern "C" size_t dppo_grpo_loss_workspace_bytes(const dppo_loss_params* p) {
    if (!p || p->T_max < 0) return 0;
    const size_t rows = (size_t)(p->T_max > 0 ? p->T_max : 1);
    return (rows * sizeof(dppo::RowTerms) + 255) & ~(size_t)255;
}

extern "C" int dppo_grpo_loss_fwd_bwd(const dppo_loss_params* p, const void* logits, const int32_t* target,
                                      const float* logp_old, const float* logp_ref,
                                      const int32_t* cu_seqlens, const int32_t* n_tokens_dev,
                                      const float* adv, const float* w, const int32_t* seg_map,
                                      void* dlogits, float* logp_out, float* lse_out, float* loss_out,
                                      void* workspace, size_t workspace_bytes, int32_t* status,
                                      void* stream) {
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: NULL params");
    if (p->T_max < 0 || p->V < 1 || p->S_max < 0)
        return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: T_max=%lld V=%d S_max=%d", (long long)p->T_max, p->V, p->S_max);
    if (p->dtype != DPPO_F32 && p->dtype != DPPO_BF16) return fail(DPPO_ERR_UNSUPPORTED, "grpo_loss: dtype %d", p->dtype);
    if (p->row_stride < p->V) return fail(DPPO_ERR_BAD_SHAPE, "grpo_loss: row_stride %lld < V %d", (long long)p->row_stride, p->V);
    if (!(p->temperature > 0.0) || !(p->eps_lo >= 0.0) || !(p->eps_hi >= 0.0) || !(p->beta == p->beta))
        return fail(DPPO_ERR_INVALID_ARG, "grpo_loss: temperature must be > 0, eps >= 0, beta a number");
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

    LossArgs a;
    a.logits = (const char*)logits; a.dlogits = (char*)dlogits;
    a.target = target; a.logp_old = logp_old; a.logp_ref = logp_ref;
    a.cu_seqlens = cu_seqlens; a.n_tokens_dev = n_tokens_dev; a.adv = adv; a.w = w; a.seg_map = seg_map;
    a.logp_out = logp_out; a.lse_out = lse_out; a.terms = (RowTerms*)workspace; a.status = status;
    a.T_max = p->T_max; a.row_bytes = (long long)p->row_stride * (long long)esize;
    a.V = p->V; a.S_max = p->S_max; a.bf16 = p->dtype == DPPO_BF16 ? 1 : 0;
    a.eps_lo = p->eps_lo; a.eps_hi = p->eps_hi; a.beta = p->beta; a.temperature = p->temperature;
    a.scale2 = (float)(1.4426950408889634 / p->temperature);
    cudaStream_t s = (cudaStream_t)stream;
    if (p->T_max > 0) {
        const int rc = launch_rows_general(a, s);
        if (rc != DPPO_OK) return rc;
    }
    return launch_loss_reduce(a, loss_out, s);
}
