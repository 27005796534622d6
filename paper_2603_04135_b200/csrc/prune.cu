// Candidate sets (Eq. 15, 17), dynamic pruning masks, discrete importance rescaling (Eq. 18) and the
// history carry-forward (Eq. 16) for one batch, in one single-block kernel.
//
// The batch is tiny (P*G of a few hundred), so the whole step is latency-bound; one block avoids any
// inter-block dependency for the retained-prompt count that every gamma_q needs.  All floating-point
// decisions and factors are explicitly rounded binary64 operations; the draws are Philox4x32-10
// (Salmon et al., SC'11) keyed by (seed) and counted by (index, domain, step).
#include "common.cuh"

namespace dppo {

constexpr int kPruneThreads = 1024;

__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t hi0 = __umulhi(M0, c[0]), lo0 = M0 * c[0];
    const uint32_t hi1 = __umulhi(M1, c[2]), lo1 = M1 * c[2];
    c[0] = hi1 ^ c[1] ^ k0;
    c[1] = lo1;
    c[2] = hi0 ^ c[3] ^ k1;
    c[3] = lo0;
}

// u in [0,1) with 53 random bits: counter (index, domain, step lo, step hi), key (seed lo, seed hi).
__device__ double philox_uniform(uint64_t seed, uint64_t step, uint32_t domain, uint32_t index) {
    uint32_t c[4] = {index, domain, (uint32_t)step, (uint32_t)(step >> 32)};
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        philox_round(c, k0, k1);
    }
    const uint64_t x = (uint64_t)c[0] | ((uint64_t)c[1] << 32);
    return (double)(x >> 11) * 0x1.0p-53;
}

__device__ __forceinline__ double draw(const double* u, uint64_t seed, uint64_t step, uint32_t domain,
                                       uint32_t index) {
    return u ? u[index] : philox_uniform(seed, step, domain, index);
}

__global__ void __launch_bounds__(kPruneThreads)
prune_and_rescale_kernel(dppo_prune_params prm, const float* __restrict__ adv,
                         const float* __restrict__ mean_abs_adv, const float* __restrict__ H_prev,
                         const double* __restrict__ u_q, const double* __restrict__ u_o,
                         uint8_t* __restrict__ cand_q, uint8_t* __restrict__ cand_o,
                         uint8_t* __restrict__ keep_q, uint8_t* __restrict__ keep_o,
                         int32_t* __restrict__ n_keep_q, int32_t* __restrict__ n_keep_o,
                         float* __restrict__ gamma_q, float* __restrict__ gamma_o,
                         float* __restrict__ w_seq, float* __restrict__ H_next) {
    __shared__ int s_keep_q;
    const int P = prm.P, G = prm.G;
    const int half = H_prev ? P / 2 : 0;                       // |B_t|
    const bool fixed = prm.mode == 1;
    const int m_q = fixed ? (int)floor(__dmul_rn(prm.r_q, (double)half)) : 0;
    // pruning probability of a prompt candidate: r_q, or the realised fraction in fixed-fraction mode
    const double Pq_cand = fixed ? (half > 0 ? __ddiv_rn((double)m_q, (double)half) : 0.0) : prm.r_q;
    if (threadIdx.x == 0) s_keep_q = 0;
    __syncthreads();

    // ---- phase 1a: prompt candidates B_t — the floor(P/2) lowest history scores, ties to the lower index
    for (int k = threadIdx.x; k < P; k += blockDim.x) {
        bool cq = false;
        if (H_prev) {
            const float hk = H_prev[k];
            int rank = 0;
            for (int j = 0; j < P; ++j) {
                const float hj = H_prev[j];
                const bool before = prm.reverse ? (hj > hk) : (hj < hk);
                rank += (before || (hj == hk && j < k)) ? 1 : 0;
            }
            cq = rank < half;
        }
        cand_q[k] = cq ? 1 : 0;
    }
    __syncthreads();

    // ---- phase 1b: prompt masks
    for (int k = threadIdx.x; k < P; k += blockDim.x) {
        bool pruned = false;
        if (cand_q[k]) {
            const double uk = draw(u_q, prm.seed, prm.step, 1u, (uint32_t)k);
            if (!fixed) {
                pruned = uk < prm.r_q;
            } else if (m_q > 0) {
                // fixed fraction: the m_q candidates with the smallest (u, index) go; draws of the
                // other candidates are re-generated rather than staged in scratch memory
                int urank = 0;
                for (int j = 0; j < P && urank < m_q; ++j) {
                    if (j == k || !cand_q[j]) continue;
                    const double uj = draw(u_q, prm.seed, prm.step, 1u, (uint32_t)j);
                    urank += (uj < uk || (uj == uk && j < k)) ? 1 : 0;
                }
                pruned = urank < m_q;
            }
        }
        keep_q[k] = pruned ? 0 : 1;
        if (!pruned) atomicAdd(&s_keep_q, 1);                  // integer count: order-independent
    }
    __syncthreads();
    const int n_q = s_keep_q;
    if (threadIdx.x == 0) *n_keep_q = n_q;

    // ---- phase 2: per prompt — completion candidates, masks, factors, history
    for (int k = threadIdx.x; k < P; k += blockDim.x) {
        const float* a = adv + (size_t)k * G;
        const size_t base = (size_t)k * G;
        const bool kq = keep_q[k] != 0;
        const double Pq = cand_q[k] ? Pq_cand : 0.0;

        double sum_abs = 0.0;
        for (int i = 0; i < G; ++i) sum_abs = __dadd_rn(sum_abs, fabs((double)a[i]));
        const double bound = __dmul_rn(sum_abs, 1.0 + 1e-12);  // tie slack on |A_i| <= mean|A|
        int n_cand = 0;
        for (int i = 0; i < G; ++i) {
            const bool low = __dmul_rn((double)G, fabs((double)a[i])) <= bound;
            const bool c = prm.reverse ? !low : low;
            cand_o[base + i] = c ? 1 : 0;
            n_cand += c ? 1 : 0;
        }
        const int m_o = fixed ? (int)floor(__dmul_rn(prm.r_o, (double)n_cand)) : 0;
        const double Po_cand = fixed ? (n_cand > 0 ? __ddiv_rn((double)m_o, (double)n_cand) : 0.0) : prm.r_o;

        int n_o = 0;
        for (int i = 0; i < G; ++i) {
            bool pruned = !kq;
            if (kq && cand_o[base + i]) {
                const double ui = draw(u_o, prm.seed, prm.step, 2u, (uint32_t)(base + i));
                if (!fixed) {
                    pruned = ui < prm.r_o;
                } else if (m_o > 0) {
                    int urank = 0;
                    for (int j = 0; j < G; ++j) {
                        if (j == i || !cand_o[base + j]) continue;
                        const double uj = draw(u_o, prm.seed, prm.step, 2u, (uint32_t)(base + j));
                        urank += (uj < ui || (uj == ui && j < i)) ? 1 : 0;
                    }
                    pruned = urank < m_o;
                }
            }
            keep_o[base + i] = pruned ? 0 : 1;
            n_o += pruned ? 0 : 1;
        }
        n_keep_o[k] = n_o;

        gamma_q[k] = kq ? __double2float_rn(__ddiv_rn(__ddiv_rn((double)n_q, (double)P),
                                                      __dsub_rn(1.0, Pq))) : 0.0f;
        for (int i = 0; i < G; ++i) {
            float go = 0.0f, ws = 0.0f;
            if (keep_o[base + i]) {
                const double Po = cand_o[base + i] ? Po_cand : 0.0;
                const double one_m_po = __dsub_rn(1.0, Po);
                go = __double2float_rn(__ddiv_rn(__ddiv_rn((double)n_o, (double)G), one_m_po));
                const double den = __dmul_rn(__dmul_rn((double)((int64_t)P * G), __dsub_rn(1.0, Pq)), one_m_po);
                ws = __double2float_rn(__ddiv_rn(1.0, den));
            }
            gamma_o[base + i] = go;
            w_seq[base + i] = ws;
        }
        H_next[k] = (kq || !H_prev) ? mean_abs_adv[k] : H_prev[k];
    }
}

// History table (Eq. 16 across epochs): one score per dataset prompt; a batch reads its prompts' scores
// before pruning and writes H_next back afterwards.
__global__ void history_gather_kernel(const float* __restrict__ table, int N, const int32_t* __restrict__ ids, int P,
                                      float* __restrict__ H_batch, int32_t* status) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= P) return;
    const int id = ids[k];
    if (id < 0 || id >= N) { set_status(status, DPPO_STATUS_BAD_INDEX); H_batch[k] = 0.0f; return; }
    H_batch[k] = table[id];
}

__global__ void history_scatter_kernel(float* __restrict__ table, int N, const int32_t* __restrict__ ids, int P,
                                       const float* __restrict__ H_next, int32_t* status) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= P) return;
    const int id = ids[k];
    if (id < 0 || id >= N) { set_status(status, DPPO_STATUS_BAD_INDEX); return; }
    table[id] = H_next[k];
}

}  // namespace dppo

extern "C" int dppo_history_gather(const float* H_table, int N, const int32_t* prompt_ids, int P, float* H_batch,
                                   int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_history_gather");
    if (N < 0 || P < 0) return dppo::fail(DPPO_ERR_INVALID_ARG, "history_gather: N=%d P=%d", N, P);
    if (P == 0) return DPPO_OK;
    if (!H_table || !prompt_ids || !H_batch) return dppo::fail(DPPO_ERR_INVALID_ARG, "history_gather: NULL array");
    dppo::history_gather_kernel<<<(P + 255) / 256, 256, 0, (cudaStream_t)stream>>>(H_table, N, prompt_ids, P, H_batch, status);
    DPPO_CHECK_LAUNCH("history_gather launch");
    return DPPO_OK;
}

extern "C" int dppo_history_scatter(float* H_table, int N, const int32_t* prompt_ids, int P, const float* H_next,
                                    int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_history_scatter");
    if (N < 0 || P < 0) return dppo::fail(DPPO_ERR_INVALID_ARG, "history_scatter: N=%d P=%d", N, P);
    if (P == 0) return DPPO_OK;
    if (!H_table || !prompt_ids || !H_next) return dppo::fail(DPPO_ERR_INVALID_ARG, "history_scatter: NULL array");
    dppo::history_scatter_kernel<<<(P + 255) / 256, 256, 0, (cudaStream_t)stream>>>(H_table, N, prompt_ids, P, H_next, status);
    DPPO_CHECK_LAUNCH("history_scatter launch");
    return DPPO_OK;
}

extern "C" int dppo_prune_and_rescale(const dppo_prune_params* p, const float* adv,
                                      const float* mean_abs_adv, const float* H_prev,
                                      const double* u_q, const double* u_o, uint8_t* cand_q,
                                      uint8_t* cand_o, uint8_t* keep_q, uint8_t* keep_o,
                                      int32_t* n_keep_q, int32_t* n_keep_o, float* gamma_q,
                                      float* gamma_o, float* w_seq, float* H_next, int32_t* status,
                                      void* stream) {
    dppo::NvtxRange nvtx_range("dppo_prune_and_rescale");
    (void)status;
    if (!p) return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: NULL params");
    if (p->P < 0 || p->G < 1) return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: P=%d G=%d", p->P, p->G);
    if ((int64_t)p->P * p->G >= (int64_t)1 << 31)
        return dppo::fail(DPPO_ERR_BAD_SHAPE, "prune_and_rescale: P*G must be below 2^31");
    if (!(p->r_q >= 0.0 && p->r_q < 1.0) || !(p->r_o >= 0.0 && p->r_o < 1.0))
        return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: r_q, r_o must lie in [0,1)");
    if (p->mode != 0 && p->mode != 1) return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: mode %d", p->mode);
    if (p->reverse != 0 && p->reverse != 1)
        return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: reverse %d", p->reverse);
    if (!n_keep_q) return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: NULL n_keep_q");
    if (p->P > 0 && (!adv || !mean_abs_adv || !cand_q || !cand_o || !keep_q || !keep_o || !n_keep_o ||
                     !gamma_q || !gamma_o || !w_seq || !H_next))
        return dppo::fail(DPPO_ERR_INVALID_ARG, "prune_and_rescale: NULL array");
    dppo::prune_and_rescale_kernel<<<1, dppo::kPruneThreads, 0, (cudaStream_t)stream>>>(
        *p, adv, mean_abs_adv, H_prev, u_q, u_o, cand_q, cand_o, keep_q, keep_o, n_keep_q, n_keep_o,
        gamma_q, gamma_o, w_seq, H_next);
    DPPO_CHECK_LAUNCH("prune_and_rescale launch");
    return DPPO_OK;
}
