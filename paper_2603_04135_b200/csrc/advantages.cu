// Group-relative advantages (Eq. 2) and the mean-|A| threshold (Eq. 14).
//
// One thread per prompt.  Every operation is an explicitly rounded binary64 intrinsic so the
// compiler can neither fuse nor reorder it: the f32 results are reproducible bit for bit, which the
// candidate test downstream (an exact tie in common cases) relies on.
#include "common.cuh"

namespace dppo {

__global__ void group_advantages_kernel(const float* __restrict__ rewards, int P, int G, int ddof,
                                        double std_eps, float* __restrict__ adv,
                                        float* __restrict__ mean_abs_adv) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= P) return;
    const float* r = rewards + (size_t)k * G;
    float* a = adv + (size_t)k * G;

    const float first = r[0];
    bool all_equal = true;
    for (int i = 1; i < G; ++i) all_equal = all_equal && (r[i] == first);
    if (all_equal || G - ddof <= 0) {
        for (int i = 0; i < G; ++i) a[i] = 0.0f;
        mean_abs_adv[k] = 0.0f;
        return;
    }
    double s = 0.0;
    for (int i = 0; i < G; ++i) s = __dadd_rn(s, (double)r[i]);
    const double mu = __ddiv_rn(s, (double)G);
    double ss = 0.0;
    for (int i = 0; i < G; ++i) {
        const double d = __dsub_rn((double)r[i], mu);
        ss = __dadd_rn(ss, __dmul_rn(d, d));
    }
    const double sigma = __dsqrt_rn(__ddiv_rn(ss, (double)(G - ddof)));
    const double denom = __dadd_rn(sigma, std_eps);
    double sum_abs = 0.0;
    for (int i = 0; i < G; ++i) {
        const double ai = __ddiv_rn(__dsub_rn((double)r[i], mu), denom);
        sum_abs = __dadd_rn(sum_abs, fabs(ai));
        a[i] = __double2float_rn(ai);
    }
    mean_abs_adv[k] = __double2float_rn(__ddiv_rn(sum_abs, (double)G));
}

}  // namespace dppo

extern "C" int dppo_group_advantages(const float* rewards, int P, int G, int std_ddof, double std_eps,
                                     float* adv, float* mean_abs_adv, int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_group_advantages");
    (void)status;
    if (P < 0 || G < 1) return dppo::fail(DPPO_ERR_INVALID_ARG, "group_advantages: P=%d G=%d", P, G);
    if (std_ddof != 0 && std_ddof != 1)
        return dppo::fail(DPPO_ERR_INVALID_ARG, "group_advantages: std_ddof must be 0 or 1");
    if (!(std_eps >= 0.0)) return dppo::fail(DPPO_ERR_INVALID_ARG, "group_advantages: std_eps < 0");
    if (P == 0) return DPPO_OK;
    if (!rewards || !adv || !mean_abs_adv)
        return dppo::fail(DPPO_ERR_INVALID_ARG, "group_advantages: NULL array");
    const int threads = 128;
    dppo::group_advantages_kernel<<<(P + threads - 1) / threads, threads, 0, (cudaStream_t)stream>>>(
        rewards, P, G, std_ddof, std_eps, adv, mean_abs_adv);
    DPPO_CHECK_LAUNCH("group_advantages launch");
    return DPPO_OK;
}
