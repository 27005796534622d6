// Internal types shared by the loss-sweep kernels (not part of the ABI).
#pragma once
#include "common.cuh"

namespace dppo {

struct RowTerms {            // one per token row, in the caller's workspace
    double loss;             // -W (surr - beta kl)
    double pg;               // -W surr
    double kl;               //  W kl
    double clipped;          // 1 if the clipped branch was strictly smaller
};

struct RowScalars {          // what pass 2 needs from the scalar stage
    float lse2_hi, lse2_lo;  // base-2 log-sum-exp of z*scale2, split hi + lo
    float g_over_tau;        // dloss/dlogp / temperature
    bool valid;              // false: bad target / segment -> the row's dlogits are zero
};

struct LossArgs {
    const char* logits;
    char* dlogits;
    const int32_t* target;
    const float* logp_old;
    const float* logp_ref;
    const int32_t* cu_seqlens;
    const int32_t* n_tokens_dev;
    const float* adv;
    const float* w;
    const int32_t* seg_map;
    float* logp_out;
    float* lse_out;
    RowTerms* terms;
    int32_t* status;
    long long T_max;
    long long row_bytes;
    int V, S_max, bf16;
    double eps_lo, eps_hi, beta, temperature;
    float scale2;            // log2(e) / temperature as the f32 both passes multiply by
};

__device__ RowScalars row_scalar_stage(const LossArgs& a, long long t, float ref2, float sum2);

int launch_rows_general(const LossArgs& a, cudaStream_t s);
int launch_loss_reduce(const LossArgs& a, float* loss_out, cudaStream_t s);

}  // namespace dppo
