// Internal types shared by the loss-sweep kernels (not part of the ABI).
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace dppo {

struct RowTerms {            // one per token row, in the caller's workspace
    double loss;             // -W (surr - beta kl)
    double pg;               // -W surr
    double kl;               //  W kl
    double clipped;          // 1 if the clipped branch was strictly smaller
};

// The per-row terms are followed, in the same workspace, by the partial sums of the final reduction.
constexpr int kReduceBlocks = 128;
inline size_t loss_rows_bytes(long long T_max) {
    const size_t rows = (size_t)(T_max > 0 ? T_max : 1);
    return (rows * sizeof(RowTerms) + 255) & ~(size_t)255;
}
inline size_t loss_terms_bytes(long long T_max) { return loss_rows_bytes(T_max) + kReduceBlocks * sizeof(RowTerms); }
inline RowTerms* loss_partials(RowTerms* terms, long long T_max) {
    return (RowTerms*)((char*)terms + loss_rows_bytes(T_max));
}

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
    const float* seq_log_ratio;   // nullable: sequence-level ratio, indexed by sequence position
    int no_length_norm;
    float scale2;            // log2(e) / temperature as the f32 both passes multiply by
    unsigned long long wait_limit_ns;   // bound of every device-side wait (on %globaltimer)
    int test_extra_tx;       // 0; the self-test of the bounded waits announces this many bytes that never arrive
};

constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // give up on a copy or a peer after 2 s
constexpr unsigned long long kSelfTestWaitLimitNs = 1000000ull;     // the self-test's waits run out after 1 ms

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

// ---- per-element arithmetic of the two row kernels that keep the exponentials (shared-memory and warp-per-row) ----
namespace packed {

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
// Packed f32 pairs (one instruction works on both halves of a 64-bit register pair).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pair_of(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpair(f32x2 p, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// Two fp16 exponentials -> two bf16 gradient entries e * sc (sc2 = the scale in both halves).
__device__ __forceinline__ uint32_t scale_pair(uint32_t h2, f32x2 sc2) {
    const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&h2));
    float lo, hi;
    unpair(mul2(pair_of(e.x, e.y), sc2), lo, hi);
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&b);
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// One 32-bit word = two bf16 logits -> their exponentials 2^(z c - r) as an fp16 pair; acc += the two (f32).
__device__ __forceinline__ uint32_t exp_pair(uint32_t w, f32x2 c2, f32x2 nr2, f32x2& acc) {
    float a, b;
    unpair(fma2(pair_of(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)), c2, nr2), a, b);
    const float ea = ex2(a), eb = ex2(b);
    acc = add2(acc, pair_of(ea, eb));
    return pack_half2(ea, eb);
}

// The same without keeping the exponentials (a forward-only call has no second pass).
__device__ __forceinline__ void exp_pair_sum(uint32_t w, f32x2 c2, f32x2 nr2, f32x2& acc) {
    float a, b;
    unpair(fma2(pair_of(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)), c2, nr2), a, b);
    acc = add2(acc, pair_of(ex2(a), ex2(b)));
}

// f32 rows: one 16-byte vector = four logits -> their exponentials 2^(z c - r), in place; acc += the four.
__device__ __forceinline__ uint4 exp_quad(uint4 q, f32x2 c2, f32x2 nr2, f32x2& acc0, f32x2& acc1) {
    float a, b, e0, e1;
    unpair(fma2(pair_of(__uint_as_float(q.x), __uint_as_float(q.y)), c2, nr2), a, b);
    e0 = ex2(a); e1 = ex2(b);
    acc0 = add2(acc0, pair_of(e0, e1));
    q.x = __float_as_uint(e0); q.y = __float_as_uint(e1);
    unpair(fma2(pair_of(__uint_as_float(q.z), __uint_as_float(q.w)), c2, nr2), a, b);
    e0 = ex2(a); e1 = ex2(b);
    acc1 = add2(acc1, pair_of(e0, e1));
    q.z = __float_as_uint(e0); q.w = __float_as_uint(e1);
    return q;
}
__device__ __forceinline__ uint4 scale_quad(uint4 q, f32x2 sc2) {
    float a, b;
    unpair(mul2(pair_of(__uint_as_float(q.x), __uint_as_float(q.y)), sc2), a, b);
    q.x = __float_as_uint(a); q.y = __float_as_uint(b);
    unpair(mul2(pair_of(__uint_as_float(q.z), __uint_as_float(q.w)), sc2), a, b);
    q.z = __float_as_uint(a); q.w = __float_as_uint(b);
    return q;
}

}  // namespace packed

// ---- scalar stage -------------------------------------------------------------------------------------
// What one token row needs besides its logits; gathered once per row (one thread, or one warp ahead of
// time while the row is still in flight).
struct RowInputs {
    double A;                // advantage of the token's sequence
    double W;                // w[seq] / |o_seq|
    double zy;               // z[y] / temperature
    double logp_old, logp_ref;
    double seq_lr;           // log of the sequence-level ratio (used when use_seq)
    int use_seq;
    int y;
    int state;               // 0 ok, else the dppo_status to report (row adds nothing, dlogits zero)
};

// load_zy = false: the caller supplies z[y] itself (the fused LM-head has no logits in memory).
__device__ __forceinline__ void row_inputs_from_segment(const LossArgs& a, long long t, int seg, RowInputs& in,
                                                        bool load_zy = true) {
    in.A = in.W = in.zy = in.logp_old = in.logp_ref = in.seq_lr = 0.0;
    in.use_seq = 0;
    in.y = a.target[t];
    in.state = 0;
    const long long seg_lo = a.cu_seqlens[seg], seg_hi = a.cu_seqlens[seg + 1];
    if (a.S_max < 1 || t < seg_lo || t >= seg_hi) { in.state = DPPO_STATUS_BAD_SEGMENTS; return; }
    if (in.y < 0 || in.y >= a.V) { in.state = DPPO_STATUS_BAD_TARGET; return; }
    const int idx = a.seg_map ? a.seg_map[seg] : seg;
    in.A = (double)a.adv[idx];
    in.W = a.no_length_norm ? (double)a.w[idx] : (double)a.w[idx] / (double)(seg_hi - seg_lo);
    if (a.seq_log_ratio) { in.use_seq = 1; in.seq_lr = (double)a.seq_log_ratio[seg]; }
    if (load_zy)
        in.zy = (double)(a.bf16 ? Elems<true>::load1(a.logits + t * a.row_bytes, in.y)
                                : Elems<false>::load1(a.logits + t * a.row_bytes, in.y)) / a.temperature;
    in.logp_old = (double)a.logp_old[t];
    in.logp_ref = (double)a.logp_ref[t];
}

// One thread: binary search for the last s with cu_seqlens[s] <= t, then the gather.
__device__ __forceinline__ void row_gather(const LossArgs& a, long long t, RowInputs& in, bool load_zy = true) {
    int lo = 0, hi = a.S_max;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)a.cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    row_inputs_from_segment(a, t, lo, in, load_zy);
}

// One warp: the same search 32 probes at a time (one memory round trip per factor of 32); lane 0
// gathers.  `in` is written by lane 0 only.
__device__ __forceinline__ void row_gather_warp(const LossArgs& a, long long t, int lane, RowInputs& in) {
    int lo = 0, hi = a.S_max;
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) >> 5;                        // probes at lo + step, lo + 2 step, ...
        const long long idx = (long long)lo + (long long)(lane + 1) * step;
        const bool le = idx < hi && (long long)a.cu_seqlens[idx] <= t;
        const int n = __popc(__ballot_sync(0xffffffffu, le));        // cu_seqlens is non-decreasing: a prefix of lanes
        lo += n * step;
        hi = min(hi, lo + step);
    }
    if (lane == 0) row_inputs_from_segment(a, t, lo, in);
}

// ref2/sum2: the row's sum of 2^(z c) is sum2 * 2^ref2 with c = log2(e)/temperature as used in pass 1.
// write: only one CTA of a cluster that shares a row stores the row's outputs.
__device__ __forceinline__ RowScalars row_finish(const LossArgs& a, long long t, const RowInputs& in, float ref2,
                                                 float sum2, bool write = true) {
    RowScalars out;
    const double lse2 = (double)ref2 + log2((double)sum2);           // base-2 log-sum-exp of z c
    const double lse = lse2 * 0.6931471805599453;                    // natural log-sum-exp of z / temperature
    out.lse2_hi = (float)lse2;
    out.lse2_lo = (float)(lse2 - (double)out.lse2_hi);
    out.g_over_tau = 0.0f;
    out.valid = false;
    RowTerms terms = {0.0, 0.0, 0.0, 0.0};
    float logp_f = 0.0f;
    if (in.state != 0) {
        if (write) set_status(a.status, in.state);
    } else {
        const double A = in.A, W = in.W;
        const double logp = in.zy - lse;
        const double rho = in.use_seq ? exp(in.seq_lr) : exp(logp - in.logp_old);
        const double d = in.logp_ref - logp;
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
    if (write) {
        a.terms[t] = terms;
        if (a.logp_out) a.logp_out[t] = logp_f;
        if (a.lse_out) a.lse_out[t] = (float)lse;
    }
    return out;
}

__device__ __forceinline__ RowScalars row_scalar_stage(const LossArgs& a, long long t, float ref2, float sum2) {
    RowInputs in;
    row_gather(a, t, in);
    return row_finish(a, t, in, ref2, sum2, true);
}

int launch_rows_general(const LossArgs& a, cudaStream_t s);
// Cluster kernel: the row is split over `cluster` CTAs that keep their slice in shared memory.
// Returns DPPO_ERR_UNSUPPORTED (nothing launched) when the shape or the device cannot take it.
// launch = false: run the checks only (shape, shared memory, cluster fit) and launch nothing.
int launch_rows_cluster(const LossArgs& a, int cluster, int threads, cudaStream_t s, bool launch = true);
// Short rows (up to 512 16-byte vectors): one warp per row, the row in registers (grpo_loss_warp.cu).
// Returns DPPO_ERR_UNSUPPORTED (nothing launched) for longer rows.
int launch_rows_warp(const LossArgs& a, cudaStream_t s, bool launch = true);
// Forward-only calls: persistent CTAs stream the rows through a shared-memory ring (grpo_loss_stream.cu).
// Returns DPPO_ERR_UNSUPPORTED (nothing launched) when dlogits are asked for.
int launch_rows_stream(const LossArgs& a, cudaStream_t s, bool launch = true);
// Calls with dlogits on dense rows of up to 32 KB: tiles of rows through a shared-memory ring, the scalar stage of
// up to 32 rows in one pass (grpo_loss_tile.cu).  Returns DPPO_ERR_UNSUPPORTED (nothing launched) for other calls.
int launch_rows_tile(const LossArgs& a, cudaStream_t s, bool launch = true);
int launch_loss_reduce(const LossArgs& a, float* loss_out, cudaStream_t s);

}  // namespace dppo
