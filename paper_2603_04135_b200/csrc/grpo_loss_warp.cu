// Loss sweep for short rows (up to 8 KB): one WARP per row, the row held in registers.
//
// With one CTA per row a short row costs more to launch than to process (the grid's launch rate, about 250 CTAs
// per microsecond, caps 2 KB rows at 1 TB/s).  Here persistent warps walk over the rows: a lane loads up to
// kVPL 16-byte vectors of the row straight into registers (coalesced, 512 bytes per warp instruction), the row
// maximum and the sum of exponentials are warp reductions, lane 0 runs the scalar stage, and the stored
// exponentials are scaled into dlogits from the same registers.  HBM sees one read and one write per element
// and nothing goes through shared memory.  The arithmetic per element is the shared-memory kernel's: packed bf16
// maximum, 2^(z c - r) once, kept as fp16 pairs (bf16 rows) or f32 (f32 rows), then a scale.
#include <cuda_fp16.h>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {
using namespace packed;
namespace warprow {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// Word `wy` of vector `jy` of a lane's row registers.  Both indices are the same in every lane (they follow from the
// sampled token's id), so a branch on them does not diverge and costs a few instructions, where selects over all
// the vectors (which keep the array in registers just the same) cost four per vector.
template <int kVPL>
__device__ __forceinline__ uint32_t pick_word(const uint4 (&d)[kVPL], int jy, int wy) {
    uint4 q = d[0];
    switch (jy) {
#define DPPO_PICK(J) case J: if (J < kVPL) q = d[J < kVPL ? J : 0]; break;
        DPPO_PICK(1) DPPO_PICK(2) DPPO_PICK(3) DPPO_PICK(4) DPPO_PICK(5) DPPO_PICK(6) DPPO_PICK(7) DPPO_PICK(8)
        DPPO_PICK(9) DPPO_PICK(10) DPPO_PICK(11) DPPO_PICK(12) DPPO_PICK(13) DPPO_PICK(14) DPPO_PICK(15)
#undef DPPO_PICK
        default: break;
    }
    switch (wy) {
        case 0: return q.x;
        case 1: return q.y;
        case 2: return q.z;
        default: return q.w;
    }
}

// The binary64 scalar stage as a call of its own: its registers are then not the whole kernel's, which is what
// lets more warps (rows in flight) share an SM.
__device__ __noinline__ RowScalars finish_row(const LossArgs& a, long long t, const RowInputs& in, float ref2, float sum2) {
    return row_finish(a, t, in, ref2, sum2, true);
}

}  // namespace warprow

using namespace warprow;

// Resident CTAs per SM the register allocation aims at: more rows in flight for the short forms.
template <bool kF32, int kVPL> constexpr int min_ctas() { return kVPL <= 4 ? 4 : kVPL == 8 ? 3 : kF32 ? 2 : 1; }

template <bool kF32, int kVPL>
__global__ void __launch_bounds__(kThreads, min_ctas<kF32, kVPL>())
grpo_loss_warp_kernel(const LossArgs a) {
    constexpr int kLog2PerVec = kF32 ? 2 : 3;               // elements per 16-byte vector: 4 f32 or 8 bf16
    constexpr uint32_t kPad = kF32 ? 0xFF800000u : 0xFF80FF80u;   // -inf: adds nothing to the maximum or the sum
    const int lane = threadIdx.x & 31;
    const int warp0 = (int)blockIdx.x * kWarps + (int)(threadIdx.x >> 5);      // the row count is below 2^31: 32-bit indices
    const int n_warps = (int)gridDim.x * kWarps;
    const int T = (int)(a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max);
    const int nvec = a.V >> kLog2PerVec;
    const int tail0 = nvec << kLog2PerVec;                  // the ragged tail: one element per lane
    const bool has_tail = tail0 + lane < a.V;
    const float c = a.scale2;

    // Every warp takes the rows in short runs of consecutive rows (up to kRun = 16), the runs dealt out round-robin over
    // the warps.  Consecutive tokens mostly belong to the same sequence, so the sequence's scalars (bounds, advantage,
    // weight) stay cached from row to row and the search of cu_seqlens runs about once per run; the sampled token's
    // logit is taken out of the registers that hold the row.  What is left on a row's dependent chain is one round
    // trip: its vectors and its three per-token scalars, all issued together.  Round-robin runs keep the rows that
    // all warps work on at any moment in one region of memory.  (Prefetching the next row into L2 was measured: no
    // gain on long inputs, 10 % slower on inputs of a few rows per warp.)
    constexpr int kRun = 16;
    // the run length (at most kRun) for which the busiest warp gets the fewest rows; ties go to the longer run
    int run = 1;
    {
        // long inputs (64 rows per warp and more) take runs of up to 16, shorter ones single rows: measured on 1-8 KB
        // rows, runs gain up to 14 % on millions of rows and lose up to 9 % on a hundred thousand
        const unsigned longest = (unsigned)T / (unsigned)n_warps >= 64u ? (unsigned)kRun : 1u;
        unsigned best = 0xffffffffu;                        // 32-bit arithmetic: T < 2^31, and 64-bit divisions are slow
        for (unsigned cand = longest; cand >= 1; --cand) {
            const unsigned runs = ((unsigned)T + cand - 1) / cand;
            const unsigned busiest = (runs + (unsigned)n_warps - 1) / (unsigned)n_warps * cand;
            if (busiest < best) { best = busiest; run = (int)cand; }
        }
    }
    int seg_lo = 0, seg_hi = 0;                             // empty: the first row looks its sequence up
    __shared__ double seg_scalars[kWarps][3];               // the cached sequence's advantage, weight, log-ratio: read
    double* seg = seg_scalars[threadIdx.x >> 5];            // once per row, so they need not occupy registers
    bool seg_ok = false;

    long long blk = warp0;
    int k = 0;
    for (int t = (int)min((long long)T, blk * run); t < T;) {
        // the row after this one
        int t_next;
        if (k + 1 < run) { t_next = t + 1; ++k; } else { blk += n_warps; k = 0; t_next = (int)min((long long)T, blk * run); }
        const char* row = a.logits + (long long)t * a.row_bytes;
        const uint4* rowv = reinterpret_cast<const uint4*>(row);
        uint4 d[kVPL];
#pragma unroll
        for (int j = 0; j < kVPL; ++j) {
            const int i = lane + 32 * j;
            d[j] = i < nvec ? __ldcs(rowv + i) : make_uint4(kPad, kPad, kPad, kPad);
        }
        const float ztail = has_tail ? Elems<!kF32>::load1(row, tail0 + lane) : -INFINITY;
        const int y_in = a.target[t];                       // the same address in every lane: one broadcast load each
        const float lp_old = a.logp_old[t], lp_ref = a.logp_ref[t];
        if (t < seg_lo || t >= seg_hi) {                    // the row is outside the cached sequence: look it up
            seg_ok = false;
            if (a.S_max >= 1) {
                int lo = 0, hi = a.S_max;
                while (hi - lo > 1) {                       // 32 probes per round trip; cu_seqlens is non-decreasing
                    const int step = (hi - lo + 31) >> 5;
                    const long long idx = (long long)lo + (long long)(lane + 1) * step;
                    const bool le = idx < hi && (long long)a.cu_seqlens[idx] <= t;
                    const int n = __popc(__ballot_sync(0xffffffffu, le));
                    lo += n * step;
                    hi = min(hi, lo + step);
                }
                seg_lo = a.cu_seqlens[lo]; seg_hi = a.cu_seqlens[lo + 1];
                if (t >= seg_lo && t < seg_hi) {
                    seg_ok = true;
                    const int idx = a.seg_map ? a.seg_map[lo] : lo;
                    if (lane == 0) {
                        seg[0] = (double)a.adv[idx];
                        seg[1] = a.no_length_norm ? (double)a.w[idx] : (double)a.w[idx] / (double)(seg_hi - seg_lo);
                        seg[2] = a.seq_log_ratio ? (double)a.seq_log_ratio[lo] : 0.0;
                    }
                    __syncwarp();
                } else {
                    seg_lo = seg_hi = 0;                    // no sequence covers this row: the next row searches again
                }
            }
        }
        // the sampled token's logit out of the registers: the lane and vector that hold element y_in
        float zy_f = 0.0f;
        const bool y_ok = y_in >= 0 && y_in < a.V;
        if (y_ok) {
            if (y_in >= tail0) {
                zy_f = __shfl_sync(0xffffffffu, ztail, y_in - tail0);
            } else {
                const int yv = y_in >> kLog2PerVec, jy = yv >> 5;
                const int wy = kF32 ? (y_in & 3) : ((y_in & 7) >> 1);
                uint32_t word = pick_word<kVPL>(d, jy, wy);
                word = __shfl_sync(0xffffffffu, word, yv & 31);
                zy_f = kF32 ? __uint_as_float(word) : __uint_as_float((y_in & 1) ? (word & 0xffff0000u) : (word << 16));
            }
        }
        RowInputs in;
        in.A = in.W = in.zy = in.logp_old = in.logp_ref = in.seq_lr = 0.0;
        in.use_seq = 0; in.y = y_in; in.state = 0;
        if (!seg_ok) in.state = DPPO_STATUS_BAD_SEGMENTS;
        else if (!y_ok) in.state = DPPO_STATUS_BAD_TARGET;
        else {
            in.A = seg[0]; in.W = seg[1];
            if (a.seq_log_ratio) { in.use_seq = 1; in.seq_lr = seg[2]; }
            in.zy = (double)zy_f / a.temperature;
            in.logp_old = (double)lp_old; in.logp_ref = (double)lp_ref;
        }

        // ---- row maximum
        float m = ztail;
        if constexpr (kF32) {
#pragma unroll
            for (int j = 0; j < kVPL; ++j)
                m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(d[j].x), __uint_as_float(d[j].y)),
                                   fmaxf(__uint_as_float(d[j].z), __uint_as_float(d[j].w))));
        } else {
            __nv_bfloat162 mx2 = __float2bfloat162_rn(-INFINITY);
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[j].x));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[j].y));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[j].z));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[j].w));
            }
            m = fmaxf(m, fmaxf(__low2float(mx2), __high2float(mx2)));
        }
        m = warp_max(m);
        const float r = m * c;                              // -inf only if the whole row is -inf
        const float nr = r > -INFINITY ? -r : 0.0f;

        // ---- exponentials 2^(z c - r) in place, and their sum (packed f32 pairs: one instruction for two elements)
        const f32x2 c2 = pair_of(c, c), nr2 = pair_of(nr, nr);
        f32x2 acc0 = pair_of(0.0f, 0.0f), acc1 = acc0;
#pragma unroll
        for (int j = 0; j < kVPL; ++j) {
            if constexpr (kF32) {
                d[j] = exp_quad(d[j], c2, nr2, acc0, acc1);
            } else {
                d[j].x = exp_pair(d[j].x, c2, nr2, acc0); d[j].y = exp_pair(d[j].y, c2, nr2, acc1);
                d[j].z = exp_pair(d[j].z, c2, nr2, acc0); d[j].w = exp_pair(d[j].w, c2, nr2, acc1);
            }
        }
        float s0, s1;
        unpair(add2(acc0, acc1), s0, s1);
        const float etail = ztail > -INFINITY ? ex2(fmaf(ztail, c, nr)) : 0.0f;
        const float s = warp_sum(s0 + s1 + etail);

        // ---- scalar stage (lane 0), broadcast of what the stores need
        RowScalars rs;
        rs.lse2_hi = 0.0f; rs.lse2_lo = 0.0f; rs.g_over_tau = 0.0f; rs.valid = false;
        int y = -1;
        if (lane == 0) {
            rs = finish_row(a, t, in, r, s);
            y = rs.valid ? in.y : -1;
        }
        const float lse2_hi = __shfl_sync(0xffffffffu, rs.lse2_hi, 0), lse2_lo = __shfl_sync(0xffffffffu, rs.lse2_lo, 0);
        const float ng = -__shfl_sync(0xffffffffu, rs.valid ? rs.g_over_tau : 0.0f, 0);
        y = __shfl_sync(0xffffffffu, y, 0);

        // ---- dlogits = g/tau (onehot - 2^(z c - lse2)) from the registers
        if (a.dlogits) {
            char* drow = a.dlogits + (long long)t * a.row_bytes;
            uint4* dst = reinterpret_cast<uint4*>(drow);
            const float sc = ng * ex2((r - lse2_hi) - lse2_lo);
            const f32x2 sc2 = pair_of(sc, sc);
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                const int i = lane + 32 * j;
                if (i < nvec) {
                    uint4 o;
                    if constexpr (kF32) {
                        o = scale_quad(d[j], sc2);
                    } else {
                        o.x = scale_pair(d[j].x, sc2); o.y = scale_pair(d[j].y, sc2);
                        o.z = scale_pair(d[j].z, sc2); o.w = scale_pair(d[j].w, sc2);
                    }
                    __stcs(dst + i, o);
                }
            }
            // the one element that also carries the onehot term: the lane that stored its vector redoes it
            const int yvec = y >= 0 ? (y >> kLog2PerVec) : -1;
            if (yvec >= 0 && yvec < nvec && (yvec & 31) == lane) {
                const int jy = yvec >> 5;
                const int wy = kF32 ? (y & 3) : ((y & 7) >> 1);
                uint32_t word = pick_word<kVPL>(d, jy, wy);
                if constexpr (kF32) {
                    reinterpret_cast<float*>(drow)[y] = fmaf(__uint_as_float(word), sc, -ng);
                } else {
                    const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&word));
                    reinterpret_cast<__nv_bfloat16*>(drow)[y] = __float2bfloat16_rn(fmaf((y & 1) ? e.y : e.x, sc, -ng));
                }
            }
            if (has_tail) {
                const int v = tail0 + lane;
                Elems<!kF32>::store1(drow, v, sc * etail - (v == y ? ng : 0.0f));
            }
        }
        t = t_next;
    }
}

// ---- host side ---------------------------------------------------------------------------------------
template <bool kF32, int kVPL>
static int launch_warp_t(const LossArgs& a, cudaStream_t s, bool launch) {
    auto kernel = grpo_loss_warp_kernel<kF32, kVPL>;
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0);
    if (e != cudaSuccess || per_sm < 1) { cudaGetLastError(); return fail(DPPO_ERR_UNSUPPORTED, "warp-per-row kernel does not fit this device"); }
    if (!launch) return DPPO_OK;
    const long long want = (a.T_max + kWarps - 1) / kWarps;
    const long long cap = (long long)sm_count() * per_sm;
    kernel<<<(unsigned)(want < cap ? want : cap), kThreads, 0, s>>>(a);
    DPPO_CHECK_LAUNCH("grpo_loss warp-per-row launch");
    return DPPO_OK;
}

template <bool kF32>
static int launch_warp_dtype(const LossArgs& a, int vpl, cudaStream_t s, bool launch) {
    if (vpl <= 2) return launch_warp_t<kF32, 2>(a, s, launch);
    if (vpl <= 4) return launch_warp_t<kF32, 4>(a, s, launch);
    if (vpl <= 8) return launch_warp_t<kF32, 8>(a, s, launch);
    return launch_warp_t<kF32, 16>(a, s, launch);
}

// Rows of up to 512 vectors (8 KB).  DPPO_ERR_UNSUPPORTED (nothing launched) for longer rows.
int launch_rows_warp(const LossArgs& a, cudaStream_t s, bool launch) {
    const int nvec = a.V >> (a.bf16 ? 3 : 2);
    if (nvec > 32 * 16) return fail(DPPO_ERR_UNSUPPORTED, "warp-per-row kernel: rows of %d vectors exceed %d", nvec, 32 * 16);
    const int vpl = (nvec + 31) / 32;
    return a.bf16 ? launch_warp_dtype<false>(a, vpl, s, launch) : launch_warp_dtype<true>(a, vpl, s, launch);
}

}  // namespace dppo
