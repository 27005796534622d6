// Loss sweep for short rows (up to 8 KB): one WARP per row, the row held in registers, several rows per warp at a time.
//
// With one CTA per row a short row costs more to launch than to process (the grid's launch rate, about 250 CTAs
// per microsecond, caps 2 KB rows at 1 TB/s).  Here persistent warps walk over the rows: a lane loads up to
// kVPL 16-byte vectors of a row straight into registers (coalesced, 512 bytes per warp instruction), the row
// maximum and the sum of exponentials are warp reductions, and the stored exponentials are scaled into dlogits
// from the same registers.  HBM sees one read and one write per element and nothing goes through shared memory.
// The arithmetic per element is the shared-memory kernel's: packed bf16 maximum, 2^(z c - r) once, kept as fp16
// pairs (bf16 rows) or f32 (f32 rows), then a scale.
//
// On rows this short the binary64 scalar stage (a logarithm, two exponentials, the clip logic) is as many
// instructions as everything else a row needs, and a warp instruction costs the same with one lane active as
// with 32.  So a warp takes a GROUP of up to kRows consecutive rows at a time: all their vectors are loaded at
// once (kRows * kVPL loads in flight per lane), the reductions run row by row, and then lane q runs the scalar
// stage of row q: one pass of the scalar stage for the whole group.  The per-token side inputs are lane-indexed
// loads (one instruction for the group), and so are the group's stores of the per-row outputs.
#include <cuda_fp16.h>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {
using namespace packed;
namespace warprow {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// Rows a warp holds at a time: 64 data registers per lane in every form.
__host__ __device__ constexpr int rows_per_group(int vpl) { return vpl <= 2 ? 8 : vpl <= 4 ? 4 : vpl <= 8 ? 2 : 1; }

// The binary64 scalar stage as a call of its own: its registers are then not the whole kernel's, which is what
// lets more warps (rows in flight) share an SM.
__device__ __noinline__ RowScalars finish_row(const LossArgs& a, long long t, const RowInputs& in, float ref2, float sum2) {
    return row_finish(a, t, in, ref2, sum2, true);
}

}  // namespace warprow

using namespace warprow;

// Resident CTAs per SM the register allocation aims at.
template <bool kF32, int kVPL> constexpr int min_ctas() { return kVPL <= 8 ? 2 : kF32 ? 2 : 1; }

template <bool kF32, int kVPL>
__global__ void __launch_bounds__(kThreads, min_ctas<kF32, kVPL>())
grpo_loss_warp_kernel(const LossArgs a) {
    constexpr int kRows = rows_per_group(kVPL);
    constexpr int kLog2PerVec = kF32 ? 2 : 3;               // elements per 16-byte vector: 4 f32 or 8 bf16
    constexpr uint32_t kPad = kF32 ? 0xFF800000u : 0xFF80FF80u;   // -inf: adds nothing to the maximum or the sum
    const int lane = threadIdx.x & 31;
    const int warp0 = (int)blockIdx.x * kWarps + (int)(threadIdx.x >> 5);      // the row count is below 2^31: 32-bit indices
    const int n_warps = (int)gridDim.x * kWarps;
    const int T = (int)(a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max);
    const int nvec = a.V >> kLog2PerVec;
    const int tail0 = nvec << kLog2PerVec;                  // the ragged tail: one element per lane
    const bool any_tail = tail0 < a.V, has_tail = tail0 + lane < a.V;
    const float c = a.scale2;

    // The groups (runs of `run` <= kRows consecutive rows) are dealt out round-robin over the warps, which keeps the
    // rows that all warps work on at any moment in one region of memory.  The group length is the one for which the
    // busiest warp has the least to do, a group counted as its rows plus kFixed rows for its pass of the scalar
    // stage: long inputs get full groups, an input of a few rows per warp is spread over more warps instead.
    int run = 1;
    if constexpr (kRows > 1) {
        constexpr unsigned kFixed = kVPL <= 2 ? 2u : 1u;
        unsigned best = 0xffffffffu;                        // 32-bit arithmetic: T < 2^31, and 64-bit divisions are slow
        for (unsigned cand = (unsigned)kRows; cand >= 1; --cand) {
            const unsigned groups = ((unsigned)T + cand - 1) / cand;
            const unsigned busiest = (groups + (unsigned)n_warps - 1) / (unsigned)n_warps * (cand + kFixed);
            if (busiest < best) { best = busiest; run = (int)cand; }
        }
    }
    // Consecutive tokens mostly belong to the same sequence, so the sequence's scalars (bounds, advantage, weight)
    // stay cached from group to group and the search of cu_seqlens runs about once per sequence.
    int seg_lo = 0, seg_hi = 0;                             // empty: the first row looks its sequence up
    __shared__ double seg_scalars[kWarps][3];               // the cached sequence's advantage, weight, log-ratio: read
    double* seg = seg_scalars[threadIdx.x >> 5];            // once per group, so they need not occupy registers
    bool seg_ok = false;
    // Row t's sequence into the cache (all lanes; cu_seqlens is non-decreasing, 32 probes per round trip).
    auto look_up = [&](int t) {
        seg_ok = false;
        seg_lo = seg_hi = 0;
        if (a.S_max < 1) return;
        int lo = 0, hi = a.S_max;
        while (hi - lo > 1) {
            const int step = (hi - lo + 31) >> 5;
            const long long idx = (long long)lo + (long long)(lane + 1) * step;
            const bool le = idx < hi && (long long)a.cu_seqlens[idx] <= t;
            const int n = __popc(__ballot_sync(0xffffffffu, le));
            lo += n * step;
            hi = min(hi, lo + step);
        }
        const int s_lo = a.cu_seqlens[lo], s_hi = a.cu_seqlens[lo + 1];
        if (t < s_lo || t >= s_hi) return;                  // no sequence covers this row: the next row searches again
        seg_lo = s_lo; seg_hi = s_hi; seg_ok = true;
        const int idx = a.seg_map ? a.seg_map[lo] : lo;
        __syncwarp();                                       // the lanes' reads of the previous sequence are done
        if (lane == 0) {
            seg[0] = (double)a.adv[idx];
            seg[1] = a.no_length_norm ? (double)a.w[idx] : (double)a.w[idx] / (double)(s_hi - s_lo);
            seg[2] = a.seq_log_ratio ? (double)a.seq_log_ratio[lo] : 0.0;
        }
        __syncwarp();
    };

    // The per-token inputs of a group (lane q: row q) are loaded one group ahead, so that the sampled token's logit,
    // whose address needs the token id, goes out together with the group's rows: one round trip per group.
    int y_next = -1;
    float lp_old_next = 0.0f, lp_ref_next = 0.0f;
    auto load_side_inputs = [&](long long g) {
        const long long t = g * run + lane;
        y_next = -1; lp_old_next = 0.0f; lp_ref_next = 0.0f;
        if (lane < run && t < T) { y_next = a.target[t]; lp_old_next = a.logp_old[t]; lp_ref_next = a.logp_ref[t]; }
    };
    load_side_inputs(warp0);

    for (long long g = warp0;; g += n_warps) {
        const long long t0l = g * run;
        if (t0l >= T) break;
        const int t0 = (int)t0l;
        const int nrow = min(run, T - t0);                  // rows of this group; row t0 + q belongs to lane q
        const bool mine = lane < nrow;
        const long long t_mine = t0l + lane;

        // ---- everything the group needs from memory, issued together: the sampled tokens' logits (one element of
        //      the row a lane answers for), the rows, and the next group's per-token inputs
        const int y_mine = y_next;
        const float lp_old = lp_old_next, lp_ref = lp_ref_next;
        const bool y_ok = mine && y_mine >= 0 && y_mine < a.V;
        float zy_raw = 0.0f;
        if (y_ok) zy_raw = Elems<!kF32>::load1(a.logits + t_mine * a.row_bytes, y_mine);
        uint4 d[kRows][kVPL];
        float ztail[kRows];
#pragma unroll
        for (int q = 0; q < kRows; ++q) {
            const char* row = a.logits + (t0l + q) * a.row_bytes;
            const uint4* rowv = reinterpret_cast<const uint4*>(row);
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                const int i = lane + 32 * j;
                d[q][j] = (q < nrow && i < nvec) ? __ldcs(rowv + i) : make_uint4(kPad, kPad, kPad, kPad);
            }
            ztail[q] = (has_tail && q < nrow) ? Elems<!kF32>::load1(row, tail0 + lane) : -INFINITY;
        }
        load_side_inputs(g + n_warps);

        // ---- row by row: maximum, exponentials 2^(z c - r) in place (packed f32 pairs: one instruction for two
        //      elements), their sum; lane q keeps row q's reference and sum
        float r_mine = 0.0f, nr_mine = 0.0f, s_mine = 0.0f;
#pragma unroll
        for (int q = 0; q < kRows; ++q) {
            if (q < nrow) {
                float m = ztail[q];
                if constexpr (kF32) {
#pragma unroll
                    for (int j = 0; j < kVPL; ++j)
                        m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(d[q][j].x), __uint_as_float(d[q][j].y)),
                                           fmaxf(__uint_as_float(d[q][j].z), __uint_as_float(d[q][j].w))));
                } else {
                    __nv_bfloat162 mx2 = __float2bfloat162_rn(-INFINITY);
#pragma unroll
                    for (int j = 0; j < kVPL; ++j) {
                        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[q][j].x));
                        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[q][j].y));
                        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[q][j].z));
                        mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[q][j].w));
                    }
                    m = fmaxf(m, fmaxf(__low2float(mx2), __high2float(mx2)));
                }
                m = warp_max(m);
                const float r = m * c;                      // -inf only if the whole row is -inf
                const float nr = r > -INFINITY ? -r : 0.0f;
                const f32x2 c2 = pair_of(c, c), nr2 = pair_of(nr, nr);
                f32x2 acc0 = pair_of(0.0f, 0.0f), acc1 = acc0;
#pragma unroll
                for (int j = 0; j < kVPL; ++j) {
                    if constexpr (kF32) {
                        d[q][j] = exp_quad(d[q][j], c2, nr2, acc0, acc1);
                    } else {
                        d[q][j].x = exp_pair(d[q][j].x, c2, nr2, acc0); d[q][j].y = exp_pair(d[q][j].y, c2, nr2, acc1);
                        d[q][j].z = exp_pair(d[q][j].z, c2, nr2, acc0); d[q][j].w = exp_pair(d[q][j].w, c2, nr2, acc1);
                    }
                }
                float s0, s1;
                unpair(add2(acc0, acc1), s0, s1);
                const float etail = ztail[q] > -INFINITY ? ex2(fmaf(ztail[q], c, nr)) : 0.0f;
                const float s = warp_sum(s0 + s1 + etail);
                if (lane == q) { r_mine = r; nr_mine = nr; s_mine = s; }
            }
        }

        // ---- the group's sequences: the usual case is that all its rows lie in the cached one
        bool seg_ok_mine = false;
        double A_mine = 0.0, W_mine = 0.0, lr_mine = 0.0;
        if (t0 >= seg_lo && t0 + nrow <= seg_hi) {
            if (mine) { seg_ok_mine = true; A_mine = seg[0]; W_mine = seg[1]; lr_mine = seg[2]; }
        } else {
#pragma unroll
            for (int q = 0; q < kRows; ++q) {
                if (q < nrow) {
                    const int t = t0 + q;
                    if (t < seg_lo || t >= seg_hi) look_up(t);
                    if (lane == q && seg_ok) { seg_ok_mine = true; A_mine = seg[0]; W_mine = seg[1]; lr_mine = seg[2]; }
                }
            }
        }

        // ---- scalar stage: lane q for row q, one pass for the group
        float sc_mine = 0.0f, ng_mine = 0.0f;
        bool fix_mine = false;
        if (mine) {
            RowInputs in;
            in.A = in.W = in.zy = in.logp_old = in.logp_ref = in.seq_lr = 0.0;
            in.use_seq = 0; in.y = y_mine; in.state = 0;
            if (!seg_ok_mine) in.state = DPPO_STATUS_BAD_SEGMENTS;
            else if (!y_ok) in.state = DPPO_STATUS_BAD_TARGET;
            else {
                in.A = A_mine; in.W = W_mine;
                if (a.seq_log_ratio) { in.use_seq = 1; in.seq_lr = lr_mine; }
                in.zy = (double)zy_raw / a.temperature;
                in.logp_old = (double)lp_old; in.logp_ref = (double)lp_ref;
            }
            const RowScalars rs = finish_row(a, t_mine, in, r_mine, s_mine);
            if (rs.valid) {
                ng_mine = -rs.g_over_tau;
                sc_mine = ng_mine * ex2((r_mine - rs.lse2_hi) - rs.lse2_lo);
                fix_mine = true;
            }
        }

        // ---- dlogits = g/tau (onehot - 2^(z c - lse2)) from the registers: row q scaled by lane q's factor
        if (a.dlogits) {
#pragma unroll
            for (int q = 0; q < kRows; ++q) {
                if (q < nrow) {
                    char* drow = a.dlogits + (t0l + q) * a.row_bytes;
                    uint4* dst = reinterpret_cast<uint4*>(drow);
                    const float sc = __shfl_sync(0xffffffffu, sc_mine, q);
                    const f32x2 sc2 = pair_of(sc, sc);
#pragma unroll
                    for (int j = 0; j < kVPL; ++j) {
                        const int i = lane + 32 * j;
                        if (i < nvec) {
                            uint4 o;
                            if constexpr (kF32) {
                                o = scale_quad(d[q][j], sc2);
                            } else {
                                o.x = scale_pair(d[q][j].x, sc2); o.y = scale_pair(d[q][j].y, sc2);
                                o.z = scale_pair(d[q][j].z, sc2); o.w = scale_pair(d[q][j].w, sc2);
                            }
                            __stcs(dst + i, o);
                        }
                    }
                    if (any_tail) {
                        const float nr = __shfl_sync(0xffffffffu, nr_mine, q);
                        if (has_tail) Elems<!kF32>::store1(drow, tail0 + lane, ztail[q] > -INFINITY ? sc * ex2(fmaf(ztail[q], c, nr)) : 0.0f);
                    }
                }
            }
            // the one element of a row that also carries the onehot term is stored again, by the lane that ran the
            // row's scalar stage, from the logit it loaded: the same exponential (rounded to fp16 where the
            // vector it sits in was) times the same factor, minus g/tau
            __syncwarp();                                   // after the other lanes' stores to the same row
            if (fix_mine) {
                float e = zy_raw > -INFINITY ? ex2(fmaf(zy_raw, c, nr_mine)) : 0.0f;
                if (!kF32 && y_mine < tail0) e = __half2float(__float2half_rn(e));
                Elems<!kF32>::store1(a.dlogits + t_mine * a.row_bytes, y_mine, fmaf(e, sc_mine, -ng_mine));
            }
        }
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
