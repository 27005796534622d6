// Forward-only loss sweep for long rows: the logits stream through shared memory exactly once and nothing waits for
// a row to be complete.
//
// A call without dlogits needs, per row, only (max, sum of exponentials), the sampled token's logit and the scalar
// stage.  The shared-memory kernel of the forward + backward sweep holds a whole row on chip because the row has to
// be written back scaled; here that is not needed, and holding it costs: a CTA's copy, reduction, exchange and scalar
// stage follow one another and overlap only with other CTAs' phases.  This kernel keeps the memory system busy by
// construction instead.  One persistent CTA per SM walks over rows t = blockIdx.x, + gridDim.x, ...:
//   producer warp   one thread issues bulk copies of consecutive 32 KB pieces of the CTA's rows into a ring of
//                   shared-memory stages (mbarrier complete_tx), running ahead across row boundaries as far as the
//                   ring allows: 192 KB in flight per SM whatever the consumers are doing
//   16 consumer     every thread keeps an ONLINE (maximum, sum of 2^(z c - max c)) pair over the vectors it sees: the
//   warps           maximum of a vector is taken first (packed bf16 max), the running pair is rescaled on the few
//                   occasions the maximum grows, then one exponential per element.  No block-wide step per piece; a
//                   warp releases a stage as soon as its own lanes are done with it.  At the end of a row the pairs are
//                   joined within each warp by shuffles and the 16 warp pairs go to a shared-memory slot
//   finisher warp   gathers the row's side inputs ahead of time, joins the 16 pairs (plus the row's ragged tail, read
//                   with plain loads), runs the binary64 scalar stage and writes the row's outputs, while the
//                   consumers are already in the next row
// HBM traffic is the algorithmic minimum (each row read once).  Every wait is bounded; on a time-out the CTA raises
// an abort flag, reports DPPO_STATUS_TIMEOUT, lets its copies in flight land (bounded) and leaves.
#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {
using namespace packed;

namespace stream {

constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 2) * 32;       // + producer warp + finisher warp
constexpr int kStages = 6;
constexpr int kStageVecs = 2048;                          // 16-byte vectors per stage: 32 KB
constexpr int kStageBytes = kStageVecs * 16;
constexpr size_t kDynSmem = (size_t)kStages * kStageBytes;

struct Shared {
    unsigned long long full[kStages];                     // the stage's bytes have landed
    unsigned long long empty[kStages];                    // all consumer warps are done with the stage
    unsigned long long row_done[2];                       // all consumer warps have stored their pair of a row
    unsigned long long row_free[2];                       // the finisher has read the slot
    float2 pair[2][kConsumerWarps];                       // per row parity: (reference r = max c, sum) of every warp
    int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// One try: the thread is suspended until the phase completes or about a microsecond has passed (a waiting warp
// then issues a handful of instructions per microsecond instead of spinning against the working warps).
constexpr uint32_t kSuspendNs = 1000;
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
    return done != 0;
}
// Bounded wait on phase `parity`; also leaves (false) when another role has raised the abort flag.  The clock and
// the abort flag are looked at once per eight tries.
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns) {
    if (try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 8; ++i)
            if (try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

// (r1, s1) (+) (r2, s2): the sum of 2^x over both parts relative to the larger reference; a part that has seen
// nothing but -inf carries r = -inf, s = 0.
__device__ __forceinline__ void join(float& r, float& s, float r2, float s2) {
    const float R = fmaxf(r, r2);
    const float a = r > -INFINITY ? s * ex2(r - R) : 0.0f;
    const float b = r2 > -INFINITY ? s2 * ex2(r2 - R) : 0.0f;
    r = R; s = a + b;
}

}  // namespace stream

using namespace stream;

template <bool kF32>
__global__ void __launch_bounds__(kThreads, 1)
grpo_loss_stream_fwd_kernel(const LossArgs a) {
    constexpr int kLog2PerVec = kF32 ? 2 : 3;
    extern __shared__ __align__(128) unsigned char ring_raw[];
    __shared__ Shared sh;
    const uint4* ring = reinterpret_cast<const uint4*>(ring_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort_flag = &sh.abort;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    const int nvec = a.V >> kLog2PerVec;
    const int n_pieces = (nvec + kStageVecs - 1) / kStageVecs;            // per row (0 for rows of fewer than one vector)
    const float c = a.scale2;

    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&sh.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&sh.empty[s])), "r"(kConsumerWarps));
        }
        for (int p = 0; p < 2; ++p) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&sh.row_done[p])), "r"(kConsumerWarps));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&sh.row_free[p])));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t g = 0;                                                // pieces issued over the CTA's lifetime
            for (long long t = blockIdx.x; t < T && !*abort_flag; t += gridDim.x) {
                const char* row = a.logits + t * a.row_bytes;
                for (int p = 0; p < n_pieces; ++p, ++g) {
                    const uint32_t s = g % kStages, use = g / kStages;
                    if (use > 0 && !wait(smem_u32(&sh.empty[s]), (use - 1) & 1, abort_flag, a.wait_limit_ns)) break;
                    const uint32_t bytes = (uint32_t)min(kStageVecs, nvec - p * kStageVecs) * 16u;
                    const uint32_t bar = smem_u32(&sh.full[s]);
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 :: "r"(bar), "r"(bytes + (g == 0 ? (uint32_t)a.test_extra_tx : 0u)) : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 :: "r"(smem_u32(ring_raw + (size_t)s * kStageBytes)), "l"(row + (size_t)p * kStageBytes), "r"(bytes), "r"(bar)
                                 : "memory");
                }
            }
            if (*abort_flag) {
                // leaving early: the copies still in flight get a bounded chance to land before the CTA's shared
                // memory goes away
                const uint32_t pending = g < (uint32_t)kStages ? g : (uint32_t)kStages;
                for (uint32_t i = 0; i < pending; ++i) {
                    const uint32_t gi = g - 1 - i;
                    const unsigned long long t0 = global_ns();
                    for (;;) {
                        uint32_t done;
                        asm volatile("{\n\t.reg .pred p;\n\t"
                                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                                     "selp.u32 %0, 1, 0, p;\n\t}"
                                     : "=r"(done) : "r"(smem_u32(&sh.full[gi % kStages])), "r"((gi / kStages) & 1) : "memory");
                        if (done || global_ns() - t0 > a.wait_limit_ns) break;
                    }
                }
            }
        }
    } else if (warp < kConsumerWarps) {
        // ------------------------------------------------------------------ consumers
        const int ctid = tid;                                              // 0 .. 511
        uint32_t g = 0, n_row = 0;
        for (long long t = blockIdx.x; t < T && !*abort_flag; t += gridDim.x, ++n_row) {
            float m = -INFINITY, nr = 0.0f;                                // running raw maximum; -m c (0 while m = -inf)
            f32x2 acc0 = pair_of(0.0f, 0.0f), acc1 = acc0;
            bool ok = true;
            for (int p = 0; p < n_pieces && ok; ++p, ++g) {
                const uint32_t s = g % kStages;
                ok = wait(smem_u32(&sh.full[s]), (g / kStages) & 1, abort_flag, a.wait_limit_ns);
                if (!ok) break;
                const uint4* stage = ring + (size_t)s * kStageVecs;
                const int nv = min(kStageVecs, nvec - p * kStageVecs);
#pragma unroll 2
                for (int i = ctid; i < nv; i += kConsumerWarps * 32) {
                    const uint4 q = stage[i];
                    float vmax;
                    if constexpr (kF32) {
                        vmax = fmaxf(fmaxf(__uint_as_float(q.x), __uint_as_float(q.y)), fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
                    } else {
                        __nv_bfloat162 mx2 = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.x), *reinterpret_cast<const __nv_bfloat162*>(&q.y));
                        mx2 = __hmax2(mx2, __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.z), *reinterpret_cast<const __nv_bfloat162*>(&q.w)));
                        vmax = fmaxf(__low2float(mx2), __high2float(mx2));
                    }
                    if (vmax > m) {                                        // rare after the first few vectors of a row
                        const float scale = ex2((m - vmax) * c);           // 0 while m is still -inf (the sums are 0 then)
                        const f32x2 sc2 = pair_of(scale, scale);
                        acc0 = mul2(acc0, sc2); acc1 = mul2(acc1, sc2);
                        m = vmax; nr = -vmax * c;
                    }
                    const f32x2 c2 = pair_of(c, c), nr2 = pair_of(nr, nr);
                    if constexpr (kF32) {
                        exp_quad(q, c2, nr2, acc0, acc1);
                    } else {
                        exp_pair_sum(q.x, c2, nr2, acc0); exp_pair_sum(q.y, c2, nr2, acc1);
                        exp_pair_sum(q.z, c2, nr2, acc0); exp_pair_sum(q.w, c2, nr2, acc1);
                    }
                }
                __syncwarp();
                if (lane == 0) arrive(smem_u32(&sh.empty[s]));             // this warp is done with the stage
            }
            if (!ok) break;
            // the warp's pair: every lane's (r, s) joined by shuffles
            float s0, s1;
            unpair(add2(acc0, acc1), s0, s1);
            float r = m > -INFINITY ? m * c : -INFINITY, s = s0 + s1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float r2 = __shfl_xor_sync(0xffffffffu, r, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
                join(r, s, r2, s2);
            }
            const uint32_t par = n_row & 1;
            if (n_row >= 2 && !wait(smem_u32(&sh.row_free[par]), ((n_row >> 1) - 1) & 1, abort_flag, a.wait_limit_ns)) break;
            if (lane == 0) {
                sh.pair[par][warp] = make_float2(r, s);
                arrive(smem_u32(&sh.row_done[par]));                       // release: the finisher's wait acquires
            }
        }
    } else {
        // ------------------------------------------------------------------ finisher
        const int tail0 = nvec << kLog2PerVec;
        uint32_t n_row = 0;
        for (long long t = blockIdx.x; t < T && !*abort_flag; t += gridDim.x, ++n_row) {
            const char* row = a.logits + t * a.row_bytes;
            RowInputs in;
            row_gather_warp(a, t, lane, in);                               // ahead of time: the row is still streaming
            float r = -INFINITY, s = 0.0f;
            if (tail0 + lane < a.V) {                                      // the row's ragged tail: fewer than 8 elements
                const float z = Elems<!kF32>::load1(row, tail0 + lane);
                if (z > -INFINITY) { r = z * c; s = 1.0f; }
            }
            const uint32_t par = n_row & 1;
            if (!wait(smem_u32(&sh.row_done[par]), (n_row >> 1) & 1, abort_flag, a.wait_limit_ns)) break;
            if (lane < kConsumerWarps) {
                const float2 p = sh.pair[par][lane];
                join(r, s, p.x, p.y);
            }
            __syncwarp();
            if (lane == 0) arrive(smem_u32(&sh.row_free[par]));            // the slot may be written again
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float r2 = __shfl_xor_sync(0xffffffffu, r, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
                join(r, s, r2, s2);
            }
            if (lane == 0) row_finish(a, t, in, r, s, true);
        }
    }

    __syncthreads();
    if (sh.abort) {
        // a wait ran out somewhere in this CTA: report it, and leave every row of the CTA as a row that adds nothing
        // (rows that were already finished included: which ones were is not worth tracking on this path)
        if (tid == 0) set_status(a.status, DPPO_STATUS_TIMEOUT);
        const RowTerms zero = {0.0, 0.0, 0.0, 0.0};
        for (long long t = (long long)blockIdx.x + (long long)tid * gridDim.x; t < T; t += (long long)kThreads * gridDim.x) {
            a.terms[t] = zero;
            if (a.logp_out) a.logp_out[t] = 0.0f;
            if (a.lse_out) a.lse_out[t] = 0.0f;
        }
    }
}

// ---- host side ---------------------------------------------------------------------------------------
template <bool kF32>
static int launch_stream_t(const LossArgs& a, cudaStream_t s, bool launch) {
    auto kernel = grpo_loss_stream_fwd_kernel<kF32>;
    static bool raised[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); dev = -1; }
    if (dev < 0 || !raised[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(DPPO_ERR_UNSUPPORTED, "streaming kernel: %zu bytes of shared memory refused", kDynSmem); }
        if (dev >= 0) raised[dev] = true;
    }
    if (!launch) return DPPO_OK;
    const long long grid = a.T_max < sm_count() ? a.T_max : sm_count();
    kernel<<<(unsigned)(grid > 0 ? grid : 1), kThreads, kDynSmem, s>>>(a);
    DPPO_CHECK_LAUNCH("grpo_loss streaming launch");
    return DPPO_OK;
}

// Forward-only calls (no dlogits) on rows of any length.  DPPO_ERR_UNSUPPORTED (nothing launched) when dlogits are
// asked for.
int launch_rows_stream(const LossArgs& a, cudaStream_t s, bool launch) {
    if (a.dlogits) return fail(DPPO_ERR_UNSUPPORTED, "streaming kernel: forward-only calls (no dlogits)");
    return a.bf16 ? launch_stream_t<false>(a, s, launch) : launch_stream_t<true>(a, s, launch);
}

}  // namespace dppo
