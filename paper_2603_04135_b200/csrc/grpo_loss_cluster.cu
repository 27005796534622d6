// Loss sweep for long bf16 rows: the row never comes back from HBM.
//
// A logit row of the full vocabulary (151,936 bf16 = 297 KB) does not fit one SM's shared memory, and
// dlogits cannot be written before the row's log-sum-exp is known.  Instead of reading the row twice,
// a thread-block cluster of C CTAs splits it: each CTA pulls its slice into shared memory with bulk
// async copies (each CTA fetches only its own slice), reduces (max, sum 2^x) over the slice, the C partial pairs are
// exchanged through distributed shared memory, every CTA repeats the cheap scalar stage, and the
// second pass runs out of shared memory straight into streaming global stores.  HBM traffic is the
// algorithmic minimum: one read and one write per element.  The exponentials of the first pass are
// written back over the logits as fp16 (they lie in (0,1], relative to the slice maximum), so the
// second pass is a scale-and-convert with no exp: one MUFU op per element in total.  Several CTAs
// per SM sit in different phases (copy in flight / reducing / storing), which is what overlaps the
// memory system with the exp work.
//
// f32 rows take the same path with 4-element vectors: the exponentials replace the logits in place as f32
// (same size, nothing to pack) and dlogits leave as f32; a full-vocabulary f32 row (594 KB) needs a cluster of 8.
#include <cuda_fp16.h>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {
using namespace packed;

constexpr int kMaxCluster = 8;
constexpr int kChunks = 1;                    // bulk copies (and mbarriers) per slice: one copy of the whole slice was
                                              // 3.5 % faster than four (fewer waits and loop prologues per row)
constexpr unsigned long long kSettleNs = 20000ull;            // after a failed exchange: time for remote stores already
                                                              // issued by the peers to land before this CTA leaves

struct ClusterStatic {
    unsigned long long bar[kChunks];          // one mbarrier per bulk copy of the slice
    unsigned long long xbar;                  // completes when every CTA's (reference, sum) pair has landed in x[]
    unsigned long long x[kMaxCluster];        // pair of CTA k: low word = reference, high word = sum (f32 bits)
    float red_a[32], red_b[32];
    RowInputs in;
    RowScalars row;
    int failed;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait on phase `parity` of an mbarrier; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    const unsigned long long t0 = global_ns();
    for (;;) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
        if (global_ns() - t0 > limit_ns) return false;
    }
}

// The cluster barrier is used once on the way in, as a start-up handshake ("my mbarriers exist"): no data rides on
// it.  Only a CTA whose exchange failed uses it a second time, on the way out (see the end of the kernel).
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// 8-byte store into CTA `rank`'s shared memory that also signals that CTA's mbarrier (8 bytes of tx).
__device__ __forceinline__ void remote_store_signal(uint32_t local_slot, uint32_t local_bar, int rank, unsigned long long v) {
    uint32_t rslot, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rslot) : "r"(local_slot), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];"
                 :: "r"(rslot), "l"(v), "r"(rbar) : "memory");
}

// kBackward = false: a forward-only call (no dlogits): the exponentials are summed and dropped.
template <int THREADS, bool kF32, bool kBackward>
__global__ void __launch_bounds__(THREADS)
grpo_loss_cluster_kernel(const LossArgs a, const int C, const int vec_per_cta) {
    constexpr int kLog2PerVec = kF32 ? 2 : 3;               // elements per 16-byte vector: 4 f32 or 8 bf16
    extern __shared__ __align__(128) unsigned char slice_raw[];
    __shared__ ClusterStatic st;
    uint4* slice = reinterpret_cast<uint4*>(slice_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = blockIdx.x % C;                        // cluster dims are (C,1,1): consecutive blocks
    const long long t = blockIdx.x / C;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    if (t >= T) return;                                     // uniform over the cluster: nobody reaches a barrier

    const int nvec = a.V >> kLog2PerVec;                    // whole 16-byte vectors of the row
    const int v0 = rank * vec_per_cta;
    const int nv = max(0, min(vec_per_cta, nvec - v0));     // vectors of this CTA's slice
    const int chunk_vec = (nv + kChunks - 1) / kChunks;
    const char* row = a.logits + t * a.row_bytes;
    const float c = a.scale2;

    // ---- issue the slice's bulk copies
    if (tid == 0) {
        st.failed = 0;
#pragma unroll
        for (int k = 0; k < kChunks; ++k)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&st.bar[k])));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&st.xbar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the exchange expects one 8-byte pair from each CTA of the cluster (its own included); the self-test of the
        // bounded waits announces one pair more than will ever be sent, so that every CTA's wait runs out
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(smem_u32(&st.xbar)), "r"(8u * (uint32_t)C + (uint32_t)a.test_extra_tx) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
#pragma unroll
        for (int k = 0; k < kChunks; ++k) {
            const int b = k * chunk_vec, e = min(nv, b + chunk_vec);
            if (e > b) {
                const uint32_t bytes = (uint32_t)(e - b) * 16u;
                const uint32_t bar = smem_u32(&st.bar[k]);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             :: "r"(smem_u32(slice + b)), "l"(row + (size_t)(v0 + b) * 16), "r"(bytes), "r"(bar)
                             : "memory");
            }
        }
    }
    __syncthreads();                                        // barriers initialised before anyone polls them
    cluster_arrive_relaxed();                               // handshake: this CTA's mbarriers exist (waited on before the exchange)

    // ---- while the slice is in flight: one warp finds the token's sequence and gathers the side inputs
    if (warp == (THREADS > 32 ? 1 : 0)) row_gather_warp(a, t, lane, st.in);

    // ---- pass 1a: slice maximum (packed bf16 max), chunk by chunk as the copies land
    __nv_bfloat162 mx2 = __float2bfloat162_rn(-INFINITY);
    float mxa = -INFINITY, mxb = -INFINITY;
    bool ok = true;
#pragma unroll
    for (int k = 0; k < kChunks; ++k) {
        const int b = k * chunk_vec, e = min(nv, b + chunk_vec);
        if (e > b) {
            bool landed = mbar_wait(smem_u32(&st.bar[k]), 0, a.wait_limit_ns);
            // a copy that is late: one more bounded chance to land before anything else happens to this CTA's
            // shared memory (the row is reported as failed either way)
            if (!landed) { mbar_wait(smem_u32(&st.bar[k]), 0, a.wait_limit_ns); ok = false; }
#pragma unroll 2
            for (int i = b + tid; i < e; i += THREADS) {
                const uint4 q = slice[i];
                if constexpr (kF32) {
                    mxa = fmaxf(mxa, fmaxf(__uint_as_float(q.x), __uint_as_float(q.y)));
                    mxb = fmaxf(mxb, fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
                } else {
                    mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&q.x));
                    mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&q.y));
                    mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&q.z));
                    mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&q.w));
                }
            }
        }
    }
    if (!ok) st.failed = 1;                                 // benign race: every writer stores 1
    float m = kF32 ? fmaxf(mxa, mxb) : fmaxf(__low2float(mx2), __high2float(mx2));
    // the row's ragged tail (V % 8 elements) belongs to the last CTA and is read from global memory
    const int tail0 = nvec << kLog2PerVec;
    float ztail = -INFINITY;
    if (rank == C - 1 && tail0 + tid < a.V) {
        ztail = Elems<!kF32>::load1(row, tail0 + tid);
        m = fmaxf(m, ztail);
    }
    m = warp_max(m);
    if (lane == 0) st.red_a[warp] = m;
    __syncthreads();
    m = st.red_a[lane < THREADS / 32 ? lane : 0];
    m = warp_max(m);                                        // every warp ends with the CTA maximum
    const float r = m * c;                                  // -inf for an empty slice

    // ---- pass 1b: sum of 2^(z c - r) over the slice
    float s = 0.0f, etail = 0.0f;
    if (nv > 0 || ztail > -INFINITY) {
        // a slice of nothing but -inf (a masked part of the vocabulary) has r = -inf: any finite offset gives its
        // exponentials the value 0 they must have, where -r would give NaN
        const float nr = r > -INFINITY ? -r : 0.0f;
        const f32x2 c2 = pair_of(c, c), nr2 = pair_of(nr, nr);
        f32x2 acc0 = pair_of(0.0f, 0.0f), acc1 = acc0;
#pragma unroll 2
        for (int i = tid; i < nv; i += THREADS) {
            const uint4 q = slice[i];
            // the exponentials replace the logits in place (bf16 rows: as fp16 pairs): the second pass needs no exp
            uint4 h;
            if constexpr (kF32) {
                h = exp_quad(q, c2, nr2, acc0, acc1);
                if constexpr (kBackward) slice[i] = h;
            } else if constexpr (kBackward) {
                h.x = exp_pair(q.x, c2, nr2, acc0); h.y = exp_pair(q.y, c2, nr2, acc1);
                h.z = exp_pair(q.z, c2, nr2, acc0); h.w = exp_pair(q.w, c2, nr2, acc1);
                slice[i] = h;
            } else {
                exp_pair_sum(q.x, c2, nr2, acc0); exp_pair_sum(q.y, c2, nr2, acc1);
                exp_pair_sum(q.z, c2, nr2, acc0); exp_pair_sum(q.w, c2, nr2, acc1);
            }
        }
        float s0, s1;
        unpair(add2(acc0, acc1), s0, s1);
        s = s0 + s1;
        if (ztail > -INFINITY) { etail = ex2(fmaf(ztail, c, -r)); s += etail; }
    }
    s = warp_sum(s);
    if (lane == 0) st.red_b[warp] = s;
    __syncthreads();

    // ---- exchange (r, s) with the other CTAs of the cluster: one remote store + signal per peer, then
    //      thread 0 waits for all C pairs on its own mbarrier and runs the scalar stage (every CTA
    //      repeats it; rank 0 writes the row's outputs)
    cluster_wait();                                         // every CTA of the cluster has initialised its mbarriers
    if (warp == 0) {
        float ss = lane < THREADS / 32 ? st.red_b[lane] : 0.0f;
        ss = warp_sum(ss);
        if (lane < C) {
            const float rr = st.failed ? __int_as_float(0x7fc00000) : r;   // a NaN reference marks a copy that timed out
            const unsigned long long v = (unsigned long long)__float_as_uint(rr) | ((unsigned long long)__float_as_uint(ss) << 32);
            remote_store_signal(smem_u32(&st.x[rank]), smem_u32(&st.xbar), lane, v);
        }
        if (lane == 0) {
            const bool arrived = mbar_wait(smem_u32(&st.xbar), 0, a.wait_limit_ns);
            float R = -INFINITY;
            bool failed = !arrived;
            for (int k = 0; k < C && arrived; ++k) {
                const float xr = __uint_as_float((uint32_t)st.x[k]);
                failed = failed || (xr != xr);
                R = fmaxf(R, xr);
            }
            float S = 0.0f;
            for (int k = 0; k < C && !failed; ++k) {
                const float xr = __uint_as_float((uint32_t)st.x[k]), xs = __uint_as_float((uint32_t)(st.x[k] >> 32));
                S += (xr == -INFINITY) ? 0.0f : xs * exp2f(xr - R);
            }
            if (failed) {
                if (rank == 0) {
                    set_status(a.status, DPPO_STATUS_TIMEOUT);
                    const RowTerms zero = {0.0, 0.0, 0.0, 0.0};
                    a.terms[t] = zero;
                    if (a.logp_out) a.logp_out[t] = 0.0f;
                    if (a.lse_out) a.lse_out[t] = 0.0f;
                }
                RowScalars bad; bad.lse2_hi = 0.0f; bad.lse2_lo = 0.0f; bad.g_over_tau = 0.0f; bad.valid = false;
                st.row = bad;
                st.failed = arrived ? 1 : 2;                 // 2: this CTA's own wait for the pairs ran out
            } else {
                st.row = row_finish(a, t, st.in, R, S, rank == 0);
            }
        }
    }
    __syncthreads();
    const RowScalars rs = st.row;

    // ---- pass 2: dlogits = g/tau (onehot - 2^(z c - lse2)), shared memory -> streaming global stores
    if (kBackward && a.dlogits) {
        char* drow = a.dlogits + t * a.row_bytes;
        uint4* dst = reinterpret_cast<uint4*>(drow) + v0;
        const float ng = rs.valid ? -rs.g_over_tau : 0.0f;
        // softmax = e * 2^(r - lse2) with e relative to this CTA's reference r (a row that failed has no lse2: its
        // gradient is written as zeros)
        const float sc = st.failed ? 0.0f : ng * ex2((r - rs.lse2_hi) - rs.lse2_lo);
        const f32x2 sc2 = pair_of(sc, sc);
        const int y = rs.valid ? a.target[t] : -1;
        const int yvec = (y >= 0 ? (y >> kLog2PerVec) : -1) - v0;   // vector of the target relative to this slice
#pragma unroll 2
        for (int i = tid; i < nv; i += THREADS) {
            const uint4 q = slice[i];
            uint4 o;
            if constexpr (kF32) {
                o = scale_quad(q, sc2);
            } else {
                o.x = scale_pair(q.x, sc2); o.y = scale_pair(q.y, sc2);
                o.z = scale_pair(q.z, sc2); o.w = scale_pair(q.w, sc2);
            }
            __stcs(dst + i, o);
        }
        // the one element that also carries the onehot term: the thread that stored its vector redoes it
        if (yvec >= 0 && yvec < nv && (yvec % THREADS) == tid) {
            if constexpr (kF32) {
                const float ey = reinterpret_cast<const float*>(slice + yvec)[y & 3];
                reinterpret_cast<float*>(drow)[y] = fmaf(ey, sc, -ng);
            } else {
                const uint32_t word = reinterpret_cast<const uint32_t*>(slice + yvec)[(y & 7) >> 1];
                const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&word));
                const float ey = (y & 1) ? e.y : e.x;
                reinterpret_cast<__nv_bfloat16*>(drow)[y] = __float2bfloat16_rn(fmaf(ey, sc, -ng));
            }
        }
        if (rank == C - 1 && tail0 + tid < a.V) {
            const int v = tail0 + tid;
            Elems<!kF32>::store1(drow, v, sc * etail - (v == y ? ng : 0.0f));
        }
    }

    // ---- way out after a failed exchange.  A CTA that has received all C pairs knows that every peer is done
    //      writing into its shared memory and simply returns.  A CTA whose own wait ran out does not: a slow peer
    //      could still send its pair, and that remote store must not land in shared memory that already belongs to
    //      another CTA.  It therefore waits on the cluster barrier, which completes once every peer has either
    //      arrived here as well (it failed too) or exited (it sends before it can exit), and then lets stores that
    //      are already under way settle.  Every wait before this point is bounded, so every peer gets that far.
    if (st.failed == 2) {                                   // written before the block barrier above: uniform
        cluster_arrive_release();
        cluster_wait_acquire();
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < kSettleNs) { }
    }
}

// ---- host side ---------------------------------------------------------------------------------------
constexpr size_t kClusterSmemMax = 220 * 1024;            // largest slice a CTA may hold

// The dynamic shared-memory limit of an instantiation is raised once per device to the largest slice any launch
// may ask for (a per-call value could be lowered by another host thread between this thread's set and its launch).
template <int THREADS, bool kF32, bool kBackward>
static int cluster_prepare_t(int C, size_t dyn_bytes, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, bool check_fit) {
    auto kernel = grpo_loss_cluster_kernel<THREADS, kF32, kBackward>;
    static bool raised[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); dev = -1; }
    if (dev < 0 || !raised[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kClusterSmemMax);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: %zu bytes of shared memory refused", kClusterSmemMax); }
        if (dev >= 0) raised[dev] = true;
    }
    cfg->blockDim = dim3(THREADS, 1, 1);
    cfg->dynamicSmemBytes = dyn_bytes;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
    // clusters handed to whichever GPC has room rather than spread evenly: 5 % faster on eight-CTA clusters (f32
    // rows of the full vocabulary), 2.5 % on four while the board is below its power limit
    attr[1].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
    cfg->attrs = attr; cfg->numAttrs = 2;
    if (check_fit) {
        int max_clusters = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&max_clusters, kernel, cfg);
        if (e != cudaSuccess || max_clusters < 1) { cudaGetLastError(); return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: cluster of %d CTAs does not fit this device", C); }
    }
    return DPPO_OK;
}

// launch = false: only the checks a launch would make (used by the kernel-choice query).
template <int THREADS, bool kF32, bool kBackward>
static int launch_cluster_tb(const LossArgs& a, int C, int vec_per_cta, size_t dyn_bytes, cudaStream_t s, bool launch) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.gridDim = dim3((unsigned)((a.T_max > 0 ? a.T_max : 1) * C), 1, 1);
    cfg.stream = s;
    const int rc = cluster_prepare_t<THREADS, kF32, kBackward>(C, dyn_bytes, &cfg, attr, true);
    if (rc != DPPO_OK || !launch) return rc;
    cudaError_t e = cudaLaunchKernelEx(&cfg, grpo_loss_cluster_kernel<THREADS, kF32, kBackward>, a, C, vec_per_cta);
    if (e != cudaSuccess) return cuda_fail(e, "grpo_loss cluster launch");
    return DPPO_OK;
}

template <int THREADS, bool kF32>
static int launch_cluster_t(const LossArgs& a, int C, int vec_per_cta, size_t dyn_bytes, cudaStream_t s, bool launch) {
    return a.dlogits ? launch_cluster_tb<THREADS, kF32, true>(a, C, vec_per_cta, dyn_bytes, s, launch)
                     : launch_cluster_tb<THREADS, kF32, false>(a, C, vec_per_cta, dyn_bytes, s, launch);
}

int launch_rows_cluster(const LossArgs& a, int C, int threads, cudaStream_t s, bool launch) {
    if (C != 1 && C != 2 && C != 4 && C != 8) return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: cluster size %d", C);
    const int log2_per_vec = a.bf16 ? 3 : 2;
    if ((a.V & ((1 << log2_per_vec) - 1)) >= threads) return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: tail");
    if (a.T_max * C >= (1ll << 31)) return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: grid too large");
    const int nvec = a.V >> log2_per_vec;
    const int vec_per_cta = (nvec + C - 1) / C;
    const size_t dyn_bytes = (size_t)(vec_per_cta > 0 ? vec_per_cta : 1) * 16;
    if (dyn_bytes > kClusterSmemMax) return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: slice of %zu bytes exceeds shared memory", dyn_bytes);
    if (dyn_bytes / kChunks + 16 >= (1u << 20)) return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: chunk too large");
    if (a.bf16) {
        switch (threads) {
            case 128: return launch_cluster_t<128, false>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 256: return launch_cluster_t<256, false>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 512: return launch_cluster_t<512, false>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 1024: return launch_cluster_t<1024, false>(a, C, vec_per_cta, dyn_bytes, s, launch);
        }
    } else {
        switch (threads) {
            case 128: return launch_cluster_t<128, true>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 256: return launch_cluster_t<256, true>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 512: return launch_cluster_t<512, true>(a, C, vec_per_cta, dyn_bytes, s, launch);
            case 1024: return launch_cluster_t<1024, true>(a, C, vec_per_cta, dyn_bytes, s, launch);
        }
    }
    return fail(DPPO_ERR_UNSUPPORTED, "cluster kernel: %d threads", threads);
}

}  // namespace dppo
