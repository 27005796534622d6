// Loss sweep for rows of up to 32 KB: tiles of consecutive rows go through a shared-memory ring, and
// the three kinds of work a row needs are done by three kinds of warps that never wait for memory.
//
// A short row is dominated by what does not scale with its length: two warp reductions and, above all, the
// binary64 scalar stage (a logarithm, two exponentials, the clip logic: several hundred instructions, and a warp
// instruction costs the same with one lane active as with 32).  A warp that loads a row, reduces it, runs the
// scalar stage and stores the row sees all of those latencies one after the other.  Here one persistent CTA per SM
// splits the work:
//   loader          one thread issues one bulk copy per TILE (up to 32 KB of consecutive rows, at most 32 units)
//                   into a ring of stages, running ahead as far as the ring allows
//   16 consumer     two groups of eight take the tiles alternately.  Pass 1 on the tile's UNITS (a unit is a row, or
//   warps           one of the equal parts of at most 2 KB of a longer row; a warp works on two units at a time):
//                   maximum, 2^(z c - r) once, kept in place as fp16 pairs (bf16 rows) or f32, the unit's (r, sum) to
//                   shared memory.  Pass 2, after pass 1 of the group's next tile: the stored exponentials times the
//                   unit's factor go to dlogits with streaming stores; the stage is then free
//   scalar warps    lane q takes row q of a tile: joins the row's units, runs the scalar stage for up to 32 rows in
//                   one pass, and leaves every unit's factor g/tau 2^(r - lse2) (and the one element per row that
//                   also carries the onehot term) for pass 2.  The rows' per-token inputs and sequences are gathered
//                   a tile ahead
// A forward-only call (no dlogits) runs pass 1 without the write-back and the scalar stage; a stage is free as soon
// as pass 1 has read it.
// HBM sees one read and one write per element.  Every wait is bounded; on a time-out the CTA raises an abort flag,
// reports DPPO_STATUS_TIMEOUT, lets its copies in flight land (bounded) and leaves all of its rows as rows that add
// nothing.
#include <cuda_fp16.h>

#include <type_traits>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {
using namespace packed;

namespace tile {

constexpr int kConsumerWarps = 16;
constexpr int kScalarWarps = 3;
constexpr int kThreads = (kConsumerWarps + kScalarWarps + 1) * 32;       // + the loader's warp
constexpr int kStages = 6;
constexpr int kStageBytes = 32768;
constexpr int kMaxUnits = 32;                             // units of a tile (and rows: one lane of a scalar warp each)
constexpr int kGroups = 2;                                // the consumer warps work in groups on alternate tiles
constexpr int kGroupWarps = kConsumerWarps / kGroups;
constexpr int kGroupSkew = 1;                             // a group runs pass 2 of a tile after pass 1 of its kGroupSkew-th next tile
constexpr int kCuCache = 6144;                            // entries of cu_seqlens kept in shared memory (24 KB)
constexpr size_t kDynSmem = (size_t)kStages * kStageBytes + (size_t)kCuCache * 4;

struct Meta {                                             // of one stage
    float2 rs[kMaxUnits];                                 // per unit: reference r = max c, sum of 2^(z c - r)
    float sc[kMaxUnits];                                  // per unit: the factor of its stored exponentials
    int fix_y[kMaxUnits];                                 // per row: the element that also carries the onehot term, or -1
    float fix_val[kMaxUnits];                             // its value
};

struct Shared {
    unsigned long long full[kStages];                     // the tile's bytes have landed
    unsigned long long p1_done[kStages];                  // the tile's group of consumer warps has finished pass 1
    unsigned long long s_done[kStages];                   // the tile's scalar stage is done
    unsigned long long free_[kStages];                    // ... and pass 2: the stage may be refilled
    Meta meta[kStages];
    int abort;
};

// How a row length maps to tiles: rows per tile R, parts per row P (units of a tile: R * P <= 32).
struct Geometry {
    int nvec;                                             // 16-byte vectors of a row that hold elements
    int part_vecs;                                        // vectors per part, at most 32 kVPL (the last part of a row may have fewer)
    int parts;                                            // parts per row
    int rows;                                             // rows per tile
};
template <int kVPL>
__host__ __device__ inline Geometry geometry(int V, int log2_per_vec, long long row_bytes) {
    Geometry g;
    g.nvec = V >> log2_per_vec;
    const long long fit = kStageBytes / (row_bytes > 0 ? row_bytes : 1);
    // parts per row: as few as keep a part within 32 kVPL vectors (more, smaller parts that would fill the 16 consumer
    // warps more evenly measured slower: a unit's fixed cost, its two warp reductions, is what counts)
    g.parts = g.nvec > 32 * kVPL ? (g.nvec + 32 * kVPL - 1) / (32 * kVPL) : 1;
    g.part_vecs = (g.nvec + g.parts - 1) / g.parts;       // equal parts (the last one may be a little shorter)
    if (g.part_vecs < 1) g.part_vecs = 1;
    const int by_units = kMaxUnits / g.parts;
    g.rows = (int)(fit < by_units ? fit : by_units);
    return g;
}

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
// Bounded wait on phase `parity`; also leaves (false) when another role has raised the abort flag.  A warp that waits
// with all its lanes takes the vote of the lanes' results, so that it leaves as a whole.  The clock and the abort
// flag are looked at once per eight tries (a try lasts up to a microsecond), not per try.
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

}  // namespace tile

using namespace tile;

// Pass 1 on N units of one warp at once, so that their instruction streams interleave (the shuffle chains of one unit
// run under the exponentials of the other): per unit the maximum, 2^(z c - r) for every element (kept in place as fp16
// pairs or f32 when write_back), and (r, sum) of the unit.
template <bool kF32, int kVPL, int N>
__device__ __forceinline__ void pass1_units(uint4* const (&src)[N], const int (&nv)[N], int lane, float c, bool write_back,
                                            float2 (&out)[N]) {
    constexpr uint32_t kPad = kF32 ? 0xFF800000u : 0xFF80FF80u;   // -inf: adds nothing to the maximum or the sum
    uint4 d[N][kVPL];
#pragma unroll
    for (int n = 0; n < N; ++n)
#pragma unroll
        for (int j = 0; j < kVPL; ++j) {
            const int i = lane + 32 * j;
            d[n][j] = i < nv[n] ? src[n][i] : make_uint4(kPad, kPad, kPad, kPad);
        }
    float m[N];
#pragma unroll
    for (int n = 0; n < N; ++n) {
        if constexpr (kF32) {
            m[n] = -INFINITY;
#pragma unroll
            for (int j = 0; j < kVPL; ++j)
                m[n] = fmaxf(m[n], fmaxf(fmaxf(__uint_as_float(d[n][j].x), __uint_as_float(d[n][j].y)),
                                         fmaxf(__uint_as_float(d[n][j].z), __uint_as_float(d[n][j].w))));
        } else {
            __nv_bfloat162 mx2 = __float2bfloat162_rn(-INFINITY);
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[n][j].x));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[n][j].y));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[n][j].z));
                mx2 = __hmax2(mx2, *reinterpret_cast<const __nv_bfloat162*>(&d[n][j].w));
            }
            m[n] = fmaxf(__low2float(mx2), __high2float(mx2));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int n = 0; n < N; ++n) m[n] = fmaxf(m[n], __shfl_xor_sync(0xffffffffu, m[n], o));
    float sum[N];
#pragma unroll
    for (int n = 0; n < N; ++n) {
        const float r = m[n] * c;                                  // -inf only if the whole unit is -inf
        const float nr = r > -INFINITY ? -r : 0.0f;
        const f32x2 c2 = pair_of(c, c), nr2 = pair_of(nr, nr);
        f32x2 acc0 = pair_of(0.0f, 0.0f), acc1 = acc0;
        if (write_back) {
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                if constexpr (kF32) {
                    d[n][j] = exp_quad(d[n][j], c2, nr2, acc0, acc1);
                } else {
                    d[n][j].x = exp_pair(d[n][j].x, c2, nr2, acc0); d[n][j].y = exp_pair(d[n][j].y, c2, nr2, acc1);
                    d[n][j].z = exp_pair(d[n][j].z, c2, nr2, acc0); d[n][j].w = exp_pair(d[n][j].w, c2, nr2, acc1);
                }
                const int i = lane + 32 * j;
                if (i < nv[n]) src[n][i] = d[n][j];
            }
        } else {
#pragma unroll
            for (int j = 0; j < kVPL; ++j) {
                if constexpr (kF32) {
                    exp_quad(d[n][j], c2, nr2, acc0, acc1);
                } else {
                    exp_pair_sum(d[n][j].x, c2, nr2, acc0); exp_pair_sum(d[n][j].y, c2, nr2, acc1);
                    exp_pair_sum(d[n][j].z, c2, nr2, acc0); exp_pair_sum(d[n][j].w, c2, nr2, acc1);
                }
            }
        }
        float s0, s1;
        unpair(add2(acc0, acc1), s0, s1);
        sum[n] = s0 + s1;
        out[n].x = r;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int n = 0; n < N; ++n) sum[n] += __shfl_xor_sync(0xffffffffu, sum[n], o);
#pragma unroll
    for (int n = 0; n < N; ++n) out[n].y = sum[n];
}

// Pass 2 on N units of one warp at once: the stored exponentials times the unit's factor, to dlogits.
template <bool kF32, int kVPL, int N>
__device__ __forceinline__ void pass2_units(const uint4* const (&src)[N], uint4* const (&dst)[N], const int (&nv)[N],
                                            const float (&sc)[N], int lane) {
    uint4 e[N][kVPL];
#pragma unroll
    for (int n = 0; n < N; ++n)
#pragma unroll
        for (int j = 0; j < kVPL; ++j) {
            const int i = lane + 32 * j;
            e[n][j] = i < nv[n] ? src[n][i] : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
    for (int n = 0; n < N; ++n) {
        const f32x2 sc2 = pair_of(sc[n], sc[n]);
#pragma unroll
        for (int j = 0; j < kVPL; ++j) {
            const int i = lane + 32 * j;
            if (i < nv[n]) {
                uint4 o;
                if constexpr (kF32) {
                    o = scale_quad(e[n][j], sc2);
                } else {
                    o.x = scale_pair(e[n][j].x, sc2); o.y = scale_pair(e[n][j].y, sc2);
                    o.z = scale_pair(e[n][j].z, sc2); o.w = scale_pair(e[n][j].w, sc2);
                }
                __stcs(dst[n] + i, o);
            }
        }
    }
}

template <bool kF32, int kVPL>
__global__ void __launch_bounds__(kThreads, 1)
grpo_loss_tile_kernel(const LossArgs a, const int rows_per_tile) {
    constexpr int kLog2PerVec = kF32 ? 2 : 3;               // elements per 16-byte vector: 4 f32 or 8 bf16
    extern __shared__ __align__(128) unsigned char ring_raw[];
    __shared__ Shared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort_flag = &sh.abort;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    const Geometry geo = geometry<kVPL>(a.V, kLog2PerVec, a.row_bytes);
    const int R = rows_per_tile, P = geo.parts;               // R <= geo.rows: fewer for a batch of less than a full tile per SM
    const float c = a.scale2;
    const bool backward = a.dlogits != nullptr;           // else forward only: pass 1 and the scalar stage
    // this CTA's tiles: tile k covers rows (blockIdx.x + k gridDim.x) R ... of the batch
    const long long total_tiles = (T + R - 1) / R;
    const int n_tiles = (long long)blockIdx.x < total_tiles ? (int)((total_tiles - 1 - blockIdx.x) / gridDim.x) + 1 : 0;
    auto tile_row0 = [&](int k) { return ((long long)blockIdx.x + (long long)k * gridDim.x) * R; };
    auto tile_rows = [&](int k) { return (int)min((long long)R, T - tile_row0(k)); };

    // cu_seqlens is searched once per tile by the scalar warps; a copy in shared memory (when its S_max + 1 entries
    // fit) turns the three or four dependent round trips of a search into a fraction of a microsecond
    int32_t* cu_copy = reinterpret_cast<int32_t*>(ring_raw + (size_t)kStages * kStageBytes);
    const bool cu_cached = a.S_max >= 1 && a.S_max + 1 <= kCuCache;
    if (cu_cached)
        for (int i = tid; i <= a.S_max; i += kThreads) cu_copy[i] = a.cu_seqlens[i];
    const int32_t* cu = cu_cached ? cu_copy : a.cu_seqlens;
    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&sh.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&sh.p1_done[s])), "r"(kGroupWarps));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&sh.s_done[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&sh.free_[s])), "r"(kGroupWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps + kScalarWarps) {
        // ------------------------------------------------------------------ loader
        if (lane == 0) {
            int k = 0;
            for (; k < n_tiles && !*abort_flag; ++k) {
                const uint32_t s = (uint32_t)k % kStages, use = (uint32_t)k / kStages;
                if (use > 0 && !wait(smem_u32(&sh.free_[s]), (use - 1) & 1, abort_flag, a.wait_limit_ns)) break;
                const uint32_t bytes = (uint32_t)tile_rows(k) * (uint32_t)a.row_bytes;
                const uint32_t bar = smem_u32(&sh.full[s]);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             :: "r"(bar), "r"(bytes + (k == 0 ? (uint32_t)a.test_extra_tx : 0u)) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             :: "r"(smem_u32(ring_raw + (size_t)s * kStageBytes)), "l"(a.logits + tile_row0(k) * a.row_bytes), "r"(bytes), "r"(bar)
                             : "memory");
            }
            if (*abort_flag) {
                // leaving early: the copies still in flight get a bounded chance to land before the CTA's shared
                // memory goes away
                const int pending = k < kStages ? k : kStages;
                for (int i = 0; i < pending; ++i) {
                    const uint32_t ki = (uint32_t)(k - 1 - i);
                    const unsigned long long t0 = global_ns();
                    while (!try_wait(smem_u32(&sh.full[ki % kStages]), (ki / kStages) & 1) && global_ns() - t0 <= a.wait_limit_ns) {}
                }
            }
        }
    } else if (warp < kConsumerWarps) {
        // ------------------------------------------------------------------ consumers
        // Two groups of eight warps take the tiles alternately (group g: tiles g, g + 2, ...), so that the groups are
        // in different phases of their tiles (one in its exponentials while the other reduces, waits or stores) instead
        // of all sixteen warps wanting the same pipe at the same time.  A warp works on its units two at a time.
        // This warp's units of a tile, the same in every tile: unit u = wid + 8 i is part u % P of row u / P.
        const int group = warp / kGroupWarps, wid = warp - group * kGroupWarps;
        constexpr int kUnitsPerWarp = kMaxUnits / kGroupWarps;
        int u_row[kUnitsPerWarp], u_nv[kUnitsPerWarp], u_e0[kUnitsPerWarp];
        uint32_t u_vec[kUnitsPerWarp];                                     // 16-byte offset of the unit inside a stage
        long long u_dst[kUnitsPerWarp];                                    // byte offset of the unit from its tile's first row
#pragma unroll
        for (int i = 0; i < kUnitsPerWarp; ++i) {
            const int u = wid + i * kGroupWarps;
            const int row = u / P, part = u - row * P;
            u_row[i] = row;
            u_nv[i] = min(geo.part_vecs, geo.nvec - part * geo.part_vecs);
            u_e0[i] = (part * geo.part_vecs) << kLog2PerVec;
            u_vec[i] = (uint32_t)row * (uint32_t)(a.row_bytes >> 4) + (uint32_t)(part * geo.part_vecs);
            u_dst[i] = (long long)row * a.row_bytes + (long long)part * geo.part_vecs * 16;
        }
        for (int j = 0; !*abort_flag; ++j) {
            const int k = group + kGroups * j;                              // pass 1 of tile k
            const int kk = k - kGroups * kGroupSkew;                        // pass 2 of tile kk
            if (k >= n_tiles && (!backward || kk >= n_tiles)) break;
            if (k < n_tiles) {
                const uint32_t s = (uint32_t)k % kStages, use = (uint32_t)k / kStages;
                if (!__all_sync(0xffffffffu, wait(smem_u32(&sh.full[s]), use & 1, abort_flag, a.wait_limit_ns))) break;
                // forward only: there is no pass 2 whose wait would tell that the scalar warp has read this stage's
                // (r, sum) of the previous round
                if (!backward && use > 0 &&
                    !__all_sync(0xffffffffu, wait(smem_u32(&sh.s_done[s]), (use - 1) & 1, abort_flag, a.wait_limit_ns))) break;
                uint4* stage = reinterpret_cast<uint4*>(ring_raw + (size_t)s * kStageBytes);
                const int units = tile_rows(k) * P;
#pragma unroll
                for (int i = 0; i < kUnitsPerWarp; i += 2) {
                    const int ua = wid + i * kGroupWarps, ub = ua + kGroupWarps;
                    if (ub < units) {
                        uint4* const src[2] = {stage + u_vec[i], stage + u_vec[i + 1]};
                        const int nv[2] = {u_nv[i], u_nv[i + 1]};
                        float2 rs[2];
                        pass1_units<kF32, kVPL, 2>(src, nv, lane, c, backward, rs);
                        if (lane == 0) { sh.meta[s].rs[ua] = rs[0]; sh.meta[s].rs[ub] = rs[1]; }
                    } else if (ua < units) {
                        uint4* const src[1] = {stage + u_vec[i]};
                        const int nv[1] = {u_nv[i]};
                        float2 rs[1];
                        pass1_units<kF32, kVPL, 1>(src, nv, lane, c, backward, rs);
                        if (lane == 0) sh.meta[s].rs[ua] = rs[0];
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    arrive(smem_u32(&sh.p1_done[s]));                       // release: the scalar warp's wait acquires
                    if (!backward) arrive(smem_u32(&sh.free_[s]));          // forward only: the stage has been read, that is all
                }
            }
            if (backward && kk >= 0 && kk < n_tiles) {
                const uint32_t s = (uint32_t)kk % kStages;
                if (!__all_sync(0xffffffffu, wait(smem_u32(&sh.s_done[s]), ((uint32_t)kk / kStages) & 1, abort_flag, a.wait_limit_ns))) break;
                const uint4* stage = reinterpret_cast<const uint4*>(ring_raw + (size_t)s * kStageBytes);
                const int units = tile_rows(kk) * P;
                const long long t0 = tile_row0(kk);
                char* tile_dst = a.dlogits + t0 * a.row_bytes;
#pragma unroll
                for (int i = 0; i < kUnitsPerWarp; i += 2) {
                    const int ua = wid + i * kGroupWarps, ub = ua + kGroupWarps;
                    if (ub < units) {
                        const uint4* const src[2] = {stage + u_vec[i], stage + u_vec[i + 1]};
                        uint4* const dst[2] = {reinterpret_cast<uint4*>(tile_dst + u_dst[i]), reinterpret_cast<uint4*>(tile_dst + u_dst[i + 1])};
                        const int nv[2] = {u_nv[i], u_nv[i + 1]};
                        const float sc[2] = {sh.meta[s].sc[ua], sh.meta[s].sc[ub]};
                        pass2_units<kF32, kVPL, 2>(src, dst, nv, sc, lane);
                    } else if (ua < units) {
                        const uint4* const src[1] = {stage + u_vec[i]};
                        uint4* const dst[1] = {reinterpret_cast<uint4*>(tile_dst + u_dst[i])};
                        const int nv[1] = {u_nv[i]};
                        const float sc[1] = {sh.meta[s].sc[ua]};
                        pass2_units<kF32, kVPL, 1>(src, dst, nv, sc, lane);
                    }
                }
                // the one element of a row that also carries the onehot term, where it lies in one of this warp's units
                __syncwarp();                                               // after the lanes' stores of the units
                if (lane < kUnitsPerWarp) {
                    int row = 0, e0 = 0, nv = 0;
#pragma unroll
                    for (int i = 0; i < kUnitsPerWarp; ++i)
                        if (lane == i) { row = u_row[i]; e0 = u_e0[i]; nv = u_nv[i]; }
                    if (wid + lane * kGroupWarps < units) {
                        const int y = sh.meta[s].fix_y[row];
                        if (y >= e0 && y < e0 + (nv << kLog2PerVec))
                            Elems<!kF32>::store1(tile_dst + (long long)row * a.row_bytes, y, sh.meta[s].fix_val[row]);
                    }
                }
                // the stage goes back to the loader: this warp's reads and writes of it come before the next copy into it
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) arrive(smem_u32(&sh.free_[s]));
            }
        }
    } else {
        // ------------------------------------------------------------------ scalar warps: lane q <-> row q of a tile
        const int first = warp - kConsumerWarps;
        // What the scalar stage needs besides (r, sum), gathered one tile ahead ("next", used as "cur") in two halves, so
        // that no load is waited for where it is issued: values stay as loaded (conversions wait for the load) and
        // the loads that depend on loaded values (the sampled logit on the token id, advantage and weight on the mapped
        // sequence index) go out a scalar stage after those.
        struct Gathered {
            long long t;
            int y;                                                          // -1 for a lane without a row
            int seg, idx, len;                                              // sequence position, mapped index, length
            float lp_old, lp_ref, adv, w, lr;
            typename std::conditional<kF32, float, __nv_bfloat16>::type zy;
            bool mine, seg_ok;
        };
        Gathered nxt, cur;
        // first half: the per-token inputs (lane-indexed loads) and the rows' sequences: the whole warp searches the
        // copy of cu_seqlens, 32 probes per step, once per sequence that the tile touches
        auto gather_first = [&](int k) {
            const long long t0 = tile_row0(k), t_end = t0 + tile_rows(k);
            nxt.t = t0 + lane;
            nxt.mine = nxt.t < t_end;
            nxt.y = -1; nxt.lp_old = 0.0f; nxt.lp_ref = 0.0f;
            if (nxt.mine) { nxt.y = a.target[nxt.t]; nxt.lp_old = a.logp_old[nxt.t]; nxt.lp_ref = a.logp_ref[nxt.t]; }
            nxt.seg_ok = false; nxt.seg = 0; nxt.len = 1;
            long long at = t0;                                              // first row not yet looked up
            while (a.S_max >= 1 && at < t_end) {
                int lo = 0, hi = a.S_max;
                while (hi - lo > 1) {
                    const int step = (hi - lo + 31) >> 5;
                    const long long idx = (long long)lo + (long long)(lane + 1) * step;
                    const bool le = idx < hi && (long long)cu[idx] <= at;
                    const int n = __popc(__ballot_sync(0xffffffffu, le));
                    lo += n * step;
                    hi = min(hi, lo + step);
                }
                const long long s_lo = cu[lo], s_hi = cu[lo + 1];
                const bool ok = at >= s_lo && at < s_hi;
                const long long upto = ok ? min(s_hi, t_end) : at + 1;      // rows [at, upto) are settled by this lookup
                if (ok && nxt.t >= at && nxt.t < upto) { nxt.seg_ok = true; nxt.seg = lo; nxt.len = (int)(s_hi - s_lo); }
                at = upto;
            }
            nxt.idx = nxt.seg;
            if (nxt.mine && nxt.seg_ok && a.seg_map) nxt.idx = a.seg_map[nxt.seg];
        };
        // second half: what needs the first half's loads.  The sampled token's logit comes from global memory: the
        // stage's copy of the row is overwritten by pass 1
        auto gather_second = [&]() {
            nxt.adv = nxt.w = nxt.lr = 0.0f;
            if (nxt.mine && nxt.seg_ok) {
                nxt.adv = a.adv[nxt.idx];
                nxt.w = a.w[nxt.idx];
                if (a.seq_log_ratio) nxt.lr = a.seq_log_ratio[nxt.seg];
            }
            nxt.zy = 0.0f;
            if (nxt.mine && nxt.y >= 0 && nxt.y < a.V)
                nxt.zy = reinterpret_cast<const decltype(nxt.zy)*>(a.logits + nxt.t * a.row_bytes)[nxt.y];
        };
        if (first < n_tiles) { gather_first(first); gather_second(); }
        for (int k = first; k < n_tiles && !*abort_flag; k += kScalarWarps) {
            const uint32_t s = (uint32_t)k % kStages;
            if (!__all_sync(0xffffffffu, wait(smem_u32(&sh.p1_done[s]), ((uint32_t)k / kStages) & 1, abort_flag, a.wait_limit_ns))) break;
            cur = nxt;
            const bool more = k + kScalarWarps < n_tiles;
            if (more) gather_first(k + kScalarWarps);                      // in flight during this tile's scalar stage
            Meta& meta = sh.meta[s];
            if (cur.mine) {
                const int u0 = lane * P;
                float r = -INFINITY, sum = 0.0f;                            // the row's units joined: sum of 2^(z c - r)
                for (int p = 0; p < P; ++p) {
                    const float2 q = meta.rs[u0 + p];
                    const float hi = fmaxf(r, q.x);
                    const float x = r > -INFINITY ? sum * ex2(r - hi) : 0.0f;
                    const float y = q.x > -INFINITY ? q.y * ex2(q.x - hi) : 0.0f;
                    r = hi; sum = x + y;
                }
                const bool y_ok = cur.y >= 0 && cur.y < a.V;
                const float zy_raw = (float)cur.zy;
                RowInputs in;
                in.A = in.W = in.zy = in.logp_old = in.logp_ref = in.seq_lr = 0.0;
                in.use_seq = 0; in.y = cur.y; in.state = 0;
                if (!cur.seg_ok) in.state = DPPO_STATUS_BAD_SEGMENTS;
                else if (!y_ok) in.state = DPPO_STATUS_BAD_TARGET;
                else {
                    in.A = (double)cur.adv;
                    in.W = a.no_length_norm ? (double)cur.w : (double)cur.w / (double)cur.len;
                    if (a.seq_log_ratio) { in.use_seq = 1; in.seq_lr = (double)cur.lr; }
                    in.zy = (double)zy_raw / a.temperature;
                    in.logp_old = (double)cur.lp_old; in.logp_ref = (double)cur.lp_ref;
                }
                const RowScalars rs = row_finish(a, cur.t, in, r, sum, true);
                const float ng = rs.valid ? -rs.g_over_tau : 0.0f;
                // dlogits = g/tau (onehot - 2^(z c - lse2)): every unit's stored exponentials times its own factor
                for (int p = 0; p < P; ++p) {
                    const float rp = meta.rs[u0 + p].x;
                    meta.sc[u0 + p] = rs.valid ? ng * ex2((rp - rs.lse2_hi) - rs.lse2_lo) : 0.0f;
                }
                int fix_y = -1;
                float fix_val = 0.0f;
                if (rs.valid) {
                    // the element that also carries the onehot term: the same exponential as pass 1 formed (rounded
                    // to fp16 where the stored ones are) times its unit's factor, minus g/tau
                    const int py = (cur.y >> kLog2PerVec) / geo.part_vecs;
                    const float rp = meta.rs[u0 + py].x;
                    const float nr = rp > -INFINITY ? -rp : 0.0f;
                    float e = zy_raw > -INFINITY ? ex2(fmaf(zy_raw, c, nr)) : 0.0f;
                    if (!kF32) e = __half2float(__float2half_rn(e));
                    fix_y = cur.y;
                    fix_val = fmaf(e, meta.sc[u0 + py], -ng);
                }
                meta.fix_y[lane] = fix_y;
                meta.fix_val[lane] = fix_val;
            }
            __syncwarp();
            if (lane == 0) arrive(smem_u32(&sh.s_done[s]));                 // release: the consumers' waits acquire
            if (more) gather_second();
        }
    }

    __syncthreads();
    if (sh.abort) {
        // a wait ran out somewhere in this CTA: report it, and leave every row of the CTA as a row that adds nothing
        // (rows that were already finished included: which ones were is not worth tracking on this path)
        if (tid == 0) set_status(a.status, DPPO_STATUS_TIMEOUT);
        const RowTerms zero = {0.0, 0.0, 0.0, 0.0};
        for (int k = 0; k < n_tiles; ++k) {
            const long long t0 = tile_row0(k);
            const int rows = tile_rows(k);
            for (int q = tid; q < rows; q += kThreads) {
                a.terms[t0 + q] = zero;
                if (a.logp_out) a.logp_out[t0 + q] = 0.0f;
                if (a.lse_out) a.lse_out[t0 + q] = 0.0f;
            }
            for (int i = tid; backward && i < rows * geo.nvec; i += kThreads) {
                const int q = i / geo.nvec, v = i - q * geo.nvec;
                reinterpret_cast<uint4*>(a.dlogits + (t0 + q) * a.row_bytes)[v] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
}

// ---- host side ---------------------------------------------------------------------------------------
template <bool kF32, int kVPL>
static int launch_tile_t(const LossArgs& a, cudaStream_t s, bool launch) {
    auto kernel = grpo_loss_tile_kernel<kF32, kVPL>;
    static bool raised[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); dev = -1; }
    if (dev < 0 || !raised[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(DPPO_ERR_UNSUPPORTED, "tile kernel: %zu bytes of shared memory refused", kDynSmem); }
        if (dev >= 0) raised[dev] = true;
    }
    if (!launch) return DPPO_OK;
    // rows per tile: as many as a stage and the 32 units allow; a batch that would leave SMs without a tile takes
    // smaller tiles instead
    const Geometry geo = geometry<kVPL>(a.V, kF32 ? 2 : 3, a.row_bytes);
    const long long per_sm = (a.T_max + sm_count() - 1) / sm_count();
    const int rows = (int)(per_sm < geo.rows ? (per_sm > 1 ? per_sm : 1) : geo.rows);
    const long long tiles = (a.T_max + rows - 1) / rows;
    const long long grid = tiles < sm_count() ? tiles : sm_count();
    kernel<<<(unsigned)(grid > 0 ? grid : 1), kThreads, kDynSmem, s>>>(a, rows);
    DPPO_CHECK_LAUNCH("grpo_loss tile launch");
    return DPPO_OK;
}

template <bool kF32>
static int launch_tile_dtype(const LossArgs& a, int nvec, cudaStream_t s, bool launch) {
    if (nvec <= 32) return launch_tile_t<kF32, 1>(a, s, launch);
    if (nvec <= 64) return launch_tile_t<kF32, 2>(a, s, launch);
    return launch_tile_t<kF32, 4>(a, s, launch);
}

// Dense rows, with dlogits or forward only: V a whole number of 16-byte vectors, the row pitch a multiple of 16 bytes and at
// most 32 KB, both matrices 16-byte aligned.  DPPO_ERR_UNSUPPORTED (nothing launched) otherwise.
int launch_rows_tile(const LossArgs& a, cudaStream_t s, bool launch) {
    const int per_vec = a.bf16 ? 8 : 4;
    if (a.V < per_vec || a.V % per_vec != 0) return fail(DPPO_ERR_UNSUPPORTED, "tile kernel: V=%d is not a whole number of 16-byte vectors", a.V);
    if (a.row_bytes % 16 != 0 || a.row_bytes > kStageBytes || a.row_bytes < (long long)a.V * (a.bf16 ? 2 : 4))
        return fail(DPPO_ERR_UNSUPPORTED, "tile kernel: row pitch of %lld bytes", a.row_bytes);
    if ((((uintptr_t)a.logits) | ((uintptr_t)a.dlogits)) & 15) return fail(DPPO_ERR_UNSUPPORTED, "tile kernel: matrices not 16-byte aligned");   // dlogits may be null
    const int nvec = a.V / per_vec;
    return a.bf16 ? launch_tile_dtype<false>(a, nvec, s, launch) : launch_tile_dtype<true>(a, nvec, s, launch);
}

}  // namespace dppo
