// Dense Prompt Packing (Section 4.3): window-based greedy packing of the retained units into rows.
//
// The packer is sequential by nature — every pick depends on the space the previous pick left — so it
// runs as ONE warp.  The pool W never has to be materialised: units enter it in stream order and
// leave it without reordering, so at any time W = { unplaced stream positions j < min(n, N_win +
// #placed) } and "pool order" is position order.  The warp therefore keeps a placed-bitmask in
// shared memory and finds the pick with a ballot over 32 positions at a time, starting at the lowest
// unplaced position.  Stream compaction (keep mask -> stream) and the cu_seqlens scan ride along.
#include "common.cuh"

namespace dppo {

constexpr int kPackMaxUnits = 1 << 21;         // units per call (a dataset of two million prompts)
constexpr int kPackSmemMask = 65536;           // up to this n_max the placed-bitmask (2048 words) sits in shared memory,
                                               // above it in the caller's workspace
constexpr int kPackSmemLens = 8192;            // stream lengths in a static shared array up to this n_max (stream in global)
constexpr int kPackSmemAll = 16384;            // stream, lengths and loss tokens all in dynamic shared memory up to this
                                               // n_max (192 KB): covers a dataset of 7.5-8.5 k prompts packed at set-up

struct PackWorkspace {                         // carved from the caller's workspace
    int32_t* stream;                           // i32 [n_max]: unit index of stream position j
    int32_t* slen;                             // i32 [n_max]: its length
    uint32_t* mask;                            // [n_max / 32] placed-bitmask, only for n_max > kPackSmemMask
};

template <bool kLensInSmem, bool kStreamInSmem, bool kMaskInSmem = true>
__global__ void __launch_bounds__(32)
pack_prompts_kernel(dppo_pack_params prm, const int32_t* __restrict__ len,
                    const uint8_t* __restrict__ keep, const int32_t* __restrict__ loss_len,
                    int32_t* __restrict__ order, int32_t* __restrict__ row_of,
                    int32_t* __restrict__ off_in_row, int32_t* __restrict__ row_fill,
                    int32_t* __restrict__ cu_seqlens, int32_t* __restrict__ counts,
                    PackWorkspace ws, int32_t* status) {
    __shared__ uint32_t placed_smem[kMaskInSmem ? kPackSmemMask / 32 : 1];
    uint32_t* placed = kMaskInSmem ? placed_smem : ws.mask;
    __shared__ int32_t lens_static[(kLensInSmem && !kStreamInSmem) ? kPackSmemLens : 1];
    extern __shared__ int32_t pack_dyn[];                      // kStreamInSmem: stream, loss tokens, lengths, [n_max] each
    int32_t* stream_s = pack_dyn;
    int32_t* sloss_s = pack_dyn + prm.n_max;
    int32_t* lens_smem = kStreamInSmem ? pack_dyn + 2 * prm.n_max : lens_static;
    const int lane = threadIdx.x;
    const int n_max = prm.n_max, L = prm.L_row;

    // ---- stream compaction, validation, output defaults
    int n = 0;
    long long total_tokens = 0;
    bool bad = false;
    for (int base = 0; base < n_max; base += 32) {
        const int u = base + lane;
        const bool in = u < n_max && (keep == nullptr || keep[u] != 0);
        const int l = in ? len[u] : 0;
        if (u < n_max) { order[u] = -1; row_of[u] = -1; off_in_row[u] = -1; row_fill[u] = 0; }
        const unsigned m = __ballot_sync(0xffffffffu, in);
        if (in) {
            const int pos = n + __popc(m & ((1u << lane) - 1u));
            if (kStreamInSmem) { stream_s[pos] = u; sloss_s[pos] = loss_len ? loss_len[u] : l; } else ws.stream[pos] = u;
            if (kLensInSmem) lens_smem[pos] = l; else ws.slen[pos] = l;
            bad = bad || l < 1 || l > L;
        }
        n += __popc(m);
        long long t = l;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        total_tokens += t;
    }
    for (int w = lane; w < (n + 31) / 32; w += 32) placed[w] = 0u;
    bad = __any_sync(0xffffffffu, bad) || total_tokens > 0x7fffffffLL;   // the token counts are reported as i32
    __syncwarp();
    if (bad) {
        if (lane == 0) { set_status(status, DPPO_STATUS_BAD_LENGTH); counts[0] = counts[1] = counts[2] = counts[3] = 0; }
        for (int p = lane; p <= n_max; p += 32) cu_seqlens[p] = 0;
        return;
    }
    const int32_t* slen = kLensInSmem ? lens_smem : ws.slen;

    // ---- greedy placement
    int n_placed = 0, lo = 0, row = 0, remaining = L, loss_cum = 0;
    if (kStreamInSmem && prm.policy == 0) {
        // Batch-sized streams, first-fit: as long as the pool lies within 64 stream positions from `base` (a
        // multiple of 32 at or below the oldest unplaced unit), lane i keeps positions base + i and base + 32 + i
        // in registers (length, unit index, loss tokens) and the two placed-masks are warp-uniform registers.  A
        // placement is then ballot -> ffs -> two shuffles, with no shared-memory round trip on its dependent
        // chain.  A wider pool (large N_win, or many later units placed over a waiting one) leaves this loop for
        // the general one below, which continues from the same state.
        int base = 0;
        int lenA, lenB, uA, uB, lsA, lsB;
        uint32_t pA = 0u, pB = 0u;
        auto load_block = [&](int b0, int& len_r, int& u_r, int& ls_r) {
            const int j = b0 + lane;
            const bool in = j < n;
            len_r = in ? lens_smem[j] : 0x7fffffff;
            u_r = in ? stream_s[j] : -1;
            ls_r = in ? sloss_s[j] : 0;
        };
        load_block(0, lenA, uA, lsA);
        load_block(32, lenB, uB, lsB);
        while (n_placed < n) {
            const int fetched = min(n, prm.N_win + n_placed);
            if (fetched - base > 64) break;
            const int jA = base + lane, jB = jA + 32;
            bool in_b = false;
            unsigned m = __ballot_sync(0xffffffffu, jA >= lo && jA < fetched && !((pA >> lane) & 1u) && lenA <= remaining);
            if (!m) {
                in_b = true;
                m = __ballot_sync(0xffffffffu, jB >= lo && jB < fetched && !((pB >> lane) & 1u) && lenB <= remaining);
            }
            if (!m) {                                            // nothing in W fits: close the row
                if (lane == 0) row_fill[row] = L - remaining;
                ++row;
                remaining = L;
                continue;
            }
            const int src = __ffs(m) - 1;
            const int l = __shfl_sync(0xffffffffu, in_b ? lenB : lenA, src);
            const int ls = __shfl_sync(0xffffffffu, in_b ? lsB : lsA, src);
            if (lane == src) {                                   // the lane that holds the unit writes its placement
                const int u = in_b ? uB : uA;
                order[n_placed] = u;
                row_of[u] = row;
                off_in_row[u] = L - remaining;
                cu_seqlens[n_placed] = loss_cum;
            }
            if (in_b) pB |= 1u << src; else pA |= 1u << src;
            loss_cum += ls;
            remaining -= l;
            ++n_placed;
            if (base + (in_b ? 32 : 0) + src == lo) {            // the oldest unit went: next unplaced position
                ++lo;
                if (lo < base + 32) {
                    const uint32_t w = ~pA & (0xffffffffu << (lo - base));
                    lo = w ? base + __ffs(w) - 1 : base + 32;
                }
                if (lo >= base + 32 && lo < base + 64) {
                    const uint32_t w = ~pB & (0xffffffffu << (lo - base - 32));
                    lo = w ? base + 32 + __ffs(w) - 1 : base + 64;
                }
                lo = min(lo, n);
                while (lo >= base + 32 && lo < n) {              // block A is used up: slide the window by 32
                    if (lane == 0) placed[base >> 5] = pA;
                    base += 32;
                    lenA = lenB; uA = uB; lsA = lsB; pA = pB;
                    load_block(base + 32, lenB, uB, lsB);
                    pB = 0u;
                }
            }
        }
        if (lane == 0) { placed[base >> 5] = pA; placed[(base >> 5) + 1] = pB; }   // state for the general loop
        __syncwarp();
    }
    while (n_placed < n) {
        const int fetched = min(n, prm.N_win + n_placed);       // stream positions that have entered W
        int pick = -1;
        if (prm.policy == 0) {                                   // first unit in pool order that fits
            for (int base = lo & ~31; base < fetched; base += 32) {
                const int j = base + lane;
                const bool ok = j >= lo && j < fetched && !((placed[j >> 5] >> (j & 31)) & 1u) && slen[j] <= remaining;
                const unsigned m = __ballot_sync(0xffffffffu, ok);
                if (m) { pick = base + __ffs(m) - 1; break; }
            }
        } else {                                                 // longest unit that fits, ties to the oldest
            long long best = -1;                                 // (len << 32) | (0x7fffffff - j)
            for (int base = lo & ~31; base < fetched; base += 32) {
                const int j = base + lane;
                const bool ok = j >= lo && j < fetched && !((placed[j >> 5] >> (j & 31)) & 1u) && slen[j] <= remaining;
                long long key = ok ? (((long long)slen[j] << 32) | (long long)(0x7fffffff - j)) : -1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
                best = max(best, key);
            }
            if (best >= 0) pick = 0x7fffffff - (int)(best & 0xffffffffLL);
        }
        if (pick < 0) {                                          // nothing in W fits: close the row
            if (lane == 0) row_fill[row] = L - remaining;
            ++row;
            remaining = L;
            continue;
        }
        const int l = slen[pick];
        if (lane == 0) {
            const int u = kStreamInSmem ? stream_s[pick] : ws.stream[pick];
            order[n_placed] = u;
            row_of[u] = row;
            off_in_row[u] = L - remaining;
            cu_seqlens[n_placed] = loss_cum;
            placed[pick >> 5] |= 1u << (pick & 31);
            loss_cum += kStreamInSmem ? sloss_s[pick] : (loss_len ? loss_len[u] : l);
        }
        loss_cum = __shfl_sync(0xffffffffu, loss_cum, 0);
        __syncwarp();
        remaining -= l;
        ++n_placed;
        if (pick == lo) {                                        // advance to the next unplaced position
            ++lo;
            while (lo < n) {
                const uint32_t w = ~placed[lo >> 5] & (0xffffffffu << (lo & 31));
                if (w) { lo = (lo & ~31) + __ffs(w) - 1; break; }
                lo = (lo & ~31) + 32;
            }
            lo = min(lo, n);
        }
    }
    const int n_rows = n > 0 ? row + 1 : 0;
    if (lane == 0) {
        if (n > 0) row_fill[row] = L - remaining;
        counts[0] = n; counts[1] = n_rows; counts[2] = (int32_t)total_tokens; counts[3] = loss_cum;
    }
    for (int p = n + lane; p <= n_max; p += 32) cu_seqlens[p] = loss_cum;
}

static size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }
constexpr int kMaxDevices = 64;

// ---- scratch for dppo_pack_prompts_static ------------------------------------------------------
// Lives in the library's device image: every GPU that loads the library holds these 32 KB until the
// process exits.  It holds the stream (the unit index of every stream position); the lengths of the stream sit
// in shared memory for streams of this size.
constexpr int kPackStaticMaxUnits = 8192;
static_assert(kPackStaticMaxUnits <= kPackSmemLens, "the static-scratch packer keeps the stream's lengths in shared memory");
static __device__ __align__(256) int32_t g_pack_static_scratch[kPackStaticMaxUnits];

static int32_t* g_pack_static_ptr[kMaxDevices];          // device address of the array, per device ordinal; it
                                                         // outlives neither cudaDeviceReset nor a new context

// Device address of the scratch array on the current device.  In host code the array's name is only a
// handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress, asked once per
// device with that device current.
static int pack_static_scratch(int32_t** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "pack_prompts_static: cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return fail(DPPO_ERR_UNSUPPORTED, "pack_prompts_static: device ordinal %d", dev);
    int32_t* p = __atomic_load_n(&g_pack_static_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        void* sym = nullptr;
        e = cudaGetSymbolAddress(&sym, g_pack_static_scratch);
        if (e != cudaSuccess || sym == nullptr) return cuda_fail(e, "pack_prompts_static: cudaGetSymbolAddress");
        p = static_cast<int32_t*>(sym);
        __atomic_store_n(&g_pack_static_ptr[dev], p, __ATOMIC_RELEASE);   // racing threads store the same value
    }
    *out = p;
    return DPPO_OK;
}

}  // namespace dppo

extern "C" size_t dppo_pack_workspace_bytes(const dppo_pack_params* p) {
    if (!p || p->n_max < 0 || p->n_max > dppo::kPackMaxUnits) return 0;
    const size_t n = (size_t)(p->n_max > 0 ? p->n_max : 1);
    return 2 * dppo::align_up(n * sizeof(int32_t)) + (p->n_max > dppo::kPackSmemMask ? dppo::align_up((n + 31) / 32 * 4) : 0);
}

extern "C" int dppo_pack_prompts(const dppo_pack_params* p, const int32_t* len, const uint8_t* keep,
                                 const int32_t* loss_len, int32_t* order, int32_t* row_of,
                                 int32_t* off_in_row, int32_t* row_fill, int32_t* cu_seqlens,
                                 int32_t* counts, void* workspace, size_t workspace_bytes,
                                 int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_pack_prompts");
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "pack_prompts: NULL params");
    if (p->n_max < 0 || p->L_row < 1 || p->N_win < 1 || (p->policy != 0 && p->policy != 1))
        return fail(DPPO_ERR_INVALID_ARG, "pack_prompts: n_max=%d L_row=%d N_win=%d policy=%d", p->n_max,
                    p->L_row, p->N_win, p->policy);
    if (p->n_max > kPackMaxUnits)
        return fail(DPPO_ERR_BAD_SHAPE, "pack_prompts: n_max=%d above the limit %d", p->n_max, kPackMaxUnits);
    if (!cu_seqlens || !counts) return fail(DPPO_ERR_INVALID_ARG, "pack_prompts: NULL cu_seqlens/counts");
    if (p->n_max > 0 && (!len || !order || !row_of || !off_in_row || !row_fill))
        return fail(DPPO_ERR_INVALID_ARG, "pack_prompts: NULL array");
    const size_t need = dppo_pack_workspace_bytes(p);
    if (!workspace || workspace_bytes < need)
        return fail(DPPO_ERR_WORKSPACE_TOO_SMALL, "pack_prompts: workspace %zu < %zu bytes", workspace_bytes, need);
    if (((uintptr_t)workspace & 15) != 0) return fail(DPPO_ERR_MISALIGNED, "pack_prompts: workspace not 16-byte aligned");
    const size_t per_array = align_up((size_t)(p->n_max > 0 ? p->n_max : 1) * sizeof(int32_t));
    PackWorkspace ws;
    ws.stream = (int32_t*)workspace;
    ws.slen = (int32_t*)((char*)workspace + per_array);
    ws.mask = (uint32_t*)((char*)workspace + 2 * per_array);          // used above kPackSmemMask units only
    cudaStream_t s = (cudaStream_t)stream;
    if (p->n_max <= kPackSmemAll) {
        // batch-sized streams: the stream and its loss-token counts sit in shared memory too, so a placement
        // costs shared-memory latency instead of two dependent global loads
        const size_t dyn = (size_t)(p->n_max > 0 ? p->n_max : 1) * 3 * sizeof(int32_t);
        // the limit is raised once per device to the largest size any call may ask for (a per-call value could be
        // lowered by another host thread between this thread's set and its launch)
        static bool raised[kMaxDevices];
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); dev = -1; }
        if (dev < 0 || !raised[dev]) {
            cudaError_t e = cudaFuncSetAttribute(pack_prompts_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)(kPackSmemAll * 3 * sizeof(int32_t)));
            if (e != cudaSuccess) return cuda_fail(e, "pack_prompts: shared memory attribute");
            if (dev >= 0) raised[dev] = true;
        }
        pack_prompts_kernel<true, true><<<1, 32, dyn, s>>>(*p, len, keep, loss_len, order, row_of, off_in_row, row_fill,
                                                         cu_seqlens, counts, ws, status);
    } else if (p->n_max <= kPackSmemMask)
        pack_prompts_kernel<false, false><<<1, 32, 0, s>>>(*p, len, keep, loss_len, order, row_of, off_in_row, row_fill,
                                                    cu_seqlens, counts, ws, status);
    else
        pack_prompts_kernel<false, false, false><<<1, 32, 0, s>>>(*p, len, keep, loss_len, order, row_of, off_in_row,
                                                                  row_fill, cu_seqlens, counts, ws, status);
    DPPO_CHECK_LAUNCH("pack_prompts launch");
    return DPPO_OK;
}

extern "C" int dppo_pack_static_max_units(void) { return dppo::kPackStaticMaxUnits; }

extern "C" int dppo_pack_prompts_static(const dppo_pack_params* p, const int32_t* len, const uint8_t* keep,
                                        const int32_t* loss_len, int32_t* order, int32_t* row_of,
                                        int32_t* off_in_row, int32_t* row_fill, int32_t* cu_seqlens,
                                        int32_t* counts, int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_pack_prompts_static");
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "pack_prompts_static: NULL params");
    if (p->n_max < 0 || p->L_row < 1 || p->N_win < 1 || (p->policy != 0 && p->policy != 1))
        return fail(DPPO_ERR_INVALID_ARG, "pack_prompts_static: n_max=%d L_row=%d N_win=%d policy=%d", p->n_max,
                    p->L_row, p->N_win, p->policy);
    if (p->n_max > kPackStaticMaxUnits)
        return fail(DPPO_ERR_BAD_SHAPE, "pack_prompts_static: n_max=%d exceeds the built-in scratch (%d units); "
                    "use dppo_pack_prompts with a caller workspace", p->n_max, kPackStaticMaxUnits);
    if (!cu_seqlens || !counts) return fail(DPPO_ERR_INVALID_ARG, "pack_prompts_static: NULL cu_seqlens/counts");
    if (p->n_max > 0 && (!len || !order || !row_of || !off_in_row || !row_fill))
        return fail(DPPO_ERR_INVALID_ARG, "pack_prompts_static: NULL array");
    int32_t* scratch = nullptr;
    const int rc = pack_static_scratch(&scratch);
    if (rc != DPPO_OK) return rc;
    PackWorkspace ws;
    ws.stream = scratch;
    ws.slen = nullptr;                                       // lengths: shared memory in this instantiation
    ws.mask = nullptr;                                       // bitmask: shared memory at this size
    // Nothing in the scratch has to start at zero: the kernel writes every stream slot it later reads.
    pack_prompts_kernel<true, false><<<1, 32, 0, (cudaStream_t)stream>>>(*p, len, keep, loss_len, order, row_of, off_in_row,
                                                                  row_fill, cu_seqlens, counts, ws, status);
    DPPO_CHECK_LAUNCH("pack_prompts_static launch");
    return DPPO_OK;
}
