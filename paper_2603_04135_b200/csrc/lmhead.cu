// Fused LM-head + GRPO loss on the 5th-generation tensor cores.
//
// The call walks over the tokens in chunks.  Per chunk:
//   logits    z = hidden W^T, tile by tile (tcgen05.mma, accumulators in tensor memory).  As each 128 x 256
//             tile leaves TMEM its per-row (max, sum of exponentials) and the sampled token's logit are kept;
//             a backward pass also keeps the exponentials themselves, relative to the tile's row maxima, as
//             fp16 in a bounded scratch (the [T x V] logits never exist in memory, not even for one chunk;
//             Eq. 1's pi_theta(o_t | ...) is a log-softmax of exactly these f32 accumulators)
//   rows      one warp per token joins the tile partials into the log-sum-exp and runs the loss's scalar stage
//   dlogits   D = g (onehot - softmax)/tau of the chunk as bf16: the stored exponentials times one factor per
//             (token, tile), no second exp
//   dhidden = D W and dW += D^T hidden: two more runs of the same GEMM core over the chunk
//
// One GEMM core serves all three contractions; an operand is K-major or MN-major as stored (W, hidden and D
// are never copied transposed), only the epilogue differs.  One persistent CTA per SM, by default paired with
// its neighbour (cta_group::2, see lm_gemm2_kernel); in the single-CTA form:
//   warp 0      TMA producer: 64-deep K slabs of A (128 rows) and of B (256 rows), 128B-swizzled, into
//               a 4-stage shared-memory ring (every CTA fetches its own operands)
//   warp 1      one thread issues tcgen05.mma (M=128, N=256, K=16 x 4 per slab) into one of two
//               256-column TMEM accumulators; tcgen05.commit releases smem stages / publishes the tile
//   warps 2-5   epilogue: each thread owns one row of the tile and reads it 32 columns at a time with
//               tcgen05.ld; while it drains accumulator b the MMA warp already fills accumulator 1-b
// Every wait is bounded; on a timeout the CTA records DPPO_STATUS_TIMEOUT, leaves its loops, frees its
// tensor memory and returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "common.cuh"
#include "grpo_loss.cuh"

namespace dppo {

constexpr int kBM = 128;                 // rows per tile (TMEM lanes)
constexpr int kBN = 256;                 // columns per tile (TMEM columns of one accumulator)
constexpr int kBK = 64;                  // K slab: 64 bf16 = one 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kStageBytesA = kBM * kBK * 2;                  // 16 KB
constexpr int kStageBytesB = kBN * kBK * 2;                  // 32 KB
constexpr int kStageBytes = kStageBytesA + kStageBytesB;
constexpr int kLmThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kChunkTokens = 9472;       // tokens whose dlogits are held in scratch at a time: 74 row tiles, so the
                                         // dhidden GEMM of a chunk has 74 x H/256 tiles = whole waves on 148 SMs
constexpr int kMaxChunkTokens = 1 << 16;

// Launch-shape choices of the call, by hidden width (from sweeps on B200 at 99,030 tokens, V = 151,936).
struct LmTune {
    int chunk_tokens;                    // tokens whose dlogits are held at a time (a multiple of 256: whole row-tile pairs)
    int sub_tokens;                      // the logits, dlogits and dW launches take a chunk in pieces of about this size
    int group_logits;                    // column tiles per group of the logits launch (0: all row tiles of two column tiles at a time)
    int group_dw;                        // the same for the dW launch (0: all column tiles of a few row tiles at a time)
    int hints;                           // two bits each (kHint...): loads of logits A, B; dhidden A, B; dW A, B; then the
                                         // stores of the exponentials and the add-reductions of dW
};
static LmTune lm_tune(int H) {
    // The hidden rows of a piece are re-read by every wave of the logits and dW launches and should stay in L2
    // between them: a piece holds at most about 48 MB of them (9472 rows at H = 2560: one piece per chunk; H = 4096:
    // two pieces of 4864 and 4608 rows, 288 ms against 300 ms for the whole call).  Chunks of 18,944 tokens, pieces of
    // a third or a quarter of a chunk, grouped tile orders and eviction hints on the loads or on the stores of the
    // exponentials and of dW were all measured within 1 % of this choice or slower.
    LmTune t = {kChunkTokens, kChunkTokens, 0, 0, 0};
    const long long rows_48mb = (48500000ll / (2ll * (H > 0 ? H : 1))) / 256 * 256;
    if (rows_48mb < kChunkTokens) t.sub_tokens = (int)(rows_48mb < 256 ? 256 : rows_48mb);
    return t;
}

struct LmShared {
    unsigned long long full[kStages];    // TMA bytes have landed in stage s
    unsigned long long empty[kStages];   // the MMAs reading stage s are done
    unsigned long long acc_full[2];      // accumulator b holds a finished tile
    unsigned long long acc_empty[2];     // the epilogue has drained accumulator b (4 warps arrive)
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ uint32_t lm_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long lm_global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool lm_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

// Bounded wait; also leaves when another role has raised the abort flag.  The clock and the flag are looked at once
// per sixteen tries (a try already suspends the thread for a short, hardware-chosen time), not per try.
__device__ __forceinline__ bool lm_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns) {
    if (lm_try(bar, parity)) return true;
    const unsigned long long t0 = lm_global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 16; ++i)
            if (lm_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (lm_global_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
}

// Bounded wait that ignores the abort flag (used on the way out).
__device__ __forceinline__ bool lm_wait_plain(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    if (lm_try(bar, parity)) return true;
    const unsigned long long t0 = lm_global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 16; ++i)
            if (lm_try(bar, parity)) return true;
        if (lm_global_ns() - t0 > limit_ns) return false;
    }
}

__device__ __forceinline__ void lm_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ float lm_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptors (descriptor version 1 = sm_100, layout type 2 = SWIZZLE_128B; addresses and
// offsets in 16-byte units).  Both layouts are made of 1024-byte swizzle atoms, 8 rows of 128 bytes, exactly as a
// 128B-swizzled TMA box with a 64-element inner extent lands them:
//   K-major   a row of the atom is 64 K-elements of one M/N index; the tile is one box of 64 K x (128 or 256)
//             rows, so 8-row groups are 1024 bytes apart (stride offset); the leading offset is unused.  The
//             next 16 K-elements are 32 bytes further along the row.
//   MN-major  a row of the atom is 64 consecutive M/N indices of one K index (the operand is stored with its
//             M/N index contiguous, i.e. it is used transposed without a transposed copy); one box holds
//             64 K x 64 M/N = 8 atoms stacked along K, 1024 bytes apart (stride offset), and the boxes of
//             successive 64-wide M/N blocks follow each other 8192 bytes apart (leading offset).  The next
//             16 K-elements are two atoms = 2048 bytes further.
constexpr int kMnBoxBytes = kBK * 64 * 2;                // 8 KB: 64 K-rows of 64 M/N elements
__device__ __forceinline__ uint64_t lm_smem_desc_k(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t lm_smem_desc_mn(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3FFF) | ((uint64_t)(kMnBoxBytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
template <bool kMn> __device__ __forceinline__ uint64_t lm_smem_desc(uint32_t smem_addr) {
    return kMn ? lm_smem_desc_mn(smem_addr) : lm_smem_desc_k(smem_addr);
}
template <bool kMn> __host__ __device__ constexpr uint64_t lm_desc_kstep() { return kMn ? (uint64_t)(2048 >> 4) : (uint64_t)(32 >> 4); }

// Instruction descriptor of kind::f16: D = f32, A = B = bf16, N = 256, M = 128 (256 for a CTA pair); bits 15 / 16
// say that A / B is MN-major.
template <bool kAMn, bool kBMn, int kM> __host__ __device__ constexpr uint32_t lm_idesc() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((kAMn ? 1u : 0u) << 15) | ((kBMn ? 1u : 0u) << 16) |
           ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kM >> 4) << 24);
}

// L2 eviction policy of an operand's loads: a tile that other CTAs (or later waves) will ask for again is kept
// (evict_last), one that is streamed through once makes room first (evict_first).
enum { kHintNone = 0, kHintEvictFirst = 1, kHintEvictLast = 2 };
__device__ __forceinline__ uint64_t lm_l2_policy(int hint) {
    uint64_t pol = 0;
    if (hint == kHintEvictFirst) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else if (hint == kHintEvictLast) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// One tiled TMA load (x = innermost coordinate, 16-byte aligned by construction: multiples of 64 elements).
// pol = 0: no hint.
__device__ __forceinline__ void lm_tma_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, uint64_t pol) {
    if (pol)
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
                     :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// The same from a CTA of a pair: the barrier may be the peer's (the pair's leader collects both CTAs' bytes).
__device__ __forceinline__ void lm_tma_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, uint64_t pol) {
    if (pol)
        asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
                     :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                     :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

// What a launch of the GEMM core covers, and the order in which its tiles are handed out.  Work item j of a CTA
// (or CTA pair) is id = its index + j * (number of CTAs or pairs); ids are laid over the n_m x n_ntiles grid of
// work items (n_m = row tiles, or row-tile pairs for CTA pairs) as
//   group == 0:  m_fast ? (m = id % n_m, n = id / n_m) : (m = id / n_ntiles, n = id % n_ntiles)
//   group  > 0:  column tiles are taken `group` at a time; within a group the ids sweep over all m with n fastest.
//                The CTAs that run together then share `group` B tiles and about (CTAs / group) A tiles: a working
//                set that fits L2 whatever the size of A, and every B tile is fetched from HBM once per launch.
struct GemmShape {
    int n_mtiles, n_ntiles, n_ksteps;
    int a_row0;                          // row offset added to A's TMA coordinate
    int m_fast;
    int group;
    int hint_a, hint_b;                  // L2 eviction hints of the operand loads (kHint...)
    int hint_c;                          // and of the epilogue's tiled stores / add-reductions
    unsigned long long wait_limit_ns;    // bound of every wait on a pipeline barrier
    int test_extra_tx;                   // 0; self-test of the bounded waits: bytes the first stage expects but never gets
};

__device__ __forceinline__ bool tile_from_id(const GemmShape& gs, long long id, int n_m, int& m, int& n) {
    if (id >= (long long)n_m * gs.n_ntiles) return false;
    if (gs.group > 0) {
        const long long per_group = (long long)gs.group * n_m;
        const int grp = (int)(id / per_group);
        const int local = (int)(id - (long long)grp * per_group);
        const int n0 = grp * gs.group;
        const int width = min(gs.group, gs.n_ntiles - n0);         // the last group may be narrower
        m = local / width; n = n0 + local % width;
    } else if (gs.m_fast) { m = (int)(id % n_m); n = (int)(id / n_m); }
    else                  { m = (int)(id / gs.n_ntiles); n = (int)(id % gs.n_ntiles); }
    return true;
}

__device__ __forceinline__ bool tile_of(const GemmShape& gs, uint32_t j, int& m, int& n) {
    return tile_from_id(gs, (long long)blockIdx.x + (long long)j * gridDim.x, gs.n_mtiles, m, n);
}

// ---- epilogue output through shared memory ---------------------------------------------------------
// An epilogue thread holds 32 consecutive f32 of ONE row, so direct stores make every warp instruction touch
// 32 different lines.  Instead each epilogue warp stages its 32 x 32 block (4 KB, rows of 128 bytes, 16-byte
// chunks XOR-swizzled with the row so that the staging writes are conflict-free) and lane 0 hands it to the
// TMA unit as one tiled store -- or a tiled f32 add-reduction -- which writes whole 128-byte runs and clips
// at the tensor's edges.  Two staging buffers per warp: the block being drained and the block being filled.
constexpr int kStageTileBytes = 32 * 32 * 4;
constexpr int kStageBytesEpi = 4 * 2 * kStageTileBytes;  // 4 epilogue warps x 2 buffers = 32 KB

struct EpiCtx {
    const CUtensorMap* map_c;            // f32 [rows x cols], 32 x 32 boxes, 128B swizzle
    uint64_t pol;                        // L2 eviction policy of the tiled stores (0: none)
    uint32_t stage;                      // this warp's two staging buffers (shared::cta address, 1024-aligned)
    uint32_t toggle;
    int lane;
};

// Block of 32 rows x 32 f32 at (column x, row y) of the tensor behind map_c; v = this lane's row.
template <bool kAdd>
__device__ __forceinline__ void lm_store_block(EpiCtx& ctx, const uint32_t (&v)[32], int x, int y) {
    if (ctx.lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the buffer filled two blocks ago has been read
    __syncwarp();
    const uint32_t buf = ctx.stage + ctx.toggle * kStageTileBytes;
    const uint32_t rowp = buf + (uint32_t)ctx.lane * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     :: "r"(rowp + (uint32_t)((j ^ (ctx.lane & 7)) << 4)), "r"(v[4 * j]), "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3])
                     : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (ctx.lane == 0) {
        if (kAdd) {
            if (ctx.pol)
                asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                             :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y), "l"(ctx.pol) : "memory");
            else
                asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                             :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y) : "memory");
        } else {
            if (ctx.pol)
                asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                             :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y), "l"(ctx.pol) : "memory");
            else
                asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                             :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y) : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    ctx.toggle ^= 1u;
}

// The same staging for 2-byte elements: a block of 32 rows x 64 fp16 (again rows of 128 bytes) is filled in two
// halves, 32 columns each (h = this lane's row of the half, 16 words of two fp16); the second half sends it.
__device__ __forceinline__ void lm_store_half_block(EpiCtx& ctx, const uint32_t (&h)[16], int half, int x, int y) {
    if (half == 0) {
        if (ctx.lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the buffer filled two blocks ago has been read
        __syncwarp();
    }
    const uint32_t buf = ctx.stage + ctx.toggle * kStageTileBytes;
    const uint32_t rowp = buf + (uint32_t)ctx.lane * 128u;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     :: "r"(rowp + (uint32_t)(((4 * half + j) ^ (ctx.lane & 7)) << 4)), "r"(h[4 * j]), "r"(h[4 * j + 1]), "r"(h[4 * j + 2]), "r"(h[4 * j + 3])
                     : "memory");
    if (half == 0) return;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (ctx.lane == 0) {
        if (ctx.pol)
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                         :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y), "l"(ctx.pol) : "memory");
        else
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                         :: "l"(ctx.map_c), "r"(buf), "r"(x), "r"(y) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    ctx.toggle ^= 1u;
}

// 32 consecutive f32 columns of this thread's TMEM lane (its tile row) into registers.
__device__ __forceinline__ void lm_tmem_load32(uint32_t (&v)[32], uint32_t taddr) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---- the GEMM core --------------------------------------------------------------------------------
// Epi (one copy per epilogue thread = per tile row), called for every tile:
//   void row_begin(int m, int n, int row)
//   void chunk(int m, int n, int row, int ch, uint32_t (&v)[32], EpiCtx& ctx)   32 accumulator columns (f32 bits)
//   void row_end(int m, int n, int row)
template <class Epi, bool kAMn, bool kBMn>
__global__ void __launch_bounds__(kLmThreads, 1)
lm_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c,
               const GemmShape gs, const Epi epi_args, int32_t* status) {
    extern __shared__ unsigned char lm_raw[];
    __shared__ LmShared sh;
    const uint32_t tiles = (lm_smem_u32(lm_raw) + 1023u) & ~1023u;      // 1024-byte aligned ring (swizzle atoms)
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sh.abort;

    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < kStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.empty[s])));
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.acc_full[b])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" :: "r"(lm_smem_u32(&sh.acc_empty[b])));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                                     // tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(lm_smem_u32(&sh.tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_a = lm_l2_policy(gs.hint_a), pol_b = lm_l2_policy(gs.hint_b);
            uint32_t it = 0;                                             // slab counter over the CTA's lifetime
            int m, n;
            for (uint32_t j = 0; tile_of(gs, j, m, n) && !*abort_flag; ++j) {
                for (int k = 0; k < gs.n_ksteps; ++k, ++it) {
                    const uint32_t s = it % kStages, use = it / kStages;
                    if (use > 0 && !lm_wait(lm_smem_u32(&sh.empty[s]), (use - 1) & 1, abort_flag, gs.wait_limit_ns)) break;
                    const uint32_t bar = lm_smem_u32(&sh.full[s]);
                    const uint32_t dst_a = tiles + s * kStageBytes, dst_b = dst_a + kStageBytesA;
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 :: "r"(bar), "r"((uint32_t)kStageBytes + (it == 0 ? (uint32_t)gs.test_extra_tx : 0u)) : "memory");
                    if (!kAMn) {
                        lm_tma_2d(dst_a, &map_a, bar, k * kBK, gs.a_row0 + m * kBM, pol_a);
                    } else {
#pragma unroll
                        for (int i = 0; i < kBM / 64; ++i) lm_tma_2d(dst_a + i * kMnBoxBytes, &map_a, bar, m * kBM + 64 * i, k * kBK, pol_a);
                    }
                    if (!kBMn) {
                        lm_tma_2d(dst_b, &map_b, bar, k * kBK, n * kBN, pol_b);
                    } else {
#pragma unroll
                        for (int i = 0; i < kBN / 64; ++i) lm_tma_2d(dst_b + i * kMnBoxBytes, &map_b, bar, n * kBN + 64 * i, k * kBK, pol_b);
                    }
                }
            }
            if (*abort_flag) {
                // leaving early: give this thread's own copies in flight a bounded chance to land before
                // the CTA (and its shared memory) goes away
                const uint32_t pending = it < (uint32_t)kStages ? it : (uint32_t)kStages;
                for (uint32_t i = 0; i < pending; ++i) {
                    const uint32_t i2 = it - 1 - i;
                    lm_wait_plain(lm_smem_u32(&sh.full[i2 % kStages]), (i2 / kStages) & 1, gs.wait_limit_ns);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0;
            int m, n;
            for (uint32_t j = 0; tile_of(gs, j, m, n) && !*abort_flag; ++j) {
                const uint32_t b = j & 1, use_b = j >> 1;
                if (use_b > 0 && !lm_wait(lm_smem_u32(&sh.acc_empty[b]), (use_b - 1) & 1, abort_flag, gs.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + b * kBN;
                bool ok = true;
                for (int k = 0; k < gs.n_ksteps; ++k, ++it) {
                    const uint32_t s = it % kStages, use = it / kStages;
                    if (!lm_wait(lm_smem_u32(&sh.full[s]), use & 1, abort_flag, gs.wait_limit_ns)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = tiles + s * kStageBytes, sb = sa + kStageBytesA;
                    const uint64_t da = lm_smem_desc<kAMn>(sa), db = lm_smem_desc<kBMn>(sb);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {              // 16 K elements per instruction
                        const uint32_t accumulate = (k > 0 || kk > 0) ? 1u : 0u;
                        asm volatile("{\n\t.reg .pred p;\n\t"
                                     "setp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                     :: "r"(d_tmem), "l"(da + kk * lm_desc_kstep<kAMn>()), "l"(db + kk * lm_desc_kstep<kBMn>()),
                                        "r"(lm_idesc<kAMn, kBMn, kBM>()), "r"(accumulate) : "memory");
                    }
                    // frees this smem stage once the MMAs issued so far have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 :: "r"(lm_smem_u32(&sh.empty[s])) : "memory");
                }
                if (!ok) break;
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             :: "r"(lm_smem_u32(&sh.acc_full[b])) : "memory");
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                                          // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        Epi epi = epi_args;                                              // per-thread copy: its state lives in registers
        EpiCtx ctx;
        ctx.map_c = &map_c; ctx.pol = lm_l2_policy(gs.hint_c);
        ctx.stage = tiles + kStages * kStageBytes + (uint32_t)q * (2 * kStageTileBytes);
        ctx.toggle = 0; ctx.lane = lane;
        int m, n;
        for (uint32_t j = 0; tile_of(gs, j, m, n); ++j) {
            const uint32_t b = j & 1, use_b = j >> 1;
            epi.row_begin(m, n, row);
            // warp-uniform outcome: the tcgen05.ld below must be executed by all 32 lanes together
            if (!__all_sync(0xffffffffu, lm_wait(lm_smem_u32(&sh.acc_full[b]), use_b & 1, abort_flag, gs.wait_limit_ns))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * kBN;
            if constexpr (Epi::kTwoPass) {                               // a first look at the whole tile (its row maxima)
#pragma unroll 1
                for (int ch = 0; ch < kBN / 32; ++ch) {
                    uint32_t v[32];
                    lm_tmem_load32(v, taddr + (uint32_t)(ch * 32));
                    epi.scan(m, n, row, ch, v);
                }
            }
#pragma unroll 1
            for (int ch = 0; ch < kBN / 32; ++ch) {
                uint32_t v[32];
                lm_tmem_load32(v, taddr + (uint32_t)(ch * 32));
                epi.chunk(m, n, row, ch, v, ctx);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) lm_arrive(lm_smem_u32(&sh.acc_empty[b]));
            epi.row_end(m, n, row);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's tiled stores are complete
    }

    // ---- common exit: nobody touches tensor memory any more, then the allocating warp frees it
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && sh.abort) set_status(status, DPPO_STATUS_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

// ---- the GEMM core on CTA pairs (cta_group::2) -------------------------------------------------------
// Two CTAs of a cluster share one 256 x 256 tile: each loads its own 128 rows of A and HALF of the B tile
// (128 rows), the leader's MMA thread issues tcgen05.mma.cta_group::2 (M = 256) which reads both halves of B
// from the two CTAs' shared memory and writes each CTA's 128 rows into that CTA's tensor memory.  Per SM
// and K slab this is 32 KB of operands instead of 48 KB for the same flops.  TMA loads signal the
// leader's `full` barrier (every CTA fetches its own operands); the tcgen05.commit arrivals go to both CTAs'
// barriers; both
// epilogues report to the leader's `acc_empty`.
constexpr int kStages2 = 6;
constexpr int kHalfBN = kBN / 2;
constexpr int kStageBytesB2 = kHalfBN * kBK * 2;             // 16 KB
constexpr int kStageBytes2 = kStageBytesA + kStageBytesB2;   // 32 KB per CTA
constexpr uint32_t kPeerMask = 0xFEFFFFFFu;                  // shared::cluster address of the pair's leader (rank bit cleared)

struct LmShared2 {
    unsigned long long full[kStages2];
    unsigned long long empty[kStages2];
    unsigned long long acc_full[2];
    unsigned long long acc_empty[2];     // the leader's copy counts 8 arrivals: 4 epilogue warps x 2 CTAs
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ bool pair_tile_of(const GemmShape& gs, uint32_t j, int& m2, int& n) {
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    return tile_from_id(gs, (long long)pair + (long long)j * npairs, (gs.n_mtiles + 1) >> 1, m2, n);
}

__device__ __forceinline__ void lm_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <class Epi, bool kAMn, bool kBMn>
__global__ void __launch_bounds__(kLmThreads, 1)
lm_gemm2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_c,
                const GemmShape gs, const Epi epi_args, int32_t* status) {
    extern __shared__ unsigned char lm_raw[];
    __shared__ LmShared2 sh;
    const uint32_t tiles = (lm_smem_u32(lm_raw) + 1023u) & ~1023u;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const bool leader = rank == 0;
    volatile int* abort_flag = &sh.abort;

    if (tid == 0) {
        sh.abort = 0;
        for (int s = 0; s < kStages2; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.empty[s])));
        }
        for (int b = 0; b < 2; ++b) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(lm_smem_u32(&sh.acc_full[b])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 8;" :: "r"(lm_smem_u32(&sh.acc_empty[b])));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                                     // both CTAs, same warp, same destination
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(lm_smem_u32(&sh.tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    lm_cluster_sync();                                                   // the peer's barriers and tensor memory exist
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            const uint64_t pol_a = lm_l2_policy(gs.hint_a), pol_b = lm_l2_policy(gs.hint_b);
            uint32_t it = 0;
            int m2, n;
            for (uint32_t j = 0; pair_tile_of(gs, j, m2, n) && !*abort_flag; ++j) {
                const int m = 2 * m2 + (int)rank;
                for (int k = 0; k < gs.n_ksteps; ++k, ++it) {
                    const uint32_t s = it % kStages2, use = it / kStages2;
                    if (use > 0 && !lm_wait(lm_smem_u32(&sh.empty[s]), (use - 1) & 1, abort_flag, gs.wait_limit_ns)) break;
                    const uint32_t bar_local = lm_smem_u32(&sh.full[s]);
                    const uint32_t bar = bar_local & kPeerMask;           // the leader's barrier collects both CTAs' bytes
                    const uint32_t dst_a = tiles + s * kStageBytes2, dst_b = dst_a + kStageBytesA;
                    if (leader)
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                     :: "r"(bar_local), "r"((uint32_t)(2 * kStageBytes2) + (it == 0 ? (uint32_t)gs.test_extra_tx : 0u)) : "memory");
                    if (!kAMn) {
                        lm_tma_2d_pair(dst_a, &map_a, bar, k * kBK, gs.a_row0 + m * kBM, pol_a);
                    } else {
#pragma unroll
                        for (int i = 0; i < kBM / 64; ++i) lm_tma_2d_pair(dst_a + i * kMnBoxBytes, &map_a, bar, m * kBM + 64 * i, k * kBK, pol_a);
                    }
                    const int nb0 = n * kBN + (int)rank * kHalfBN;       // this CTA's half of the B tile
                    if (!kBMn) {
                        lm_tma_2d_pair(dst_b, &map_b, bar, k * kBK, nb0, pol_b);
                    } else {
#pragma unroll
                        for (int i = 0; i < kHalfBN / 64; ++i) lm_tma_2d_pair(dst_b + i * kMnBoxBytes, &map_b, bar, nb0 + 64 * i, k * kBK, pol_b);
                    }
                }
            }
            if (*abort_flag && leader) {
                // leaving early: the leader's `full` barriers count the copies of both CTAs, so the leader gives the
                // copies still in flight a bounded chance to land; its peer cannot leave before it (the cluster
                // barrier on the way out), so neither CTA's shared memory goes away under a copy
                const uint32_t pending = it < (uint32_t)kStages2 ? it : (uint32_t)kStages2;
                for (uint32_t i = 0; i < pending; ++i) {
                    const uint32_t i2 = it - 1 - i;
                    lm_wait_plain(lm_smem_u32(&sh.full[i2 % kStages2]), (i2 / kStages2) & 1, gs.wait_limit_ns);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            uint32_t it = 0;
            int m2, n;
            for (uint32_t j = 0; pair_tile_of(gs, j, m2, n) && !*abort_flag; ++j) {
                const uint32_t b = j & 1, use_b = j >> 1;
                if (use_b > 0 && !lm_wait(lm_smem_u32(&sh.acc_empty[b]), (use_b - 1) & 1, abort_flag, gs.wait_limit_ns)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + b * kBN;
                bool ok = true;
                for (int k = 0; k < gs.n_ksteps; ++k, ++it) {
                    const uint32_t s = it % kStages2, use = it / kStages2;
                    if (!lm_wait(lm_smem_u32(&sh.full[s]), use & 1, abort_flag, gs.wait_limit_ns)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t sa = tiles + s * kStageBytes2, sb = sa + kStageBytesA;
                    const uint64_t da = lm_smem_desc<kAMn>(sa), db = lm_smem_desc<kBMn>(sb);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        const uint32_t accumulate = (k > 0 || kk > 0) ? 1u : 0u;
                        asm volatile("{\n\t.reg .pred p;\n\t"
                                     "setp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                     :: "r"(d_tmem), "l"(da + kk * lm_desc_kstep<kAMn>()), "l"(db + kk * lm_desc_kstep<kBMn>()),
                                        "r"(lm_idesc<kAMn, kBMn, 2 * kBM>()), "r"(accumulate) : "memory");
                    }
                    // frees this stage in BOTH CTAs once the MMAs issued so far have read it
                    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                                 :: "r"(lm_smem_u32(&sh.empty[s])), "h"((unsigned short)3) : "memory");
                }
                if (!ok) break;
                asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                             :: "r"(lm_smem_u32(&sh.acc_full[b])), "h"((unsigned short)3) : "memory");
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int q = warp & 3;
        const int row = q * 32 + lane;
        Epi epi = epi_args;
        EpiCtx ctx;
        ctx.map_c = &map_c; ctx.pol = lm_l2_policy(gs.hint_c);
        ctx.stage = tiles + kStages2 * kStageBytes2 + (uint32_t)q * (2 * kStageTileBytes);
        ctx.toggle = 0; ctx.lane = lane;
        int m2, n;
        for (uint32_t j = 0; pair_tile_of(gs, j, m2, n); ++j) {
            const int m = 2 * m2 + (int)rank;
            const uint32_t b = j & 1, use_b = j >> 1;
            epi.row_begin(m, n, row);
            if (!__all_sync(0xffffffffu, lm_wait(lm_smem_u32(&sh.acc_full[b]), use_b & 1, abort_flag, gs.wait_limit_ns))) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * kBN;
            if constexpr (Epi::kTwoPass) {                               // a first look at the whole tile (its row maxima)
#pragma unroll 1
                for (int ch = 0; ch < kBN / 32; ++ch) {
                    uint32_t v[32];
                    lm_tmem_load32(v, taddr + (uint32_t)(ch * 32));
                    epi.scan(m, n, row, ch, v);
                }
            }
#pragma unroll 1
            for (int ch = 0; ch < kBN / 32; ++ch) {
                uint32_t v[32];
                lm_tmem_load32(v, taddr + (uint32_t)(ch * 32));
                epi.chunk(m, n, row, ch, v, ctx);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)                                               // the leader's MMA thread waits for all 8 warps
                asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" :: "r"(lm_smem_u32(&sh.acc_empty[b]) & kPeerMask) : "memory");
            epi.row_end(m, n, row);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---- common exit: both CTAs are done with tensor memory and with each other's barriers, then free
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    lm_cluster_sync();
    if (tid == 0 && sh.abort) set_status(status, DPPO_STATUS_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

// ---- epilogues ------------------------------------------------------------------------------------
struct RowInfo {             // what the backward needs from the forward, per token
    float lse2_hi, lse2_lo;  // base-2 log-sum-exp of z * scale2
    float f;                 // dlogits[t, v] = -f * E'[t, v]: f = (dloss/dlogp / temperature) * 2^(ref - lse2); 0 for rows
                             // that add nothing (no token, bad target, out of range)
    int y;                   // target, -1 if the row is invalid
};

// Forward, one chunk of tokens: each 128 x 256 logits tile leaves behind, per token row, the tile's
// (max, sum 2^(x - max)) of x = z * scale2 and the sampled token's logit if it lies in the tile.  The tiles of a
// row are combined by lm_rows_kernel.  This form keeps nothing else (forward-only calls).
struct EpiPartial {
    static constexpr bool kTwoPass = false;
    float2* part;            // [chunk tokens x n_ntiles]
    float* zy_out;           // [chunk tokens]
    const int32_t* target;
    const int32_t* n_tokens_dev;
    long long T_max, t0, tc;
    int V, n_ntiles;
    float c;
    // per-thread state
    float m2, s, zy;
    int y;
    bool live, hit;
    __device__ __forceinline__ void row_begin(int m, int, int row) {
        const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
        const long long r = (long long)m * kBM + row;
        live = r < tc && t0 + r < T;
        y = live ? target[t0 + r] : -1;
        m2 = -INFINITY; s = 0.0f; zy = 0.0f; hit = false;
    }
    __device__ __forceinline__ void chunk(int m, int n, int row, int ch, uint32_t (&v)[32], EpiCtx& ctx) {
        const int col0 = n * kBN + ch * 32;
        const int valid = V - col0;                                  // columns of this chunk inside the vocabulary
        if (valid <= 0 || !live) return;
        const int yrel = y - col0;                                   // selects, not an indexed read: v stays in registers
        hit = hit || (yrel >= 0 && yrel < 32);
        float cm = -INFINITY;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const float raw = __uint_as_float(v[j]);
            zy = (j == yrel) ? raw : zy;
            const float x = (j < valid) ? raw * c : -INFINITY;
            v[j] = __float_as_uint(x);
            cm = fmaxf(cm, x);
        }
        if (cm > m2) { s *= lm_ex2(m2 - cm); m2 = cm; }
        float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            acc0 += lm_ex2(__uint_as_float(v[j]) - m2);
            acc1 += lm_ex2(__uint_as_float(v[j + 1]) - m2);
        }
        s += acc0 + acc1;
    }
    __device__ __forceinline__ void row_end(int m, int n, int row) {
        if (!live) return;
        const long long r = (long long)m * kBM + row;
        part[r * n_ntiles + n] = make_float2(m2, s);
        if (hit) zy_out[r] = zy;
    }
};

// The same for a call with a backward pass.  The exponentials are formed ONCE, relative to a per-row reference
// that is known before the GEMM starts: the sampled token's own logit (ref2[t] = scale2 * hidden[t] . W[y_t],
// one dot product per token, see lm_ref_kernel).  e = 2^(x - ref2) is added up for the log-sum-exp and kept, as
// bf16, in a chunk-sized scratch E' [chunk tokens x V]; the f32 logits are never written out.  Because the
// reference is the same for a whole row, softmax = e * 2^(ref2 - lse2) is a ROW scaling of E', and so is the
// gradient: with the one entry E'[t, y_t] replaced by e_y - 2^(lse2 - ref2) (lm_rows_ref_kernel),
//     dlogits[t, :] = -f_t * E'[t, :],   f_t = (dloss/dlogp / temperature) * 2^(ref2 - lse2).
// The two gradient contractions therefore read E' itself: dhidden = -diag(f) (E' W) scales the accumulator rows
// in its epilogue, dW = E'^T (-diag(f) hidden) takes pre-scaled hidden rows (kept transposed: the token axis is
// the contraction's K).  No dlogits pass, no second copy.
// The row maximum is never below the sampled token's logit, so e >= 1 for the largest entry; bf16 has the exponent
// range of f32, and the exponent is clamped at 100 so that sums of V such entries times weights stay far from the
// f32 overflow in the two contractions.  A row counts as in range while its sum stays below 2^96, i.e. while its
// sampled token has a log-prob above about -66 (any token a sampler could have drawn); rows beyond that are
// reported by the rows kernel and get a zero gradient.
constexpr float kMaxExp2 = 100.0f;
constexpr float kMaxRowSum = 7.9e28f;        // 2^96

struct EpiExpRef {
    static constexpr bool kTwoPass = false;
    float* sums;             // [piece tokens x n_ntiles] sum of e over the tile's columns
    float* zy_out;           // [piece tokens]
    const float* ref2;       // [T] the rows' references
    const int32_t* target;
    const int32_t* n_tokens_dev;
    long long T_max, t0, tc;
    int V, n_ntiles;
    float c;
    // per-thread state
    float nref, s, zy;
    int y;
    bool live, hit;
    __device__ __forceinline__ void row_begin(int m, int, int row) {
        const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
        const long long r = (long long)m * kBM + row;
        live = r < tc && t0 + r < T;
        y = live ? target[t0 + r] : -1;
        nref = live ? -ref2[t0 + r] : 0.0f;
        s = 0.0f; zy = 0.0f; hit = false;
    }
    __device__ __forceinline__ void chunk(int m, int n, int row, int ch, uint32_t (&v)[32], EpiCtx& ctx) {
        const int col0 = n * kBN + ch * 32;
        const int valid = live ? V - col0 : 0;                       // rows without a token are written as zeros
        const int y0 = m * kBM + row - ctx.lane;                     // first row of this warp's block
        if (y0 >= tc || V - (col0 & ~63) <= 0) return;               // nothing of this 64-column block exists (whole warp)
        const int yrel = y - col0;
        hit = hit || (yrel >= 0 && yrel < 32);
        uint32_t h[16];
        float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            const float r0 = __uint_as_float(v[j]), r1 = __uint_as_float(v[j + 1]);
            zy = (j == yrel) ? r0 : zy;
            zy = (j + 1 == yrel) ? r1 : zy;
            const float e0 = (j < valid) ? lm_ex2(fminf(fmaf(r0, c, nref), kMaxExp2)) : 0.0f;
            const float e1 = (j + 1 < valid) ? lm_ex2(fminf(fmaf(r1, c, nref), kMaxExp2)) : 0.0f;
            acc0 += e0; acc1 += e1;
            const __nv_bfloat162 p = __floats2bfloat162_rn(e0, e1);
            h[j >> 1] = *reinterpret_cast<const uint32_t*>(&p);
        }
        s += acc0 + acc1;
        lm_store_half_block(ctx, h, ch & 1, col0 & ~63, y0);        // clipped at V and at the piece's last row
    }
    __device__ __forceinline__ void row_end(int m, int n, int row) {
        if (!live) return;
        const long long r = (long long)m * kBM + row;
        sums[r * n_ntiles + n] = s;
        if (hit) zy_out[r] = zy;
    }
};

// The rows' references for a backward call: ref2[t] = scale2 * (hidden[t] . W[y_t]) in f32, one warp per token
// (0 for a row without a token or with a target outside the vocabulary).  It only has to be NEAR the logit the
// tensor cores will produce for that entry: any value works as a reference, the log-prob itself uses the GEMM's.
__global__ void __launch_bounds__(256)
lm_ref_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ W, const int32_t* __restrict__ target,
              const int32_t* __restrict__ n_tokens_dev, long long T_max, int V, int H, float c, float* __restrict__ ref2) {
    const long long t = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (t >= T_max) return;
    const long long T = n_tokens_dev ? min((long long)*n_tokens_dev, T_max) : T_max;
    const int y = t < T ? target[t] : -1;
    if (y < 0 || y >= V) { if (lane == 0) ref2[t] = 0.0f; return; }
    const uint4* hr = reinterpret_cast<const uint4*>(hidden + t * H);
    const uint4* wr = reinterpret_cast<const uint4*>(W + (long long)y * H);
    float acc = 0.0f;
    for (int i = lane; i < H / 8; i += 32) {                         // H is a multiple of 64
        const uint4 a = hr[i], b = wr[i];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc = fmaf(__uint_as_float(aw[k] << 16), __uint_as_float(bw[k] << 16), acc);
            acc = fmaf(__uint_as_float(aw[k] & 0xffff0000u), __uint_as_float(bw[k] & 0xffff0000u), acc);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) ref2[t] = acc * c;
}

// One warp per token of the chunk: the row's tile partials -> base-2 log-sum-exp, then the loss's scalar
// stage (lane 0) -> per-row loss terms, logp, lse and what the backward needs.
constexpr int kRowsWarps = 8;

__global__ void __launch_bounds__(kRowsWarps * 32)
lm_rows_kernel(const LossArgs a, const float2* __restrict__ part, const float* __restrict__ zy,
               long long t0, long long tc, int n_ntiles) {
    const long long r = (long long)blockIdx.x * kRowsWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= tc) return;
    const long long t = t0 + r;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    if (t >= T) return;                                              // no token here
    float M = -INFINITY, S = 0.0f;
    for (int i = lane; i < n_ntiles; i += 32) {
        const float2 q = part[r * n_ntiles + i];                     // every tile holds a vocabulary column: q.x is finite
        const float Mn = fmaxf(M, q.x);
        S = (M == -INFINITY ? 0.0f : S * lm_ex2(M - Mn)) + q.y * lm_ex2(q.x - Mn);
        M = Mn;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float Mo = __shfl_xor_sync(0xffffffffu, M, o), So = __shfl_xor_sync(0xffffffffu, S, o);
        const float Mn = fmaxf(M, Mo);
        S = (M == -INFINITY ? 0.0f : S * lm_ex2(M - Mn)) + (Mo == -INFINITY ? 0.0f : So * lm_ex2(Mo - Mn));
        M = Mn;
    }
    if (lane == 0) {
        RowInputs in;
        row_gather(a, t, in, false);
        if (in.state == 0) in.zy = (double)zy[r] / a.temperature;
        row_finish(a, t, in, M, S, true);
    }
}

// Backward: one warp per token of the piece.  The tile sums of the row -> base-2 log-sum-exp (reference + log2 of
// their sum, added in a fixed order), the loss's scalar stage (lane 0), then what turns E' into the gradient:
// the row factor f and the replacement of the sampled token's entry.  A row whose sum has left the range of the reference (the sampled token's log-prob below about -66) is
// reported as DPPO_STATUS_RANGE, adds nothing to the loss and gets a zero gradient.
__global__ void __launch_bounds__(kRowsWarps * 32)
lm_rows_ref_kernel(const LossArgs a, const float* __restrict__ sums, const float* __restrict__ zy,
                   const float* __restrict__ ref2, RowInfo* __restrict__ info, long long t0, long long tc, int n_ntiles,
                   __nv_bfloat16* __restrict__ E, long long lde) {
    const long long r = (long long)blockIdx.x * kRowsWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= tc) return;
    const long long t = t0 + r;
    const long long T = a.n_tokens_dev ? min((long long)*a.n_tokens_dev, a.T_max) : a.T_max;
    if (t < T) {
        float S = 0.0f;
        for (int i = lane; i < n_ntiles; i += 32) S += sums[r * n_ntiles + i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xffffffffu, S, o);
        if (lane == 0) {
            const float ref = ref2[t];
            RowInfo ri; ri.lse2_hi = 0.0f; ri.lse2_lo = 0.0f; ri.f = 0.0f; ri.y = -1;
            RowInputs in;
            row_gather(a, t, in, false);
            // log2(S) is how far the log-sum-exp lies above the reference; S >= about 1 since the row holds the
            // sampled token's own entry
            const bool in_range = S > 0.0f && S < kMaxRowSum;         // no entry of the row reached the clamp
            if (in.state == 0 && !in_range) {
                set_status(a.status, DPPO_STATUS_RANGE);
                const RowTerms zero = {0.0, 0.0, 0.0, 0.0};
                a.terms[t] = zero;
                if (a.logp_out) a.logp_out[t] = 0.0f;
                if (a.lse_out) a.lse_out[t] = 0.0f;
            } else {
                if (in.state == 0) in.zy = (double)zy[r] / a.temperature;
                const RowScalars rs = row_finish(a, t, in, ref, in_range ? S : 1.0f, true);
                if (rs.valid && rs.g_over_tau != 0.0f) {
                    ri.lse2_hi = rs.lse2_hi; ri.lse2_lo = rs.lse2_lo; ri.y = in.y;
                    ri.f = rs.g_over_tau * lm_ex2((ref - rs.lse2_hi) - rs.lse2_lo);
                    // the sampled token's entry carries the onehot term: -f (e_y - 2^(lse2 - ref)) = g - f e_y
                    const float ey = lm_ex2(fminf(fmaf(zy[r], a.scale2, -ref), kMaxExp2));
                    E[r * lde + in.y] = __float2bfloat16_rn(ey - lm_ex2((rs.lse2_hi - ref) + rs.lse2_lo));
                }
            }
            info[t] = ri;
        }
    } else if (lane == 0) {                                            // no token here: the backward sees f = 0
        RowInfo z; z.lse2_hi = 0.0f; z.lse2_lo = 0.0f; z.f = 0.0f; z.y = -1;
        info[t] = z;
    }
}

// The piece's operand of the dW contraction, K-major (the token axis contiguous, which is what the tensor core
// reads fastest): hsT[k, r] = -f[t0 + r] * hidden[t0 + r, k] as bf16, row pitch ld (a multiple of 64; the columns
// tc .. ld - 1 are written as zeros).  One CTA transposes a tile of 64 tokens x 64 hidden columns through
// shared memory: 16-byte loads along the hidden rows, 16-byte stores along the token axis.
constexpr int kTrTile = 64;
__global__ void __launch_bounds__(256)
lm_scaled_hidden_t_kernel(const __nv_bfloat16* __restrict__ hidden, const RowInfo* __restrict__ info, long long t0,
                          long long tc, int H, __nv_bfloat16* __restrict__ hsT, long long ld) {
    __shared__ __align__(16) unsigned short tile[kTrTile][kTrTile + 8];          // [hidden column][token], padded rows
    const long long r0 = (long long)blockIdx.x * kTrTile;
    const int k0 = blockIdx.y * kTrTile;
    for (int v = threadIdx.x; v < kTrTile * (kTrTile / 8); v += 256) {
        const int row = v >> 3, kv = (v & 7) * 8;
        const long long r = r0 + row;
        float nf = 0.0f;
        if (r < tc) nf = -info[t0 + r].f;
        uint4 x = make_uint4(0u, 0u, 0u, 0u);
        if (nf != 0.0f && k0 + kv < H) x = *reinterpret_cast<const uint4*>(hidden + (t0 + r) * H + k0 + kv);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(nf * __uint_as_float(w[k] << 16), nf * __uint_as_float(w[k] & 0xffff0000u));
            const uint32_t o = nf != 0.0f ? *reinterpret_cast<const uint32_t*>(&b2) : 0u;
            tile[kv + 2 * k][row] = (unsigned short)(o & 0xffffu);
            tile[kv + 2 * k + 1][row] = (unsigned short)(o >> 16);
        }
    }
    __syncthreads();
    for (int v = threadIdx.x; v < kTrTile * (kTrTile / 8); v += 256) {
        const int k = v >> 3, rv = (v & 7) * 8;
        if (k0 + k < H && r0 + rv < ld)
            *reinterpret_cast<uint4*>(hsT + (long long)(k0 + k) * ld + r0 + rv) = *reinterpret_cast<const uint4*>(&tile[k][rv]);
    }
}

// C[rows x ldc] = -f[row] * acc as bf16 (dhidden: the accumulator is E' W, the row factor turns E' into dlogits).
struct EpiStoreScaledBf16 {
    static constexpr bool kTwoPass = false;
    __nv_bfloat16* C;
    const RowInfo* info;         // per token; indexed by output row
    long long ldc, row0, rows;   // output row of tile row 0; rows that exist in C
    int cols;
    float nf;
    __device__ __forceinline__ void row_begin(int m, int, int row) {
        const long long r = row0 + (long long)m * kBM + row;
        nf = r < rows ? -info[r].f : 0.0f;
    }
    __device__ __forceinline__ void chunk(int m, int n, int row, int ch, uint32_t (&v)[32], EpiCtx&) {
        const long long r = row0 + (long long)m * kBM + row;
        const int col0 = n * kBN + ch * 32;
        if (r >= rows || col0 >= cols) return;
        __nv_bfloat16* dst = C + r * ldc + col0;
        if (col0 + 32 <= cols) {
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const __nv_bfloat162 b2 = __floats2bfloat162_rn(nf * __uint_as_float(v[2 * j]), nf * __uint_as_float(v[2 * j + 1]));
                pk[j] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            uint4* d4 = reinterpret_cast<uint4*>(dst);
            d4[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            d4[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            d4[2] = make_uint4(pk[8], pk[9], pk[10], pk[11]);
            d4[3] = make_uint4(pk[12], pk[13], pk[14], pk[15]);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) if (col0 + j < cols) dst[j] = __float2bfloat16_rn(nf * __uint_as_float(v[j]));
        }
    }
    __device__ __forceinline__ void row_end(int, int, int) {}
};

// C (f32, the tensor behind the kernel's output map) = or += acc (dW, accumulated over the token chunks; the
// add is done by the memory system, nothing is read back).
struct EpiAccumF32 {
    static constexpr bool kTwoPass = false;
    long long rows;
    int cols, accumulate;
    __device__ __forceinline__ void row_begin(int, int, int) {}
    __device__ __forceinline__ void chunk(int m, int n, int row, int ch, uint32_t (&v)[32], EpiCtx& ctx) {
        const int col0 = n * kBN + ch * 32;
        const int y0 = m * kBM + row - ctx.lane;                     // first row of this warp's block
        if (y0 >= rows || col0 >= cols) return;                      // the same for the whole warp
        if (accumulate) lm_store_block<true>(ctx, v, col0, y0);
        else            lm_store_block<false>(ctx, v, col0, y0);
    }
    __device__ __forceinline__ void row_end(int, int, int) {}
};

// out (bf16) = in (f32), 8 elements per thread; n is a multiple of 8.
__global__ void __launch_bounds__(256)
lm_f32_to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, long long n) {
    const long long i = ((long long)blockIdx.x * 256 + threadIdx.x) * 8;
    if (i >= n) return;
    const float4 a = *reinterpret_cast<const float4*>(in + i), b = *reinterpret_cast<const float4*>(in + i + 4);
    const __nv_bfloat162 b0 = __floats2bfloat162_rn(a.x, a.y), b1 = __floats2bfloat162_rn(a.z, a.w);
    const __nv_bfloat162 b2 = __floats2bfloat162_rn(b.x, b.y), b3 = __floats2bfloat162_rn(b.z, b.w);
    uint4 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&b0); pk.y = *reinterpret_cast<const uint32_t*>(&b1);
    pk.z = *reinterpret_cast<const uint32_t*>(&b2); pk.w = *reinterpret_cast<const uint32_t*>(&b3);
    *reinterpret_cast<uint4*>(out + i) = pk;
}

// out (f32) = in (bf16), 8 elements per thread; n is a multiple of 8.
__global__ void __launch_bounds__(256)
lm_bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ in, float* __restrict__ out, long long n) {
    const long long i = ((long long)blockIdx.x * 256 + threadIdx.x) * 8;
    if (i >= n) return;
    const uint4 q = *reinterpret_cast<const uint4*>(in + i);
    *reinterpret_cast<float4*>(out + i) = make_float4(__uint_as_float(q.x << 16), __uint_as_float(q.x & 0xffff0000u),
                                                       __uint_as_float(q.y << 16), __uint_as_float(q.y & 0xffff0000u));
    *reinterpret_cast<float4*>(out + i + 4) = make_float4(__uint_as_float(q.z << 16), __uint_as_float(q.z & 0xffff0000u),
                                                           __uint_as_float(q.w << 16), __uint_as_float(q.w & 0xffff0000u));
}

// ---- host side -----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 [rows x cols] with row pitch ld elements; boxes of 64 columns x box_rows rows, 128B swizzle, zero fill
// outside [rows x cols].
static int make_map(CUtensorMap* map, const void* base, long long rows, long long cols, long long ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled failed with %d", (int)r);
    return DPPO_OK;
}

// f32 [rows x cols] with row pitch ld elements as the target of the epilogue's tiled stores: 32 x 32 boxes
// (128-byte rows), 128B swizzle.
static int make_map_out(CUtensorMap* map, const void* base, long long rows, long long cols, long long ld) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled (output) failed with %d", (int)r);
    return DPPO_OK;
}

// bf16 [rows x cols] with row pitch ld elements as the target of the half-block stores: boxes of 64 columns x 32
// rows (128-byte rows), 128B swizzle.
static int make_map_out_bf16(CUtensorMap* map, const void* base, long long rows, long long cols, long long ld) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {64, 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(DPPO_ERR_CUDA, "lmhead: cuTensorMapEncodeTiled (exponentials) failed with %d", (int)r);
    return DPPO_OK;
}

constexpr size_t kLmDynSmem = (size_t)kStages * kStageBytes + kStageBytesEpi + 1024;

template <class Epi, bool kAMn, bool kBMn>
static int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmShape& gs, const Epi& epi,
                       int32_t* status, cudaStream_t s, const char* what) {
    auto kernel = lm_gemm_kernel<Epi, kAMn, kBMn>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLmDynSmem);
    if (e != cudaSuccess) return cuda_fail(e, "lmhead: shared memory attribute");
    const long long work = (long long)gs.n_mtiles * gs.n_ntiles;
    const int grid = (int)(work < sm_count() ? work : sm_count());
    if (grid < 1) return DPPO_OK;
    kernel<<<grid, kLmThreads, kLmDynSmem, s>>>(ma, mb, mc, gs, epi, status);
    cudaError_t e2 = cudaGetLastError();
    if (e2 != cudaSuccess) return cuda_fail(e2, what);
    return DPPO_OK;
}

constexpr size_t kLmDynSmem2 = (size_t)kStages2 * kStageBytes2 + kStageBytesEpi + 1024;
static_assert(kLmDynSmem <= 232448 - 256 && kLmDynSmem2 <= 232448 - 256, "ring + staging must fit one CTA's shared memory");

// CTA-pair version: `mb_half` is B's tensor map with 128-row boxes.
template <class Epi, bool kAMn, bool kBMn>
static int launch_gemm2(const CUtensorMap& ma, const CUtensorMap& mb_half, const CUtensorMap& mc, const GemmShape& gs, const Epi& epi,
                        int32_t* status, cudaStream_t s, const char* what) {
    auto kernel = lm_gemm2_kernel<Epi, kAMn, kBMn>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLmDynSmem2);
    if (e != cudaSuccess) return cuda_fail(e, "lmhead: shared memory attribute");
    const long long n_m2 = (gs.n_mtiles + 1) / 2;
    const long long work = n_m2 * gs.n_ntiles;
    const long long max_pairs = sm_count() / 2;
    const int pairs = (int)(work < max_pairs ? work : max_pairs);
    if (pairs < 1) return DPPO_OK;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(kLmThreads, 1, 1);
    cfg.dynamicSmemBytes = kLmDynSmem2;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kernel, ma, mb_half, mc, gs, epi, status);
    if (e != cudaSuccess) return cuda_fail(e, what);
    return DPPO_OK;
}

// An MN-major operand's map has 64 x 64 boxes whatever the tile (mb_half == mb then).  mc: the f32 output of
// the epilogues that store through the TMA unit (any valid map for the others).
template <class Epi, bool kAMn, bool kBMn>
static int run_gemm(bool pair, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mb_half, const CUtensorMap& mc,
                    const GemmShape& gs,
                    const Epi& epi, int32_t* status, cudaStream_t s, const char* what) {
    return pair ? launch_gemm2<Epi, kAMn, kBMn>(ma, mb_half, mc, gs, epi, status, s, what)
                : launch_gemm<Epi, kAMn, kBMn>(ma, mb, mc, gs, epi, status, s, what);
}

static long long round_up(long long x, long long m) { return (x + m - 1) / m * m; }

struct LmWorkspace {
    size_t terms, info, ref, part, zy, e, hs, dw32, total;   // byte offsets and the total
    long long ld_v;                              // pitch of E' (vocabulary)
    int n_ntiles;
};

// A chunk of tc tokens is taken in ceil(tc / sub) pieces of equal size, rounded up to whole row-tile pairs (the
// last piece takes what is left): the size of a piece.
static long long lm_piece_tokens(long long tc, int sub) {
    if (sub < 256) sub = 256;
    const long long n_pieces = (tc + sub - 1) / sub;
    return n_pieces <= 1 ? tc : round_up((tc + n_pieces - 1) / n_pieces, 256);
}

static LmWorkspace lm_layout(const dppo_lmhead_params* p, bool backward) {
    LmWorkspace w;
    const long long T = p->loss.T_max > 0 ? p->loss.T_max : 1;
    auto al = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    const LmTune tune = lm_tune(p->H);
    const size_t rows_d = (size_t)(T < tune.chunk_tokens ? round_up(T, kBM) : tune.chunk_tokens);   // rows of the dlogits scratch
    // rows of the per-piece buffers: no piece of any chunk is longer than the piece size rounded up to a tile pair
    const size_t rows = (size_t)std::min(round_up((long long)rows_d, 256), round_up(std::max(tune.sub_tokens, 256), 256));
    w.ld_v = round_up(p->loss.V, 8);
    w.n_ntiles = (p->loss.V + kBN - 1) / kBN;
    size_t off = 0;
    w.terms = off; off += al(loss_terms_bytes(T));
    w.info = off;  off += al((size_t)T * sizeof(RowInfo));
    w.ref = off;   off += backward ? al((size_t)T * sizeof(float)) : 0;
    w.part = off;  off += al(rows * w.n_ntiles * sizeof(float2));
    w.zy = off;    off += al(rows * sizeof(float));
    w.e = w.hs = w.dw32 = off;
    if (backward) {
        w.e = off;   off += al(rows_d * w.ld_v * 2);                  // E' of a chunk
        w.hs = off;  off += al((size_t)round_up((long long)rows, 64) * (size_t)p->H * 2);   // (-f * hidden)^T of a piece
        if (p->dW_dtype == DPPO_BF16) { w.dw32 = off; off += al((size_t)p->loss.V * p->H * 4); }   // dW is accumulated in f32
    }
    w.total = off;
    return w;
}

}  // namespace dppo

extern "C" size_t dppo_lmhead_workspace_bytes(const dppo_lmhead_params* p) {
    if (!p || p->loss.T_max < 0 || p->loss.V < 1 || p->H < 1) return 0;
    return dppo::lm_layout(p, p->backward != 0).total;
}

extern "C" int dppo_lmhead_grpo_loss(const dppo_lmhead_params* p, const void* hidden, const void* W,
                                     const int32_t* target, const float* logp_old, const float* logp_ref,
                                     const int32_t* cu_seqlens, const int32_t* n_tokens_dev, const float* adv,
                                     const float* w, const int32_t* seg_map, void* dhidden, void* dW,
                                     float* logp_out, float* lse_out, float* loss_out, void* workspace,
                                     size_t workspace_bytes, int32_t* status, void* stream) {
    dppo::NvtxRange nvtx_range("dppo_lmhead_grpo_loss");
    using namespace dppo;
    if (!p) return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL params");
    const dppo_loss_params& lp = p->loss;
    if (lp.T_max < 0 || lp.V < 1 || lp.S_max < 0 || p->H < 1)
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: T_max=%lld V=%d S_max=%d H=%d", (long long)lp.T_max, lp.V, lp.S_max, p->H);
    if (p->H % kBK != 0) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: H=%d must be a multiple of %d", p->H, kBK);
    if (lp.dtype != DPPO_BF16) return fail(DPPO_ERR_UNSUPPORTED, "lmhead: hidden and W must be bf16");
    if (!(lp.temperature > 0.0) || !(lp.eps_lo >= 0.0) || !(lp.eps_hi >= 0.0) || !(lp.beta == lp.beta))
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: temperature must be > 0, eps >= 0, beta a number");
    if ((lp.no_length_norm != 0 && lp.no_length_norm != 1) || (lp.seq_log_ratio && lp.no_length_norm))
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: no_length_norm / seq_log_ratio");
    if (lp.T_max >= ((int64_t)1 << 31) - kMaxChunkTokens) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: T_max too large");
    if (p->variant != 0 && p->variant != 1 && p->variant != 100 && p->variant != 101)
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: variant %d", p->variant);
    if (p->dW_dtype != DPPO_F32 && p->dW_dtype != DPPO_BF16) return fail(DPPO_ERR_INVALID_ARG, "lmhead: dW_dtype %d", p->dW_dtype);
    if ((p->accumulate_dW != 0 && p->accumulate_dW != 1) || p->reserved != 0)
        return fail(DPPO_ERR_INVALID_ARG, "lmhead: accumulate_dW %d reserved %d", p->accumulate_dW, p->reserved);
    const bool backward = p->backward != 0;
    if (backward && (!dhidden || !dW)) return fail(DPPO_ERR_INVALID_ARG, "lmhead: backward requested but dhidden / dW is NULL");
    if (!backward && (dhidden || dW)) return fail(DPPO_ERR_INVALID_ARG, "lmhead: dhidden / dW given but params.backward is 0");
    if (!loss_out) return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL loss_out");
    if (lp.T_max > 0) {
        if (!hidden || !W || !target || !logp_old || !logp_ref || !cu_seqlens || !adv || !w)
            return fail(DPPO_ERR_INVALID_ARG, "lmhead: NULL array");
        if (lp.S_max < 1) return fail(DPPO_ERR_BAD_SHAPE, "lmhead: tokens but no sequences (S_max=0)");
        if (((uintptr_t)hidden & 15) || ((uintptr_t)W & 15) || ((uintptr_t)dhidden & 15) || ((uintptr_t)dW & 15))
            return fail(DPPO_ERR_MISALIGNED, "lmhead: hidden / W / dhidden / dW not 16-byte aligned");
    }
    const LmWorkspace lay = lm_layout(p, backward);
    if (!workspace || workspace_bytes < lay.total)
        return fail(DPPO_ERR_WORKSPACE_TOO_SMALL, "lmhead: workspace %zu < %zu bytes", workspace_bytes, lay.total);
    if ((uintptr_t)workspace & 1023) return fail(DPPO_ERR_MISALIGNED, "lmhead: workspace not 1024-byte aligned");
    char* ws = (char*)workspace;

    LossArgs a;
    a.logits = nullptr; a.dlogits = nullptr;
    a.target = target; a.logp_old = logp_old; a.logp_ref = logp_ref;
    a.cu_seqlens = cu_seqlens; a.n_tokens_dev = n_tokens_dev; a.adv = adv; a.w = w; a.seg_map = seg_map;
    a.logp_out = logp_out; a.lse_out = lse_out; a.terms = (RowTerms*)(ws + lay.terms); a.status = status;
    a.T_max = lp.T_max; a.row_bytes = 0; a.V = lp.V; a.S_max = lp.S_max; a.bf16 = 1;
    a.eps_lo = lp.eps_lo; a.eps_hi = lp.eps_hi; a.beta = lp.beta; a.temperature = lp.temperature;
    a.scale2 = (float)(1.4426950408889634 / lp.temperature);
    a.seq_log_ratio = lp.seq_log_ratio; a.no_length_norm = lp.no_length_norm;
    a.wait_limit_ns = kDefaultWaitLimitNs; a.test_extra_tx = 0;
    cudaStream_t s = (cudaStream_t)stream;
    const int H = p->H, V = lp.V;
    const long long T = lp.T_max;          // host-side bound; rows at or past the device-side count carry g = 0
    if (T > 0) {
        const bool pair = p->variant % 100 != 1;   // CTA pairs sharing the B tile unless the single-CTA core is forced
        const bool self_test = p->variant >= 100;  // every CTA's first pipeline wait runs out (see dppo_lmhead_params.variant)
        GemmShape gs0 = {};
        gs0.wait_limit_ns = self_test ? kSelfTestWaitLimitNs : kDefaultWaitLimitNs;
        gs0.test_extra_tx = self_test ? 16 : 0;
        alignas(64) CUtensorMap map_h, map_w, map_w_half;
        int rc = make_map(&map_h, hidden, T, H, H, kBM);
        if (rc != DPPO_OK) return rc;
        rc = make_map(&map_w, W, V, H, H, kBN);
        if (rc != DPPO_OK) return rc;
        rc = make_map(&map_w_half, W, V, H, H, kHalfBN);
        if (rc != DPPO_OK) return rc;
        RowInfo* info = (RowInfo*)(ws + lay.info);
        float2* part = (float2*)(ws + lay.part);
        float* zy = (float*)(ws + lay.zy);
        __nv_bfloat16* E = (__nv_bfloat16*)(ws + lay.e);                               // E' of the current chunk
        __nv_bfloat16* hs = (__nv_bfloat16*)(ws + lay.hs);
        float* ref2 = (float*)(ws + lay.ref);
        alignas(64) CUtensorMap map_w_mn;                                              // W as [K = V][N = H]
        alignas(64) CUtensorMap map_dw;
        if (backward) {
            rc = make_map(&map_w_mn, W, V, H, H, 64);
            if (rc != DPPO_OK) return rc;
            rc = make_map_out(&map_dw, p->dW_dtype == DPPO_BF16 ? (void*)(ws + lay.dw32) : dW, V, H, H);
            if (rc != DPPO_OK) return rc;
            // the rows' references: the sampled tokens' own logits
            lm_ref_kernel<<<(unsigned)((T + 7) / 8), 256, 0, s>>>((const __nv_bfloat16*)hidden, (const __nv_bfloat16*)W, target,
                                                               n_tokens_dev, T, V, H, a.scale2, ref2);
            DPPO_CHECK_LAUNCH("lmhead reference launch");
            if (p->accumulate_dW && p->dW_dtype == DPPO_BF16) {        // the f32 sum starts from the caller's bf16 dW
                const long long n = (long long)V * H;
                lm_bf16_to_f32_kernel<<<(unsigned)((n / 8 + 255) / 256), 256, 0, s>>>((const __nv_bfloat16*)dW, (float*)(ws + lay.dw32), n);
                DPPO_CHECK_LAUNCH("lmhead dW conversion launch");
            }
        }

        const LmTune tune = lm_tune(H);
        const long long chunk = tune.chunk_tokens;
        long long n_dw = 0;                                                            // dW launches so far
        for (long long t0 = 0; t0 < T; t0 += chunk) {
            const long long tc = (T - t0) < chunk ? (T - t0) : chunk;                   // tokens in this chunk
            const long long piece = lm_piece_tokens(tc, tune.sub_tokens);
            for (long long s0 = t0; s0 < t0 + tc; s0 += piece) {
                const long long ts = (t0 + tc - s0) < piece ? (t0 + tc - s0) : piece;   // tokens in this piece
                const long long hs_ld = round_up(ts, 64);                              // row pitch of (-f hidden)^T
                // (1) logits of the piece, tile by tile.  Forward only: per-tile (max, sum) of every row and z[y].
                //     Backward: the exponentials relative to the rows' references, as bf16, into the piece's rows of
                //     E' [tc x V], their per-tile sums and z[y]
                GemmShape g1 = gs0;
                g1.n_mtiles = (int)((ts + kBM - 1) / kBM); g1.n_ntiles = lay.n_ntiles; g1.n_ksteps = H / kBK;
                g1.a_row0 = (int)s0; g1.m_fast = 1;                                    // neighbours share the W tile
                g1.group = tune.group_logits; g1.hint_a = tune.hints & 3; g1.hint_b = (tune.hints >> 2) & 3;
                g1.hint_c = (tune.hints >> 12) & 3;
                __nv_bfloat16* Ep = E + (s0 - t0) * lay.ld_v;
                if (backward) {
                    EpiExpRef e1 = {};
                    e1.sums = (float*)part; e1.zy_out = zy; e1.ref2 = ref2; e1.target = target; e1.n_tokens_dev = n_tokens_dev;
                    e1.T_max = T; e1.t0 = s0; e1.tc = ts; e1.V = V; e1.n_ntiles = lay.n_ntiles; e1.c = a.scale2;
                    alignas(64) CUtensorMap map_e;
                    rc = make_map_out_bf16(&map_e, Ep, ts, V, lay.ld_v);
                    if (rc != DPPO_OK) return rc;
                    rc = run_gemm<EpiExpRef, false, false>(pair, map_h, map_w, map_w_half, map_e, g1, e1, status, s, "lmhead logits launch");
                } else {
                    EpiPartial e1 = {};
                    e1.part = part; e1.zy_out = zy; e1.target = target; e1.n_tokens_dev = n_tokens_dev;
                    e1.T_max = T; e1.t0 = s0; e1.tc = ts; e1.V = V; e1.n_ntiles = lay.n_ntiles; e1.c = a.scale2;
                    rc = run_gemm<EpiPartial, false, false>(pair, map_h, map_w, map_w_half, map_h, g1, e1, status, s, "lmhead logits launch");
                }
                if (rc != DPPO_OK) return rc;
                // (2) rows: log-sum-exp, logp, loss terms; backward: the row factors f, the sampled tokens' entries of
                //     E' and the piece's -f * hidden
                if (!backward) {
                    lm_rows_kernel<<<(unsigned)((ts + kRowsWarps - 1) / kRowsWarps), kRowsWarps * 32, 0, s>>>(
                        a, part, zy, s0, ts, lay.n_ntiles);
                    DPPO_CHECK_LAUNCH("lmhead rows launch");
                    continue;
                }
                lm_rows_ref_kernel<<<(unsigned)((ts + kRowsWarps - 1) / kRowsWarps), kRowsWarps * 32, 0, s>>>(
                    a, (const float*)part, zy, ref2, info, s0, ts, lay.n_ntiles, Ep, lay.ld_v);
                DPPO_CHECK_LAUNCH("lmhead rows launch");
                lm_scaled_hidden_t_kernel<<<dim3((unsigned)(hs_ld / kTrTile), (unsigned)((H + kTrTile - 1) / kTrTile)), 256, 0, s>>>(
                    (const __nv_bfloat16*)hidden, info, s0, ts, H, hs, hs_ld);
                DPPO_CHECK_LAUNCH("lmhead transposed operand launch");
                // (3) dW (+)= E'^T (-f hidden)[s0 : s0+ts, :]   (M = V, N = H, K = tokens of the piece; E' MN-major,
                //     (-f hidden)^T K-major); the K range stops at the piece: both maps have ts tokens and fill with
                //     zeros beyond
                alignas(64) CUtensorMap map_e_mn, map_hs_k, map_hs_k_half;
                rc = make_map(&map_e_mn, Ep, ts, V, lay.ld_v, 64);
                if (rc != DPPO_OK) return rc;
                rc = make_map(&map_hs_k, hs, H, ts, hs_ld, kBN);
                if (rc != DPPO_OK) return rc;
                rc = make_map(&map_hs_k_half, hs, H, ts, hs_ld, kHalfBN);
                if (rc != DPPO_OK) return rc;
                GemmShape g3 = gs0;
                g3.n_mtiles = (V + kBM - 1) / kBM; g3.n_ntiles = (H + kBN - 1) / kBN; g3.n_ksteps = (int)((ts + kBK - 1) / kBK);
                g3.group = tune.group_dw; g3.hint_a = (tune.hints >> 8) & 3; g3.hint_b = (tune.hints >> 10) & 3;
                g3.hint_c = (tune.hints >> 14) & 3;
                EpiAccumF32 e3 = {};
                e3.rows = V; e3.cols = H; e3.accumulate = (n_dw > 0 || p->accumulate_dW) ? 1 : 0;
                rc = run_gemm<EpiAccumF32, true, false>(pair, map_e_mn, map_hs_k, map_hs_k_half, map_dw, g3, e3, status, s, "lmhead dW launch");
                if (rc != DPPO_OK) return rc;
                ++n_dw;
            }
            if (!backward) continue;
            // (4) dhidden[t0 : t0+tc, :] = -diag(f) (E' W)   (M = tokens of the chunk, N = H, K = V; E' K-major, W MN-major)
            alignas(64) CUtensorMap map_e_k;
            rc = make_map(&map_e_k, E, tc, V, lay.ld_v, kBM);
            if (rc != DPPO_OK) return rc;
            GemmShape g2 = gs0;
            g2.n_mtiles = (int)((tc + kBM - 1) / kBM); g2.n_ntiles = (H + kBN - 1) / kBN; g2.n_ksteps = (V + kBK - 1) / kBK;
            g2.hint_a = (tune.hints >> 4) & 3; g2.hint_b = (tune.hints >> 6) & 3;
            EpiStoreScaledBf16 e2 = {};
            e2.C = (__nv_bfloat16*)dhidden; e2.info = info; e2.ldc = H; e2.row0 = t0; e2.rows = T; e2.cols = H;
            rc = run_gemm<EpiStoreScaledBf16, false, true>(pair, map_e_k, map_w_mn, map_w_mn, map_e_k, g2, e2, status, s, "lmhead dhidden launch");
            if (rc != DPPO_OK) return rc;
        }
        if (backward && p->dW_dtype == DPPO_BF16) {
            const long long n = (long long)V * H;
            lm_f32_to_bf16_kernel<<<(unsigned)((n / 8 + 255) / 256), 256, 0, s>>>((const float*)(ws + lay.dw32), (__nv_bfloat16*)dW, n);
            DPPO_CHECK_LAUNCH("lmhead dW conversion launch");
        }
    }
    return launch_loss_reduce(a, loss_out, s);
}
