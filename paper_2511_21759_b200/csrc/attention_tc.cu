// Bidirectional block-query attention on the tcgen05 tensor cores (head dim 128): the refresh prefill and
// the decode step over several block copies.
//
// Work item: up to 128 consecutive query rows x one head (x one key split in a decode step).
//   refresh: keys = every row of the sequence (fresh q/k/v of the same forward; nothing is read from the
//            cache, the refresh is what writes it); the output is final.
//   step:    the rows of all copies of one block (a StepTile).  Key splits 0 .. ks-2 stream the cached
//            K/V of the positions outside the block, visible to every row; the last split takes the fresh
//            rows, one key tile per source copy: a row sees its own copy's tile and, in the decoded-share
//            layout, the decoded rows of copy 0's tile.  Copies stay mutually invisible through this
//            per-row key mask, no mask tensor exists.  Outputs are per-split (max, sum, unnormalised
//            output) partials merged in split order by the merge kernel of attention.cu.
// No causal mask.  One pass over the key tiles of 64; per tile S = Q K^T is one 128 x 64 x 128 tcgen05.mma group
// whose fp32 result lives in TMEM, and thread r owns TMEM lane r = query row r (no cross-thread reduction):
//   the tile's largest visible score moves the row's shift M - an INTEGER in the log2 domain - only when it exceeds
//   M by more than a slack of 4 (so P < 16); then O (in TMEM) and the row sum are multiplied by the exact power of two
//   2^(M_old - M_new), once the previous P V has been added;
//   P = exp2(S - M), row sums, P rounded to a two-term bf16 sum (value + remainder, as in the
//   mma.sync kernel) and written to shared memory as the A operand of O += P V
//   (128 x 128 x 64, V taken MN-major straight from its [key][dim] tile), O in TMEM.
// Exact softmax (rescaling by powers of two changes no bit of a normal number).  Warp-specialised: warps 0..3 = softmax (one query row per thread),
// warp 4 lane 0 = MMA issuer, warp 5 lane 0 = loader (TMA: boxes of 64 rows x 64 columns with the 128-byte
// swizzle land in the canonical operand layout, two 64-column atoms per 128-wide row; rows past a buffer's
// end read as zero, rows that are not keys of this work item are masked in the softmax and hold finite
// values, the K/V cache being zeroed when a session is created).  S is double buffered in TMEM and K in
// shared memory, so S(t + 1) is computed while the softmax warps work on tile t and P V(t) while they work
// on tile t + 1; the roles meet only through mbarriers.  Two CTAs share an SM (112 KB of shared memory, 256
// TMEM columns each).  Every mbarrier wait is bounded; on expiry the CTA records ODB_ERR_TIMEOUT, every
// role stops, the CTA releases its TMEM and exits.
#include "odb_internal.cuh"

namespace odb {

namespace {

constexpr int kTQ = 128;   // query rows per work item (MMA M)
constexpr int kTK = 64;    // keys per tile
constexpr int kHD = 128;
constexpr int kThreads = 192;   // 4 softmax warps, MMA warp, loader warp

constexpr uint32_t kQBytes = kTQ * kHD * 2;          // 32 KB: two atoms of 128 rows x 128 B
constexpr uint32_t kKBytes = kTK * kHD * 2;          // 16 KB: two atoms of 64 rows x 128 B
constexpr uint32_t kPBytes = kTQ * kTK * 2;          // 16 KB: one atom of 128 rows x 128 B
constexpr uint32_t kSmemBytes = kQBytes + 3 * kKBytes + 2 * kPBytes + 128;   // the dynamic region starts 1024-aligned
constexpr uint32_t kTmemCols = 256;                  // S0: columns 0..63, O: 64..191, S1: 192..255

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// one box of 64 rows x 64 columns (8 KB): rows row0.., columns col0..
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* tmap, uint64_t* bar, int col0, int row0) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(col0), "r"(row0)
        : "memory");
}

// asks L2 for the same box (no shared-memory destination, nothing to wait for)
__device__ __forceinline__ void tma_prefetch_box(const CUtensorMap* tmap, int col0, int row0) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(reinterpret_cast<uint64_t>(tmap)),
                 "r"(col0), "r"(row0)
                 : "memory");
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

// Bounded wait (shared implementation): false if the CTA has been aborted or the limit expired.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* cta_abort, int* status) {
    return mbar_wait_bounded(bar, parity, cta_abort, status);
}

// K-major operand, rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_k_major(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(1) << 16;                   // leading byte offset (unused with swizzle)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;           // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                   // descriptor version of this architecture
    d |= static_cast<uint64_t>(2) << 61;                   // 128-byte swizzle
    return d;
}

// MN-major operand: 64 contiguous elements (128 bytes) of the N dimension per K row, 128-byte swizzle;
// 8-K-row groups 1024 bytes apart (stride offset), 64-element N groups `n_group_bytes` apart (leading offset)
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t saddr, uint32_t n_group_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(n_group_bytes >> 4) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// bf16 x bf16 -> fp32, A K-major, B K-major or MN-major
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
          "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),
          "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),
          "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
        "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]),
        "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]),
        "r"(v[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

struct alignas(8) TcShared {
    uint64_t q_full;       // Q tile landed                                   (loader -> MMA)
    uint64_t k_full[2];    // key tile landed in K buffer 0 / 1                (loader -> MMA)
    uint64_t k_empty[2];   // the MMAs have read K buffer 0 / 1                (MMA -> loader)
    uint64_t v_full;       // V tile landed                                    (loader -> MMA)
    uint64_t v_empty;      // the MMAs have read the V tile                    (MMA -> loader)
    uint64_t s_full[2];    // S = Q K^T into S buffer 0 / 1 has completed      (MMA -> softmax)
    uint64_t s_empty[2];   // the softmax warps have read S buffer 0 / 1       (softmax -> MMA, 4 arrivals)
    uint64_t p_full;       // P is in shared memory                            (softmax -> MMA, 4 arrivals)
    uint64_t p_empty;      // the MMAs have read P                             (MMA -> softmax)
    uint64_t o_full;       // the last O += P V has completed                  (MMA -> softmax)
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 2^x for x <= 0 on the special-function unit (flushes to zero far below zero, which is the wanted value)
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One key tile of a work item: 64 consecutive rows of a [rows][128]-column view starting at row0, of which
// the first `valid` are keys.  src: 0 = fresh k / v rows of this forward, 1 = the K/V cache.
struct KeyTile {
    int src, row0, v_row0, valid;
    int copy;          // fresh tile of a step: the source copy; -1 otherwise (visible to every row)
};

struct TcArgs {
    const QTile* qtiles;          // refresh work items
    const StepTile* stiles;       // step work items
    const int32_t* row_flags;
    __nv_bfloat16* o;             // refresh: final output [M][H * 128]
    float* part_o; float* part_ml;   // step: split partials [ks][M][H][128], [ks][M][H][2]
    int layer, n_layers, H, max_seq, M;
};

template <bool STEP>
__global__ void __launch_bounds__(kThreads) attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                                                                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_c,
                                                                TcArgs a, int* status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* sQ = smem_raw;
    uint8_t* sK0 = sQ + kQBytes;         // key tiles with even index
    uint8_t* sK1 = sK0 + kKBytes;        // key tiles with odd index
    uint8_t* sV = sK1 + kKBytes;
    uint8_t* sPh = sV + kKBytes;         // P, rounded to bf16
    uint8_t* sPl = sPh + kPBytes;        // P minus its rounded value, rounded to bf16
    TcShared* sh = reinterpret_cast<TcShared*>(sPl + kPBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* cta_abort = &sh->abort;

    pdl_launch_dependents();
    if ((smem_u32(smem_raw) & 1023u) != 0) {                // the swizzled tiles need 1024-byte alignment
        if (tid == 0) atomicExch(status, ODB_ERR_CUDA);
        pdl_wait();
        return;
    }
    if (tid == 0) {
        mbar_init(&sh->q_full, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sh->k_full[b], 1);
            mbar_init(&sh->k_empty[b], 1);
            mbar_init(&sh->s_full[b], 1);
            mbar_init(&sh->s_empty[b], 4);
        }
        mbar_init(&sh->v_full, 1);
        mbar_init(&sh->v_empty, 1);
        mbar_init(&sh->p_full, 4);
        mbar_init(&sh->p_empty, 1);
        mbar_init(&sh->o_full, 1);
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_s0 = sh->tmem_base;                // 64 columns
    const uint32_t tmem_o = sh->tmem_base + 64;            // 128 columns
    const uint32_t tmem_s1 = sh->tmem_base + 192;          // 64 columns

    pdl_wait();   // q, k, v of this layer come from the preceding kernel
    const int head = blockIdx.y;
    const int z = blockIdx.z, ks = gridDim.z;
    // ---- the work item: query rows and key tiles ----
    int q_row0, nq, ntiles;
    int f0 = 0, NK = 0;                                     // refresh: keys = fresh rows [f0, f0 + NK)
    int cA = 0, cB0 = 0, cB1 = 0, nA_t = 0, t_first = 0;    // step, cached split: positions [0, cA) and [cB0, cB1)
    int c_row = 0;                                          // step: row of position 0 of this head's keys in the cache view
    bool fresh_split = false;
    const bool single = STEP && ks == 1;                    // step without key splits
    int n_cached = 0;                                       // step: cached key tiles of this CTA (they come first)
    const StepTile* stp = nullptr;
    if constexpr (!STEP) {
        const QTile t = a.qtiles[blockIdx.x];
        q_row0 = t.q_row0; nq = t.nq; f0 = t.f0; NK = t.n0;
        ntiles = (NK + kTK - 1) / kTK;
    } else {
        stp = a.stiles + blockIdx.x;
        q_row0 = stp->slab_row0[0];
        nq = stp->slab_row0[stp->n_slabs - 1] + stp->slab_n[stp->n_slabs - 1] - q_row0;   // the slabs are consecutive rows
        cA = stp->cA; cB0 = stp->cB0; cB1 = stp->cB1;
        nA_t = (cA + kTK - 1) / kTK;
        const int nct = nA_t + (cB1 - cB0 + kTK - 1) / kTK;
        if (single) {
            // one CTA takes every key of the item: the cached tiles, then the fresh ones; its output is final
            n_cached = nct;
            ntiles = nct + stp->n_src;
        } else {
            fresh_split = z == ks - 1;
            const int tp = (nct + ks - 2) / (ks - 1);
            t_first = fresh_split ? 0 : z * tp;
            n_cached = fresh_split ? 0 : max(0, min(nct, t_first + tp) - t_first);
            ntiles = fresh_split ? stp->n_src : n_cached;
        }
        c_row = ((stp->seq * a.n_layers + a.layer) * 2 * a.H + head) * a.max_seq;   // K; V is H * max_seq rows further
    }
    auto key_tile = [&](int i) {
        KeyTile kt;
        kt.copy = -1;
        if constexpr (!STEP) {
            kt.src = 0; kt.row0 = f0 + i * kTK; kt.v_row0 = kt.row0; kt.valid = min(kTK, NK - i * kTK);
        } else if (i >= n_cached) {
            const int f = i - n_cached;
            kt.src = 0; kt.row0 = stp->src_row0[f]; kt.v_row0 = kt.row0; kt.valid = stp->src_n[f]; kt.copy = stp->src_copy[f];
        } else {
            const int j = t_first + i;
            const int pos0 = j < nA_t ? j * kTK : cB0 + (j - nA_t) * kTK;
            const int end = j < nA_t ? cA : cB1;
            kt.src = 1; kt.row0 = c_row + pos0; kt.v_row0 = kt.row0 + a.H * a.max_seq; kt.valid = min(kTK, end - pos0);
        }
        return kt;
    };
    const float scale_log2 = rsqrtf(static_cast<float>(kHD)) * 1.4426950408889634f;
    auto wait = [&](uint64_t* bar, uint32_t& phase) {
        const bool ok = mbar_wait(bar, phase, cta_abort, status);
        phase ^= 1u;
        return ok;
    };

    if (warp == 5) {
        // ================= loader =================
        if (lane == 0) {
            const int col0 = head * kHD;
            // 64 rows x 128 columns: one box per 64-column atom (the cache view has 128 columns per row)
            auto load_k = [&](int tile) {
                if (tile >= ntiles) return;
                const int b = tile & 1;
                const KeyTile kt = key_tile(tile);
                const uint32_t dst = smem_u32(b ? sK1 : sK0);
                mbar_expect_tx(&sh->k_full[b], kKBytes);
                tma_box(dst, kt.src ? &tm_c : &tm_k, &sh->k_full[b], kt.src ? 0 : col0, kt.row0);
                tma_box(dst + kTK * 128, kt.src ? &tm_c : &tm_k, &sh->k_full[b], kt.src ? 64 : col0 + 64, kt.row0);
            };
            auto load_v = [&](int tile) {
                if (tile >= ntiles) return;
                const KeyTile kt = key_tile(tile);
                const uint32_t dst = smem_u32(sV);
                mbar_expect_tx(&sh->v_full, kKBytes);
                tma_box(dst, kt.src ? &tm_c : &tm_v, &sh->v_full, kt.src ? 0 : col0, kt.v_row0);
                tma_box(dst + kTK * 128, kt.src ? &tm_c : &tm_v, &sh->v_full, kt.src ? 64 : col0 + 64, kt.v_row0);
            };
            // Two K buffers and one V buffer cover little of a load's latency from HBM: every load also asks L2 for
            // the tile kAhead tiles further on, so that the load that later fills a buffer comes from L2.
            constexpr int kAhead = 3;
            auto hint_k = [&](int tile) {
                if (tile >= ntiles) return;
                const KeyTile kt = key_tile(tile);
                tma_prefetch_box(kt.src ? &tm_c : &tm_k, kt.src ? 0 : col0, kt.row0);
                tma_prefetch_box(kt.src ? &tm_c : &tm_k, kt.src ? 64 : col0 + 64, kt.row0);
            };
            auto hint_v = [&](int tile) {
                if (tile >= ntiles) return;
                const KeyTile kt = key_tile(tile);
                tma_prefetch_box(kt.src ? &tm_c : &tm_v, kt.src ? 0 : col0, kt.v_row0);
                tma_prefetch_box(kt.src ? &tm_c : &tm_v, kt.src ? 64 : col0 + 64, kt.v_row0);
            };
            uint32_t ph_ke[2] = {0, 0}, ph_ve = 0;
            bool ok = true;
            // Q: rows 0..63 and 64..127 of each atom
            mbar_expect_tx(&sh->q_full, kQBytes);
            tma_box(smem_u32(sQ), &tm_q, &sh->q_full, col0, q_row0);
            tma_box(smem_u32(sQ) + 64 * 128, &tm_q, &sh->q_full, col0, q_row0 + 64);
            tma_box(smem_u32(sQ) + kTQ * 128, &tm_q, &sh->q_full, col0 + 64, q_row0);
            tma_box(smem_u32(sQ) + kTQ * 128 + 64 * 128, &tm_q, &sh->q_full, col0 + 64, q_row0 + 64);
            load_k(0);
            load_v(0);
            load_k(1);
            for (int t = 1; t < 1 + kAhead; ++t) hint_v(t);
            for (int t = 2; t < 2 + kAhead; ++t) hint_k(t);
            // S(tile) completes long before P V(tile) (the softmax of the tile lies between them), and S(tile + 2) is
            // issued right behind P V(tile): the K buffer is refilled first, so that its load runs during that softmax
            for (int tile = 0; tile < ntiles && ok; ++tile) {
                const int b = tile & 1;
                if (tile + 2 < ntiles) {
                    ok = wait(&sh->k_empty[b], ph_ke[b]);        // S(tile) has read this buffer
                    if (!ok) break;
                    load_k(tile + 2);
                    hint_k(tile + 2 + kAhead);
                }
                if (tile + 1 < ntiles) {
                    ok = wait(&sh->v_empty, ph_ve);             // P V(tile) has read the V tile
                    if (!ok) break;
                    load_v(tile + 1);
                    hint_v(tile + 1 + kAhead);
                }
            }
        }
    } else if (warp == 4) {
        // ================= MMA issuer =================
        if (lane == 0 && ntiles > 0) {
            constexpr uint32_t idesc_s = instr_desc(kTQ, kTK, 0);
            constexpr uint32_t idesc_o = instr_desc(kTQ, kHD, 1);
            uint32_t ph_q = 0, ph_kf[2] = {0, 0}, ph_se[2] = {0, 0}, ph_vf = 0, ph_pf = 0;
            bool ok = wait(&sh->q_full, ph_q);
            // S(tile) = Q K^T over the 128-wide head dim: 8 MMAs of K = 16 into S buffer tile & 1
            auto issue_s = [&](int tile) {
                const int b = tile & 1;
                const uint32_t qa = smem_u32(sQ), kb = smem_u32(b ? sK1 : sK0);
                const uint32_t ts = b ? tmem_s1 : tmem_s0;
#pragma unroll
                for (int kk = 0; kk < kHD / 16; ++kk) {
                    const uint32_t atom = kk >> 2, within = (kk & 3) * 32;
                    umma(ts, desc_k_major(qa + atom * (kTQ * 128) + within), desc_k_major(kb + atom * (kTK * 128) + within),
                         idesc_s, kk > 0 ? 1u : 0u);
                }
                umma_commit(&sh->k_empty[b]);
                umma_commit(&sh->s_full[b]);
            };
            auto issue_pv = [&](int tile, bool last) {
                const uint32_t pa = smem_u32(sPh), pb = smem_u32(sPl), vb = smem_u32(sV);
#pragma unroll
                for (int kk = 0; kk < kTK / 16; ++kk) {             // 16 keys per MMA
                    const uint64_t bdesc = desc_mn_major(vb + kk * 2048, kTK * 128);
                    umma(tmem_o, desc_k_major(pa + kk * 32), bdesc, idesc_o, (tile > 0 || kk > 0) ? 1u : 0u);
                    umma(tmem_o, desc_k_major(pb + kk * 32), bdesc, idesc_o, 1u);
                }
                umma_commit(&sh->v_empty);
                umma_commit(&sh->p_empty);
                if (last) umma_commit(&sh->o_full);
            };
            for (int tile = 0; tile < ntiles && ok; ++tile) {
                const int b = tile & 1;
                ok = wait(&sh->k_full[b], ph_kf[b]);
                if (ok && tile >= 2) ok = wait(&sh->s_empty[b], ph_se[b]);   // S(tile - 2) has been read
                if (!ok) break;
                tc_fence_after();
                issue_s(tile);
                if (tile > 0) {                                      // P V of the previous tile, behind S(tile)
                    ok = wait(&sh->p_full, ph_pf);
                    if (ok) ok = wait(&sh->v_full, ph_vf);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(tile - 1, false);
                }
            }
            if (ok) {
                ok = wait(&sh->p_full, ph_pf);
                if (ok) ok = wait(&sh->v_full, ph_vf);
                if (ok) {
                    tc_fence_after();
                    issue_pv(ntiles - 1, true);
                }
            }
        }
    } else {
        // ================= softmax: thread r = query row r = TMEM lane r =================
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;   // this warp's TMEM lanes
        uint32_t ph_sf[2] = {0, 0}, ph_pe = 0, ph_of = 0;
        bool ok = true;
        int my_copy = -1, stage2 = 0;
        if constexpr (STEP) {
            stage2 = stp->stage2;
            const int grow = q_row0 + tid;
            for (int sl = 0; sl < stp->n_slabs; ++sl)
                if (grow >= stp->slab_row0[sl] && grow < stp->slab_row0[sl] + stp->slab_n[sl]) my_copy = stp->slab_copy[sl];
        }
        // which of the tile's 64 keys this row sees (bit j = key j).  Every lane of a warp calls this for the
        // same tile: the branch that uses the ballots is uniform.
        auto tile_mask = [&](const KeyTile& kt) -> unsigned long long {
            const unsigned long long all = kt.valid >= 64 ? ~0ull : ((1ull << kt.valid) - 1ull);
            if (kt.copy < 0) return all;                            // cached keys, or a refresh
            unsigned long long shared = 0ull;
            if constexpr (STEP) {
                if (stage2 && kt.copy == 0) {                        // decoded rows of copy 0, shared with every copy
                    const bool d0 = lane < kt.valid && (a.row_flags[kt.row0 + lane] & kRowDecoded);
                    const bool d1 = lane + 32 < kt.valid && (a.row_flags[kt.row0 + lane + 32] & kRowDecoded);
                    const unsigned lo = __ballot_sync(0xffffffffu, d0), hi = __ballot_sync(0xffffffffu, d1);
                    shared = (static_cast<unsigned long long>(hi) << 32 | lo) & all;
                }
            }
            return kt.copy == my_copy ? all : shared;
        };
        // ---- one pass over the key tiles: online softmax.  The row's shift M is an INTEGER in the log2 domain, so
        // that moving it rescales O and the row sum by an exact power of two; it moves only when a tile's maximum
        // exceeds it by more than kSlack (P then stays below 2^kSlack), which after the first tiles is rare. ----
        constexpr float kSlack = 4.0f;
        float M_row = -INFINITY;                                     // no visible key yet
        float l_row = 0.f;
        const uint32_t ph_base = smem_u32(sPh) + tid * 128, pl_base = smem_u32(sPl) + tid * 128;
        for (int tile = 0; tile < ntiles && ok; ++tile) {
            const int b = tile & 1;
            const KeyTile kt = key_tile(tile);
            const unsigned long long mask = tile_mask(kt);
            ok = wait(&sh->s_full[b], ph_sf[b]);
            if (!ok) break;
            tc_fence_after();
            // a whole tile of cached keys (or of a refresh) is seen by every row: no per-key test (the softmax
            // warps are bound by the instructions they issue per key)
            const bool full = kt.copy < 0 && kt.valid >= 64;
            float m_t = -INFINITY;                                   // largest visible score of the tile
            uint32_t sv[2][32];                                      // the row's 64 scores: read from TMEM once
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t (&v)[32] = sv[half];
                tmem_ld32((b ? tmem_s1 : tmem_s0) + lane_base + half * 32, v);
                if (full) {
                    float m0 = m_t, m1 = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        m0 = fmaxf(m0, fmaxf(__uint_as_float(v[j]), __uint_as_float(v[j + 1])));
                        m1 = fmaxf(m1, fmaxf(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])));
                    }
                    m_t = fmaxf(m0, m1);
                } else {
                    const unsigned m32 = static_cast<unsigned>(mask >> (half * 32));
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if ((m32 >> j) & 1u) m_t = fmaxf(m_t, __uint_as_float(v[j]));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->s_empty[b]);             // S(tile) is in registers
            float factor = 1.0f;                                     // what O and the row sum so far are multiplied by
            const float mt_log2 = m_t * scale_log2;                  // -inf: the row sees no key of this tile
            if (mt_log2 > M_row + kSlack) {                          // also the first visible key (M_row = -inf)
                const float M_new = ceilf(mt_log2);
                if (M_row != -INFINITY) factor = exp2f(M_row - M_new);   // an exact power of two
                M_row = M_new;
            }
            const bool rescale = __any_sync(0xffffffffu, factor != 1.0f);
            const float m_log2 = M_row == -INFINITY ? 0.f : M_row;   // a row that has seen no key: every P is masked to 0
            uint32_t hi[32], lo[32];                                 // row `tid` of P: 64 keys as bf16 pairs
            float l_tile = 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const uint32_t (&v)[32] = sv[half];
                const unsigned m32 = full ? 0xffffffffu : static_cast<unsigned>(mask >> (half * 32));
                float l0 = 0.f, l1 = 0.f;
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const int j = 2 * u;
                    // arguments are <= kSlack: the hardware exponential needs no range handling (far below zero it returns 0)
                    float p0 = ex2_approx(fmaf(__uint_as_float(v[j]), scale_log2, -m_log2));
                    float p1 = ex2_approx(fmaf(__uint_as_float(v[j + 1]), scale_log2, -m_log2));
                    if (!full) {
                        p0 = ((m32 >> j) & 1u) ? p0 : 0.f;
                        p1 = ((m32 >> (j + 1)) & 1u) ? p1 : 0.f;
                    }
                    l0 += p0;
                    l1 += p1;
                    const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                    const uint32_t hb = *reinterpret_cast<const uint32_t*>(&h);
                    // the bf16 halves widened back to fp32 are the bit patterns themselves, shifted into place
                    const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - __uint_as_float(hb << 16),
                                                                   p1 - __uint_as_float(hb & 0xffff0000u));
                    hi[half * 16 + u] = hb;
                    lo[half * 16 + u] = *reinterpret_cast<const uint32_t*>(&l);
                }
                l_tile += l0 + l1;
            }
            if (tile > 0) {
                ok = wait(&sh->p_empty, ph_pe);                      // P V(tile - 1) has read P and has been added to O
                if (!ok) break;
                if (rescale) {                                       // warp-uniform; rows that keep their shift multiply by 1
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < kHD / 32; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tmem_o + lane_base + c * 32, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * factor);
                        tmem_st32(tmem_o + lane_base + c * 32, v);
                    }
                    tc_fence_before();
                }
            }
            l_row = l_row * factor + l_tile;
#pragma unroll
            for (int c = 0; c < 8; ++c) {                            // 8 keys = one 16-byte chunk
                const uint32_t off = static_cast<uint32_t>((c ^ (tid & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ph_base + off), "r"(hi[4 * c]), "r"(hi[4 * c + 1]),
                             "r"(hi[4 * c + 2]), "r"(hi[4 * c + 3])
                             : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(pl_base + off), "r"(lo[4 * c]), "r"(lo[4 * c + 1]),
                             "r"(lo[4 * c + 2]), "r"(lo[4 * c + 3])
                             : "memory");
            }
            proxy_fence();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->p_full);
        }
        const float m_log2 = M_row == -INFINITY ? 0.f : M_row;      // the shift the row's sum and output carry
        if (ok && ntiles > 0) ok = wait(&sh->o_full, ph_of);
        if (ok) {
            tc_fence_after();
            const int d = a.H * kHD;
            const int row = q_row0 + tid;
            if (!STEP || single) {
                const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
                __nv_bfloat16* orow = a.o + static_cast<size_t>(row) * d + head * kHD;
#pragma unroll 1
                for (int c = 0; c < kHD / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tmem_o + lane_base + c * 32, v);
                    if (tid < nq) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint4 pk;
                            __nv_bfloat162 x0 = __floats2bfloat162_rn(__uint_as_float(v[j]) * inv, __uint_as_float(v[j + 1]) * inv);
                            __nv_bfloat162 x1 = __floats2bfloat162_rn(__uint_as_float(v[j + 2]) * inv, __uint_as_float(v[j + 3]) * inv);
                            __nv_bfloat162 x2 = __floats2bfloat162_rn(__uint_as_float(v[j + 4]) * inv, __uint_as_float(v[j + 5]) * inv);
                            __nv_bfloat162 x3 = __floats2bfloat162_rn(__uint_as_float(v[j + 6]) * inv, __uint_as_float(v[j + 7]) * inv);
                            pk.x = *reinterpret_cast<const uint32_t*>(&x0);
                            pk.y = *reinterpret_cast<const uint32_t*>(&x1);
                            pk.z = *reinterpret_cast<const uint32_t*>(&x2);
                            pk.w = *reinterpret_cast<const uint32_t*>(&x3);
                            *reinterpret_cast<uint4*>(orow + c * 32 + j) = pk;
                        }
                    }
                }
            } else {
                // split partial: unnormalised output, (max in the log2 domain, sum); a split that saw no key has sum 0
                const size_t pr = (static_cast<size_t>(z) * a.M + row) * a.H + head;
                if (tid < nq) *reinterpret_cast<float2*>(a.part_ml + pr * 2) = make_float2(m_log2, l_row);
                if (ntiles > 0) {
                    float* po = a.part_o + pr * kHD;
#pragma unroll 1
                    for (int c = 0; c < kHD / 32; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tmem_o + lane_base + c * 32, v);
                        if (tid < nq) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<float4*>(po + c * 32 + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                                          __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh->tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <bool STEP>
cudaError_t launch_tc(dim3 grid, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, const __nv_bfloat16* cache,
                      size_t cache_rows, const TcArgs& ta, int* status, cudaStream_t st) {
    static std::atomic<unsigned long long> attr_done{0};
    {
        cudaError_t e0 = set_smem_limit_once(attr_done, attention_tc_kernel<STEP>, static_cast<int>(kSmemBytes));
        if (e0 != cudaSuccess) return e0;
    }
    // the fresh q / k / v of this forward: [M][H * 128] bf16, rows beyond M read as zero; the cache as rows of 128
    CUtensorMap tq, tk, tv, tc;
    const int d = ta.H * kHD;
    cudaError_t e = make_rows_tmap(&tq, q, ta.M, d, 64);
    if (e == cudaSuccess) e = make_rows_tmap(&tk, k, ta.M, d, 64);
    if (e == cudaSuccess) e = make_rows_tmap(&tv, v, ta.M, d, 64);
    if (e == cudaSuccess) e = STEP ? make_rows_tmap(&tc, cache, cache_rows, kHD, 64) : make_rows_tmap(&tc, k, ta.M, d, 64);
    if (e != cudaSuccess) return e;
    return launch_kernel(attention_tc_kernel<STEP>, grid, dim3(kThreads), kSmemBytes, st, tq, tk, tv, tc, ta, status);
}

}  // namespace

// Refresh attention on the tensor cores: a.tiles = work items of up to 128 query rows whose keys are the
// fresh rows [f0, f0 + n0) (cA = cB0 = cB1 = n1 = 0), head dim 128.
cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st) {
    if (a.n_tiles == 0) return cudaSuccess;
    if (a.hd != kHD) return cudaErrorInvalidValue;
    TcArgs ta{};
    ta.qtiles = a.tiles;
    ta.row_flags = a.row_flags;
    ta.o = a.o;
    ta.layer = a.layer; ta.n_layers = a.n_layers; ta.H = a.H; ta.max_seq = a.max_seq; ta.M = a.M;
    return launch_tc<false>(dim3(a.n_tiles, a.H), a.q, a.k, a.v, nullptr, 0, ta, status, st);
}

// Decode-step attention over StepTiles on the tensor cores (head dim 128); cache_rows = rows of the K/V cache
// viewed as [rows][128] (batch x layers x 2 x heads x max_seq).  ksplit = 1: every work item is one CTA over all of its
// keys and writes the final output; ksplit >= 2: partials only, the caller merges them.
cudaError_t launch_step_attention_tc(const StepAttnArgs& a, size_t cache_rows, int* status, cudaStream_t st) {
    if (a.n_tiles == 0) return cudaSuccess;
    if (a.hd != kHD || a.ksplit < 1 || a.ksplit > 8) return cudaErrorInvalidValue;
    TcArgs ta{};
    ta.stiles = a.tiles;
    ta.row_flags = a.row_flags;
    ta.o = a.o;                                            // written when there is no key split
    ta.part_o = a.part_o; ta.part_ml = a.part_ml;
    ta.layer = a.layer; ta.n_layers = a.n_layers; ta.H = a.H; ta.max_seq = a.max_seq; ta.M = a.M;
    return launch_tc<true>(dim3(a.n_tiles, a.H, a.ksplit), a.q, a.k, a.v, a.cache, cache_rows, ta, status, st);
}

}  // namespace odb
