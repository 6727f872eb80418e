// Weight-streaming GEMM for sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM -> registers.
//
// Computes, for every K split s,   partial[s][m][n] = sum_{k in split s} x[m][k] * w[n][k]
// with x the bf16 activations [M][K] (few rows: block_len * copies in a decode step; all
// positions in a refresh) and w a bf16 weight matrix [N][K].  The 128-row side of the tensor
// core tile is given to the WEIGHTS (they are the large, streamed operand) and the activation
// rows ride on the MMA's N dimension (32..256), so a 32-row decode step wastes no tensor-core
// rows and every weight byte is fetched from HBM exactly once.
//
// Weights are stored PACKED: tile (n-tile of 128 rows, k-block of 64 columns) is one contiguous
// 16 KB chunk, tiles of a row of tiles consecutive in k.  A CTA therefore reads one sequential
// stream of whole DRAM pages; with the plain row-major layout each TMA box gathers 128 separate
// 128-byte pieces 2K bytes apart and HBM delivers little more than half its bandwidth (measured).
//
// One CTA = one 128 x BN output tile over one K range.  Warp 0 lane 0 issues TMA loads into a
// ring of shared-memory stages, warp 1 lane 0 issues the MMAs (accumulator in TMEM) and frees
// stages through tcgen05.commit, warps 2..5 read the accumulator back (tcgen05.ld) and store
// fp32 partials.  Splits are reduced later in a fixed order by the consumer kernel, so results
// are run-to-run identical.  Every mbarrier wait is bounded: on expiry the CTA records
// ODB_ERR_TIMEOUT, stops issuing work, releases its TMEM and exits.
#include <stdlib.h>

#include "odb_internal.cuh"
#include "tcgen05_common.cuh"

namespace odb {

namespace {

struct alignas(8) GemmShared {
    uint64_t full[16];
    uint64_t empty[16];
    uint64_t acc_full;
    uint32_t tmem_base;
    int abort;
    float scale[256];      // RowScale of the tile's activation rows
};

// BN: activation rows per tile (MMA N): 32, 64, 128 or 256.
// SWIGLU: the weight is the gate/up matrix packed with gate and up rows interleaved in groups of
// 64 (tile t = gate rows [64t, 64t+64) then up rows [64t, 64t+64)); the epilogue pairs TMEM lane r
// (gate) with lane r + 64 (up) through shared memory and stores bf16(silu(gate) * up) to
// g[m][64 t + r]; N is then the FFN width F and there is no K split.
constexpr int EPI_PARTIAL = 0, EPI_SWIGLU = 1, EPI_CONF = 3;

template <int BN, int EPI, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
            float* __restrict__ partial, __nv_bfloat16* __restrict__ act_out, RowScale rs,
            ConfEpilogue ce, int M, int N, int nkb_total, int nkb_per_split, int stages,
            int l2_prefetch, int pair_tiles_x, int pair_tiles_y,
            int* status, const __grid_constant__ PeerOut po) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    constexpr uint32_t kABytes = kBM * kBK * 2;
    constexpr int kBRows = PAIR ? BN / 2 : BN;        // activation rows this CTA stages
    constexpr uint32_t kBBytes = kBRows * kBK * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kTxBytes = PAIR ? 2 * kStageBytes : kStageBytes;   // bytes reported to a full barrier
    constexpr uint32_t kTmemCols = BN < 32 ? 32 : BN;
    const uint32_t pair_rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = pair_rank == 0;

    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GemmShared* sh = reinterpret_cast<GemmShared*>(tiles + static_cast<size_t>(stages) * kStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Work unit of this CTA.  Single CTAs: grid (weight tiles, row tiles, K splits).  Pairs: grid (2, row tiles of
    // a group, weight-tile pairs x row-tile groups x K splits), scheduled in that order: the row tiles of a group
    // run side by side on one weight-tile pair (its weights come from HBM once, from L2 for the other row
    // tiles), and a group's activation rows (a few MB) stay in L2 while every weight-tile pair passes over them.
    const int n_pairs = PAIR ? pair_tiles_x >> 1 : 0;
    const int n_tile = PAIR ? 2 * static_cast<int>(blockIdx.z % n_pairs) + static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x);
    const int n_tiles = PAIR ? pair_tiles_x : static_cast<int>(gridDim.x);
    const int m_groups = PAIR ? (pair_tiles_y + static_cast<int>(gridDim.y) - 1) / static_cast<int>(gridDim.y) : 1;
    const int m_tile = PAIR ? static_cast<int>((blockIdx.z / n_pairs) % m_groups) * static_cast<int>(gridDim.y) + static_cast<int>(blockIdx.y)
                            : static_cast<int>(blockIdx.y);
    if (PAIR && m_tile >= pair_tiles_y) {   // ragged last group: both CTAs of the pair leave together
        if (po.n > 0 && threadIdx.x == 0) {
            pdl_wait();   // the arrival counter is shared with the previous exchanging launch: count only once that one is complete
            tp_arrive_and_signal(po, gridDim.x * gridDim.y * gridDim.z);
        }
        return;
    }
    const int n0 = n_tile * kBM;
    const int m0 = m_tile * BN;
    const int split = PAIR ? static_cast<int>(blockIdx.z / (n_pairs * m_groups)) : static_cast<int>(blockIdx.z);
    const int kb0 = split * nkb_per_split;
    int nkb = nkb_total - kb0;
    if (nkb > nkb_per_split) nkb = nkb_per_split;
    volatile int* cta_abort = &sh->abort;
    // packed weights: tile (n-tile, k-block) is the contiguous 16 KB chunk number n_tile * nkb_total + k_block
    const int wtile0 = n_tile * nkb_total + kb0;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(&sh->full[i], 1);
            mbar_init(&sh->empty[i], 1);
        }
        mbar_init(&sh->acc_full, 1);
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_w)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_x)) : "memory");
    }
    if (warp == 1) {   // whole warp: allocate the accumulator's TMEM columns
        __syncwarp();
        if constexpr (PAIR) {   // the same warp of both CTAs allocates the same columns in both SMs
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                         "r"(kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                         "r"(kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if constexpr (PAIR) cluster_barrier();   // the peer's barriers are initialised before anything signals them
    const uint32_t tmem_acc = sh->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            // The weights do not depend on the preceding kernel: fill the ring with weight tiles
            // first, then wait for the predecessor and fetch the activation tiles.
            const int pre = nkb < stages ? nkb : stages;
            const int mb = m0 + static_cast<int>(pair_rank) * kBRows;   // first activation row this CTA stages
            for (int i = 0; i < pre; ++i) {
                if (leader) mbar_expect_tx(&sh->full[i], kTxBytes);
                if constexpr (PAIR)
                    tma_load_3d_pair(tiles + static_cast<size_t>(i) * kStageBytes, &tmap_w, &sh->full[i], 0, 0, wtile0 + i,
                                     kEvictFirst);
                else
                    tma_load_3d(tiles + static_cast<size_t>(i) * kStageBytes, &tmap_w, &sh->full[i], 0, 0, wtile0 + i,
                                kEvictFirst);
            }
            // and ask L2 for the weight tiles that follow, so that HBM keeps streaming while the
            // predecessor (a short elementwise kernel) is still running
            int pf = nkb - pre;
            if (pf > l2_prefetch) pf = l2_prefetch;
            for (int i = pre; i < pre + pf; ++i)
                asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(
                                 reinterpret_cast<uint64_t>(&tmap_w)),
                             "r"(0), "r"(0), "r"(wtile0 + i)
                             : "memory");
            pdl_wait();
            for (int i = 0; i < pre; ++i) {
                if constexpr (PAIR)
                    tma_load_2d_pair(tiles + static_cast<size_t>(i) * kStageBytes + kABytes, &tmap_x, &sh->full[i],
                                     (kb0 + i) * kBK, mb, kEvictLast);
                else
                    tma_load_2d(tiles + static_cast<size_t>(i) * kStageBytes + kABytes, &tmap_x, &sh->full[i], (kb0 + i) * kBK,
                                mb, kEvictLast);
            }
            int issued = pre;
            for (int i = pre; i < nkb; ++i) {
                const int st = i % stages;
                const uint32_t ph = static_cast<uint32_t>(i / stages) & 1u;
                if (!mbar_wait(&sh->empty[st], ph ^ 1u, cta_abort, status)) break;
                uint8_t* a_dst = tiles + static_cast<size_t>(st) * kStageBytes;
                uint8_t* b_dst = a_dst + kABytes;
                if (leader) mbar_expect_tx(&sh->full[st], kTxBytes);
                if constexpr (PAIR) {
                    tma_load_3d_pair(a_dst, &tmap_w, &sh->full[st], 0, 0, wtile0 + i, kEvictFirst);
                    tma_load_2d_pair(b_dst, &tmap_x, &sh->full[st], (kb0 + i) * kBK, mb, kEvictLast);
                } else {
                    tma_load_3d(a_dst, &tmap_w, &sh->full[st], 0, 0, wtile0 + i, kEvictFirst);
                    tma_load_2d(b_dst, &tmap_x, &sh->full[st], (kb0 + i) * kBK, mb, kEvictLast);
                }
                issued = i + 1;
            }
            if (*cta_abort && leader) {
                // aborted: let the copies still in flight land before the CTA's shared memory goes away (the
                // peer of a pair cannot observe its own copies; it is held by the cluster barrier at the end)
                const int first = issued > stages ? issued - stages : 0;
                for (int i = first; i < issued; ++i) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait_parity(&sh->full[i % stages], static_cast<uint32_t>(i / stages) & 1u) &&
                           clock64() - t0 < kWaitLimitCycles / 8) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            // ---- MMA issuer (the leader's, for both CTAs of a pair) ----
            constexpr uint32_t idesc = make_instr_desc(PAIR ? 2 * kBM : kBM, BN);
            bool ok = true;
            for (int i = 0; i < nkb && ok; ++i) {
                const int st = i % stages;
                const uint32_t ph = static_cast<uint32_t>(i / stages) & 1u;
                ok = mbar_wait(&sh->full[st], ph, cta_abort, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(tiles + static_cast<size_t>(st) * kStageBytes);
                const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                for (int k = 0; k < kBK / kUmmaK; ++k) {
                    if constexpr (PAIR)
                        umma_bf16_pair(tmem_acc, make_smem_desc(a_addr + k * kUmmaK * 2), make_smem_desc(b_addr + k * kUmmaK * 2),
                                       idesc, (i > 0 || k > 0) ? 1u : 0u);
                    else
                        umma_bf16(tmem_acc, make_smem_desc(a_addr + k * kUmmaK * 2), make_smem_desc(b_addr + k * kUmmaK * 2),
                                  idesc, (i > 0 || k > 0) ? 1u : 0u);
                }
                // frees the stage (in both CTAs of a pair) once these MMAs have read it
                if constexpr (PAIR) umma_commit_pair(&sh->empty[st]);
                else umma_commit(&sh->empty[st]);
            }
            if (ok) {
                if constexpr (PAIR) umma_commit_pair(&sh->acc_full);
                else umma_commit(&sh->acc_full);
            }
        }
    } else {
        // ---- epilogue: warps 2..5 own TMEM lanes 32*(warp%4) .. +31 ----
        const int q = warp & 3;
        pdl_wait();   // the previous reader of the output buffer has finished; the predecessor's results are visible
        if (rs.ssq) {   // uniform: row scalars of this tile's activation rows, computed while the main loop runs
            for (int i = threadIdx.x - 64; i < BN; i += 128) sh->scale[i] = m0 + i < M ? row_scale_of(rs, m0 + i) : 1.0f;
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        const bool ok = nkb > 0 && mbar_wait(&sh->acc_full, 0, cta_abort, status);   // nkb == 0: empty K split
        if (ok) tc_fence_after();
        if constexpr (EPI == EPI_PARTIAL) {
            const int n = n0 + q * 32 + lane;
            if (ok) {
                const size_t split_off = static_cast<size_t>(split) * M * N;
                float* out = partial + split_off;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tmem_acc + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c * 32), v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (po.n == 0) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + c * 32 + j;
                            const float sc = rs.ssq ? sh->scale[c * 32 + j] : 1.0f;
                            if (n < N && m < M) out[static_cast<size_t>(m) * N + n] = __uint_as_float(v[j]) * sc;
                        }
                    } else {
                        // tensor-parallel partial sums: the tile goes to the receive buffer of every rank
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int m = m0 + c * 32 + j;
                            if (n < N && m < M) {
                                const size_t off = split_off + static_cast<size_t>(m) * N + n;
#pragma unroll 1
                                for (int r = 0; r < po.n; ++r) po.partial[r][off] = __uint_as_float(v[j]);
                            }
                        }
                    }
                }
            }
            if (po.n > 0) {   // uniform: the tile's stores of all four warps, then one arrival for the CTA
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (threadIdx.x == 64) tp_arrive_and_signal(po, gridDim.x * gridDim.y * gridDim.z);
            }
        } else if constexpr (EPI == EPI_CONF) {
            // LM head fused with the confidence reduction: the logits of this tile (128 vocabulary
            // entries x BN rows) never leave the SM.  They are transposed through shared memory so that
            // four threads scan one row's 128 logits (32 each, ascending ids, online max / sum of exp /
            // argmax); the four are merged in id order and one (max, sum, argmax) triple per (row, tile)
            // is stored.  The RMSNorm scalar of the row is applied first; [MASK] and padding are skipped.
            float* xch = reinterpret_cast<float*>(tiles);           // [32 rows][129]
            const int t = threadIdx.x - 64;                            // 0..127
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                if (ok) {
                    tmem_ld32(tmem_acc + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c * 32), v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) xch[j * 129 + q * 32 + lane] = ok ? __uint_as_float(v[j]) : 0.f;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const int m_l = t >> 2, part = t & 3;
                const int m = m0 + c * 32 + m_l;
                const float sc = rs.ssq ? sh->scale[c * 32 + m_l] : 1.0f;
                float mx = -INFINITY, sum = 0.f;
                int idx = 0x7fffffff;
#pragma unroll 8
                for (int i = 0; i < 32; ++i) {
                    const int n = n0 + part * 32 + i;
                    const int id = n + ce.tile0 * kBM;                  // vocabulary id (a shard starts at tile0)
                    const float l = xch[m_l * 129 + part * 32 + i] * sc;
                    if (n < N && id != ce.mask_id) {
                        if (l > mx) {
                            sum = sum * expf(mx - l) + 1.0f;            // first element: 0 * exp(-inf) + 1
                            mx = l;
                            idx = id;
                        } else {
                            sum += expf(l - mx);
                        }
                    }
                }
#pragma unroll
                for (int o = 1; o < 4; o <<= 1) {
                    const float om = __shfl_down_sync(0xffffffffu, mx, o, 4);
                    const float os = __shfl_down_sync(0xffffffffu, sum, o, 4);
                    const int oi = __shfl_down_sync(0xffffffffu, idx, o, 4);
                    if (part + o < 4) conf_merge(mx, sum, idx, om, os, oi);
                }
                if (ok && part == 0 && m < M) {
                    ConfPartial p;
                    p.m = mx; p.s = sum; p.idx = idx;
                    if (po.n == 0) {
                        ce.part[static_cast<size_t>(m) * n_tiles + n_tile] = p;
                    } else {
                        for (int r = 0; r < po.n; ++r) po.conf[r][static_cast<size_t>(m) * ce.tiles_total + ce.tile0 + n_tile] = p;
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            if (po.n > 0 && t == 0) tp_arrive_and_signal(po, gridDim.x * gridDim.y * gridDim.z);   // behind the loop's last barrier
        } else {
            // all MMAs have completed, so the stage ring is free: use it to hand the up values over.
            // Every epilogue warp executes every barrier, whether or not its wait succeeded.
            float* xch = reinterpret_cast<float*>(tiles);           // [64][33]
            const int f = n_tile * 64 + (q & 1) * 32 + lane;          // FFN feature of this lane's pair
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                if (ok) {
                    tmem_ld32(tmem_acc + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c * 32), v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                }
                if (ok && q >= 2) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) xch[((q & 1) * 32 + lane) * 33 + j] = __uint_as_float(v[j]);
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (ok && q < 2) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int m = m0 + c * 32 + j;
                        const float sc = rs.ssq ? sh->scale[c * 32 + j] : 1.0f;
                        if (m < M && f < N) {
                            const float gate = __uint_as_float(v[j]) * sc;
                            const float up = xch[((q & 1) * 32 + lane) * 33 + j] * sc;
                            act_out[static_cast<size_t>(m) * N + f] = __float2bfloat16_rn(gate / (1.0f + expf(-gate)) * up);
                        }
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
        }
    }
    pdl_wait();   // every thread: keeps completion of the launch chain transitive
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_barrier();   // neither CTA's shared memory or TMEM goes away while its peer may touch it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if constexpr (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(kTmemCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(kTmemCols) : "memory");
    }
}

__global__ void reduce_partials_kernel(const float* __restrict__ partial, int splits, size_t stride,
                                       float* __restrict__ out, size_t n) {
    const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float acc = partial[i];
    for (int s = 1; s < splits; ++s) acc += partial[s * stride + i];
    out[i] = acc;
}

// ---- tensor maps -----------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 [rows][K] row-major, box = 64 K-elements x box_rows rows, 128-byte swizzle, zero fill.
cudaError_t make_tmap_2d(CUtensorMap* out, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return cudaErrorNotSupported;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK), static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Packed weight [n_tiles * k_blocks][128][64] bf16: one tile = 16 KB contiguous, rows of 128 bytes.
cudaError_t make_tmap_packed(CUtensorMap* out, const void* base, int N, int K) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return cudaErrorNotSupported;
    const cuuint64_t ntiles = static_cast<cuuint64_t>((N + kBM - 1) / kBM) * ((K + kBK - 1) / kBK);
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(kBK), static_cast<cuuint64_t>(kBM), ntiles};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(kBK) * 2, static_cast<cuuint64_t>(kBK) * kBM * 2};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(kBK), static_cast<cuuint32_t>(kBM), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// dst[((tn * KB + kb) * 128 + r) * 64 + c] = src[(tn * 128 + r) * K + kb * 64 + c], zero beyond N or K
__global__ void pack_weight_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int N, int K,
                                   int KB) {
    const size_t chunk = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;   // 8 elements (16 bytes) each
    const size_t total = static_cast<size_t>((N + kBM - 1) / kBM) * KB * kBM * (kBK / 8);
    if (chunk >= total) return;
    const int c8 = static_cast<int>(chunk % (kBK / 8));
    const int r = static_cast<int>((chunk / (kBK / 8)) % kBM);
    const size_t tile = chunk / (kBK / 8) / kBM;
    const int kb = static_cast<int>(tile % KB);
    const int tn = static_cast<int>(tile / KB);
    const int n = tn * kBM + r, k = kb * kBK + c8 * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (n < N && k < K) v = *reinterpret_cast<const uint4*>(src + static_cast<size_t>(n) * K + k);   // K % 8 == 0
    reinterpret_cast<uint4*>(dst)[chunk] = v;
}

// Gate/up variant: src is [2F][K] = gate rows then up rows; packed tile t holds gate rows
// [64t, 64t+64) in its rows 0..63 and up rows [64t, 64t+64) in its rows 64..127.
__global__ void pack_gate_up_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int F, int K,
                                    int KB) {
    const size_t chunk = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    const size_t total = static_cast<size_t>((F + 63) / 64) * KB * kBM * (kBK / 8);
    if (chunk >= total) return;
    const int c8 = static_cast<int>(chunk % (kBK / 8));
    const int r = static_cast<int>((chunk / (kBK / 8)) % kBM);
    const size_t tile = chunk / (kBK / 8) / kBM;
    const int kb = static_cast<int>(tile % KB);
    const int t = static_cast<int>(tile / KB);
    const int f = t * 64 + (r & 63), k = kb * kBK + c8 * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (f < F && k < K) v = *reinterpret_cast<const uint4*>(src + (static_cast<size_t>(r < 64 ? 0 : F) + f) * K + k);
    reinterpret_cast<uint4*>(dst)[chunk] = v;
}

// CTA pairs (cta_group::2) are used whenever the number of weight tiles is even (ODB_GEMM_PAIR=0 turns them off).
bool pair_enabled() {
    static int v = -1;
    if (v < 0) {
        const char* e = getenv("ODB_GEMM_PAIR");
        v = e ? atoi(e) : 1;
    }
    return v != 0;
}

int pick_bn(int M, bool pair) {
    static int max_bn = -1;
    if (max_bn < 0) {
        const char* e = getenv("ODB_GEMM_MAX_BN");
        max_bn = e ? atoi(e) : 0;
    }
    // Up to 128 rows per tile two CTAs share an SM (one's epilogue overlaps the other's main loop).  A CTA
    // pair stages only half of the rows per CTA, so it affords 256-row tiles at the same occupancy.
    int bn = M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : pair ? 256 : 128;
    if (max_bn > 0 && bn > max_bn) bn = max_bn;
    return bn;
}

template <int BN, int EPI, bool PAIR>
cudaError_t launch_bn(const GemmArgs& a, cudaStream_t st) {
    constexpr bool SWIGLU = EPI == EPI_SWIGLU;
    constexpr int kBRows = PAIR ? BN / 2 : BN;
    CUtensorMap tmx;
    cudaError_t e = make_tmap_2d(&tmx, a.x, a.M, a.K, kBRows);
    if (e != cudaSuccess) return e;
    const int nkb_total = (a.K + kBK - 1) / kBK;
    const int nkb_per_split = (nkb_total + a.splits - 1) / a.splits;
    const uint32_t stage_bytes = kBM * kBK * 2 + kBRows * kBK * 2;
    // two CTAs per SM as long as two accumulators fit TMEM and a CTA stages at most 128 rows
    const uint32_t budget = kBRows <= 128 ? 100 * 1024 : 200 * 1024;
    int stages = static_cast<int>(budget / stage_bytes);
    if (stages > 16) stages = 16;
    if (stages > nkb_per_split) stages = nkb_per_split < 2 ? 2 : nkb_per_split;
    const size_t smem = static_cast<size_t>(stages) * stage_bytes + sizeof(GemmShared) + 1024;
    static std::atomic<unsigned long long> attr_done{0};
    e = set_smem_limit_once(attr_done, gemm_kernel<BN, EPI, PAIR>, 227 * 1024);
    if (e != cudaSuccess) return e;
    // SWIGLU: N is the FFN width and a weight tile holds 64 gate + 64 up rows
    dim3 grid(SWIGLU ? (a.N + 63) / 64 : (a.N + kBM - 1) / kBM, (a.M + BN - 1) / BN, a.splits);
    static int l2_prefetch = -1;
    if (l2_prefetch < 0) {
        const char* env = getenv("ODB_GEMM_L2_PREFETCH");
        l2_prefetch = env ? atoi(env) : 0;   // measured: prefetching into L2 slows the step down
    }
    if constexpr (PAIR) {
        if (grid.x & 1) return cudaErrorInvalidValue;
        const int tiles_x = static_cast<int>(grid.x), tiles_y = static_cast<int>(grid.y);
        // row tiles per group: 8 x 256 rows x K x 2 B stay in L2 (measured at 128 row tiles: groups of 2 / 4 / 8 / 16
        // give 430 / 414 / 404 / 407 ms of GEMM time per refresh, no grouping 475, one row tile per weight pass 462)
        const int group = tiles_y < 8 ? tiles_y : 8;
        const int m_groups = (tiles_y + group - 1) / group;
        if (static_cast<size_t>(tiles_x / 2) * m_groups * a.splits > 65535) return cudaErrorInvalidValue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2, group, (tiles_x / 2) * m_groups * a.splits);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;   // neighbouring weight tiles form the pair
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pdl_enabled() ? 2 : 1;
        return cudaLaunchKernelEx(&cfg, gemm_kernel<BN, EPI, PAIR>, a.tmap_w, tmx, a.partial, a.act_out, a.row_scale, a.conf,
                                  a.M, a.N, nkb_total, nkb_per_split, stages, pdl_enabled() ? l2_prefetch : 0, tiles_x, tiles_y, a.status, a.peers);
    } else {
        return launch_kernel(gemm_kernel<BN, EPI, PAIR>, grid, dim3(kThreads), smem, st, a.tmap_w, tmx, a.partial, a.act_out,
                             a.row_scale, a.conf, a.M, a.N, nkb_total, nkb_per_split, stages,
                             pdl_enabled() ? l2_prefetch : 0, 0, 0, a.status, a.peers);
    }
}

template <int EPI>
cudaError_t launch_epi(const GemmArgs& a, int bn, bool pair, cudaStream_t st) {
    if (pair) {
        switch (bn) {
            case 32: return launch_bn<32, EPI, true>(a, st);
            case 64: return launch_bn<64, EPI, true>(a, st);
            case 128: return launch_bn<128, EPI, true>(a, st);
            default: return launch_bn<256, EPI, true>(a, st);
        }
    }
    switch (bn) {
        case 32: return launch_bn<32, EPI, false>(a, st);
        case 64: return launch_bn<64, EPI, false>(a, st);
        case 128: return launch_bn<128, EPI, false>(a, st);
        default: return launch_bn<256, EPI, false>(a, st);
    }
}

// Whether a projection of M activation rows with n_tiles weight tiles runs as CTA pairs.  Measured on the
// 8B shape: with many rows (refresh, 768..1024 rows: tensor/L2 bound) pairs with 256-row tiles are 11 %
// faster than single CTAs with 128-row tiles; up to 128 rows (decode steps: HBM bound) the pair's extra
// synchronisation costs more than the halved activation traffic saves (3.55 vs 3.41 ms at 32 rows).
bool use_pair(int M, int n_tiles) {
    static int min_rows = -1;
    if (min_rows < 0) {
        const char* e = getenv("ODB_GEMM_PAIR_MIN_ROWS");
        min_rows = e ? atoi(e) : 128;
    }
    return pair_enabled() && M > min_rows && (n_tiles & 1) == 0;
}

}  // namespace

cudaError_t make_weight_tmap(CUtensorMap* out, const void* w, int N, int K) { return make_tmap_packed(out, w, N, K); }

cudaError_t make_rows_tmap(CUtensorMap* out, const void* base, int rows, int cols, int box_rows) {
    return make_tmap_2d(out, base, rows, cols, box_rows);
}

size_t packed_weight_bytes(int N, int K) {
    return static_cast<size_t>((N + kBM - 1) / kBM) * ((K + kBK - 1) / kBK) * kBM * kBK * 2;
}

size_t packed_gate_up_bytes(int F, int K) {
    return static_cast<size_t>((F + 63) / 64) * ((K + kBK - 1) / kBK) * kBM * kBK * 2;
}

cudaError_t make_gate_up_tmap(CUtensorMap* out, const void* w, int F, int K) {
    return make_tmap_packed(out, w, ((F + 63) / 64) * kBM, K);
}

cudaError_t launch_pack_gate_up(const void* src, void* dst, int F, int K, cudaStream_t st) {
    const int KB = (K + kBK - 1) / kBK;
    const size_t chunks = packed_gate_up_bytes(F, K) / 16;
    pack_gate_up_kernel<<<static_cast<unsigned>((chunks + 255) / 256), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(src), static_cast<__nv_bfloat16*>(dst), F, K, KB);
    return cudaGetLastError();
}

cudaError_t launch_pack_weight(const void* src, void* dst, int N, int K, cudaStream_t st) {
    const int KB = (K + kBK - 1) / kBK;
    const size_t chunks = packed_weight_bytes(N, K) / 16;
    pack_weight_kernel<<<static_cast<unsigned>((chunks + 255) / 256), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(src), static_cast<__nv_bfloat16*>(dst), N, K, KB);
    return cudaGetLastError();
}

bool pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char* e = getenv("ODB_PDL");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v != 0;
}

static int target_ctas() {
    static int v = 0;
    if (!v) {
        const char* e = getenv("ODB_GEMM_TARGET_CTAS");
        v = e ? atoi(e) : 2 * 148;
        if (v < 1) v = 2 * 148;
    }
    return v;
}

int gemm_pick_splits(int M, int N, int K) {
    const int n_tiles = (N + kBM - 1) / kBM;
    const int bn = pick_bn(M, use_pair(M, n_tiles));
    const int tiles = n_tiles * ((M + bn - 1) / bn);
    const int nkb = (K + kBK - 1) / kBK;
    // all work units must be resident at once (two CTA slots per SM) and equal in size: a
    // second, partly filled wave would double the kernel's time
    if (M > 128) {
        // many rows (refresh): compute bound, and every K split costs M x N fp32 partials written and
        // read back, so split only when the tiles alone cannot occupy the SMs
        static int big_target = 0;
        if (!big_target) {
            const char* e = getenv("ODB_GEMM_BIG_TARGET_CTAS");
            big_target = e ? atoi(e) : 296;
        }
        int sp = tiles >= big_target ? 1 : big_target / tiles;
        if (sp > nkb / 8) sp = nkb / 8;
        return sp < 1 ? 1 : sp;
    }
    int splits = target_ctas() / tiles;
    if (splits > nkb / 4) splits = nkb / 4;
    if (splits > 16) splits = 16;
    if (splits < 1) splits = 1;
    // no empty split: ceil(nkb/splits) * (splits-1) < nkb
    while (splits > 1 && ((nkb + splits - 1) / splits) * (splits - 1) >= nkb) --splits;
    return splits;
}

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st) {
    const bool swiglu = a.act_out != nullptr;
    // The gate/up projection has no K split to balance its CTAs over the SMs (192 tiles on 148 SMs at the 8B
    // shape: some SMs stage for two CTAs), so from 65 rows up it also runs as pairs, each CTA staging half of
    // the activation rows (measured at 128 rows: step 4.84 -> 4.72 ms; at 32 rows pairs lose, 3.27 vs 3.26).
    const bool pair = use_pair(a.M, swiglu ? (a.N + 63) / 64 : (a.N + kBM - 1) / kBM) ||
                      (swiglu && a.M > 64 && pair_enabled() && (((a.N + 63) / 64) & 1) == 0);
    const int bn = pick_bn(a.M, pair);
    if (swiglu) {
        if (a.splits != 1) return cudaErrorInvalidValue;
        return launch_epi<EPI_SWIGLU>(a, bn, pair, st);
    }
    if (a.conf.part) {
        if (a.splits != 1) return cudaErrorInvalidValue;
        return launch_epi<EPI_CONF>(a, bn, pair, st);
    }
    return launch_epi<EPI_PARTIAL>(a, bn, pair, st);
}

cudaError_t launch_reduce_partials(const float* partial, int splits, size_t stride, float* out, size_t n,
                                   cudaStream_t st) {
    reduce_partials_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(partial, splits, stride, out, n);
    return cudaGetLastError();
}

}  // namespace odb
