// Persistent decode-step kernel: the whole forward of one block-decode step in ONE cooperative launch.
//
// Why: a decode step of the 8B shape streams 15 GB of weights through four projections per layer.  As separate
// kernels the projections reach 92 % of the HBM rate when chained, but every short kernel between them
// (RMSNorm, RoPE, attention, merge) is a synchronisation point at which the weight stream stops.  Here one CTA
// per SM stays resident for the whole step:
//   * warp 0 (one thread) is the TMA producer.  It walks the CTA's share of the weight tiles of ALL projections
//     of the step in order and keeps a ring of shared-memory stages full; it does not stop at a phase boundary:
//     while the consumers are in a short phase it fills the ring with the next projection's weights.  Only the
//     small activation tile of a stage has to wait until the phase that produces it is complete.
//   * warp 1 (one thread) issues the tcgen05 MMAs (weights = 128-row operand, activation rows = N operand,
//     fp32 accumulator in TMEM, two accumulators so that the next output tile starts while one is read back).
//   * warps 2..5 read accumulators back (fp32 partial tiles, or the LM head's softmax statistics) and run the
//     short phases between the projections: residual + split reduction + RMSNorm operand, RoPE, block-query
//     attention (the same body as the stand-alone kernel), key-split merge, SwiGLU.
// Work split: the (weight tile, k-block) units of a projection are cut into one contiguous range per CTA
// (even to within one unit, whatever the number of tiles); a CTA's range covers parts of one to three output
// tiles, each part gives one fp32 partial tile, and the consumer of the projection adds the parts of a tile
// in CTA order, so results do not depend on timing.
// Phases are separated by grid-wide barriers: one word per barrier (zeroed before the launch), one arrival per
// CTA, bounded polling.  The launch is cooperative with one CTA per SM, so every CTA a barrier waits for is
// resident.  Every wait in the kernel (mbarrier, grid barrier) is bounded: on expiry ODB_ERR_TIMEOUT is recorded
// in the status word, which every poller also watches, all roles of all CTAs stop, TMEM is released and the
// kernel exits normally.
#include <stdlib.h>

#include "odb_internal.cuh"
#include "tcgen05_common.cuh"
#include "attention_body.cuh"

namespace odb {

namespace {

constexpr int kPThreads = 192;        // warp 0 producer, warp 1 MMA issuer, warps 2..5 workers
constexpr int kWorkers = 128;
constexpr int kMaxStages = 12;
constexpr int kAccCols = 128;         // TMEM columns per accumulator (two accumulators)

struct alignas(8) PShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort;
    float red[8];
    float scale[128];
};

struct WorkerSync {
    static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void red_release_add(unsigned int* p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// ---- the fixed work split -------------------------------------------------------------------------------
// Units of a projection, tile-major: u = tile * nkb + kb.  CTA c of G owns [c U / G, (c + 1) U / G).
__device__ __forceinline__ int owner_of(long long u, long long U, int G) {
    return static_cast<int>(((u + 1) * G - 1) / U);
}
// the parts of output tile `tile`: the CTAs first .. first + n - 1 each hold one partial tile, in k order
__device__ __forceinline__ void tile_parts(int tile, int nkb, int n_tiles, int G, int& first, int& n) {
    const long long U = static_cast<long long>(n_tiles) * nkb;
    first = owner_of(static_cast<long long>(tile) * nkb, U, G);
    n = owner_of(static_cast<long long>(tile + 1) * nkb - 1, U, G) - first + 1;
}

// One contiguous piece of a CTA's range inside one output tile.
struct Segment {
    int g, tile, kb0, nkb, part;   // projection, output tile, first k-block, k-blocks, index of the partial tile
};

// Walks the segments of CTA `cta` over all projections, in order.
struct Schedule {
    const PGemmDesc* gemms;
    int n_gemms, G, cta;
    int g;
    long long u, hi;
    int nkb_g, n_tiles_g, conf_g, use_g;

    __device__ void init(const PGemmDesc* gm, int n, int G_, int cta_) {
        gemms = gm; n_gemms = n; G = G_; cta = cta_;
        g = -1; u = hi = 0;
    }
    __device__ bool load_gemm() {   // advances to the next projection with a non-empty range
        while (u >= hi) {
            if (++g >= n_gemms) return false;
            n_tiles_g = gemms[g].n_tiles; nkb_g = gemms[g].nkb; conf_g = gemms[g].conf; use_g = gemms[g].g_use;
            if (cta >= use_g) {
                u = hi = 0;       // a tiny projection is divided over the first use_g CTAs only
            } else if (conf_g) {   // whole tiles: the epilogue reduces a complete column of logits
                u = static_cast<long long>(cta) * n_tiles_g / use_g * nkb_g;
                hi = static_cast<long long>(cta + 1) * n_tiles_g / use_g * nkb_g;
            } else {
                const long long U = static_cast<long long>(n_tiles_g) * nkb_g;
                u = cta * U / use_g;
                hi = (cta + 1) * U / use_g;
            }
        }
        return true;
    }
    __device__ bool next(Segment& s) {
        if (!load_gemm()) return false;
        s.g = g;
        s.tile = static_cast<int>(u / nkb_g);
        s.kb0 = static_cast<int>(u % nkb_g);
        long long n = nkb_g - s.kb0;
        if (n > hi - u) n = hi - u;
        s.nkb = static_cast<int>(n);
        s.part = conf_g ? 0 : cta - owner_of(static_cast<long long>(s.tile) * nkb_g, static_cast<long long>(n_tiles_g) * nkb_g, use_g);
        u += n;
        return true;
    }
};

// grid barriers of the step, in order; `per_layer` barriers per layer
__device__ __forceinline__ int bars_per_layer(int ksplit) { return ksplit > 1 ? 10 : 9; }
// the barrier after which the activation operand of projection g is complete
__device__ __forceinline__ int gate_of(int g, int n_layers, int ksplit) {
    const int nb = bars_per_layer(ksplit);
    const int l = g >> 2, j = g & 3;
    if (l >= n_layers) return n_layers * nb;                          // LM head: after the final norm
    const int o_gate = ksplit > 1 ? 4 : 3;
    return l * nb + (j == 0 ? 0 : j == 1 ? o_gate : j == 2 ? o_gate + 2 : o_gate + 4);
}

// Polls until barrier word `id` has reached G arrivals.  One thread.  False on abort / expiry.
__device__ __forceinline__ bool poll_barrier(const StepPersistentArgs& A, int id, int G, volatile int* cta_abort) {
    const unsigned int* w = A.bars + id;
    if (ld_acquire_u32(w) >= static_cast<unsigned int>(G)) return true;
    const long long t0 = clock64();
    unsigned int spins = 0;
    while (ld_acquire_u32(w) < static_cast<unsigned int>(G)) {
        if (*cta_abort) return false;
        if ((++spins & 15u) == 0) {
            if (*reinterpret_cast<volatile int*>(A.status) != 0) { *cta_abort = 1; return false; }   // another CTA gave up
            if (clock64() - t0 > kWaitLimitCycles) {
                *cta_abort = 1;
                atomicExch(A.status, ODB_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// mbarrier wait that also watches the step's status word (another CTA's expiry ends this one's waits too)
__device__ __forceinline__ bool pwait(uint64_t* bar, uint32_t parity, volatile int* cta_abort, int* status) {
    if (mbar_try_wait_parity(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned int spins = 0;
    while (!mbar_try_wait_parity(bar, parity)) {
        if (*cta_abort) return false;
        if ((++spins & 63u) == 0) {
            if (*reinterpret_cast<volatile int*>(status) != 0) { *cta_abort = 1; return false; }
            if (clock64() - t0 > kWaitLimitCycles) {
                *cta_abort = 1;
                atomicExch(status, ODB_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// ---- the short phases (128 worker threads, tid 0..127) -----------------------------------------------------

constexpr int kMaxParts = 8;   // partial tiles per output tile (the host's split keeps it below)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ void mul4(float4& a, float s) { a.x *= s; a.y *= s; a.z *= s; a.w *= s; }

// sum over the parts of the output tile that holds column `col` of row `row`: partial[part][M][Np]
__device__ __forceinline__ float4 sum_parts(const float* partial, const PGemmDesc& pg, int M, int row, int col) {
    int first, n;
    tile_parts(col >> 7, pg.nkb, pg.n_tiles, pg.g_use, first, n);
    const size_t Np = static_cast<size_t>(pg.n_tiles) * 128;
    const float* p = partial + static_cast<size_t>(row) * Np + col;
    float4 t[kMaxParts];
#pragma unroll
    for (int s = 0; s < kMaxParts; ++s)
        if (s < n) t[s] = ldcg4(p + static_cast<size_t>(s) * M * Np);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s = 0; s < kMaxParts; ++s)
        if (s < n) add4(acc, t[s]);
    return acc;
}

// Residual stream += the parts of the preceding projection (prev), or := the token embeddings (layer 0);
// operand a = bf16(h * gain); per (row, 1024-column slice) the sum of squares for the consumer's 1 / rms.
__device__ __noinline__ void norm_phase(const StepPersistentArgs& A, PShared* sh, int tid, int cta, int G, const float* gain,
                           const PGemmDesc* prev, bool from_embed) {
    const int d = A.d, slices = (d + kNormSliceCols - 1) / kNormSliceCols;
    const int n_items = A.M * slices;
    const int warp = tid >> 5, lane = tid & 31;
    for (int it = cta; it < n_items; it += G) {
        const int row = it / slices, sl = it % slices;
        float ss = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int i = sl * (kNormSliceCols / 4) + half * kWorkers + tid;   // float4 index within the row
            if (i < (d >> 2)) {
                const int col = i << 2;
                float4 v;
                if (from_embed) {
                    const uint2 e = *reinterpret_cast<const uint2*>(A.embed + static_cast<size_t>(A.row_tok[row]) * d + col);
                    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.x));
                    const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.y));
                    v = make_float4(lo.x, lo.y, hi.x, hi.y);
                } else {
                    v = ldcg4(A.h + static_cast<size_t>(row) * d + col);
                }
                if (prev) add4(v, sum_parts(A.partial, *prev, A.M, row, col));
                if (prev || from_embed) *reinterpret_cast<float4*>(A.h + static_cast<size_t>(row) * d + col) = v;
                ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                if (gain) {
                    const float4 g = *reinterpret_cast<const float4*>(gain + col);
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z * g.z, v.w * g.w);
                    uint2 pk;
                    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
                    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(A.a + static_cast<size_t>(row) * d + col) = pk;
                }
            }
        }
        ss = warp_sum(ss);
        WorkerSync::sync();
        if (lane == 0) sh->red[warp] = ss;
        WorkerSync::sync();
        if (tid == 0) A.ssq[static_cast<size_t>(row) * slices + sl] = sh->red[0] + sh->red[1] + sh->red[2] + sh->red[3];
    }
}

__device__ __forceinline__ float row_scale_cg(const StepPersistentArgs& A, int row) {
    const int slices = (A.d + kNormSliceCols - 1) / kNormSliceCols;
    float t = 0.f;
    for (int i = 0; i < slices; ++i) t += __ldcg(A.ssq + static_cast<size_t>(row) * slices + i);
    return 1.0f / sqrtf(t * (1.0f / static_cast<float>(A.d)) + A.rms_eps);
}

__device__ __forceinline__ uint2 pack4(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(c, d);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    return pk;
}

// Parts of the QKV projection -> x 1/rms -> rotate q and k (rotate-half pairing) -> bf16 q, k, v rows.
__device__ __noinline__ void rope_phase(const StepPersistentArgs& A, const PGemmDesc& pq, int tid, int cta, int G) {
    const int d = A.d, half = A.hd / 2;
    const int quads = d / 8, chunks = (quads + kWorkers - 1) / kWorkers;
    const int n_items = A.M * chunks;
    for (int it = cta; it < n_items; it += G) {
        const int row = it / chunks;
        const int t = ((it % chunks) * kWorkers + tid) * 4;       // first of four rotation pairs
        if (t >= d / 2) continue;
        const int head = t / half, i = t % half;
        const int e0 = head * A.hd + i, e1 = e0 + half;
        float4 q0 = sum_parts(A.partial, pq, A.M, row, e0), q1 = sum_parts(A.partial, pq, A.M, row, e1);
        float4 k0 = sum_parts(A.partial, pq, A.M, row, d + e0), k1 = sum_parts(A.partial, pq, A.M, row, d + e1);
        float4 v0 = sum_parts(A.partial, pq, A.M, row, 2 * d + e0), v1 = sum_parts(A.partial, pq, A.M, row, 2 * d + e1);
        const float inv = row_scale_cg(A, row);
        const float2* rope = A.rope + static_cast<size_t>(A.row_pos[row]) * half;
        const float4 c01 = *reinterpret_cast<const float4*>(rope + i);
        const float4 c23 = *reinterpret_cast<const float4*>(rope + i + 2);
        mul4(q0, inv); mul4(q1, inv); mul4(k0, inv); mul4(k1, inv); mul4(v0, inv); mul4(v1, inv);
        const size_t o = static_cast<size_t>(row) * d;
        *reinterpret_cast<uint2*>(A.q + o + e0) = pack4(q0.x * c01.x - q1.x * c01.y, q0.y * c01.z - q1.y * c01.w,
                                                        q0.z * c23.x - q1.z * c23.y, q0.w * c23.z - q1.w * c23.w);
        *reinterpret_cast<uint2*>(A.q + o + e1) = pack4(q1.x * c01.x + q0.x * c01.y, q1.y * c01.z + q0.y * c01.w,
                                                        q1.z * c23.x + q0.z * c23.y, q1.w * c23.z + q0.w * c23.w);
        *reinterpret_cast<uint2*>(A.k + o + e0) = pack4(k0.x * c01.x - k1.x * c01.y, k0.y * c01.z - k1.y * c01.w,
                                                        k0.z * c23.x - k1.z * c23.y, k0.w * c23.z - k1.w * c23.w);
        *reinterpret_cast<uint2*>(A.k + o + e1) = pack4(k1.x * c01.x + k0.x * c01.y, k1.y * c01.z + k0.y * c01.w,
                                                        k1.z * c23.x + k0.z * c23.y, k1.w * c23.z + k0.w * c23.w);
        *reinterpret_cast<uint2*>(A.v + o + e0) = pack4(v0.x, v0.y, v0.z, v0.w);
        *reinterpret_cast<uint2*>(A.v + o + e1) = pack4(v1.x, v1.y, v1.z, v1.w);
    }
}

// Merge of the key splits of the attention, in split order (the arithmetic of attention_combine_kernel).
__device__ __noinline__ void combine_phase(const StepPersistentArgs& A, int tid, int cta, int G) {
    const int hd = A.hd, H = A.H, M = A.M, ks = A.ksplit;
    const int tpi = hd / 4, ipr = kWorkers / tpi;               // threads per (row, head) item, items per round
    const int n_items = M * H;
    const size_t zs = static_cast<size_t>(M) * H;
    for (int b0 = cta * ipr; b0 < n_items; b0 += G * ipr) {
        const int item = b0 + tid / tpi;
        if (item >= n_items) continue;
        const int d4 = (tid % tpi) * 4;
        const size_t base = item;                                  // row * H + head
        float2 ml[8];
        float4 v[8];
#pragma unroll
        for (int z = 0; z < 8; ++z)
            if (z < ks) ml[z] = __ldcg(reinterpret_cast<const float2*>(A.part_ml + (z * zs + base) * 2));
#pragma unroll
        for (int z = 0; z < 8; ++z)
            if (z < ks) v[z] = ldcg4(A.part_o + (z * zs + base) * hd + d4);
        float mmax = -INFINITY;
#pragma unroll
        for (int z = 0; z < 8; ++z)
            if (z < ks && ml[z].y > 0.f) mmax = fmaxf(mmax, ml[z].x);
        float L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int z = 0; z < 8; ++z) {
            if (z < ks && ml[z].y > 0.f) {
                const float wt = exp2f(ml[z].x - mmax);
                L += ml[z].y * wt;
                acc.x += v[z].x * wt; acc.y += v[z].y * wt; acc.z += v[z].z * wt; acc.w += v[z].w * wt;
            }
        }
        const float inv = L > 0.f ? 1.0f / L : 0.f;
        *reinterpret_cast<uint2*>(A.o + base * hd + d4) = pack4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
}

// Parts of the gate/up projection (tile t = 64 gate features then their 64 up features) -> x 1/rms ->
// g = bf16(silu(gate) * up).
__device__ __noinline__ void swiglu_phase(const StepPersistentArgs& A, const PGemmDesc& pg, int tid, int cta, int G) {
    const int F = A.F, chunks = (F + 4 * kWorkers - 1) / (4 * kWorkers);
    const int n_items = A.M * chunks;
    for (int it = cta; it < n_items; it += G) {
        const int row = it / chunks;
        const int f = ((it % chunks) * kWorkers + tid) * 4;
        if (f >= F) continue;
        const int col = (f >> 6) * 128 + (f & 63);
        const float4 gate = sum_parts(A.partial, pg, A.M, row, col);
        const float4 up = sum_parts(A.partial, pg, A.M, row, col + 64);
        const float sc = row_scale_cg(A, row);
        const float g0 = gate.x * sc, g1 = gate.y * sc, g2 = gate.z * sc, g3 = gate.w * sc;
        *reinterpret_cast<uint2*>(A.g + static_cast<size_t>(row) * F + f) =
            pack4(g0 / (1.0f + expf(-g0)) * (up.x * sc), g1 / (1.0f + expf(-g1)) * (up.y * sc),
                  g2 / (1.0f + expf(-g2)) * (up.z * sc), g3 / (1.0f + expf(-g3)) * (up.w * sc));
    }
}

// Attention work items (query tile, head, key split) of this CTA.  The cached key tiles of the first item are
// requested before `wait_rope` (the grid barrier behind the RoPE phase) is called.
template <int HD, class WaitFn>
__device__ __noinline__ void attention_phase(const StepPersistentArgs& A, const AttnArgs& aa, uint8_t* scratch, int tid, int cta, int G,
                                             WaitFn wait_rope) {
    const int n_attn = A.n_qtiles * A.H * A.ksplit;
    for (int it = cta; it < n_attn; it += G) {
        const int z = it % A.ksplit, head = (it / A.ksplit) % A.H, qt = it / (A.ksplit * A.H);
        const QTile t = A.tiles[qt];
        attention_item<HD, WorkerSync>(aa, t, head, z, tid, scratch, true, wait_rope);
        WorkerSync::sync();                              // the tiles in shared memory are free for the next item
    }
    wait_rope();
}

// ---- the kernel -----------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kPThreads, 1) step_persistent_kernel(const __grid_constant__ StepPersistentArgs A) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int BN = A.BN, S = A.stages;
    const uint32_t kABytes = kBM * kBK * 2;
    const uint32_t stage_bytes = kABytes + static_cast<uint32_t>(BN) * kBK * 2;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* scratch = ring + static_cast<size_t>(S) * stage_bytes;                 // attention tiles / logit transpose
    PShared* sh = reinterpret_cast<PShared*>(scratch + A.scratch_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = static_cast<int>(gridDim.x), cta = static_cast<int>(blockIdx.x);
    const int n_gemms = 4 * A.n_layers + (A.with_lm ? 1 : 0);   // the table always has the LM head's slot (its gain is the final norm's)
    volatile int* cta_abort = &sh->abort;

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&sh->full[i], 1);
            mbar_init(&sh->empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->acc_full[i], 1);
            mbar_init(&sh->acc_empty[i], 4);      // one arrival per worker warp
        }
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // whole warp: both accumulators' TMEM columns
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(2 * kAccCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer: weight tiles run ahead of the phase, activation tiles follow their gate ----
            Schedule sw, sa;
            sw.init(A.gemms, n_gemms, G, cta);
            sa.init(A.gemms, n_gemms, G, cta);
            Segment segw{}, sega{};
            int lw = 0, la = 0;                      // k-blocks left in the current segment of each cursor
            bool have_w = sw.next(segw), have_a = sa.next(sega);
            if (have_w) lw = segw.nkb;
            if (have_a) la = sega.nkb;
            long long it_w = 0, it_a = 0;            // stages given their weight tile / their activation tile
            int gate_known = -1;                     // highest barrier id seen complete
            long long t_idle = clock64();
            while (have_a) {
                bool progress = false;
                if (have_w) {
                    const int st = static_cast<int>(it_w % S);
                    const uint32_t ph = static_cast<uint32_t>(it_w / S) & 1u;
                    if (mbar_try_wait_parity(&sh->empty[st], ph ^ 1u)) {
                        const PGemmDesc* pg = A.gemms + segw.g;
                        mbar_expect_tx(&sh->full[st], stage_bytes);
                        tma_load_3d(ring + static_cast<size_t>(st) * stage_bytes, &pg->tmap_w, &sh->full[st], 0, 0,
                                    segw.tile * pg->nkb + segw.kb0 + (segw.nkb - lw), kEvictFirst);
                        ++it_w;
                        if (--lw == 0) {
                            have_w = sw.next(segw);
                            if (have_w) lw = segw.nkb;
                        }
                        progress = true;
                    }
                }
                if (it_a < it_w) {
                    const int gate = gate_of(sega.g, A.n_layers, A.ksplit);
                    bool open = gate <= gate_known;
                    if (!open && ld_acquire_u32(A.bars + gate) >= static_cast<unsigned int>(G)) {
                        gate_known = gate;
                        fence_proxy_async_all();     // the operand was written with ordinary stores by other CTAs
                        open = true;
                    }
                    if (open) {
                        const int st = static_cast<int>(it_a % S);
                        const PGemmDesc* pg = A.gemms + sega.g;
                        tma_load_2d(ring + static_cast<size_t>(st) * stage_bytes + kABytes, &pg->tmap_x, &sh->full[st],
                                    (sega.kb0 + (sega.nkb - la)) * kBK, 0, kEvictLast);
                        ++it_a;
                        if (--la == 0) {
                            have_a = sa.next(sega);
                            if (have_a) la = sega.nkb;
                        }
                        progress = true;
                    }
                }
                if (progress) {
                    t_idle = clock64();
                } else {
                    if (*cta_abort) break;
                    if (*reinterpret_cast<volatile int*>(A.status) != 0) { *cta_abort = 1; break; }
                    if (clock64() - t_idle > kWaitLimitCycles) {
                        *cta_abort = 1;
                        atomicExch(A.status, ODB_ERR_TIMEOUT);
                        break;
                    }
                }
            }
            if (*cta_abort) {
                // stages whose weight tile was requested but whose activation tile never will be: their barrier
                // cannot complete, but the weight copies must land before the shared memory goes away
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {   // ~1 ms: far beyond any copy in flight
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            const uint32_t idesc = make_instr_desc(kBM, BN);
            Schedule sm;
            sm.init(A.gemms, n_gemms, G, cta);
            Segment seg{};
            long long it = 0, seg_idx = 0;
            bool ok = true;
            while (ok && sm.next(seg)) {
                const int buf = static_cast<int>(seg_idx & 1);
                ok = pwait(&sh->acc_empty[buf], (static_cast<uint32_t>(seg_idx >> 1) & 1u) ^ 1u, cta_abort, A.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tacc = tmem_base + static_cast<uint32_t>(buf * kAccCols);
                for (int i = 0; i < seg.nkb && ok; ++i, ++it) {
                    const int st = static_cast<int>(it % S);
                    ok = pwait(&sh->full[st], static_cast<uint32_t>(it / S) & 1u, cta_abort, A.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(ring + static_cast<size_t>(st) * stage_bytes);
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k = 0; k < kBK / kUmmaK; ++k)
                        umma_bf16(tacc, make_smem_desc(a_addr + k * kUmmaK * 2), make_smem_desc(b_addr + k * kUmmaK * 2), idesc,
                                  (i > 0 || k > 0) ? 1u : 0u);
                    umma_commit(&sh->empty[st]);
                }
                if (ok) umma_commit(&sh->acc_full[buf]);
                ++seg_idx;
            }
        }
    } else {
        // ---- workers: accumulator read-back and the short phases ----
        const int tid = threadIdx.x - 64;
        const int q = warp & 3;                         // TMEM lanes 32 q .. 32 q + 31
        Schedule se;
        se.init(A.gemms, n_gemms, G, cta);
        Segment seg{};
        bool have = se.next(seg);
        long long seg_idx = 0;
        int bar_id = 0;
        bool ok = true;

        auto arrive = [&]() {
            __threadfence();
            fence_proxy_async_all();                    // our ordinary stores before other CTAs' TMA loads of them
            WorkerSync::sync();
            if (tid == 0) red_release_add(A.bars + bar_id, 1u);
        };
        auto wait = [&]() {
            if (tid == 0) poll_barrier(A, bar_id, G, cta_abort);
            WorkerSync::sync();
            ++bar_id;
            if (*cta_abort) ok = false;
        };
        // read back every segment this CTA has in projection g
        auto epilogue = [&](int g) {
            const PGemmDesc& pg = A.gemms[g];
            const size_t Np = static_cast<size_t>(pg.n_tiles) * 128;
            if (pg.conf && ok) {
                for (int i = tid; i < BN; i += kWorkers) sh->scale[i] = i < A.M ? row_scale_cg(A, i) : 1.0f;
                WorkerSync::sync();
            }
            while (have && seg.g == g) {
                const int buf = static_cast<int>(seg_idx & 1);
                const bool got = ok && pwait(&sh->acc_full[buf], static_cast<uint32_t>(seg_idx >> 1) & 1u, cta_abort, A.status);
                if (got) tc_fence_after();
                const uint32_t tacc = tmem_base + static_cast<uint32_t>(buf * kAccCols) + (static_cast<uint32_t>(q * 32) << 16);
                if (!pg.conf) {
                    if (got) {
                        float* out = A.partial + static_cast<size_t>(seg.part) * A.M * Np + static_cast<size_t>(seg.tile) * 128 + q * 32 + lane;
#pragma unroll 1
                        for (int c = 0; c < BN / 32; ++c) {
                            uint32_t v[32];
                            tmem_ld32(tacc + static_cast<uint32_t>(c * 32), v);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int m = c * 32 + j;
                                if (m < A.M) out[static_cast<size_t>(m) * Np] = __uint_as_float(v[j]);
                            }
                        }
                    }
                } else {
                    // LM head: softmax statistics of this vocabulary tile per row; the logits never leave the SM
                    float* xch = reinterpret_cast<float*>(scratch);   // [32 rows][129]
                    const int n0 = seg.tile * 128;
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        uint32_t v[32];
                        if (got) {
                            tmem_ld32(tacc + static_cast<uint32_t>(c * 32), v);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) xch[j * 129 + q * 32 + lane] = got ? __uint_as_float(v[j]) : 0.f;
                        WorkerSync::sync();
                        const int m_l = tid >> 2, part = tid & 3;
                        const int m = c * 32 + m_l;
                        const float sc = sh->scale[c * 32 + m_l];
                        float mx = -INFINITY, sum = 0.f;
                        int idx = 0x7fffffff;
#pragma unroll 8
                        for (int i = 0; i < 32; ++i) {
                            const int n = n0 + part * 32 + i;
                            const float l = xch[m_l * 129 + part * 32 + i] * sc;
                            if (n < A.vocab && n != A.mask_id) {
                                if (l > mx) {
                                    sum = sum * expf(mx - l) + 1.0f;
                                    mx = l;
                                    idx = n;
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
                        if (got && part == 0 && m < A.M) {
                            ConfPartial p;
                            p.m = mx; p.s = sum; p.idx = idx;
                            A.conf_part[static_cast<size_t>(m) * pg.n_tiles + seg.tile] = p;
                        }
                        WorkerSync::sync();
                    }
                }
                if (got) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&sh->acc_empty[buf])) : "memory");
                } else {
                    ok = false;
                }
                ++seg_idx;
                have = se.next(seg);
            }
        };

        AttnArgs aa;
        aa.tiles = A.tiles; aa.n_tiles = A.n_qtiles;
        aa.q = A.q; aa.k = A.k; aa.v = A.v; aa.cache = A.cache; aa.row_flags = A.row_flags; aa.o = A.o;
        aa.part_o = A.part_o; aa.part_ml = A.part_ml;
        aa.n_layers = A.n_layers; aa.H = A.H; aa.hd = A.hd; aa.max_seq = A.max_seq; aa.M = A.M; aa.ksplit = A.ksplit;
        aa.early = 1;
        aa.pf = L2Prefetch{nullptr, 0};
        for (int l = 0; l < A.n_layers && ok; ++l) {
            const PGemmDesc* g0 = A.gemms + 4 * l;
            // residual (+ the previous layer's down projection, or the embeddings) -> operand of QKV
            norm_phase(A, sh, tid, cta, G, g0[0].gain, l > 0 ? g0 - 1 : nullptr, l == 0);
            arrive(); wait();
            epilogue(4 * l);
            arrive(); wait();
            if (ok) rope_phase(A, g0[0], tid, cta, G);
            arrive();
            // attention: cached key tiles are requested before the wait for q and the fresh k / v
            {
                aa.layer = l;
                bool waited = false;
                auto wait_rope = [&]() {
                    if (!waited) { wait(); waited = true; }
                };
                if (!ok) wait_rope();
                else if (A.hd == 128) attention_phase<128>(A, aa, scratch, tid, cta, G, wait_rope);
                else attention_phase<64>(A, aa, scratch, tid, cta, G, wait_rope);
            }
            arrive(); wait();
            if (A.ksplit > 1) {
                if (ok) combine_phase(A, tid, cta, G);
                arrive(); wait();
            }
            epilogue(4 * l + 1);
            arrive(); wait();
            if (ok) norm_phase(A, sh, tid, cta, G, g0[2].gain, g0 + 1, false);
            arrive(); wait();
            epilogue(4 * l + 2);
            arrive(); wait();
            if (ok) swiglu_phase(A, g0[2], tid, cta, G);
            arrive(); wait();
            epilogue(4 * l + 3);
            arrive(); wait();
        }
        // the last down projection into the residual stream; operand of the LM head
        if (ok) norm_phase(A, sh, tid, cta, G, A.gemms[4 * A.n_layers].gain, A.gemms + 4 * A.n_layers - 1, false);
        if (A.with_lm) {
            arrive(); wait();
            epilogue(4 * A.n_layers);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kAccCols) : "memory");
    }
}

size_t ring_budget(int scratch_bytes) { return 227 * 1024 - 1024 - sizeof(PShared) - 64 - static_cast<size_t>(scratch_bytes); }

}  // namespace

int step_persistent_grid() {
    static int sms[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!sms[dev]) {
        int n = 0, coop = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return 0;
        sms[dev] = n;
    }
    return sms[dev];
}

size_t step_persistent_table_bytes(int n_layers) { return sizeof(PGemmDesc) * (4 * static_cast<size_t>(n_layers) + 1); }
size_t step_persistent_barrier_bytes(int n_layers) { return sizeof(unsigned int) * (10 * static_cast<size_t>(n_layers) + 2); }

bool step_persistent_supported(int M, int d, int F, int hd) {
    static int enabled = -1;
    if (enabled < 0) {
        const char* e = getenv("ODB_PERSISTENT");
        enabled = (e && e[0] == '1') ? 1 : 0;   // off unless asked for
    }
    return enabled && M >= 1 && M <= 128 && d % 8 == 0 && F % 4 == 0 && (hd == 64 || hd == 128) && step_persistent_grid() > 0;
}

cudaError_t step_persistent_configure(StepPersistentArgs& a) {
    a.BN = a.M <= 32 ? 32 : a.M <= 64 ? 64 : 128;
    const size_t attn = a.hd == 128 ? attention_smem_bytes<128>() : attention_smem_bytes<64>();
    const size_t xch = 32 * 129 * sizeof(float);
    a.scratch_bytes = static_cast<int>(((attn > xch ? attn : xch) + 1023) / 1024 * 1024);
    const size_t stage = kBM * kBK * 2 + static_cast<size_t>(a.BN) * kBK * 2;
    size_t stages = ring_budget(a.scratch_bytes) / stage;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    a.stages = static_cast<int>(stages);
    a.n_bars = a.n_layers * (a.ksplit > 1 ? 10 : 9) + 1;
    return cudaSuccess;
}

void step_persistent_fill_desc(PGemmDesc& d, const CUtensorMap& tmap_w, const CUtensorMap& tmap_x, const float* gain, int n_tiles,
                               int nkb, int conf, int grid) {
    d.tmap_w = tmap_w;
    d.tmap_x = tmap_x;
    d.gain = gain;
    d.n_tiles = n_tiles;
    d.nkb = nkb;
    d.conf = conf;
    // a CTA's range is at least a sixth of a tile's k-blocks long: an output tile has at most 8 parts
    const long long U = static_cast<long long>(n_tiles) * nkb;
    const long long per = (nkb + 5) / 6;
    long long use = conf ? n_tiles : U / (per < 1 ? 1 : per);
    if (use > grid) use = grid;
    if (use < 1) use = 1;
    d.g_use = static_cast<int>(use);
    for (int& p : d.pad) p = 0;
}

cudaError_t launch_step_persistent(const StepPersistentArgs& a, cudaStream_t st) {
    const int grid = step_persistent_grid();
    if (grid <= 0) return cudaErrorNotSupported;
    const size_t stage = kBM * kBK * 2 + static_cast<size_t>(a.BN) * kBK * 2;
    const size_t smem = 1024 + static_cast<size_t>(a.stages) * stage + a.scratch_bytes + sizeof(PShared) + 64;
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = set_smem_limit_once(attr_done, step_persistent_kernel, 227 * 1024);
    if (e != cudaSuccess) return e;
    // every CTA a grid barrier waits for must be resident: one per SM, checked against the occupancy the
    // device reports for this configuration
    static int fits[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !fits[dev]) {
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, step_persistent_kernel, kPThreads, 227 * 1024 - 1024);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
        fits[dev] = 1;
    }
    e = cudaMemsetAsync(a.bars, 0, sizeof(unsigned int) * a.n_bars, st);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kPThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, step_persistent_kernel, a);
}

}  // namespace odb
