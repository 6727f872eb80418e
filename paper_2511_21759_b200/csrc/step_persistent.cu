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
constexpr int kPartsTiles = 256;      // output tiles per projection the parts table holds
constexpr int kTmemCols = 512;        // all of the SM's tensor memory: two sets of interleaved accumulators
constexpr long long kStatusPeriodCycles = 400000;   // ~0.2 ms between looks at the step's status word while waiting

struct alignas(8) PShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort;
    int bars_passed;      // grid barriers this CTA's workers have passed (the producer's gates, read without leaving the SM)
    float red[8];
    float scale[128];
    // The kernel's arguments, for the phase functions that are not inlined: handed a reference to the parameter
    // block they would read a copy of it in local memory, which the SM's small L1 (almost all of it is carved out
    // as shared memory here) cannot hold.
    StepPersistentArgs args;
    uint8_t nparts[4][kPartsTiles];   // parts per output tile of the four projections of a layer (the same in every layer)
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

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Non-blocking test of an mbarrier phase.  (mbarrier.try_wait may suspend the thread for a system-dependent time
// when the phase is not complete; the producer has two things to look after and must not sleep on one of them.)
__device__ __forceinline__ bool mbar_test_parity(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// ---- the fixed work split -------------------------------------------------------------------------------
// Units of a projection, tile-major: u = tile * nkb + kb.  CTA c of G owns [c U / G, (c + 1) U / G).
// All of it in 32-bit arithmetic (the host checks U * G < 2^31): these run in single-thread loops.
__device__ __forceinline__ int owner_of(uint32_t u, uint32_t U, uint32_t G) { return static_cast<int>(((u + 1) * G - 1) / U); }
// the parts of output tile `tile`: the CTAs first .. first + n - 1 each hold one partial tile, in k order
__device__ __forceinline__ void tile_parts(int tile, int nkb, int n_tiles, int G, int& first, int& n) {
    const uint32_t U = static_cast<uint32_t>(n_tiles) * nkb;
    first = owner_of(static_cast<uint32_t>(tile) * nkb, U, G);
    n = owner_of(static_cast<uint32_t>(tile + 1) * nkb - 1, U, G) - first + 1;
}

// One contiguous piece of a CTA's range inside one output tile.
struct Segment {
    int g, tile, kb0, nkb, part;   // projection, output tile, first k-block, k-blocks, index of the partial tile
};

// Walks the segments of CTA `cta` over all projections, in order.
struct Schedule {
    const PGemmDesc* gemms;
    int n_gemms, cta;
    int g;
    uint32_t u, hi;
    int nkb_g, n_tiles_g, conf_g, use_g;

    __device__ void init(const PGemmDesc* gm, int n, int cta_) {
        gemms = gm; n_gemms = n; cta = cta_;
        g = -1; u = hi = 0;
    }
    __device__ bool load_gemm() {   // advances to the next projection with a non-empty range
        while (u >= hi) {
            if (++g >= n_gemms) return false;
            n_tiles_g = gemms[g].n_tiles; nkb_g = gemms[g].nkb; conf_g = gemms[g].conf; use_g = gemms[g].g_use;
            if (cta >= use_g) {
                u = hi = 0;       // a tiny projection is divided over the first use_g CTAs only
            } else if (conf_g) {   // whole tiles: the epilogue reduces a complete column of logits
                u = static_cast<uint32_t>(cta) * n_tiles_g / use_g * nkb_g;
                hi = static_cast<uint32_t>(cta + 1) * n_tiles_g / use_g * nkb_g;
            } else {
                const uint32_t U = static_cast<uint32_t>(n_tiles_g) * nkb_g;
                u = static_cast<uint32_t>(cta) * U / use_g;
                hi = static_cast<uint32_t>(cta + 1) * U / use_g;
            }
        }
        return true;
    }
    // with_part: also the index of the partial tile (only the read-back needs it)
    __device__ bool next(Segment& s, bool with_part) {
        if (!load_gemm()) return false;
        s.g = g;
        s.tile = static_cast<int>(u / nkb_g);
        s.kb0 = static_cast<int>(u - static_cast<uint32_t>(s.tile) * nkb_g);
        uint32_t n = nkb_g - s.kb0;
        if (n > hi - u) n = hi - u;
        s.nkb = static_cast<int>(n);
        s.part = (conf_g || !with_part) ? 0
                                        : cta - owner_of(static_cast<uint32_t>(s.tile) * nkb_g, static_cast<uint32_t>(n_tiles_g) * nkb_g, use_g);
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
    // the status word lives in global memory: a look at it stalls this thread for a memory round trip, so it is
    // consulted only after the wait has lasted kStatusPeriodCycles, and then once per period
    const long long t0 = clock64();
    long long t_next = t0 + kStatusPeriodCycles;
    while (!mbar_try_wait_parity(bar, parity)) {
        if (*cta_abort) return false;
        const long long now = clock64();
        if (now > t_next) {
            t_next = now + kStatusPeriodCycles;
            if (*reinterpret_cast<volatile int*>(status) != 0) { *cta_abort = 1; return false; }
            if (now - t0 > kWaitLimitCycles) {
                *cta_abort = 1;
                atomicExch(status, ODB_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// ---- the short phases (128 worker threads, tid 0..127) -----------------------------------------------------

constexpr int kMaxParts = 8;      // partial tiles per output tile (the host's split keeps it at or below)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ void mul4(float4& a, float s) { a.x *= s; a.y *= s; a.z *= s; a.w *= s; }

// The parts of one float4 of a projection's output, partial[part][M][Np]: all requested at once, then added in
// part order.  Every short phase is a few dependent memory round trips long, so what matters is that a thread
// has all the loads of all its items in flight before it uses the first.
template <int MAXP>
struct Parts {
    float4 t[MAXP];
    int n;
    __device__ __forceinline__ void load(const float* partial, size_t Np, int M, int row, int col, int n_) {
        n = n_;
        const float* p = partial + static_cast<size_t>(row) * Np + col;
#pragma unroll
        for (int s = 0; s < MAXP; ++s)
            if (s < n) t[s] = ldcg4(p + static_cast<size_t>(s) * M * Np);
    }
    __device__ __forceinline__ float4 sum() const {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < MAXP; ++s)
            if (s < n) add4(acc, t[s]);
        return acc;
    }
};

__device__ __forceinline__ uint2 pack4(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(c, d);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    return pk;
}

__device__ __forceinline__ float row_scale_cg(const StepPersistentArgs& A, int row) {
    const int slices = (A.d + kNormSliceCols - 1) / kNormSliceCols;
    float t = 0.f;
    for (int i = 0; i < slices; ++i) t += __ldcg(A.ssq + static_cast<size_t>(row) * slices + i);
    return 1.0f / sqrtf(t * (1.0f / static_cast<float>(A.d)) + A.rms_eps);
}

// Residual stream += the parts of the preceding projection (kind pj of the parts table, -1: none), or := the
// token embeddings (layer 0); operand a = bf16(h * gain); per (row, 1024-column slice) the sum of squares for
// the consumer's 1 / rms.
template <int MAXP>
__device__ __noinline__ void norm_phase(const StepPersistentArgs& A, PShared* sh, int tid, int cta, int G, const float* gain,
                                        const PGemmDesc* prev, int pj, bool from_embed) {
    const int d = A.d, slices = (d + kNormSliceCols - 1) / kNormSliceCols;
    const int n_items = A.M * slices;
    const int warp = tid >> 5, lane = tid & 31;
    const size_t Np = prev ? static_cast<size_t>(prev->n_tiles) * 128 : 0;
    for (int it = cta; it < n_items; it += G) {
        const int row = it / slices, sl = it % slices;
        float4 v[2];
        Parts<MAXP> pp[2];
        int col[2];
        bool in[2];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int i = sl * (kNormSliceCols / 4) + half * kWorkers + tid;   // float4 index within the row
            in[half] = i < (d >> 2);
            col[half] = i << 2;
            pp[half].n = 0;
            if (!in[half]) continue;
            if (from_embed) {
                const uint2 e = *reinterpret_cast<const uint2*>(A.embed + static_cast<size_t>(A.row_tok[row]) * d + col[half]);
                const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.x));
                const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.y));
                v[half] = make_float4(lo.x, lo.y, hi.x, hi.y);
            } else {
                v[half] = ldcg4(A.h + static_cast<size_t>(row) * d + col[half]);
            }
            if (prev) pp[half].load(A.partial, Np, A.M, row, col[half], sh->nparts[pj][col[half] >> 7]);
        }
        float ss = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            if (!in[half]) continue;
            float4 x = v[half];
            if (prev) add4(x, pp[half].sum());
            if (prev || from_embed) *reinterpret_cast<float4*>(A.h + static_cast<size_t>(row) * d + col[half]) = x;
            ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
            if (gain) {
                const float4 g = *reinterpret_cast<const float4*>(gain + col[half]);
                *reinterpret_cast<uint2*>(A.a + static_cast<size_t>(row) * d + col[half]) = pack4(x.x * g.x, x.y * g.y, x.z * g.z, x.w * g.w);
            }
        }
        ss = warp_sum(ss);
        WorkerSync::sync();
        if (lane == 0) sh->red[warp] = ss;
        WorkerSync::sync();
        if (tid == 0) A.ssq[static_cast<size_t>(row) * slices + sl] = sh->red[0] + sh->red[1] + sh->red[2] + sh->red[3];
    }
}

// Parts of the QKV projection -> x 1/rms -> rotate q and k (rotate-half pairing) -> bf16 q, k, v rows.
// One thread per four rotation pairs of one row; all threads of the grid share the rows x pairs evenly.
template <int MAXP>
__device__ __noinline__ void rope_phase(const StepPersistentArgs& A, PShared* sh, const PGemmDesc& pq, int tid, int cta, int G) {
    const int d = A.d, half = A.hd / 2, quads = d / 8;
    const int total = A.M * quads;
    const size_t Np = static_cast<size_t>(pq.n_tiles) * 128;
    for (int item = cta * kWorkers + tid; item < total; item += G * kWorkers) {
        const int row = item / quads;
        const int t = (item - row * quads) * 4;                   // first of four rotation pairs
        const int head = t / half, i = t - head * half;
        const int e0 = head * A.hd + i, e1 = e0 + half;
        const float inv = row_scale_cg(A, row);
        const float2* rope = A.rope + static_cast<size_t>(A.row_pos[row]) * half;
        const float4 c01 = *reinterpret_cast<const float4*>(rope + i);
        const float4 c23 = *reinterpret_cast<const float4*>(rope + i + 2);
        const size_t o = static_cast<size_t>(row) * d;
        auto rotate_store = [&](__nv_bfloat16* dst, float4 x0, float4 x1) {
            mul4(x0, inv); mul4(x1, inv);
            *reinterpret_cast<uint2*>(dst + o + e0) = pack4(x0.x * c01.x - x1.x * c01.y, x0.y * c01.z - x1.y * c01.w,
                                                            x0.z * c23.x - x1.z * c23.y, x0.w * c23.z - x1.w * c23.w);
            *reinterpret_cast<uint2*>(dst + o + e1) = pack4(x1.x * c01.x + x0.x * c01.y, x1.y * c01.z + x0.y * c01.w,
                                                            x1.z * c23.x + x0.z * c23.y, x1.w * c23.z + x0.w * c23.w);
        };
        Parts<MAXP> a0, a1, b0, b1;
        a0.load(A.partial, Np, A.M, row, e0, sh->nparts[0][e0 >> 7]);
        a1.load(A.partial, Np, A.M, row, e1, sh->nparts[0][e1 >> 7]);
        b0.load(A.partial, Np, A.M, row, d + e0, sh->nparts[0][(d + e0) >> 7]);
        b1.load(A.partial, Np, A.M, row, d + e1, sh->nparts[0][(d + e1) >> 7]);
        if constexpr (MAXP <= 4) {
            Parts<MAXP> c0, c1;
            c0.load(A.partial, Np, A.M, row, 2 * d + e0, sh->nparts[0][(2 * d + e0) >> 7]);
            c1.load(A.partial, Np, A.M, row, 2 * d + e1, sh->nparts[0][(2 * d + e1) >> 7]);
            rotate_store(A.q, a0.sum(), a1.sum());
            rotate_store(A.k, b0.sum(), b1.sum());
            float4 v0 = c0.sum(), v1 = c1.sum();
            mul4(v0, inv); mul4(v1, inv);
            *reinterpret_cast<uint2*>(A.v + o + e0) = pack4(v0.x, v0.y, v0.z, v0.w);
            *reinterpret_cast<uint2*>(A.v + o + e1) = pack4(v1.x, v1.y, v1.z, v1.w);
        } else {
            rotate_store(A.q, a0.sum(), a1.sum());
            rotate_store(A.k, b0.sum(), b1.sum());
            a0.load(A.partial, Np, A.M, row, 2 * d + e0, sh->nparts[0][(2 * d + e0) >> 7]);
            a1.load(A.partial, Np, A.M, row, 2 * d + e1, sh->nparts[0][(2 * d + e1) >> 7]);
            float4 v0 = a0.sum(), v1 = a1.sum();
            mul4(v0, inv); mul4(v1, inv);
            *reinterpret_cast<uint2*>(A.v + o + e0) = pack4(v0.x, v0.y, v0.z, v0.w);
            *reinterpret_cast<uint2*>(A.v + o + e1) = pack4(v1.x, v1.y, v1.z, v1.w);
        }
    }
}

// Merge of the key splits of the attention, in split order (the arithmetic of attention_combine_kernel).
// One thread per four output elements; two of them at a time.
__device__ __noinline__ void combine_phase(const StepPersistentArgs& A, int tid, int cta, int G) {
    const int hd = A.hd, ks = A.ksplit;
    const int tpi = hd / 4;
    const int total = A.M * A.H * tpi;
    const size_t zs = static_cast<size_t>(A.M) * A.H;
    const int stride = G * kWorkers;
    for (int it0 = cta * kWorkers + tid; it0 < total; it0 += 2 * stride) {
        float2 ml[2][8];
        float4 v[2][8];
        size_t base[2];
        int d4[2];
        bool in[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int it = it0 + u * stride;
            in[u] = it < total;
            base[u] = in[u] ? it / tpi : 0;                        // row * H + head
            d4[u] = in[u] ? (it % tpi) * 4 : 0;
#pragma unroll
            for (int z = 0; z < 8; ++z)
                if (in[u] && z < ks) {
                    ml[u][z] = __ldcg(reinterpret_cast<const float2*>(A.part_ml + (z * zs + base[u]) * 2));
                    v[u][z] = ldcg4(A.part_o + (z * zs + base[u]) * hd + d4[u]);
                }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (!in[u]) continue;
            float mmax = -INFINITY;
#pragma unroll
            for (int z = 0; z < 8; ++z)
                if (z < ks && ml[u][z].y > 0.f) mmax = fmaxf(mmax, ml[u][z].x);
            float L = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int z = 0; z < 8; ++z) {
                if (z < ks && ml[u][z].y > 0.f) {
                    const float wt = exp2f(ml[u][z].x - mmax);
                    L += ml[u][z].y * wt;
                    acc.x += v[u][z].x * wt; acc.y += v[u][z].y * wt; acc.z += v[u][z].z * wt; acc.w += v[u][z].w * wt;
                }
            }
            const float inv = L > 0.f ? 1.0f / L : 0.f;
            *reinterpret_cast<uint2*>(A.o + base[u] * hd + d4[u]) = pack4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        }
    }
}

// Parts of the gate/up projection (tile t = 64 gate features then their 64 up features) -> x 1/rms ->
// g = bf16(silu(gate) * up).  One thread per four features of one row, UN of them at a time.
template <int MAXP, int UN>
__device__ __noinline__ void swiglu_phase(const StepPersistentArgs& A, PShared* sh, const PGemmDesc& pg, int tid, int cta, int G) {
    const int F = A.F, f4 = F / 4;
    const int total = A.M * f4;
    const size_t Np = static_cast<size_t>(pg.n_tiles) * 128;
    const int stride = G * kWorkers;
    for (int it0 = cta * kWorkers + tid; it0 < total; it0 += UN * stride) {
        Parts<MAXP> gate[UN], up[UN];
        float sc[UN];
        int row[UN], f[UN];
        bool in[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int it = it0 + u * stride;
            in[u] = it < total;
            gate[u].n = up[u].n = 0;
            if (!in[u]) continue;
            row[u] = it / f4;
            f[u] = (it - row[u] * f4) * 4;
            const int col = (f[u] >> 6) * 128 + (f[u] & 63);
            const int n = sh->nparts[2][f[u] >> 6];
            gate[u].load(A.partial, Np, A.M, row[u], col, n);
            up[u].load(A.partial, Np, A.M, row[u], col + 64, n);
            sc[u] = row_scale_cg(A, row[u]);
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            if (!in[u]) continue;
            const float4 gt = gate[u].sum(), uu = up[u].sum();
            const float s_ = sc[u];
            const float g0 = gt.x * s_, g1 = gt.y * s_, g2 = gt.z * s_, g3 = gt.w * s_;
            *reinterpret_cast<uint2*>(A.g + static_cast<size_t>(row[u]) * F + f[u]) =
                pack4(g0 / (1.0f + expf(-g0)) * (uu.x * s_), g1 / (1.0f + expf(-g1)) * (uu.y * s_),
                      g2 / (1.0f + expf(-g2)) * (uu.z * s_), g3 / (1.0f + expf(-g3)) * (uu.w * s_));
        }
    }
}

// The wait half of a grid barrier, for the 128 workers: thread 0 polls, tells the CTA's producer that the operand
// behind the barrier is complete, then all workers meet.
__device__ __forceinline__ void grid_wait(const StepPersistentArgs& A, PShared* sh, int bar_id, int G, int cta, int tid) {
    if (tid == 0) {
        if (poll_barrier(A, bar_id, G, &sh->abort))
            asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(&sh->bars_passed)), "r"(bar_id + 1) : "memory");
        if (A.timing) A.timing[(static_cast<size_t>(cta) * A.n_bars + bar_id) * 2 + 1] = global_timer_ns();
    }
    WorkerSync::sync();
}

// Attention work items (query tile, head, key split) of this CTA.  The cached key tiles of the first item are
// requested before the wait at grid barrier `bar_id` (the one behind the RoPE phase), which happens in here.
template <int HD>
__device__ __noinline__ void attention_phase(const StepPersistentArgs& A, PShared* sh, uint8_t* scratch, int layer, int bar_id, int tid,
                                             int cta, int G) {
    AttnArgs aa;
    aa.tiles = A.tiles; aa.n_tiles = A.n_qtiles;
    aa.q = A.q; aa.k = A.k; aa.v = A.v; aa.cache = A.cache; aa.row_flags = A.row_flags; aa.o = A.o;
    aa.part_o = A.part_o; aa.part_ml = A.part_ml;
    aa.layer = layer; aa.n_layers = A.n_layers; aa.H = A.H; aa.hd = A.hd; aa.max_seq = A.max_seq; aa.M = A.M; aa.ksplit = A.ksplit;
    aa.early = 1;
    aa.pf = L2Prefetch{nullptr, 0};
    bool waited = false;
    auto wait_rope = [&]() {
        if (!waited) grid_wait(A, sh, bar_id, G, cta, tid);
        waited = true;
    };
    const int n_attn = A.n_qtiles * A.H * A.ksplit;
    for (int it = cta; it < n_attn; it += G) {
        const int z = it % A.ksplit, head = (it / A.ksplit) % A.H, qt = it / (A.ksplit * A.H);
        const QTile t = A.tiles[qt];
        attention_item<HD, WorkerSync>(aa, t, head, z, tid, scratch, true, wait_rope);
        WorkerSync::sync();                              // the tiles in shared memory are free for the next item
        if (sh->abort) break;
    }
    wait_rope();
}

// 32 columns of this warp's TMEM lanes, summed over the n_acc interleaved accumulators (BN columns apart), in order
__device__ __forceinline__ void load_acc_sum(uint32_t taddr, int BN, int n_acc, float (&acc)[32]) {
    uint32_t v[32];
    tmem_ld32(taddr, v);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = __uint_as_float(v[j]);
    for (int a = 1; a < n_acc; ++a) {
        tmem_ld32(taddr + static_cast<uint32_t>(a * BN), v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[j] += __uint_as_float(v[j]);
    }
}

// ---- the kernel -----------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kPThreads, 1) step_persistent_kernel(const __grid_constant__ StepPersistentArgs A) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int BN = A.BN, S = A.stages;
    // Consecutive tcgen05.mma into ONE accumulator form a dependent chain, and with so few activation rows an MMA
    // is all pipeline latency: a single chain takes ~0.7 us per 16 KB weight tile, half of what HBM delivers to an
    // SM.  The k-blocks of a segment therefore rotate over NACC independent accumulators, summed at read-back.
    const int NACC = BN <= 64 ? 4 : 2;
    const int acc_set_cols = NACC * BN;                 // one set; two sets: a segment is read back while the next runs
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
        sh->bars_passed = 0;
        sh->args = A;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // whole warp: both accumulators' TMEM columns
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(kTmemCols)
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
            // A cursor walks this CTA's units; everything that is constant over a segment is kept in registers, and
            // stage index and phase are stepped, never divided: this thread's instruction count per tile bounds
            // the rate a single producer can sustain.
            struct Cursor {
                Schedule s;
                Segment seg;
                bool have;
                int left;                 // k-blocks left in the segment
                const CUtensorMap* tw;
                const CUtensorMap* tx;
                int wtile, kcol, gate;    // next packed weight tile, next activation column, gate of the projection
            };
            auto advance = [&](Cursor& c) {
                c.have = c.s.next(c.seg, false);
                if (!c.have) return;
                const PGemmDesc* pg = A.gemms + c.seg.g;
                c.left = c.seg.nkb;
                c.tw = &pg->tmap_w;
                c.tx = &pg->tmap_x;
                c.wtile = c.seg.tile * pg->nkb + c.seg.kb0;
                c.kcol = c.seg.kb0 * kBK;
                c.gate = gate_of(c.seg.g, A.n_layers, A.ksplit);
            };
            Cursor cw, ca, cp;
            cw.s.init(A.gemms, n_gemms, cta);
            ca.s.init(A.gemms, n_gemms, cta);
            cp.s.init(A.gemms, n_gemms, cta);
            advance(cw);
            advance(ca);
            cp.have = false;
            if (A.l2_ahead > 0) advance(cp);
            uint32_t it_w = 0, it_a = 0, it_p = 0;   // weight tiles / activation tiles given to stages; tiles asked of L2
            int st_w = 0, st_a = 0;
            uint32_t ph_w = 0;
            // optional: HBM -> L2 runs l2_ahead tiles in front of L2 -> shared memory
            auto l2_prefetch_to = [&](uint32_t upto) {
                while (cp.have && static_cast<int32_t>(upto - it_p) > 0) {
                    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(
                                     reinterpret_cast<uint64_t>(cp.tw)),
                                 "r"(0), "r"(0), "r"(cp.wtile)
                                 : "memory");
                    ++it_p;
                    ++cp.wtile;
                    if (--cp.left == 0) advance(cp);
                }
            };
            if (A.l2_ahead > 0) l2_prefetch_to(static_cast<uint32_t>(A.l2_ahead));
            int gates_open = 0;                      // grid barriers known complete (from the workers of this CTA)
            long long t_idle = clock64(), t_next = t_idle + kStatusPeriodCycles;
            bool idle = false;
            while (ca.have) {
                bool progress = false;
                if (cw.have && mbar_test_parity(&sh->empty[st_w], ph_w ^ 1u)) {
                    mbar_expect_tx(&sh->full[st_w], stage_bytes);
                    tma_load_3d(ring + static_cast<size_t>(st_w) * stage_bytes, cw.tw, &sh->full[st_w], 0, 0, cw.wtile, kEvictFirst);
                    if (++st_w == S) { st_w = 0; ph_w ^= 1u; }
                    ++it_w;
                    ++cw.wtile;
                    if (--cw.left == 0) advance(cw);
                    if (A.l2_ahead > 0) l2_prefetch_to(it_w + static_cast<uint32_t>(A.l2_ahead));
                    progress = true;
                }
                if (it_a != it_w) {
                    bool open = ca.gate < gates_open;
                    if (!open) {
                        int passed;
                        asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(passed) : "r"(smem_u32(&sh->bars_passed)) : "memory");
                        if (passed > gates_open) {
                            gates_open = passed;
                            fence_proxy_async_all();     // the operand was written with ordinary stores by other CTAs
                            open = ca.gate < gates_open;
                        }
                    }
                    if (open) {
                        tma_load_2d(ring + static_cast<size_t>(st_a) * stage_bytes + kABytes, ca.tx, &sh->full[st_a], ca.kcol, 0, kEvictLast);
                        if (++st_a == S) st_a = 0;
                        ++it_a;
                        ca.kcol += kBK;
                        if (--ca.left == 0) advance(ca);
                        progress = true;
                    }
                }
                if (progress) {
                    idle = false;
                } else {
                    if (*cta_abort) break;
                    const long long now = clock64();
                    if (!idle) {
                        idle = true;
                        t_idle = now;
                        t_next = now + kStatusPeriodCycles;
                    } else if (now > t_next) {   // rarely: the look at the status word costs a memory round trip
                        t_next = now + kStatusPeriodCycles;
                        if (*reinterpret_cast<volatile int*>(A.status) != 0) { *cta_abort = 1; break; }
                        if (now - t_idle > kWaitLimitCycles) {
                            *cta_abort = 1;
                            atomicExch(A.status, ODB_ERR_TIMEOUT);
                            break;
                        }
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
            sm.init(A.gemms, n_gemms, cta);
            Segment seg{};
            uint32_t seg_idx = 0, ph = 0;
            int st = 0;
            bool ok = true;
            while (ok && sm.next(seg, false)) {
                const int buf = static_cast<int>(seg_idx & 1u);
                ok = pwait(&sh->acc_empty[buf], ((seg_idx >> 1) & 1u) ^ 1u, cta_abort, A.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tset = tmem_base + static_cast<uint32_t>(buf * acc_set_cols);
                int ai = 0;                                     // accumulator of the set this k-block goes to
                for (int i = 0; i < seg.nkb && ok; ++i) {
                    const uint32_t tacc = tset + static_cast<uint32_t>(ai * BN);
                    if (++ai == NACC) ai = 0;
                    ok = pwait(&sh->full[st], ph, cta_abort, A.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(ring + static_cast<size_t>(st) * stage_bytes);
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k = 0; k < kBK / kUmmaK; ++k)
                        umma_bf16(tacc, make_smem_desc(a_addr + k * kUmmaK * 2), make_smem_desc(b_addr + k * kUmmaK * 2), idesc,
                                  (i >= NACC || k > 0) ? 1u : 0u);
                    umma_commit(&sh->empty[st]);
                    if (++st == S) { st = 0; ph ^= 1u; }
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
        se.init(A.gemms, n_gemms, cta);
        Segment seg{};
        bool have = se.next(seg, true);
        uint32_t seg_idx = 0;
        int bar_id = 0;
        bool ok = true;

        auto arrive = [&](bool feeds_tma = false) {
            // ordinary stores to a buffer that other CTAs' TMA loads will read (a, o, g) are ordered before them
            // by a proxy fence on the writing side; the other hand-overs are read with ordinary loads
            if (feeds_tma) asm volatile("fence.proxy.async.global;" ::: "memory");
            WorkerSync::sync();
            if (tid == 0) {
                __threadfence();                        // cumulative: covers the stores of the 127 threads behind the barrier
                red_release_add(A.bars + bar_id, 1u);
                if (A.timing) A.timing[(static_cast<size_t>(cta) * A.n_bars + bar_id) * 2] = global_timer_ns();
            }
        };
        auto wait = [&]() {
            grid_wait(A, sh, bar_id, G, cta, tid);
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
                const int buf = static_cast<int>(seg_idx & 1u);
                const bool got = ok && pwait(&sh->acc_full[buf], (seg_idx >> 1) & 1u, cta_abort, A.status);
                if (got) tc_fence_after();
                const uint32_t tacc = tmem_base + static_cast<uint32_t>(buf * acc_set_cols) + (static_cast<uint32_t>(q * 32) << 16);
                const int n_acc = seg.nkb < NACC ? seg.nkb : NACC;      // accumulators this segment has written
                if (!pg.conf) {
                    if (got) {
                        float* out = A.partial + static_cast<size_t>(seg.part) * A.M * Np + static_cast<size_t>(seg.tile) * 128 + q * 32 + lane;
#pragma unroll 1
                        for (int c = 0; c < BN / 32; ++c) {
                            float acc[32];
                            load_acc_sum(tacc + static_cast<uint32_t>(c * 32), BN, n_acc, acc);
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int m = c * 32 + j;
                                if (m < A.M) out[static_cast<size_t>(m) * Np] = acc[j];
                            }
                        }
                    }
                } else {
                    // LM head: softmax statistics of this vocabulary tile per row; the logits never leave the SM
                    float* xch = reinterpret_cast<float*>(scratch);   // [32 rows][129]
                    const int n0 = seg.tile * 128;
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        float acc[32];
                        if (got) load_acc_sum(tacc + static_cast<uint32_t>(c * 32), BN, n_acc, acc);
#pragma unroll
                        for (int j = 0; j < 32; ++j) xch[j * 129 + q * 32 + lane] = got ? acc[j] : 0.f;
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
                have = se.next(seg, true);
            }
        };

        const StepPersistentArgs& SA = sh->args;
        // parts per output tile of the four projections of a layer (identical in every layer)
        for (int j = 0; j < 4; ++j) {
            const PGemmDesc& pj = A.gemms[j];
            for (int t = tid; t < pj.n_tiles && t < kPartsTiles; t += kWorkers) {
                int first, n;
                tile_parts(t, pj.nkb, pj.n_tiles, pj.g_use, first, n);
                sh->nparts[j][t] = static_cast<uint8_t>(n);
            }
        }
        WorkerSync::sync();

#define ODB_BY_PARTS(mp, CALL)  \
    do {                        \
        if ((mp) <= 2) { CALL(2); } else if ((mp) <= 4) { CALL(4); } else { CALL(8); } \
    } while (0)
#define ODB_NORM_DOWN(P) norm_phase<P>(SA, sh, tid, cta, G, g0[0].gain, g0 - 1, 3, false)
#define ODB_NORM_O(P) norm_phase<P>(SA, sh, tid, cta, G, g0[2].gain, g0 + 1, 1, false)
#define ODB_ROPE(P) rope_phase<P>(SA, sh, g0[0], tid, cta, G)
#define ODB_SWIGLU(P) swiglu_phase<P, (P <= 2 ? 4 : P <= 4 ? 2 : 1)>(SA, sh, g0[2], tid, cta, G)
#define ODB_NORM_FINAL(P) norm_phase<P>(SA, sh, tid, cta, G, A.gemms[4 * A.n_layers].gain, A.gemms + 4 * A.n_layers - 1, 3, false)

        for (int l = 0; l < A.n_layers && ok; ++l) {
            const PGemmDesc* g0 = A.gemms + 4 * l;
            // residual (+ the previous layer's down projection, or the embeddings) -> operand of QKV
            if (l == 0) norm_phase<2>(SA, sh, tid, cta, G, g0[0].gain, nullptr, 0, true);
            else ODB_BY_PARTS(A.maxp[3], ODB_NORM_DOWN);
            arrive(true); wait();
            epilogue(4 * l);
            arrive(); wait();
            if (ok) ODB_BY_PARTS(A.maxp[0], ODB_ROPE);
            arrive();
            // attention: cached key tiles are requested before the wait for q and the fresh k / v
            if (ok) {
                if (A.hd == 128) attention_phase<128>(SA, sh, scratch, l, bar_id, tid, cta, G);
                else attention_phase<64>(SA, sh, scratch, l, bar_id, tid, cta, G);
                ++bar_id;
                if (*cta_abort) ok = false;
            } else {
                wait();
            }
            arrive(A.ksplit == 1); wait();                // without key splits the attention wrote o itself
            if (A.ksplit > 1) {
                if (ok) combine_phase(SA, tid, cta, G);
                arrive(true); wait();
            }
            epilogue(4 * l + 1);
            arrive(); wait();
            if (ok) ODB_BY_PARTS(A.maxp[1], ODB_NORM_O);
            arrive(true); wait();
            epilogue(4 * l + 2);
            arrive(); wait();
            if (ok) ODB_BY_PARTS(A.maxp[2], ODB_SWIGLU);
            arrive(true); wait();
            epilogue(4 * l + 3);
            arrive(); wait();
        }
        // the last down projection into the residual stream; operand of the LM head
        if (ok) ODB_BY_PARTS(A.maxp[3], ODB_NORM_FINAL);
        if (A.with_lm) {
            arrive(true); wait();
            epilogue(4 * A.n_layers);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
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
    static int stage_cap = -1;
    if (stage_cap < 0) {
        const char* e = getenv("ODB_PERSISTENT_STAGES");
        stage_cap = e ? atoi(e) : 0;
    }
    if (stage_cap >= 2 && stages > static_cast<size_t>(stage_cap)) stages = stage_cap;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    a.stages = static_cast<int>(stages);
    a.n_bars = a.n_layers * (a.ksplit > 1 ? 10 : 9) + 1;
    static int l2_ahead = -1;
    if (l2_ahead < 0) {
        const char* e = getenv("ODB_PERSISTENT_L2_AHEAD");
        l2_ahead = e ? atoi(e) : 0;
    }
    a.l2_ahead = l2_ahead;
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
    d.g_use = (U + 1) * grid < (1ll << 31) ? static_cast<int>(use) : 0;   // 0: beyond the kernel's 32-bit unit arithmetic
    for (int& p : d.pad) p = 0;
}

int step_persistent_max_parts(const PGemmDesc& d) {
    if (d.g_use < 1 || d.conf) return 1;
    const long long U = static_cast<long long>(d.n_tiles) * d.nkb;
    auto owner = [&](long long u) { return static_cast<int>(((u + 1) * d.g_use - 1) / U); };
    int mx = 1;
    for (int t = 0; t < d.n_tiles; ++t) {
        const int n = owner(static_cast<long long>(t + 1) * d.nkb - 1) - owner(static_cast<long long>(t) * d.nkb) + 1;
        if (n > mx) mx = n;
    }
    return mx;
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
