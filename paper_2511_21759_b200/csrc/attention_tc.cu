// Bidirectional attention of a refresh prefill on the tcgen05 tensor cores (head dim 128).
//
// Work item: 128 query rows of one sequence x one head; keys = every row of that sequence (fresh q/k/v
// of the same forward, nothing is read from the cache: the refresh is what writes it).  No causal mask.
// Two passes over the key tiles of 64, both with S = Q K^T as one 128 x 64 x 128 tcgen05.mma group whose
// fp32 result lives in TMEM:
//   pass 1  row maxima of S (thread r owns TMEM lane r = query row r: no cross-thread reduction);
//   pass 2  P = exp2(S - max), row sums, P rounded to a two-term bf16 sum (value + remainder, as in the
//           mma.sync kernel) and written to shared memory as the A operand of O += P V
//           (128 x 128 x 64, V taken MN-major straight from its [key][dim] tile), O in TMEM.
// Exact softmax, no rescaling of O.  Q, K, V tiles are staged with 16-byte cp.async in the canonical
// 128-byte-swizzled layout the MMA descriptors expect (two 64-column atoms per 128-wide row).
// S is double buffered in TMEM and K in shared memory: the MMAs of tile t + 1 are issued before the
// softmax of tile t.  Two CTAs share an SM (112 KB of shared memory, 256 TMEM columns each).  Every
// mbarrier wait is bounded; on expiry the CTA records ODB_ERR_TIMEOUT, stops issuing work, releases its
// TMEM and exits.
#include "odb_internal.cuh"

namespace odb {

namespace {

constexpr int kTQ = 128;   // query rows per work item (MMA M)
constexpr int kTK = 64;    // keys per tile
constexpr int kHD = 128;
constexpr int kThreads = 128;
constexpr long long kWaitLimitCycles = 4000000000ll;

constexpr uint32_t kQBytes = kTQ * kHD * 2;          // 32 KB: two atoms of 128 rows x 128 B
constexpr uint32_t kKBytes = kTK * kHD * 2;          // 16 KB: two atoms of 64 rows x 128 B
constexpr uint32_t kPBytes = kTQ * kTK * 2;          // 16 KB: one atom of 128 rows x 128 B
constexpr uint32_t kSmemBytes = kQBytes + 3 * kKBytes + 2 * kPBytes + 64;   // the dynamic region starts 1024-aligned
constexpr uint32_t kTmemCols = 256;                  // S0: columns 0..63, O: 64..191, S1: 192..255

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;   // size 0: destination is zero filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the CTA has been aborted or the limit expired.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* cta_abort, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*cta_abort) return false;
        if (clock64() - t0 > kWaitLimitCycles) {
            *cta_abort = 1;
            atomicExch(status, ODB_ERR_TIMEOUT);
            return false;
        }
    }
    return true;
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

struct alignas(8) TcShared {
    uint64_t bar_s[2];     // S = Q K^T into S buffer 0 / 1 has completed
    uint64_t bar_o;        // O += P V of the current tile has completed
    uint32_t tmem_base;
    int abort;
};

// swizzled position of the 16-byte chunk `chunk` (0..15 across the 128-wide row) of row `row` in a tile of
// `rows` rows: two atoms (columns 0..63, 64..127), each rows x 128 bytes, chunk index XOR (row mod 8)
__device__ __forceinline__ uint32_t tile_off(int rows, int row, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * rows * 128 + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(kThreads) attention_tc_kernel(AttnArgs a, int* status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* sQ = smem_raw;
    uint8_t* sK0 = sQ + kQBytes;         // key tiles with even index
    uint8_t* sK1 = sK0 + kKBytes;        // key tiles with odd index
    uint8_t* sV = sK1 + kKBytes;
    uint8_t* sPh = sV + kKBytes;         // P, rounded to bf16
    uint8_t* sPl = sPh + kPBytes;        // P minus its rounded value, rounded to bf16
    TcShared* sh = reinterpret_cast<TcShared*>(sPl + kPBytes);

    const int tid = threadIdx.x, warp = tid >> 5;
    volatile int* cta_abort = &sh->abort;

    pdl_launch_dependents();
    if ((smem_u32(smem_raw) & 1023u) != 0) {                // the swizzled tiles need 1024-byte alignment
        if (tid == 0) atomicExch(status, ODB_ERR_CUDA);
        pdl_wait();
        return;
    }
    if (tid == 0) {
        mbar_init(&sh->bar_s[0], 1);
        mbar_init(&sh->bar_s[1], 1);
        mbar_init(&sh->bar_o, 1);
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
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
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;   // this warp's TMEM lanes

    pdl_wait();   // q, k, v of this layer come from the preceding kernel
    const QTile t = a.tiles[blockIdx.x];
    const int head = blockIdx.y;
    const int d = a.H * kHD;
    const int NK = t.n0;                                   // keys: rows f0 .. f0 + n0 of the forward
    const int ntiles = (NK + kTK - 1) / kTK;
    const __nv_bfloat16* qsrc = a.q + static_cast<size_t>(t.q_row0) * d + head * kHD;
    const __nv_bfloat16* ksrc = a.k + static_cast<size_t>(t.f0) * d + head * kHD;
    const __nv_bfloat16* vsrc = a.v + static_cast<size_t>(t.f0) * d + head * kHD;

    auto load_kv = [&](const __nv_bfloat16* src, uint8_t* dst, int tile) {
        const uint32_t dbase = smem_u32(dst);
        for (int c = tid; c < kTK * 16; c += kThreads) {
            const int key = c >> 4, ch = c & 15;
            const int kv = tile * kTK + key;
            const bool ok = kv < NK;
            cp_async16(dbase + tile_off(kTK, key, ch), ok ? src + static_cast<size_t>(kv) * d + ch * 8 : src, ok);
        }
    };
    auto commit = [] { asm volatile("cp.async.commit_group;" ::: "memory"); };
    // copies landed (this thread's), visible to the tensor core, and every thread is here
    auto publish = [] {
        proxy_fence();
        tc_fence_before();
        __syncthreads();
    };

    // ---- Q, first two key tiles ----
    {
        const uint32_t qb = smem_u32(sQ);
        for (int c = tid; c < kTQ * 16; c += kThreads) {
            const int r = c >> 4, ch = c & 15;
            const bool ok = r < t.nq;
            cp_async16(qb + tile_off(kTQ, r, ch), ok ? qsrc + static_cast<size_t>(r) * d + ch * 8 : qsrc, ok);
        }
    }
    load_kv(ksrc, sK0, 0);
    commit();
    if (1 < ntiles) load_kv(ksrc, sK1, 1);
    commit();

    constexpr uint32_t idesc_s = instr_desc(kTQ, kTK, 0);
    constexpr uint32_t idesc_o = instr_desc(kTQ, kHD, 1);
    const float scale_log2 = rsqrtf(static_cast<float>(kHD)) * 1.4426950408889634f;
    uint32_t ph_s[2] = {0, 0}, ph_o = 0;                   // mbarrier phases
    bool ok = true;

    // S(tile) = Q K^T over the 128-wide head dim: 8 MMAs of K = 16 into S buffer tile & 1
    auto issue_s = [&](int tile) {
        const uint32_t qa = smem_u32(sQ), kb = smem_u32((tile & 1) ? sK1 : sK0);
        const uint32_t ts = (tile & 1) ? tmem_s1 : tmem_s0;
#pragma unroll
        for (int kk = 0; kk < kHD / 16; ++kk) {
            const uint32_t atom = kk >> 2, within = (kk & 3) * 32;
            umma(ts, desc_k_major(qa + atom * (kTQ * 128) + within), desc_k_major(kb + atom * (kTK * 128) + within), idesc_s,
                 kk > 0 ? 1u : 0u);
        }
        umma_commit(&sh->bar_s[tile & 1]);
    };

    // ---- pass 1: row maxima ----
    float m_row = -INFINITY;
    asm volatile("cp.async.wait_group 1;" ::: "memory");   // Q and key tile 0 landed
    publish();
    if (tid == 0) {
        tc_fence_after();
        issue_s(0);
    }
    for (int tile = 0; tile < ntiles && ok; ++tile) {
        const int b = tile & 1;
        if (tile + 1 < ntiles) {                            // S(tile + 1) runs while S(tile) is read back
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            publish();                                      // also: every thread has read S(tile - 1) out of that buffer
            if (tid == 0) {
                tc_fence_after();
                issue_s(tile + 1);
            }
        }
        ok = mbar_wait(&sh->bar_s[b], ph_s[b], cta_abort, status);
        ph_s[b] ^= 1u;
        if (!ok) break;
        tc_fence_after();
        if (tile + 2 < ntiles) load_kv(ksrc, b ? sK1 : sK0, tile + 2);   // the MMAs have read this buffer
        commit();
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32((b ? tmem_s1 : tmem_s0) + lane_base + half * 32, v);
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (tile * kTK + half * 32 + j < NK) m_row = fmaxf(m_row, __uint_as_float(v[j]));
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    ok = ok && !*cta_abort;

    // ---- pass 2: P = exp2(S - max), O += P V ----
    const float m_log2 = m_row * scale_log2;
    float l_row = 0.f;
    if (ok) {
        load_kv(ksrc, sK0, 0);
        commit();
        load_kv(vsrc, sV, 0);
        commit();
        if (1 < ntiles) load_kv(ksrc, sK1, 1);
        commit();
        asm volatile("cp.async.wait_group 2;" ::: "memory");   // key tile 0 landed
        publish();
        if (tid == 0) {
            tc_fence_after();
            issue_s(0);
        }
    }
    for (int tile = 0; tile < ntiles && ok; ++tile) {
        const int b = tile & 1;
        if (tile > 0) {
            ok = mbar_wait(&sh->bar_o, ph_o, cta_abort, status);   // P and V of the previous tile have been read
            ph_o ^= 1u;
            if (!ok) break;
            load_kv(vsrc, sV, tile);
            commit();
            asm volatile("cp.async.wait_group 1;" ::: "memory");   // key tile + 1 landed (V may be in flight)
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        publish();                                          // also: every thread has read S(tile - 1)
        if (tid == 0 && tile + 1 < ntiles) {
            tc_fence_after();
            issue_s(tile + 1);
        }
        ok = mbar_wait(&sh->bar_s[b], ph_s[b], cta_abort, status);
        ph_s[b] ^= 1u;
        if (!ok) break;
        tc_fence_after();
        if (tile + 2 < ntiles) load_kv(ksrc, b ? sK1 : sK0, tile + 2);
        commit();
        // thread r: row r of S -> P (two bf16 terms) into the swizzled A-operand tiles
        const uint32_t ph_base = smem_u32(sPh) + tid * 128, pl_base = smem_u32(sPl) + tid * 128;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32((b ? tmem_s1 : tmem_s0) + lane_base + half * 32, v);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {                         // 8 keys = one 16-byte chunk
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int j = c4 * 8 + u * 2;
                    const int key = tile * kTK + half * 32 + j;
                    const float p0 = key < NK ? exp2f(__uint_as_float(v[j]) * scale_log2 - m_log2) : 0.f;
                    const float p1 = key + 1 < NK ? exp2f(__uint_as_float(v[j + 1]) * scale_log2 - m_log2) : 0.f;
                    l_row += p0 + p1;
                    const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                    const float2 hf = __bfloat1622float2(h);
                    const __nv_bfloat162 l = __floats2bfloat162_rn(p0 - hf.x, p1 - hf.y);
                    hi[u] = *reinterpret_cast<const uint32_t*>(&h);
                    lo[u] = *reinterpret_cast<const uint32_t*>(&l);
                }
                const uint32_t off = static_cast<uint32_t>(((half * 4 + c4) ^ (tid & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ph_base + off), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]),
                             "r"(hi[3])
                             : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(pl_base + off), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]),
                             "r"(lo[3])
                             : "memory");
            }
        }
        asm volatile("cp.async.wait_group 1;" ::: "memory");        // V tile landed (key tile + 2 may be in flight)
        publish();
        if (tid == 0) {
            tc_fence_after();
            const uint32_t pa = smem_u32(sPh), pb = smem_u32(sPl), vb = smem_u32(sV);
#pragma unroll
            for (int kk = 0; kk < kTK / 16; ++kk) {                  // 16 keys per MMA
                const uint64_t bdesc = desc_mn_major(vb + kk * 2048, kTK * 128);
                umma(tmem_o, desc_k_major(pa + kk * 32), bdesc, idesc_o, (tile > 0 || kk > 0) ? 1u : 0u);
                umma(tmem_o, desc_k_major(pb + kk * 32), bdesc, idesc_o, 1u);
            }
            umma_commit(&sh->bar_o);
        }
    }
    if (ok) ok = mbar_wait(&sh->bar_o, ph_o, cta_abort, status);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (ok) {
        tc_fence_after();
        const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
        __nv_bfloat16* orow = a.o + static_cast<size_t>(t.q_row0 + tid) * d + head * kHD;
#pragma unroll 1
        for (int c = 0; c < kHD / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(tmem_o + lane_base + c * 32, v);
            if (tid < t.nq) {
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
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh->tmem_base), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

// Refresh attention on the tensor cores: a.tiles = work items of up to 128 query rows whose keys are the
// fresh rows [f0, f0 + n0) (cA = cB0 = cB1 = n1 = 0), head dim 128.
cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st) {
    if (a.n_tiles == 0) return cudaSuccess;
    if (a.hd != kHD) return cudaErrorInvalidValue;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    return launch_kernel(attention_tc_kernel, dim3(a.n_tiles, a.H), dim3(kThreads), kSmemBytes, st, a, status);
}

}  // namespace odb
