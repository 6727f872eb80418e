// Bidirectional block-query attention.
//
// A work item (QTile) is up to 64 query rows sharing one key set: cached K/V of the positions
// outside the block (read from the cache written by the refresh), followed by fresh K/V rows
// of the same forward (the copy's own block rows; in the decoded-share layout also copy 0's
// rows at decoded positions; in a refresh every row of the sequence).  No causal mask.
// grid = (tiles, heads, key splits); each CTA streams its share of the keys in tiles of 64
// through shared memory with 16-byte cp.async loads (double buffered, XOR-swizzled rows) and
// runs an online-softmax on mma.sync m16n8k16 bf16 tiles (fp32 scores, statistics and output
// accumulator; probabilities enter the P.V product as a two-term bf16 sum).  With more than one key
// split the unnormalised partial outputs and (max, sum) pairs are merged in split order by a
// second kernel, so the result does not depend on scheduling.
#include "odb_internal.cuh"
#include "attention_body.cuh"

namespace odb {

namespace {

struct CtaSync {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};

template <int HD>
__global__ void __launch_bounds__(kAttnThreads) attention_kernel(AttnArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    pdl_launch_dependents();
    l2_prefetch_slice(a.pf, (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x, gridDim.x * gridDim.y * gridDim.z);
    if (!a.early) pdl_wait();                          // the tile table itself is written by the predecessor chain
    const QTile t = a.tiles[blockIdx.x];
    bool waited = !a.early;
    attention_item<HD, CtaSync>(a, t, blockIdx.y, blockIdx.z, threadIdx.x, smem, a.early != 0, [&]() {
        if (!waited) pdl_wait();
        waited = true;
    });
}

// ---------------------------------------------------------------------------------------------
// Decode-step attention for several block copies at once ("query rows sharing the cached KV").
//
// grid (step tiles, heads, ksplit), 256 threads = 8 warps, warp w = slab w of the StepTile (16 query
// rows of one copy).  Splits 0 .. ks-2 stream a contiguous range of the cached K/V tiles of the
// positions outside the block: each tile is loaded ONCE and used by every copy in the item.  The
// last split handles the fresh keys, one tile per source copy; a slab takes part only in the tiles
// of copies it may see (its own copy; copy 0's decoded rows in the decoded-share layout), so the
// copies stay mutually invisible without any mask tensor.  Partials go to the same (max, sum,
// output) workspace as the plain kernel's and are merged by attention_combine_kernel.
// ---------------------------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(256) step_attention_kernel(StepAttnArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int CH = HD / 8;
    constexpr int kTileBytes = kTileK * HD * 2;
    uint8_t* sQ = smem;                              // [128][HD]: slab w = rows 16 w .. 16 w + 15
    uint8_t* sK = sQ + 128 * HD * 2;                 // [2][64][HD]
    uint8_t* sV = sK + 2 * kTileBytes;               // [2][64][HD]
    uint8_t* sValid = sV + 2 * kTileBytes;           // [2][64]: 0 invalid, 1 valid, 2 valid and decoded

    pdl_launch_dependents();
    // the tile table and the K/V cache were complete before this step's launch chain began: the splits
    // that stream cached keys request their first two tiles before waiting for the predecessor
    const StepTile& t = a.tiles[blockIdx.x];
    const int head = blockIdx.y;
    const int z = blockIdx.z, ks = gridDim.z;
    const bool fresh_cta = z == ks - 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d = a.H * HD;
    const int n_cache = t.cA + (t.cB1 - t.cB0);
    const int nct = (n_cache + kTileK - 1) / kTileK;
    const int tp = (nct + ks - 2) / (ks - 1);
    const int t0 = fresh_cta ? 0 : z * tp;
    const int t1 = fresh_cta ? t.n_src : min(nct, t0 + tp);

    const size_t per_kv = static_cast<size_t>(a.H) * a.max_seq * HD;
    const __nv_bfloat16* ck = a.cache + (static_cast<size_t>(t.seq) * a.n_layers + a.layer) * 2 * per_kv +
                              static_cast<size_t>(head) * a.max_seq * HD;
    const __nv_bfloat16* cv = ck + per_kv;

    auto load_tile = [&](int tile, int buf) {
        for (int c = threadIdx.x; c < kTileK * CH; c += 256) {
            const int key = c / CH, ch = c % CH;
            bool ok;
            int flag = 1;
            const __nv_bfloat16 *ksrc = a.q, *vsrc = a.q;
            if (!fresh_cta) {
                const int kv = tile * kTileK + key;
                ok = kv < n_cache;
                const int pos = kv < t.cA ? kv : t.cB0 + (kv - t.cA);
                if (ok) {
                    ksrc = ck + static_cast<size_t>(pos) * HD + ch * 8;
                    vsrc = cv + static_cast<size_t>(pos) * HD + ch * 8;
                }
            } else {
                ok = key < t.src_n[tile];
                if (ok) {
                    const int row = t.src_row0[tile] + key;
                    ksrc = a.k + static_cast<size_t>(row) * d + head * HD + ch * 8;
                    vsrc = a.v + static_cast<size_t>(row) * d + head * HD + ch * 8;
                    if (a.row_flags[row] & kRowDecoded) flag = 2;
                }
            }
            cp_async16(sK + buf * kTileBytes + swz<HD>(key, ch), ksrc, ok);
            cp_async16(sV + buf * kTileBytes + swz<HD>(key, ch), vsrc, ok);
            if (ch == 0) sValid[buf * kTileK + key] = ok ? flag : 0;
        }
    };
    // four cp.async groups: cached tiles t0 and t0 + 1 (before the wait), then Q with the fresh split's
    // first tile, then its second
    if (!fresh_cta && t0 < t1) load_tile(t0, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (!fresh_cta && t0 + 1 < t1) load_tile(t0 + 1, 1);
    asm volatile("cp.async.commit_group;" ::: "memory");
    pdl_wait();
    l2_prefetch_slice(a.pf, (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x, gridDim.x * gridDim.y * gridDim.z);
    // ---- Q: slab w holds the rows slab_row0[w] .. + slab_n[w] ----
    for (int c = threadIdx.x; c < 128 * CH; c += 256) {
        const int r = c / CH, ch = c % CH;
        const int sl = r >> 4, rr = r & 15;
        const bool ok = sl < t.n_slabs && rr < t.slab_n[sl];
        const __nv_bfloat16* src = ok ? a.q + static_cast<size_t>(t.slab_row0[sl] + rr) * d + head * HD + ch * 8 : a.q;
        cp_async16(sQ + swz<HD>(r, ch), src, ok);
    }
    if (fresh_cta && t0 < t1) load_tile(t0, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (fresh_cta && t0 + 1 < t1) load_tile(t0 + 1, 1);
    asm volatile("cp.async.commit_group;" ::: "memory");

    const bool warp_active = warp < t.n_slabs;
    const int my_copy = warp_active ? t.slab_copy[warp] : -1;
    float o_acc[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    const float scale_log2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;
    const uint32_t qbase = smem_u32(sQ);
    const int j = lane >> 3, r8 = lane & 7;

    for (int tile = t0; tile < t1; ++tile) {
        const int buf = (tile - t0) & 1;
        if (tile + 1 < t1) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        // which keys of this tile may this slab see?  cached: all; fresh of its own copy: all;
        // fresh of copy 0 (decoded-share layout): the decoded ones; fresh of another copy: none
        int need = 1;                                   // minimum sValid value that counts as visible
        bool take = warp_active;
        if (fresh_cta && warp_active) {
            const int sc = t.src_copy[tile];
            if (sc == my_copy) need = 1;
            else if (t.stage2 && sc == 0) need = 2;
            else take = false;
        }
        if (take) {
            const uint32_t kbase = smem_u32(sK + buf * kTileBytes);
            const uint32_t vbase = smem_u32(sV + buf * kTileBytes);
            const uint8_t* valid = sValid + buf * kTileK;
            float s[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
            for (int kq = 0; kq < HD / 16; ++kq) {
                uint32_t qa[4];
                ldmatrix_x4(qa, qbase + swz<HD>(warp * 16 + r8 + (j & 1) * 8, kq * 2 + (j >> 1)));
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t kb[4];
                    ldmatrix_x4(kb, kbase + swz<HD>(np * 16 + r8 + (j >> 1) * 8, kq * 2 + (j & 1)));
                    mma_bf16(s[2 * np], qa, kb[0], kb[1]);
                    mma_bf16(s[2 * np + 1], qa, kb[2], kb[3]);
                }
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
                    s[nt][e] = valid[col] >= need ? s[nt][e] * scale_log2 : -INFINITY;
                }
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                float mx = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(s[nt][2 * r], s[nt][2 * r + 1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run[r], mx);
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float corr = exp2f(m_run[r] - m_use);
                m_run[r] = m_new;
                float rs = 0.f;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    const float p0 = exp2f(s[nt][2 * r] - m_use);
                    const float p1 = exp2f(s[nt][2 * r + 1] - m_use);
                    s[nt][2 * r] = p0;
                    s[nt][2 * r + 1] = p1;
                    rs += p0 + p1;
                }
                l_run[r] = l_run[r] * corr + rs;
#pragma unroll
                for (int i = 0; i < HD / 8; ++i) {
                    o_acc[i][2 * r] *= corr;
                    o_acc[i][2 * r + 1] *= corr;
                }
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t pa[4], pl[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float x0 = s[2 * kk + (u >> 1)][(u & 1) * 2], x1 = s[2 * kk + (u >> 1)][(u & 1) * 2 + 1];
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(x0, x1);
                    const float2 hf = __bfloat1622float2(hi);
                    pa[u] = *reinterpret_cast<const uint32_t*>(&hi);
                    pl[u] = pack_bf16(x0 - hf.x, x1 - hf.y);
                }
#pragma unroll
                for (int dp = 0; dp < HD / 16; ++dp) {
                    uint32_t vb[4];
                    ldmatrix_x4_trans(vb, vbase + swz<HD>(kk * 16 + r8 + (j & 1) * 8, dp * 2 + (j >> 1)));
                    mma_bf16(o_acc[2 * dp], pa, vb[0], vb[1]);
                    mma_bf16(o_acc[2 * dp + 1], pa, vb[2], vb[3]);
                    mma_bf16(o_acc[2 * dp], pl, vb[0], vb[1]);
                    mma_bf16(o_acc[2 * dp + 1], pl, vb[2], vb[3]);
                }
            }
        }
        if (tile + 2 < t1) {
            __syncthreads();                               // everyone is done with this buffer
            load_tile(tile + 2, buf);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (!warp_active) return;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int qr = (lane >> 2) + r * 8;
        if (qr >= t.slab_n[warp]) continue;
        const int row = t.slab_row0[warp] + qr;
        const size_t pr = (static_cast<size_t>(z) * a.M + row) * a.H + head;
        float* po = a.part_o + pr * HD + (lane & 3) * 2;
#pragma unroll
        for (int nt = 0; nt < HD / 8; ++nt)
            *reinterpret_cast<float2*>(po + nt * 8) = make_float2(o_acc[nt][2 * r], o_acc[nt][2 * r + 1]);
        if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + pr * 2) = make_float2(m_run[r], l_run[r]);
    }
}

// grid (M, H), block HD / 4: merge the key splits in split order.  The (max, sum) pairs of all
// splits are read first, then the partial outputs as float4 in groups of four independent loads.
__global__ void attention_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                         __nv_bfloat16* __restrict__ o, int M, int H, int hd, int ksplit) {
    pdl_launch_dependents();
    pdl_wait();
    const int row = blockIdx.x, head = blockIdx.y, d4 = threadIdx.x * 4;
    const size_t zs = static_cast<size_t>(M) * H, base = static_cast<size_t>(row) * H + head;
    constexpr int kMaxSplit = 8;                         // the launcher never uses more
    float2 ml[kMaxSplit];
#pragma unroll
    for (int z = 0; z < kMaxSplit; ++z)
        if (z < ksplit) ml[z] = *reinterpret_cast<const float2*>(part_ml + (z * zs + base) * 2);
    float4 v[kMaxSplit];
#pragma unroll
    for (int z = 0; z < kMaxSplit; ++z)
        if (z < ksplit) v[z] = *reinterpret_cast<const float4*>(part_o + (z * zs + base) * hd + d4);
    float mmax = -INFINITY;
#pragma unroll
    for (int z = 0; z < kMaxSplit; ++z)
        if (z < ksplit && ml[z].y > 0.f) mmax = fmaxf(mmax, ml[z].x);
    float L = 0.f;
    float4 acc = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int z = 0; z < kMaxSplit; ++z) {
        if (z < ksplit && ml[z].y > 0.f) {
            const float wt = exp2f(ml[z].x - mmax);
            L += ml[z].y * wt;
            acc.x += v[z].x * wt; acc.y += v[z].y * wt; acc.z += v[z].z * wt; acc.w += v[z].w * wt;
        }
    }
    const float inv = L > 0.f ? 1.0f / L : 0.f;
    __nv_bfloat16* op = o + base * hd + d4;
    *reinterpret_cast<__nv_bfloat162*>(op) = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    *reinterpret_cast<__nv_bfloat162*>(op + 2) = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
}

template <int HD>
cudaError_t launch_hd(const AttnArgs& a, cudaStream_t st) {
    const size_t smem = kTileQ * HD * 2 + 4 * kTileK * HD * 2 + 2 * kTileK;
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = set_smem_limit_once(attr_done, attention_kernel<HD>, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    dim3 grid(a.n_tiles, a.H, a.ksplit);
    if (a.ksplit > 8) return cudaErrorInvalidValue;
    e = launch_kernel(attention_kernel<HD>, grid, dim3(kAttnThreads), smem, st, a);
    if (e != cudaSuccess || a.ksplit == 1) return e;
    return launch_kernel(attention_combine_kernel, dim3(a.M, a.H), dim3(HD / 4), 0, st, static_cast<const float*>(a.part_o),
                         static_cast<const float*>(a.part_ml), a.o, a.M, a.H, HD, a.ksplit);
}

}  // namespace

template <int HD>
cudaError_t launch_step_hd(const StepAttnArgs& a, cudaStream_t st) {
    const size_t smem = 128 * HD * 2 + 4 * kTileK * HD * 2 + 2 * kTileK;
    static std::atomic<unsigned long long> attr_done{0};
    cudaError_t e = set_smem_limit_once(attr_done, step_attention_kernel<HD>, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    e = launch_kernel(step_attention_kernel<HD>, dim3(a.n_tiles, a.H, a.ksplit), dim3(256), smem, st, a);
    if (e != cudaSuccess) return e;
    return launch_kernel(attention_combine_kernel, dim3(a.M, a.H), dim3(HD / 4), 0, st, static_cast<const float*>(a.part_o),
                         static_cast<const float*>(a.part_ml), a.o, a.M, a.H, HD, a.ksplit);
}

// merges the key-split partials (part_o, part_ml) of M rows x H heads in split order into the bf16 output
cudaError_t launch_attention_combine(const float* part_o, const float* part_ml, __nv_bfloat16* o, int M, int H, int hd,
                                     int ksplit, cudaStream_t st) {
    return launch_kernel(attention_combine_kernel, dim3(M, H), dim3(hd / 4), 0, st, part_o, part_ml, o, M, H, hd, ksplit);
}

cudaError_t launch_step_attention(const StepAttnArgs& a, cudaStream_t st) {
    if (a.n_tiles == 0) return cudaSuccess;
    if (a.ksplit < 2 || a.ksplit > 8) return cudaErrorInvalidValue;
    return a.hd == 128 ? launch_step_hd<128>(a, st) : launch_step_hd<64>(a, st);
}

cudaError_t launch_attention(const AttnArgs& a, cudaStream_t st) {
    if (a.n_tiles == 0) return cudaSuccess;
    return a.hd == 128 ? launch_hd<128>(a, st) : launch_hd<64>(a, st);
}

}  // namespace odb
