// The body of the block-query attention (one work item = query tile x head x key split), shared by the
// stand-alone kernel and the persistent decode-step kernel.  See attention.cu for the method.
#pragma once

#include "odb_internal.cuh"

namespace odb {

namespace {

constexpr int kTileQ = 64;
constexpr int kTileK = 64;
constexpr int kAttnThreads = 128;

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;   // size 0: destination is zero filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(sz) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// byte offset of the 16-byte chunk `chunk` of row `row` in a tile with HD bf16 per row
template <int HD>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return static_cast<uint32_t>(row * HD * 2 + ((chunk ^ (row & 7)) << 4));
}

// One work item of the attention: query tile t, one head, key split z of a.ksplit, executed by kAttnThreads
// threads (tid = 0 .. 127) that synchronise through Sync::sync() (the whole CTA in the stand-alone kernel, a
// named barrier of the worker warps inside the persistent step kernel).  smem: attention_smem_bytes<HD>() bytes,
// 128-byte aligned.  wait_inputs() returns once q and the fresh k / v of this forward are visible; with `early`
// the cached key tiles (complete before the forward began) are requested before it is called.
template <int HD>
constexpr size_t attention_smem_bytes() { return kTileQ * HD * 2 + 4 * kTileK * HD * 2 + 2 * kTileK; }

template <int HD, class Sync, class Wait>
__device__ __forceinline__ void attention_item(const AttnArgs& a, const QTile& t, int head, int z, int tid, uint8_t* smem,
                                               bool early, Wait wait_inputs) {
    constexpr int CH = HD / 8;                       // 16-byte chunks per row
    constexpr int kTileBytes = kTileK * HD * 2;
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + kTileQ * HD * 2;              // [2][64][HD]
    uint8_t* sV = sK + 2 * kTileBytes;               // [2][64][HD]
    uint8_t* sValid = sV + 2 * kTileBytes;           // [2][64]

    // early (decode steps): the tile table and the K/V cache were complete before this forward began, so
    // cached key tiles are requested before waiting for the producer of q and of the fresh k / v
    if (!early) wait_inputs();
    const int warp = tid >> 5, lane = tid & 31;
    const int d = a.H * HD;

    const int nA = t.cA, nB = t.cB1 - t.cB0;
    const int NK = nA + nB + t.n0 + t.n1;
    const int ntiles = (NK + kTileK - 1) / kTileK;
    const int tps = (ntiles + a.ksplit - 1) / a.ksplit;
    const int t0 = z * tps;
    const int t1 = min(ntiles, t0 + tps);

    const size_t per_kv = static_cast<size_t>(a.H) * a.max_seq * HD;
    const __nv_bfloat16* ck = a.cache + (static_cast<size_t>(t.seq) * a.n_layers + a.layer) * 2 * per_kv +
                              static_cast<size_t>(head) * a.max_seq * HD;
    const __nv_bfloat16* cv = ck + per_kv;

    auto load_tile = [&](int tile, int buf) {
        for (int c = tid; c < kTileK * CH; c += kAttnThreads) {
            const int key = c / CH, ch = c % CH;
            int kv = tile * kTileK + key;
            bool ok = kv < NK;
            const __nv_bfloat16* ks = a.q;
            const __nv_bfloat16* vs = a.q;
            if (ok) {
                if (kv < nA + nB) {
                    const int pos = kv < nA ? kv : t.cB0 + (kv - nA);
                    ks = ck + static_cast<size_t>(pos) * HD + ch * 8;
                    vs = cv + static_cast<size_t>(pos) * HD + ch * 8;
                } else {
                    kv -= nA + nB;
                    int row;
                    if (kv < t.n0) {
                        row = t.f0 + kv;
                    } else {
                        row = t.f1 + (kv - t.n0);
                        ok = (a.row_flags[row] & kRowDecoded) != 0;
                    }
                    ks = a.k + static_cast<size_t>(row) * d + head * HD + ch * 8;
                    vs = a.v + static_cast<size_t>(row) * d + head * HD + ch * 8;
                }
            }
            cp_async16(sK + buf * kTileBytes + swz<HD>(key, ch), ok ? ks : a.q, ok);
            cp_async16(sV + buf * kTileBytes + swz<HD>(key, ch), ok ? vs : a.q, ok);
            if (ch == 0) sValid[buf * kTileK + key] = ok ? 1 : 0;
        }
    };

    // The first two tiles are requested at once, later ones one iteration ahead.  Four cp.async groups:
    // the two tiles if they hold cached keys only (before the wait), then Q with whatever is left of
    // tile t0, then what is left of tile t0 + 1.
    bool pre0 = false, pre1 = false;
    if (early) {
        pre0 = t0 < t1 && (t0 + 1) * kTileK <= nA + nB;
        pre1 = t0 + 1 < t1 && (t0 + 2) * kTileK <= nA + nB;
        if (pre0) load_tile(t0, 0);
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (pre1) load_tile(t0 + 1, 1);
        asm volatile("cp.async.commit_group;" ::: "memory");
        wait_inputs();
    }
    // ---- Q tile ----
    for (int c = tid; c < kTileQ * CH; c += kAttnThreads) {
        const int r = c / CH, ch = c % CH;
        const bool ok = r < t.nq;
        const __nv_bfloat16* src = ok ? a.q + static_cast<size_t>(t.q_row0 + r) * d + head * HD + ch * 8 : a.q;
        cp_async16(sQ + swz<HD>(r, ch), src, ok);
    }
    if (t0 < t1 && !pre0) load_tile(t0, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (t0 + 1 < t1 && !pre1) load_tile(t0 + 1, 1);
    asm volatile("cp.async.commit_group;" ::: "memory");

    float o_acc[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o_acc[i][0] = o_acc[i][1] = o_acc[i][2] = o_acc[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    const float scale_log2 = rsqrtf(static_cast<float>(HD)) * 1.4426950408889634f;
    const bool warp_active = warp * 16 < t.nq;

    for (int tile = t0; tile < t1; ++tile) {
        const int buf = (tile - t0) & 1;
        if (tile + 1 < t1) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
        Sync::sync();                                   // tile `tile` has landed
        if (warp_active) {

        const uint32_t kbase = smem_u32(sK + buf * kTileBytes);
        const uint32_t vbase = smem_u32(sV + buf * kTileBytes);
        const uint32_t qbase = smem_u32(sQ);
        const uint8_t* valid = sValid + buf * kTileK;

        float s[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
        const int j = lane >> 3, r8 = lane & 7;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            uint32_t qa[4];
            ldmatrix_x4(qa, qbase + swz<HD>(warp * 16 + r8 + (j & 1) * 8, ks * 2 + (j >> 1)));
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t kb[4];
                ldmatrix_x4(kb, kbase + swz<HD>(np * 16 + r8 + (j >> 1) * 8, ks * 2 + (j & 1)));
                mma_bf16(s[2 * np], qa, kb[0], kb[1]);
                mma_bf16(s[2 * np + 1], qa, kb[2], kb[3]);
            }
        }
        // mask, scale into the log2 domain
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
                s[nt][e] = valid[col] ? s[nt][e] * scale_log2 : -INFINITY;
            }
        }
        // online softmax, rows lane/4 (e = 0,1) and lane/4 + 8 (e = 2,3)
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
        // O += P V.  P is fed to the tensor core as a sum of two bf16 terms (value rounded to bf16
        // plus the rounded remainder), so the product carries ~16 significant bits of P instead of
        // 8: with near-uniform attention the output is a small average of large terms and a bare
        // bf16 P would cost a full bf16 step of the result.
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
        }   // warp_active
        if (tile + 2 < t1) {
            Sync::sync();                               // everyone is done with this buffer
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
        const int qr = warp * 16 + (lane >> 2) + r * 8;
        if (qr >= t.nq) continue;
        const int row = t.q_row0 + qr;
        if (a.ksplit == 1) {
            const float inv = l_run[r] > 0.f ? 1.0f / l_run[r] : 0.f;
            __nv_bfloat16* o = a.o + static_cast<size_t>(row) * d + head * HD + (lane & 3) * 2;
#pragma unroll
            for (int nt = 0; nt < HD / 8; ++nt)
                *reinterpret_cast<__nv_bfloat162*>(o + nt * 8) =
                    __floats2bfloat162_rn(o_acc[nt][2 * r] * inv, o_acc[nt][2 * r + 1] * inv);
        } else {
            const size_t pr = (static_cast<size_t>(z) * a.M + row) * a.H + head;
            float* po = a.part_o + pr * HD + (lane & 3) * 2;
#pragma unroll
            for (int nt = 0; nt < HD / 8; ++nt)
                *reinterpret_cast<float2*>(po + nt * 8) = make_float2(o_acc[nt][2 * r], o_acc[nt][2 * r + 1]);
            if ((lane & 3) == 0) *reinterpret_cast<float2*>(a.part_ml + pr * 2) = make_float2(m_run[r], l_run[r]);
        }
    }
}

}  // namespace

}  // namespace odb
