// Small memory-bound kernels between the GEMMs: embedding gather, residual + split-K reduction
// + RMSNorm operand, split-K reduction + RoPE + K/V cache scatter, and the vocab-wide confidence
// reduction (SwiGLU lives in the gate/up GEMM's epilogue).  All reductions run in a fixed order (bitwise reproducible).
#include "odb_internal.cuh"

namespace odb {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(c, d);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    return pk;
}

// block-wide sum, same value returned to every thread; `red` has >= 32 floats
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += red[w];
    return t;
}

__global__ void embed_kernel(const __nv_bfloat16* __restrict__ embed, const int32_t* __restrict__ row_tok,
                             float* __restrict__ h, int d) {
    pdl_launch_dependents();
    pdl_wait();
    const int row = blockIdx.x;
    const __nv_bfloat16* src = embed + static_cast<size_t>(row_tok[row]) * d;
    float* dst = h + static_cast<size_t>(row) * d;
    for (int i = threadIdx.x * 2; i < d; i += blockDim.x * 2) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(src + i);
        *reinterpret_cast<float2*>(dst + i) = __bfloat1622float2(v);
    }
}

// grid (output rows, slices of kNormSliceCols columns), one float4 per thread: the part of RMSNorm that is
// not a row scalar.  x = residual stream row (after adding the split-K partials of the preceding projection
// in split order; all splits are requested at once, one memory round trip); writes bf16(x * gain) as the
// projection's operand and this slice's sum(x^2) for the projection's consumer.
__global__ void __launch_bounds__(kNormSliceCols / 4) rmsnorm_kernel(float* __restrict__ h, const float* __restrict__ partial,
                                                                     int splits, size_t pstride, const float* __restrict__ gain,
                                                                     __nv_bfloat16* __restrict__ out, float* __restrict__ ssq,
                                                                     const int32_t* __restrict__ row_map, int d, L2Prefetch pf,
                                                                     TpWait tw) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    tp_wait_flags(tw);   // tensor parallelism: the partials of every rank have arrived
    l2_prefetch_slice(pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
    const int orow = blockIdx.x;
    const int row = row_map ? row_map[orow] : orow;
    const int i = blockIdx.y * (kNormSliceCols / 4) + threadIdx.x;   // float4 index within the row
    float ss = 0.f;
    if (i < (d >> 2)) {
        float* hr = h + static_cast<size_t>(row) * d;
        float4 v = reinterpret_cast<const float4*>(hr)[i];
        if (partial) {
            const float* p = partial + static_cast<size_t>(row) * d + 4 * i;
            float4 t[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (u < splits) t[u] = *reinterpret_cast<const float4*>(p + static_cast<size_t>(u) * pstride);
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (u < splits) { v.x += t[u].x; v.y += t[u].y; v.z += t[u].z; v.w += t[u].w; }
            reinterpret_cast<float4*>(hr)[i] = v;
        }
        ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        const float4 g = reinterpret_cast<const float4*>(gain)[i];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * g.x, v.y * g.y);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(v.z * g.z, v.w * g.w);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&lo);
        pk.y = *reinterpret_cast<const uint32_t*>(&hi);
        reinterpret_cast<uint2*>(out + static_cast<size_t>(orow) * d)[i] = pk;
    }
    const float total = block_sum(ss, red);
    if (threadIdx.x == 0) ssq[static_cast<size_t>(orow) * gridDim.y + blockIdx.y] = total;
}

// The same for many rows (a refresh): kNormRows rows per block, every load of the thread's rows and splits in
// flight at once, so that the kernel runs nearer memory speed instead of at one short round trip per block
// (768 rows x 4096, three splits: 21 -> 14.5 us per launch).  Same sums in the same order per row.
constexpr int kNormRows = 4;
constexpr int kNormRowsMaxSplits = 4;
__global__ void __launch_bounds__(kNormSliceCols / 4) rmsnorm_rows_kernel(float* __restrict__ h, const float* __restrict__ partial,
                                                                          int splits, size_t pstride,
                                                                          const float* __restrict__ gain,
                                                                          __nv_bfloat16* __restrict__ out, float* __restrict__ ssq,
                                                                          const int32_t* __restrict__ row_map, int rows_out, int d,
                                                                          TpWait tw) {
    __shared__ float red[kNormRows][32];
    pdl_launch_dependents();
    pdl_wait();
    tp_wait_flags(tw);
    const int i = blockIdx.y * (kNormSliceCols / 4) + threadIdx.x;   // float4 index within the row
    const int orow0 = blockIdx.x * kNormRows;
    const bool in = i < (d >> 2);
    float4 v[kNormRows], t[kNormRows][kNormRowsMaxSplits];
    int row[kNormRows];
#pragma unroll
    for (int r = 0; r < kNormRows; ++r) {
        const int orow = orow0 + r;
        row[r] = orow < rows_out ? (row_map ? row_map[orow] : orow) : -1;
    }
#pragma unroll
    for (int r = 0; r < kNormRows; ++r) {
        if (!in || row[r] < 0) continue;
        v[r] = reinterpret_cast<const float4*>(h + static_cast<size_t>(row[r]) * d)[i];
        if (partial) {
            const float* p = partial + static_cast<size_t>(row[r]) * d + 4 * i;
#pragma unroll
            for (int u = 0; u < kNormRowsMaxSplits; ++u)
                if (u < splits) t[r][u] = *reinterpret_cast<const float4*>(p + static_cast<size_t>(u) * pstride);
        }
    }
    float4 g = make_float4(0.f, 0.f, 0.f, 0.f);
    if (in) g = reinterpret_cast<const float4*>(gain)[i];
    float ss[kNormRows];
#pragma unroll
    for (int r = 0; r < kNormRows; ++r) {
        ss[r] = 0.f;
        if (!in || row[r] < 0) continue;
        float4 x = v[r];
        if (partial) {
#pragma unroll
            for (int u = 0; u < kNormRowsMaxSplits; ++u)
                if (u < splits) { x.x += t[r][u].x; x.y += t[r][u].y; x.z += t[r][u].z; x.w += t[r][u].w; }
            reinterpret_cast<float4*>(h + static_cast<size_t>(row[r]) * d)[i] = x;
        }
        ss[r] = x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        reinterpret_cast<uint2*>(out + static_cast<size_t>(orow0 + r) * d)[i] = pack4_bf16(x.x * g.x, x.y * g.y, x.z * g.z, x.w * g.w);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
#pragma unroll
    for (int r = 0; r < kNormRows; ++r) {
        const float w = warp_sum(ss[r]);
        if (lane == 0) red[r][warp] = w;
    }
    __syncthreads();
    if (threadIdx.x < kNormRows && orow0 + threadIdx.x < rows_out) {
        float total = 0.f;
        for (int w = 0; w < nw; ++w) total += red[threadIdx.x][w];
        ssq[static_cast<size_t>(orow0 + threadIdx.x) * gridDim.y + blockIdx.y] = total;
    }
}

// More than 64 rows: grid (rows, chunks), one thread per FOUR consecutive rotation pairs (float4 loads, 8-byte
// stores; 1.5 x the throughput of the one-pair kernel below, which stays the faster one on the few rows of a
// decode step, where the kernel is a single memory round trip on the dependency chain).  Sums the
// QKV partials in split order, applies the RMSNorm scalar, rotates q and k (rotate-half pairing: element i
// pairs with i + hd/2; angle = pos * theta^(-2i/hd), table precomputed), rounds to bf16 and writes the
// row-major fresh q/k/v; in a refresh also the K/V cache [seq][layer][k|v][head][pos][hd].  hd/2 is a
// multiple of 4, so the four pairs of a thread lie in one head.

__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ void scale4(float4& a, float s) { a.x *= s; a.y *= s; a.z *= s; a.w *= s; }

__global__ void qkv_rope_vec4_kernel(QkvRopeArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    l2_prefetch_slice(a.pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
    const int row = blockIdx.x;
    const int d = a.H * a.hd, half = a.hd / 2;
    const int pos = a.row_pos[row];
    const int seq = a.row_seq[row];
    const float* p0 = a.partial + static_cast<size_t>(row) * 3 * d;
    const float2* rope = a.rope + static_cast<size_t>(pos) * half;
    __nv_bfloat16* ck = nullptr;
    __nv_bfloat16* cv = nullptr;
    if (a.cache) {
        const size_t per_kv = static_cast<size_t>(a.H) * a.max_seq * a.hd;
        ck = a.cache + (static_cast<size_t>(seq) * a.n_layers + a.layer) * 2 * per_kv;
        cv = ck + per_kv;
    }
    const float inv = row_scale_of(a.scale, row);   // scalar of the RMSNorm folded behind the projection
    for (int t = (blockIdx.y * blockDim.x + threadIdx.x) * 4; t < d / 2; t += gridDim.y * blockDim.x * 4) {
        const int head = t / half, i = t % half;
        const int e0 = head * a.hd + i, e1 = e0 + half;
        float4 q0 = {0.f, 0.f, 0.f, 0.f}, q1 = q0, k0 = q0, k1 = q0, v0 = q0, v1 = q0;
        for (int sb = 0; sb < a.splits; sb += 2) {
            float4 tt[2][6];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (sb + u < a.splits) {
                    const float* p = p0 + static_cast<size_t>(sb + u) * a.pstride;
                    tt[u][0] = *reinterpret_cast<const float4*>(p + e0); tt[u][1] = *reinterpret_cast<const float4*>(p + e1);
                    tt[u][2] = *reinterpret_cast<const float4*>(p + d + e0); tt[u][3] = *reinterpret_cast<const float4*>(p + d + e1);
                    tt[u][4] = *reinterpret_cast<const float4*>(p + 2 * d + e0); tt[u][5] = *reinterpret_cast<const float4*>(p + 2 * d + e1);
                }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (sb + u < a.splits) {
                    add4(q0, tt[u][0]); add4(q1, tt[u][1]); add4(k0, tt[u][2]); add4(k1, tt[u][3]); add4(v0, tt[u][4]); add4(v1, tt[u][5]);
                }
            }
        }
        scale4(q0, inv); scale4(q1, inv); scale4(k0, inv); scale4(k1, inv); scale4(v0, inv); scale4(v1, inv);
        const float4 c01 = *reinterpret_cast<const float4*>(rope + i);       // (cos, sin) of pairs i, i + 1
        const float4 c23 = *reinterpret_cast<const float4*>(rope + i + 2);   // and of pairs i + 2, i + 3
        const uint2 rq0 = pack4_bf16(q0.x * c01.x - q1.x * c01.y, q0.y * c01.z - q1.y * c01.w, q0.z * c23.x - q1.z * c23.y,
                                     q0.w * c23.z - q1.w * c23.w);
        const uint2 rq1 = pack4_bf16(q1.x * c01.x + q0.x * c01.y, q1.y * c01.z + q0.y * c01.w, q1.z * c23.x + q0.z * c23.y,
                                     q1.w * c23.z + q0.w * c23.w);
        const uint2 rk0 = pack4_bf16(k0.x * c01.x - k1.x * c01.y, k0.y * c01.z - k1.y * c01.w, k0.z * c23.x - k1.z * c23.y,
                                     k0.w * c23.z - k1.w * c23.w);
        const uint2 rk1 = pack4_bf16(k1.x * c01.x + k0.x * c01.y, k1.y * c01.z + k0.y * c01.w, k1.z * c23.x + k0.z * c23.y,
                                     k1.w * c23.z + k0.w * c23.w);
        const uint2 rv0 = pack4_bf16(v0.x, v0.y, v0.z, v0.w), rv1 = pack4_bf16(v1.x, v1.y, v1.z, v1.w);
        const size_t o = static_cast<size_t>(row) * d;
        *reinterpret_cast<uint2*>(a.q + o + e0) = rq0; *reinterpret_cast<uint2*>(a.q + o + e1) = rq1;
        *reinterpret_cast<uint2*>(a.k + o + e0) = rk0; *reinterpret_cast<uint2*>(a.k + o + e1) = rk1;
        *reinterpret_cast<uint2*>(a.v + o + e0) = rv0; *reinterpret_cast<uint2*>(a.v + o + e1) = rv1;
        if (ck) {
            const size_t c = (static_cast<size_t>(head) * a.max_seq + pos) * a.hd;
            *reinterpret_cast<uint2*>(ck + c + i) = rk0; *reinterpret_cast<uint2*>(ck + c + i + half) = rk1;
            *reinterpret_cast<uint2*>(cv + c + i) = rv0; *reinterpret_cast<uint2*>(cv + c + i + half) = rv1;
        }
    }
}

// grid (rows, pair chunks), one thread per rotation pair.  Sums the QKV partials, rotates q and k (rotate-half pairing: element i
// pairs with i + hd/2; angle = pos * theta^(-2i/hd), table precomputed), rounds to bf16 and
// writes the row-major fresh q/k/v; in a refresh also the K/V cache [seq][layer][k|v][head][pos][hd].
__global__ void qkv_rope_kernel(QkvRopeArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    l2_prefetch_slice(a.pf, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y);
    const int row = blockIdx.x;
    const int d = a.H * a.hd, half = a.hd / 2;
    const int pos = a.row_pos[row];
    const int seq = a.row_seq[row];
    const float* p0 = a.partial + static_cast<size_t>(row) * 3 * d;
    const float2* rope = a.rope + static_cast<size_t>(pos) * half;
    __nv_bfloat16* ck = nullptr;
    __nv_bfloat16* cv = nullptr;
    if (a.cache) {
        const size_t per_kv = static_cast<size_t>(a.H) * a.max_seq * a.hd;
        ck = a.cache + (static_cast<size_t>(seq) * a.n_layers + a.layer) * 2 * per_kv;
        cv = ck + per_kv;
    }
    for (int t = blockIdx.y * blockDim.x + threadIdx.x; t < d / 2; t += gridDim.y * blockDim.x) {
        const int head = t / half, i = t % half;
        const int e0 = head * a.hd + i, e1 = e0 + half;
        float q0 = 0.f, q1 = 0.f, k0 = 0.f, k1 = 0.f, v0 = 0.f, v1 = 0.f;
        for (int sb = 0; sb < a.splits; sb += 4) {
            float t[4][6];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (sb + u < a.splits) {
                    const float* p = p0 + static_cast<size_t>(sb + u) * a.pstride;
                    t[u][0] = p[e0]; t[u][1] = p[e1];
                    t[u][2] = p[d + e0]; t[u][3] = p[d + e1];
                    t[u][4] = p[2 * d + e0]; t[u][5] = p[2 * d + e1];
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (sb + u < a.splits) {
                    q0 += t[u][0]; q1 += t[u][1]; k0 += t[u][2]; k1 += t[u][3]; v0 += t[u][4]; v1 += t[u][5];
                }
            }
        }
        const float inv = row_scale_of(a.scale, row);   // scalar of the RMSNorm folded behind the projection
        q0 *= inv; q1 *= inv; k0 *= inv; k1 *= inv; v0 *= inv; v1 *= inv;
        const float2 cs = rope[i];
        const __nv_bfloat16 rq0 = __float2bfloat16_rn(q0 * cs.x - q1 * cs.y);
        const __nv_bfloat16 rq1 = __float2bfloat16_rn(q1 * cs.x + q0 * cs.y);
        const __nv_bfloat16 rk0 = __float2bfloat16_rn(k0 * cs.x - k1 * cs.y);
        const __nv_bfloat16 rk1 = __float2bfloat16_rn(k1 * cs.x + k0 * cs.y);
        const __nv_bfloat16 rv0 = __float2bfloat16_rn(v0), rv1 = __float2bfloat16_rn(v1);
        const size_t o = static_cast<size_t>(row) * d;
        a.q[o + e0] = rq0; a.q[o + e1] = rq1;
        a.k[o + e0] = rk0; a.k[o + e1] = rk1;
        a.v[o + e0] = rv0; a.v[o + e1] = rv1;
        if (ck) {
            const size_t c = (static_cast<size_t>(head) * a.max_seq + pos) * a.hd;
            ck[c + i] = rk0; ck[c + i + half] = rk1;
            cv[c + i] = rv0; cv[c + i + half] = rv1;
        }
    }
}

// Greedy token (lowest id on ties, [MASK] excluded) and its softmax probability
// conf = 1 / sum_j exp(l_j - l_max) per row of logits.  Phase 1: grid (rows, chunks), every block
// makes one online pass (running max / rescaled sum / argmax) over its slice of the vocabulary
// and writes a (max, sum, argmax) triple; phase 2 merges a row's triples in chunk order.
__global__ void __launch_bounds__(256) confidence_partial_kernel(const float* __restrict__ logits, int V, int mask_id,
                                                                 int chunk, ConfPartial* __restrict__ part) {
    __shared__ float sm[8], ss[8];
    __shared__ int si[8];
    pdl_launch_dependents();
    pdl_wait();
    const float* l = logits + static_cast<size_t>(blockIdx.x) * V;
    const int lo = blockIdx.y * chunk, hi = min(V, lo + chunk);
    float m = -INFINITY, s = 0.f;
    int idx = 0x7fffffff;
    for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const float v = l[i];
        if (i == mask_id) continue;
        if (v > m) {
            s = s * expf(m - v) + 1.0f;                 // first element: s = 0 * exp(-inf) + 1
            m = v;
            idx = i;
        } else {
            s += expf(v - m);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o);
        const float os = __shfl_xor_sync(0xffffffffu, s, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        conf_merge(m, s, idx, om, os, oi);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { sm[warp] = m; ss[warp] = s; si[warp] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (blockDim.x >> 5); ++w) conf_merge(m, s, idx, sm[w], ss[w], si[w]);
        ConfPartial p;
        p.m = m; p.s = s; p.idx = idx;
        part[static_cast<size_t>(blockIdx.x) * gridDim.y + blockIdx.y] = p;
    }
}

// One block of 128 threads per row: thread t merges triples t, t + 128, ... in ascending order, the lanes of
// a warp are merged by a fixed shuffle tree (an earlier lane's triple is always the left operand) and the
// four warps in warp order.
__global__ void __launch_bounds__(128) confidence_final_kernel(const ConfPartial* __restrict__ part, int chunks, int rows,
                                                              float* __restrict__ conf, int32_t* __restrict__ tok, TpWait tw) {
    __shared__ float sm[4], ss[4];
    __shared__ int si[4];
    pdl_launch_dependents();
    pdl_wait();
    tp_wait_flags(tw);   // tensor parallelism: every rank's vocabulary tiles have arrived
    const int row = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const ConfPartial* p = part + static_cast<size_t>(row) * chunks;
    float m = -INFINITY, s = 0.f;
    int idx = 0x7fffffff;
    for (int c = threadIdx.x; c < chunks; c += 128) conf_merge(m, s, idx, p[c].m, p[c].s, p[c].idx);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float om = __shfl_down_sync(0xffffffffu, m, o);
        const float os = __shfl_down_sync(0xffffffffu, s, o);
        const int oi = __shfl_down_sync(0xffffffffu, idx, o);
        if (lane + o < 32) conf_merge(m, s, idx, om, os, oi);
    }
    if (lane == 0) { sm[warp] = m; ss[warp] = s; si[warp] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 4; ++w) conf_merge(m, s, idx, sm[w], ss[w], si[w]);
        conf[row] = 1.0f / s;
        tok[row] = idx;
    }
}

// grid (rows, feature chunks of 256): one FFN feature per thread
__global__ void __launch_bounds__(256) swiglu_combine_kernel(const float* __restrict__ partial, int splits, size_t pstride,
                                                             RowScale scale, __nv_bfloat16* __restrict__ g, int F) {
    pdl_launch_dependents();
    pdl_wait();
    const int m = blockIdx.x;
    const int f = blockIdx.y * 256 + threadIdx.x;
    if (f >= F) return;
    const int tiles = (F + 63) / 64;
    const size_t col = static_cast<size_t>(f >> 6) * 128 + (f & 63);   // the gate entry; its up entry sits 64 further
    const float* p = partial + static_cast<size_t>(m) * tiles * 128 + col;
    float gate = 0.f, up = 0.f;
    for (int sb = 0; sb < splits; sb += 8) {
        float t[8][2];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (sb + u < splits) { t[u][0] = p[(sb + u) * pstride]; t[u][1] = p[(sb + u) * pstride + 64]; }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (sb + u < splits) { gate += t[u][0]; up += t[u][1]; }
    }
    const float sc = row_scale_of(scale, m);
    gate *= sc;
    up *= sc;
    g[static_cast<size_t>(m) * F + f] = __float2bfloat16_rn(gate / (1.0f + expf(-gate)) * up);
}

// Read-only streaming probe: every thread reads 16-byte vectors grid-stride over the buffer and folds them into
// one word, written out only if it has an (impossible) value, so that the loads cannot be removed.
__global__ void __launch_bounds__(512) read_stream_kernel(const uint4* __restrict__ src, size_t n_vec, unsigned int* sink) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    unsigned int acc = 0;
    size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n_vec; i += 4 * stride) {
        const uint4 a = __ldcs(src + i), b = __ldcs(src + i + stride), c = __ldcs(src + i + 2 * stride), d = __ldcs(src + i + 3 * stride);
        acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 a = __ldcs(src + i);
        acc ^= a.x ^ a.y ^ a.z ^ a.w;
    }
    if (acc == 0x9E3779B9u && sink) atomicAdd(sink, 1u);
}

// The same probe through the copy engine the projections use: one thread per CTA keeps a ring of kBulkStages
// bulk copies (global -> shared, completion on an mbarrier) of kBulkChunk bytes in flight over the CTA's
// contiguous share of the buffer; nothing consumes the bytes.  Waits are bounded: on expiry the thread stops
// issuing, waits (bounded again) for the copies it has in flight, and reports through `status`.
constexpr int kBulkStages = 7;
constexpr int kBulkChunk = 16384;

__global__ void __launch_bounds__(32) bulk_read_stream_kernel(const uint8_t* __restrict__ src, long long chunks_per_cta, int* status) {
    extern __shared__ __align__(1024) uint8_t ring[];
    __shared__ __align__(8) uint64_t full[kBulkStages];
    __shared__ int abort_flag, drain_status;
    if (threadIdx.x != 0) return;
    abort_flag = 0;
    for (int i = 0; i < kBulkStages; ++i)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&full[i])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint8_t* base = src + static_cast<size_t>(blockIdx.x) * chunks_per_cta * kBulkChunk;
    auto issue = [&](long long i, int st) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&full[st])), "r"(kBulkChunk) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_u32(ring + static_cast<size_t>(st) * kBulkChunk)),
                     "l"(base + static_cast<size_t>(i) * kBulkChunk), "r"(kBulkChunk), "r"(smem_u32(&full[st]))
                     : "memory");
    };
    const long long pre = chunks_per_cta < kBulkStages ? chunks_per_cta : kBulkStages;
    uint32_t in_flight = 0;   // bit s: stage s holds a copy that has not been waited for
    for (long long i = 0; i < pre; ++i) { issue(i, static_cast<int>(i)); in_flight |= 1u << i; }
    long long issued = pre;
    int st = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (long long i = 0; i < chunks_per_cta; ++i) {
        if (!mbar_wait_bounded(&full[st], ph, &abort_flag, status)) { ok = false; break; }
        in_flight &= ~(1u << st);
        if (issued < chunks_per_cta) { issue(issued, st); ++issued; in_flight |= 1u << st; }
        if (++st == kBulkStages) { st = 0; ph ^= 1; }
    }
    if (!ok) {   // wait (bounded) for the copies still in flight before the shared memory is given back
        drain_status = 0;
        for (int s = 0; s < kBulkStages; ++s) {
            if (!(in_flight & (1u << s))) continue;
            abort_flag = 0;
            mbar_wait_bounded(&full[s], s >= st ? ph : ph ^ 1, &abort_flag, &drain_status);   // stages behind the ring position are one phase on
        }
    }
}

}  // namespace

cudaError_t launch_bulk_read_stream(const void* src, size_t bytes, int grid, int* status, size_t* streamed, cudaStream_t st) {
    const long long chunks_per_cta = static_cast<long long>(bytes / (static_cast<size_t>(grid) * kBulkChunk));
    if (chunks_per_cta < 1) return cudaErrorInvalidValue;
    const int smem = kBulkStages * kBulkChunk;
    static std::atomic<unsigned long long> limit_set{0};
    cudaError_t e = set_smem_limit_once(limit_set, bulk_read_stream_kernel, smem);
    if (e != cudaSuccess) return e;
    *streamed = static_cast<size_t>(chunks_per_cta) * grid * kBulkChunk;
    bulk_read_stream_kernel<<<grid, 32, smem, st>>>(static_cast<const uint8_t*>(src), chunks_per_cta, status);
    return cudaGetLastError();
}

cudaError_t launch_swiglu_combine(const float* partial, int splits, size_t pstride, const RowScale& scale, __nv_bfloat16* g,
                                  int M, int F, cudaStream_t st) {
    return launch_kernel(swiglu_combine_kernel, dim3(M, (F + 255) / 256), dim3(256), 0, st, partial, splits, pstride, scale, g, F);
}

cudaError_t launch_read_stream(const void* src, size_t bytes, unsigned int* sink, int grid, cudaStream_t st) {
    read_stream_kernel<<<grid, 512, 0, st>>>(static_cast<const uint4*>(src), bytes / 16, sink);
    return cudaGetLastError();
}

// First kernel of a forward.  Launched WITHOUT programmatic stream serialization: it starts only when
// everything enqueued before it (the row and tile tables, the previous accept) has completed, and every
// later kernel of the chain starts after this one has started.  That is what allows the attention
// kernels to read the tile table and the K/V cache before their own griddepcontrol.wait.
cudaError_t launch_embed(const __nv_bfloat16* embed, const int32_t* row_tok, float* h, int M, int d, cudaStream_t st) {
    embed_kernel<<<dim3(M), dim3(256), 0, st>>>(embed, row_tok, h, d);
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(float* h, const float* partial, int splits, size_t pstride, const float* gain,
                           __nv_bfloat16* out, float* ssq, const int32_t* row_map, int rows_out, int d, L2Prefetch pf,
                           cudaStream_t st, const TpWait& tw) {
    if (splits > 16) return cudaErrorInvalidValue;
    const int slices = (d + kNormSliceCols - 1) / kNormSliceCols;
    if (rows_out >= 256 && splits <= kNormRowsMaxSplits)
        return launch_kernel(rmsnorm_rows_kernel, dim3((rows_out + kNormRows - 1) / kNormRows, slices), dim3(kNormSliceCols / 4), 0,
                             st, h, partial, splits, pstride, gain, out, ssq, row_map, rows_out, d, tw);
    return launch_kernel(rmsnorm_kernel, dim3(rows_out, slices), dim3(kNormSliceCols / 4), 0, st, h, partial, splits, pstride,
                         gain, out, ssq, row_map, d, pf, tw);
}

cudaError_t launch_qkv_rope(const QkvRopeArgs& a, cudaStream_t st) {
    if (a.M > 64) {   // measured at 128 rows: 0.97 vs 1.09 ms of elementwise time per step; at 32 rows the one-pair kernel wins
        const int quads = a.H * a.hd / 8;             // four rotation pairs per thread
        const int threads = quads >= 128 ? 128 : 32 * ((quads + 31) / 32);
        return launch_kernel(qkv_rope_vec4_kernel, dim3(a.M, (quads + threads - 1) / threads), dim3(threads), 0, st, a);
    }
    const int pairs = a.H * a.hd / 2;
    return launch_kernel(qkv_rope_kernel, dim3(a.M, (pairs + 255) / 256), dim3(256), 0, st, a);
}

cudaError_t launch_confidence_final(const ConfPartial* part, int chunks, int rows, float* conf, int32_t* tok,
                                    cudaStream_t st, const TpWait& tw) {
    return launch_kernel(confidence_final_kernel, dim3(rows), dim3(128), 0, st, part, chunks, rows, conf, tok, tw);
}

cudaError_t launch_confidence(const float* logits, int rows, int V, int mask_id, float* conf, int32_t* tok,
                              void* scratch, cudaStream_t st) {
    // enough blocks to fill the machine; a chunk is a multiple of 256 so that threads stay coalesced
    int chunks = (4 * 148 + rows - 1) / rows;
    if (chunks > kConfMaxChunks) chunks = kConfMaxChunks;
    int chunk = ((V + chunks - 1) / chunks + 255) / 256 * 256;
    chunks = (V + chunk - 1) / chunk;
    ConfPartial* part = static_cast<ConfPartial*>(scratch);
    cudaError_t e = launch_kernel(confidence_partial_kernel, dim3(rows, chunks), dim3(256), 0, st, logits, V, mask_id, chunk,
                                  part);
    if (e != cudaSuccess) return e;
    return launch_confidence_final(part, chunks, rows, conf, tok, st);
}

}  // namespace odb
