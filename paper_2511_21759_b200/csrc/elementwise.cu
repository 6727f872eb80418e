// Small memory-bound kernels between the GEMMs: embedding gather, residual + split-K reduction
// + RMSNorm, split-K reduction + RoPE + K/V cache scatter, split-K reduction + SwiGLU, and the
// vocab-wide confidence reduction.  All reductions run in a fixed order (bitwise reproducible).
#include "odb_internal.cuh"

namespace odb {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
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
    const int row = blockIdx.x;
    const __nv_bfloat16* src = embed + static_cast<size_t>(row_tok[row]) * d;
    float* dst = h + static_cast<size_t>(row) * d;
    for (int i = threadIdx.x * 2; i < d; i += blockDim.x * 2) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(src + i);
        *reinterpret_cast<float2*>(dst + i) = __bfloat1622float2(v);
    }
}

// One block per output row.  y = x / sqrt(mean(x^2) + eps) * gain, x = residual stream row
// (after adding the split-K partials of the preceding projection in split order).
__global__ void rmsnorm_kernel(float* __restrict__ h, const float* __restrict__ partial, int splits, size_t pstride,
                               const float* __restrict__ gain, __nv_bfloat16* __restrict__ out,
                               const int32_t* __restrict__ row_map, int d, float eps) {
    __shared__ float red[32];
    const int orow = blockIdx.x;
    const int row = row_map ? row_map[orow] : orow;
    float* hr = h + static_cast<size_t>(row) * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = hr[i];
        if (partial) {
            const float* p = partial + static_cast<size_t>(row) * d + i;
            for (int s = 0; s < splits; ++s) v += p[s * pstride];
            hr[i] = v;
        }
        ss += v * v;
    }
    const float total = block_sum(ss, red);
    const float inv = 1.0f / sqrtf(total / static_cast<float>(d) + eps);
    __nv_bfloat16* o = out + static_cast<size_t>(orow) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) o[i] = __float2bfloat16_rn(hr[i] * inv * gain[i]);
}

// One block per row.  Sums the QKV partials, rotates q and k (rotate-half pairing: element i
// pairs with i + hd/2; angle = pos * theta^(-2i/hd), table precomputed), rounds to bf16 and
// writes the row-major fresh q/k/v; in a refresh also the K/V cache [seq][layer][k|v][head][pos][hd].
__global__ void qkv_rope_kernel(QkvRopeArgs a) {
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
    for (int t = threadIdx.x; t < d / 2; t += blockDim.x) {
        const int head = t / half, i = t % half;
        const int e0 = head * a.hd + i, e1 = e0 + half;
        float q0 = 0.f, q1 = 0.f, k0 = 0.f, k1 = 0.f, v0 = 0.f, v1 = 0.f;
        for (int s = 0; s < a.splits; ++s) {
            const float* p = p0 + s * a.pstride;
            q0 += p[e0]; q1 += p[e1];
            k0 += p[d + e0]; k1 += p[d + e1];
            v0 += p[2 * d + e0]; v1 += p[2 * d + e1];
        }
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

// g[m][f] = bf16( silu(gate) * up ), gate = sum_s partial[s][m][f], up = sum_s partial[s][m][F + f]
__global__ void swiglu_kernel(const float* __restrict__ partial, int splits, size_t pstride,
                              __nv_bfloat16* __restrict__ g, int M, int F) {
    const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<size_t>(M) * F) return;
    const int m = static_cast<int>(idx / F), f = static_cast<int>(idx % F);
    const float* p = partial + static_cast<size_t>(m) * 2 * F;
    float gate = 0.f, up = 0.f;
    for (int s = 0; s < splits; ++s) {
        gate += p[s * pstride + f];
        up += p[s * pstride + F + f];
    }
    const float act = gate / (1.0f + expf(-gate));
    g[idx] = __float2bfloat16_rn(act * up);
}

// One block per row of logits: greedy token (lowest id on ties, [MASK] excluded) and its
// softmax probability conf = 1 / sum_j exp(l_j - l_max).
__global__ void confidence_kernel(const float* __restrict__ logits, int V, int mask_id, float* __restrict__ conf,
                                  int32_t* __restrict__ tok) {
    __shared__ float red_v[32];
    __shared__ int red_i[32];
    __shared__ float red[32];
    const float* l = logits + static_cast<size_t>(blockIdx.x) * V;
    float best = -INFINITY;
    int besti = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
        const float v = (i == mask_id) ? -INFINITY : l[i];
        if (v > best) { best = v; besti = i; }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
        if (ov > best || (ov == best && oi < besti)) { best = ov; besti = oi; }
    }
    if (lane == 0) { red_v[warp] = best; red_i[warp] = besti; }
    __syncthreads();
    best = red_v[0]; besti = red_i[0];
    for (int w = 1; w < nw; ++w)
        if (red_v[w] > best || (red_v[w] == best && red_i[w] < besti)) { best = red_v[w]; besti = red_i[w]; }
    float sum = 0.f;
    for (int i = threadIdx.x; i < V; i += blockDim.x)
        if (i != mask_id) sum += expf(l[i] - best);
    const float total = block_sum(sum, red);
    if (threadIdx.x == 0) {
        conf[blockIdx.x] = 1.0f / total;
        tok[blockIdx.x] = besti;
    }
}

}  // namespace

cudaError_t launch_embed(const __nv_bfloat16* embed, const int32_t* row_tok, float* h, int M, int d, cudaStream_t st) {
    embed_kernel<<<M, 256, 0, st>>>(embed, row_tok, h, d);
    return cudaGetLastError();
}

cudaError_t launch_rmsnorm(float* h, const float* partial, int splits, size_t pstride, const float* gain,
                           __nv_bfloat16* out, const int32_t* row_map, int rows_out, int d, float eps,
                           cudaStream_t st) {
    rmsnorm_kernel<<<rows_out, 256, 0, st>>>(h, partial, splits, pstride, gain, out, row_map, d, eps);
    return cudaGetLastError();
}

cudaError_t launch_qkv_rope(const QkvRopeArgs& a, cudaStream_t st) {
    qkv_rope_kernel<<<a.M, 256, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_swiglu(const float* partial, int splits, size_t pstride, __nv_bfloat16* g, int M, int F,
                          cudaStream_t st) {
    const size_t n = static_cast<size_t>(M) * F;
    swiglu_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(partial, splits, pstride, g, M, F);
    return cudaGetLastError();
}

cudaError_t launch_confidence(const float* logits, int rows, int V, int mask_id, float* conf, int32_t* tok,
                              cudaStream_t st) {
    confidence_kernel<<<rows, 1024, 0, st>>>(logits, V, mask_id, conf, tok);
    return cudaGetLastError();
}

}  // namespace odb
