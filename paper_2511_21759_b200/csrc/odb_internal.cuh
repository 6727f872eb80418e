// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/odb.h"

#include <atomic>
#include <utility>

namespace odb {

// cudaFuncSetAttribute is a setting of one device: `done` (one word per kernel, kept by the caller) remembers
// for which device indices the kernel already has its dynamic shared-memory limit.  The device is the current
// one, which must be the device of the stream the launch goes to.
template <class Kernel>
cudaError_t set_smem_limit_once(std::atomic<unsigned long long>& done, Kernel kernel, int bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = dev >= 0 && dev < 64 ? 1ull << dev : 0ull;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && bit) done.fetch_or(bit, std::memory_order_release);
    return e;
}

// ---------------------------------------------------------------------------------------
// programmatic dependent launch: every kernel of a forward lets its successor start early
// (launch_dependents at entry) and waits for its predecessor's results (wait) only where it
// first needs them, so prologues, tensor-map fetches and weight prefetches overlap the
// predecessor's tail.  Every such kernel executes pdl_wait() before it exits, which keeps the
// completion order of the chain transitive.
// ---------------------------------------------------------------------------------------

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

bool pdl_enabled();   // ODB_PDL=0 in the environment turns the launch attribute off

// A byte range of the NEXT GEMM's packed weights that a short kernel asks L2 to fetch while it
// runs: HBM would otherwise sit idle between two weight-streaming GEMMs.  Fire and forget.
struct L2Prefetch {
    const void* ptr;
    unsigned long long bytes;
};

#ifdef __CUDACC__
// Block `cta` of `n_ctas` requests its share of the range in 32 KB bulk prefetches (thread 0).
__device__ __forceinline__ void l2_prefetch_slice(const L2Prefetch& pf, int cta, int n_ctas) {
    if (pf.bytes == 0 || threadIdx.x != 0) return;
    constexpr unsigned long long kChunk = 32768;
    const unsigned long long n_chunks = (pf.bytes + kChunk - 1) / kChunk;
    for (unsigned long long c = cta; c < n_chunks; c += n_ctas) {
        const unsigned long long off = c * kChunk;
        const unsigned sz = static_cast<unsigned>((pf.bytes - off < kChunk ? pf.bytes - off : kChunk) & ~15ull);
        if (sz)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(static_cast<const char*>(pf.ptr) + off), "r"(sz)
                         : "memory");
    }
}
#endif

template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                          Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// ---------------------------------------------------------------------------------------
// session-wide device state
// ---------------------------------------------------------------------------------------

constexpr int kMaxBlock = 64;
constexpr int kMaxLoopIters = 64;   // iterations of one device-resident loop (a block needs at most its length)

// Per-sequence control state, resident on the device and mirrored on the host after every
// odb_unmask_accept.  Positions are absolute (prompt position 0 first).
struct SeqState {
    int32_t active;
    int32_t in_fwd;               // took part in the forward last built (refresh or step)
    int32_t P, T;                 // prompt length, current total length (prompt + response)
    int32_t block_idx, s, e;      // current block [s, e)
    int32_t n_masked;             // masked positions left in [s, e)
    int32_t block_iter;           // iterations taken in the current block (0: the refresh's accept comes next)
    // speculative candidates for the next step (Section 4.2): offsets inside the block and the
    // tokens they would be filled with, most confident first
    int32_t n_ranks;
    int32_t rank_off[ODB_MAX_RANKS];
    int32_t rank_tok[ODB_MAX_RANKS];
    // copies of the next step: bit r-1 of copy_mask[c] set <=> copy c fills rank r
    int32_t n_copies;
    int32_t copy_mask[ODB_MAX_COPIES];
    int32_t stage2;               // decoded-share layout (Section 4.2.2) for the next step
    // row table placement of the step last built
    int32_t row0, n_rows;
    int32_t copy_row0[ODB_MAX_COPIES];
    int32_t copy_nrows[ODB_MAX_COPIES];
    // placement of the last refresh's outputs: conf/tok of position p at lm_row0 + (p - lm_s)
    int32_t lm_row0, lm_s, lm_n;
};

// One attention work item: up to 64 query rows that share one key set.
// Keys, in order: cached positions [0, cA) and [cB0, cB1) of sequence `seq`, then the fresh
// rows [f0, f0 + n0) (all visible), then the fresh rows [f1, f1 + n1) of which only those
// flagged kRowDecoded are visible (decoded tokens of copy 0 shared with a speculative copy).
struct QTile {
    int32_t q_row0, nq;
    int32_t seq;
    int32_t cA, cB0, cB1;
    int32_t f0, n0;
    int32_t f1, n1;
};

// A decode-step attention work item: up to 8 slabs of 16 query rows, each slab inside one block copy
// of one sequence, all sharing the sequence's cached keys (positions [0, cA) and [cB0, cB1)) - the
// cached K/V tiles are loaded once for every copy in the item.  Fresh keys: the rows of the copies
// listed in src_*; a slab of copy c sees source copy c (all rows) and, in the decoded-share layout,
// source copy 0 (only rows flagged kRowDecoded).
struct StepTile {
    int32_t seq;
    int32_t cA, cB0, cB1;
    int32_t n_slabs;
    int32_t slab_copy[8], slab_row0[8], slab_n[8];   // copy id, first global row, valid rows (<= 16)
    int32_t n_src;
    int32_t src_copy[ODB_MAX_COPIES], src_row0[ODB_MAX_COPIES], src_n[ODB_MAX_COPIES];
    int32_t stage2;
};

constexpr int kRowDecoded = 1;   // row_flags bit: the row's position is decoded in the committed state

// ---------------------------------------------------------------------------------------
// kernel launchers (each enqueues on `st`; returns cudaError_t of the launch)
// ---------------------------------------------------------------------------------------

struct TmaEncoder;   // wraps the driver's tensor-map encode entry point

// The row scalar of an RMSNorm folded behind a projection, kept as the partial sums of x^2 its producer
// wrote (one per 1024-column slice of the row): scale[m] = 1 / sqrt(sum_t ssq[m * slots + t] / d + eps),
// summed in slot order.  ssq null: scale 1.
struct RowScale {
    const float* ssq = nullptr;
    int slots = 0;
    float inv_d = 0.f, eps = 0.f;
};
constexpr int kNormSliceCols = 1024;   // columns of a row one RMSNorm block handles

#ifdef __CUDACC__
__device__ __forceinline__ float row_scale_of(const RowScale& rs, int m) {
    if (!rs.ssq) return 1.0f;
    const float* p = rs.ssq + static_cast<size_t>(m) * rs.slots;
    float t = 0.f;
    for (int i = 0; i < rs.slots; ++i) t += p[i];
    return 1.0f / sqrtf(t * rs.inv_d + rs.eps);
}
#endif

// Softmax statistics of a slice of one row of logits: running max, sum of exp(l - max), argmax
// (lowest id on ties; [MASK] excluded by the producer).  Merged in a fixed order.
struct ConfPartial {
    float m, s;
    int idx;
};

#ifdef __CUDACC__
__device__ __forceinline__ void conf_merge(float& m, float& s, int& idx, float om, float os, int oi) {
    if (om == -INFINITY) return;                       // the other side saw nothing
    if (m == -INFINITY) { m = om; s = os; idx = oi; return; }
    if (om > m) {
        s = s * expf(m - om) + os;
        m = om;
        idx = oi;
    } else {
        s += os * expf(om - m);
        if (om == m && oi < idx) idx = oi;
    }
}
#endif

// Epilogue of the LM-head projection: instead of logits, the softmax statistics of each 128-feature
// tile per activation row; see EPI_CONF in gemm_tcgen05.cu.  part non-null selects it.
struct ConfEpilogue {
    ConfPartial* part = nullptr;   // [M][n_tiles]
    int mask_id = -1;              // feature excluded from the statistics (a global vocabulary id)
    // tensor-parallel shard of the vocabulary: this launch's tile t is global tile tile0 + t of tiles_total
    // (row stride of `part`), its feature n is vocabulary id 128 * tile0 + n; tiles_total == 0: no shard
    int tile0 = 0, tiles_total = 0;
};

// Tensor-parallel destinations of an epilogue: the same fp32 partial tiles (or confidence statistics) are stored to
// n buffers, one per rank, this rank's own among them (plain stores; the others are peer memory).  n == 0: none.
// When every CTA of the launch has stored its tiles, the last one to arrive advances this rank's sequence counter of
// exchange `kind` and raises this rank's flag of that kind to the new number on every rank (flag words of a rank:
// [kind][source rank]; kind 0 / 1 = the two receive slots of partial sums, 2 = the confidence statistics; a flag
// holds the number of exchanges of that kind its source has completed).  All numbers live on the device, so the
// launches carry no per-call values and can be replayed from a CUDA graph.
constexpr int kTpMaxWorld = 8;
constexpr int kTpKinds = 3;
// words of a rank's flag region: [kTpKinds][kTpMaxWorld] flags, then the arrival counter, then [kTpKinds] sequence counters
constexpr int kTpArriveWord = kTpKinds * kTpMaxWorld;
constexpr int kTpSeqWord = kTpArriveWord + 1;
constexpr int kTpFlagWords = kTpSeqWord + kTpKinds;
struct PeerOut {
    float* partial[kTpMaxWorld] = {};        // each fp32 [splits][M][N], already offset to this rank's block
    ConfPartial* conf[kTpMaxWorld] = {};     // each [M][tiles_total]
    unsigned int* flags[kTpMaxWorld] = {};   // every rank's flag region
    int n = 0, rank = 0, kind = 0;
    int alone = 0;   // measurement: the flags of ALL sources are raised on this rank itself (a rank timed without peers)
};

// The consumer's side: wait until this rank's flags [kind][0 .. world) have reached the number of exchanges of that
// kind this rank has itself completed (every rank performs the same exchanges; the consumer starts after this
// rank's own producer has finished), plus `bias` (test: 1 = a number nobody has signalled).  world == 0: nothing.
struct TpWait {
    const unsigned int* region = nullptr;    // this rank's flag region
    int kind = 0;
    unsigned int bias = 0;
    int world = 0;
    long long limit_cycles = 0;
    int* status = nullptr;
};

#ifdef __CUDACC__
__device__ __forceinline__ void st_release_sys(unsigned int* p, unsigned int v) {
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_sys(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Called by ONE thread of a CTA after the CTA's storing threads have met at a barrier: counts the CTA in and - in
// the last CTA of the launch - raises the flags.  Ordering: the CTA's stores -> CTA barrier -> this thread's
// GPU-scope fence -> arrival (atomic) -> observed by the last arriver -> its system-scope fence -> release store of
// the flag at system scope -> the consumer's acquire load at system scope.  Causality order is transitive across
// the scopes, so a consumer that sees the flag sees every CTA's stores; only the last arriver pays for a
// system-scope fence (one per CTA, 296 of them per launch, measured 6 us per projection).
__device__ __forceinline__ void tp_arrive_and_signal(const PeerOut& po, unsigned int total_ctas) {
    unsigned int* own = po.flags[po.rank];
    __threadfence();
    const unsigned int before = atomicAdd(own + kTpArriveWord, 1u);
    if (before + 1 != total_ctas) return;
    own[kTpArriveWord] = 0;              // the next launch that uses the counter comes after this one in the stream
    const unsigned int seq = atomicAdd(own + kTpSeqWord + po.kind, 1u) + 1u;
    __threadfence_system();              // every CTA's fence happened before its arrival, which this thread has observed
    for (int r = 0; r < po.n; ++r) {
        if (po.alone) st_release_sys(own + po.kind * kTpMaxWorld + r, seq);
        else st_release_sys(po.flags[r] + po.kind * kTpMaxWorld + po.rank, seq);
    }
}
// Called by every thread of a block before it reads what the peers stored: threads 0 .. world-1 each poll one
// source's flag (bounded; on expiry the status word gets ODB_ERR_TIMEOUT and the block carries on with whatever the
// buffers hold), then the block meets.  Sequence numbers only grow; the signed difference survives a wrap.
__device__ __forceinline__ void tp_wait_flags(const TpWait& tw) {
    if (tw.world == 0) return;
    if (static_cast<int>(threadIdx.x) < tw.world) {
        const unsigned int want = *reinterpret_cast<const volatile unsigned int*>(tw.region + kTpSeqWord + tw.kind) + tw.bias;
        const unsigned int* f = tw.region + tw.kind * kTpMaxWorld + threadIdx.x;
        const long long t0 = clock64();
        while (static_cast<int>(ld_acquire_sys(f) - want) < 0) {
            if (clock64() - t0 > tw.limit_cycles) {
                atomicExch(tw.status, ODB_ERR_TIMEOUT);
                break;
            }
            __nanosleep(32);
        }
    }
    __syncthreads();
}
#endif

// Weight-streaming GEMM: partial[s][M][N] (fp32) = x[M][K_s] * w[N][K_s]^T for each K split s.
struct GemmArgs {
    CUtensorMap tmap_w;    // packed bf16 weight tiles [n_tile * k_blocks][128][64], 128B swizzle
    const void* x;         // bf16 [M][K] device
    float* partial;        // fp32 [splits][M][N]
    __nv_bfloat16* act_out; // non-null: gate/up GEMM with the SwiGLU epilogue, writes bf16 [M][N = F]; splits == 1
    ConfEpilogue conf;                  // conf.part non-null: LM head fused with the confidence statistics, splits == 1
    RowScale row_scale;                 // per activation row m: the output is multiplied by scale[m]
                                        // (the 1/rms of an RMSNorm folded behind the projection); needs splits == 1
    PeerOut peers;                      // peers.n > 0: the partial tiles (or statistics) go to these buffers instead
    int M, N, K;
    int splits;
    int* status;           // device status word
};
int gemm_pick_splits(int M, int N, int K);

// Test entry: one block performs the consumers' flag wait (tensor_parallel.cu).
cudaError_t launch_tp_wait(const TpWait& tw, cudaStream_t st);
cudaError_t make_weight_tmap(CUtensorMap* out, const void* w_packed, int N, int K);
// bf16 [rows][cols] row-major; box = 64 columns x box_rows rows, 128-byte swizzle, rows beyond `rows` read as zero
cudaError_t make_rows_tmap(CUtensorMap* out, const void* base, int rows, int cols, int box_rows);
size_t packed_weight_bytes(int N, int K);
size_t packed_gate_up_bytes(int F, int K);
cudaError_t make_gate_up_tmap(CUtensorMap* out, const void* w_packed, int F, int K);
cudaError_t launch_pack_gate_up(const void* src_gate_then_up, void* dst_packed, int F, int K, cudaStream_t st);
cudaError_t launch_pack_weight(const void* src_row_major, void* dst_packed, int N, int K, cudaStream_t st);
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st);
cudaError_t launch_reduce_partials(const float* partial, int splits, size_t stride, float* out, size_t n,
                                   cudaStream_t st);

// read-only streaming kernel over `bytes` of src (a multiple of 16), `grid` blocks of 512 threads
cudaError_t launch_read_stream(const void* src, size_t bytes, unsigned int* sink, int grid, cudaStream_t st);
// bulk-copy ring probe; *streamed = the bytes one launch reads (whole chunks per CTA); `status` is a device word
cudaError_t launch_bulk_read_stream(const void* src, size_t bytes, int grid, int* status, size_t* streamed, cudaStream_t st);
cudaError_t launch_embed(const __nv_bfloat16* embed, const int32_t* row_tok, float* h, int M, int d,
                         cudaStream_t st);
// The part of RMSNorm that is not a row scalar, for rows r = map ? map[i] : i of the residual stream:
// h[r] += sum_s partial[s][r] (if partial; split order), out[i] = bf16(h[r] * gain) is the projection's
// operand, ssq[i][t] = sum of h[r]^2 over the t-th slice of kNormSliceCols columns; the projection's consumer
// multiplies its fp32 output by 1 / sqrt(sum_t ssq / d + eps) (RowScale; the scalar commutes with the matrix
// product).  splits <= 16.
cudaError_t launch_rmsnorm(float* h, const float* partial, int splits, size_t pstride, const float* gain,
                           __nv_bfloat16* out, float* ssq, const int32_t* row_map, int rows_out, int d, L2Prefetch pf,
                           cudaStream_t st, const TpWait& tw = TpWait());
// SwiGLU of a gate/up projection that ran with K splits (few weight tiles: a tensor-parallel shard): partial is fp32
// [splits][M][tiles * 128] in the packed gate/up order (tile t = gate features [64t, 64t+64), then the same up
// features); g[m][f] = bf16(silu(gate) * up) with gate, up = the split sums (split order) times the row scalar.
cudaError_t launch_swiglu_combine(const float* partial, int splits, size_t pstride, const RowScale& scale, __nv_bfloat16* g,
                                  int M, int F, cudaStream_t st);
struct QkvRopeArgs {
    const float* partial; int splits; size_t pstride;      // [splits][M][3d]
    RowScale scale;                                        // scalar of the preceding RMSNorm
    const float2* rope;                                    // [max_seq][hd/2] (cos, sin)
    const int32_t* row_pos; const int32_t* row_seq;
    __nv_bfloat16 *q, *k, *v;                              // [M][d]
    __nv_bfloat16* cache;                                  // NULL: do not write the cache
    int layer, n_layers, H, hd, max_seq, M;
    L2Prefetch pf;
};
cudaError_t launch_qkv_rope(const QkvRopeArgs& a, cudaStream_t st);
cudaError_t launch_confidence_final(const ConfPartial* part, int chunks, int rows, float* conf, int32_t* tok,
                                    cudaStream_t st, const TpWait& tw = TpWait());

// scratch: rows * kConfMaxChunks * 12 bytes of per-chunk (max, sum, argmax) triples
constexpr int kConfMaxChunks = 64;
cudaError_t launch_confidence(const float* logits, int rows, int V, int mask_id, float* conf, int32_t* tok,
                              void* scratch, cudaStream_t st);

struct AttnArgs {
    const QTile* tiles; int n_tiles;
    const __nv_bfloat16 *q, *k, *v;       // fresh rows [M][H*hd]
    const __nv_bfloat16* cache;           // [batch][L][2][H][max_seq][hd]
    const int32_t* row_flags;
    __nv_bfloat16* o;                     // [M][H*hd]
    float* part_o; float* part_ml;        // split workspaces [ks][M][H][hd], [ks][M][H][2]
    int layer, n_layers, H, hd, max_seq, M, ksplit;
    int early = 0;                        // 1: tiles and cache were complete before the launch chain began (decode steps)
    L2Prefetch pf;
};
cudaError_t launch_attention(const AttnArgs& a, cudaStream_t st);
// refresh attention on the tcgen05 tensor cores (head dim 128): a.tiles = work items of up to 128 query rows
// whose keys are the fresh rows [f0, f0 + n0); status = device status word (bounded waits)
cudaError_t launch_attention_tc(const AttnArgs& a, int* status, cudaStream_t st);

// Decode-step attention over StepTiles (copies of a block share the cached K/V loads).
struct StepAttnArgs {
    const StepTile* tiles; int n_tiles;
    const __nv_bfloat16 *q, *k, *v;       // fresh rows [M][H*hd]
    const __nv_bfloat16* cache;
    const int32_t* row_flags;
    __nv_bfloat16* o;
    float* part_o; float* part_ml;        // split workspaces, merged by attention_combine
    int layer, n_layers, H, hd, max_seq, M, ksplit;   // ksplit >= 2: the last split handles the fresh keys
    L2Prefetch pf;
};
cudaError_t launch_step_attention(const StepAttnArgs& a, cudaStream_t st);
// the same work items on the tcgen05 tensor cores (head dim 128): writes the split partials only;
// cache_rows = rows of the K/V cache viewed as [rows][128]
cudaError_t launch_step_attention_tc(const StepAttnArgs& a, size_t cache_rows, int* status, cudaStream_t st);
cudaError_t launch_attention_combine(const float* part_o, const float* part_ml, __nv_bfloat16* o, int M, int H, int hd,
                                     int ksplit, cudaStream_t st);

// ---------------------------------------------------------------------------------------
// Persistent decode-step kernel (step_persistent.cu): ONE cooperative launch runs the whole forward of a
// decode step of up to 128 query rows - every projection, RMSNorm, RoPE, attention and the LM head with its
// confidence statistics - on one CTA per SM.  The k-blocks of every projection are divided evenly over the
// CTAs (fixed assignment, partial tiles reduced in CTA order); a TMA producer warp per CTA keeps a ring of
// shared-memory stages filled with weight tiles and runs ahead of the phase its consumers are in, so HBM keeps
// streaming across the hand-overs between phases, which are grid-wide barriers with a bounded wait.
// ---------------------------------------------------------------------------------------
struct alignas(64) PGemmDesc {   // one projection of the step; an array of these lives in device memory
    CUtensorMap tmap_w;          // packed weight tiles
    CUtensorMap tmap_x;          // its bf16 activation rows [rows][K], box 64 x BN
    const float* gain;           // gain of the RMSNorm that produces its operand (QKV, gate/up, LM head), else null
    int32_t n_tiles, nkb;        // weight tiles of 128 rows, k-blocks of 64
    int32_t conf;                // 1: LM head, tile aligned, epilogue = softmax statistics per vocabulary tile
    int32_t g_use;               // CTAs its units are divided over (all of them unless the projection is tiny: a
                                 // CTA's range is never shorter than a sixth of a tile's k-blocks, so that an
                                 // output tile has at most 8 parts)
    int32_t pad[10];
};
struct StepPersistentArgs {
    const PGemmDesc* gemms;      // [4 * n_layers (qkv, o, gate/up, down per layer) + with_lm]
    int n_layers, M, BN, stages, scratch_bytes;
    int maxp[4];                 // most parts any output tile of the layer's four projections has
    int l2_ahead;                // weight tiles the producer asks L2 for ahead of the one it loads into shared memory
    int d, F, H, hd, vocab, mask_id, with_lm;
    float rms_eps;
    const __nv_bfloat16* embed;
    const int32_t* row_tok; const int32_t* row_pos; const int32_t* row_flags;
    float* h; __nv_bfloat16* a; float* ssq;
    __nv_bfloat16 *q, *k, *v, *o, *g;
    float* partial;
    const float2* rope;
    const __nv_bfloat16* cache; int max_seq;
    const QTile* tiles; int n_qtiles, ksplit;
    float* part_o; float* part_ml;
    ConfPartial* conf_part;
    unsigned int* bars;          // one word per grid barrier, zero when the kernel starts
    int n_bars;
    int* status;
    unsigned long long* timing;  // measurement only (null: off): [cta][barrier][arrived, passed] global timer in ns
};
// bytes of the PGemmDesc table and of the barrier words for a model of n_layers layers
size_t step_persistent_table_bytes(int n_layers);
size_t step_persistent_barrier_bytes(int n_layers);
// whether this step can run as the persistent kernel (shape limits, cooperative launch available on the device)
bool step_persistent_supported(int M, int d, int F, int hd);
// rows per MMA tile and ring depth for M rows; fills a.BN, a.stages, a.scratch_bytes, a.n_bars
cudaError_t step_persistent_configure(StepPersistentArgs& a);
// CTAs of the launch (the SM count of the current device; 0: no cooperative launch there)
int step_persistent_grid();
void step_persistent_fill_desc(PGemmDesc& d, const CUtensorMap& tmap_w, const CUtensorMap& tmap_x, const float* gain, int n_tiles,
                               int nkb, int conf, int grid);
// most parts an output tile of this projection has under the kernel's split
int step_persistent_max_parts(const PGemmDesc& d);
// zeroes the barrier words and launches the kernel (cooperative, one CTA per SM) on st
cudaError_t launch_step_persistent(const StepPersistentArgs& a, cudaStream_t st);

// control kernels (control.cu)
struct ControlBuffers {
    SeqState* state;          // [batch]
    int32_t* x;               // [batch][max_seq] token ids
    int32_t max_seq;
    int32_t* row_tok; int32_t* row_pos; int32_t* row_seq; int32_t* row_copy; int32_t* row_flags;
    int32_t* lm_rows;         // rows whose logits are needed
    QTile* tiles;
    QTile* big_tiles;         // refresh: the same rows cut into work items of up to 128 query rows
    StepTile* step_tiles;     // decode steps with more than one copy
    const float* conf; const int32_t* tok;   // outputs of the last forward, per logit row
    const float* noise;       // [batch][kMaxLoopIters][kMaxBlock] uniform deviates of the stochastic reverse step
    odb_result* results;      // [batch] device copy
    // pinned host memory the accept kernel writes its outcome to (state, results, the status word): the host
    // reads them after synchronising the stream, no copy is enqueued
    SeqState* host_state; odb_result* host_results; int* host_status;
    const int* status;        // device status word
};
// block_index[seq] < 0: the sequence takes no part in this refresh
cudaError_t launch_build_refresh_rows(const ControlBuffers& c, int batch, const int32_t* block_index, int block_len,
                                      cudaStream_t st);
cudaError_t launch_build_step_rows(const ControlBuffers& c, int batch, int mask_id, cudaStream_t st);

// Number of StepTiles of a sequence's step: copies packed in order into items of <= 8 slabs of 16 rows.
__host__ __device__ inline int step_tiles_of_counts(int n_copies, int rows_copy0, int rows_other) {
    int tiles = 0, slabs = 0;
    for (int cp = 0; cp < n_copies; ++cp) {
        const int need = ((cp == 0 ? rows_copy0 : rows_other) + 15) / 16;
        if (slabs == 0 || slabs + need > 8) { ++tiles; slabs = 0; }
        slabs += need;
    }
    return tiles;
}

// Shape of the row table of the next step, summed over the sequences that take part in it: everything a
// step's launch configuration depends on.  Evaluated by the host before it enqueues a step and by the
// device-resident loop, which goes on only while the shape it was recorded for still holds.
struct StepShape {
    int32_t rows, tiles, step_tiles, multi;
};
__host__ __device__ inline void step_shape_add(StepShape& sh, const SeqState& st) {
    if (!st.active || st.n_masked <= 0) return;
    const int B = st.e - st.s;
    sh.rows += st.stage2 ? B + (st.n_copies - 1) * st.n_masked : st.n_copies * B;
    sh.tiles += st.n_copies;
    if (st.n_copies > 1) sh.multi = 1;
    sh.step_tiles += step_tiles_of_counts(st.n_copies, B, st.stage2 ? st.n_masked : B);
}
// dry: model without LM head; commits nothing, only lays out the next step
cudaError_t launch_accept(const ControlBuffers& c, int batch, const odb_decode_params& p, int after_refresh,
                          int mask_id, int eos_id, int dry, cudaStream_t st);

// Control words of the device-resident block loop (a CUDA graph whose body, one step and its accept, sits in a
// WHILE node).  The accept kernel of the body appends the per-sequence results of iteration i to
// host_log[i][batch], and its last block decides whether the body runs again: iterations < max_iters, a masked
// position left, no device error, and the next step's row table has the shape the body was recorded for.
struct LoopControl {
    cudaGraphConditionalHandle handle;
    int32_t* iter;          // device: iterations completed since the loop was launched
    int32_t* arrivals;      // device: accept blocks that have finished the current iteration
    const int32_t* max_iters;   // device: iteration limit of this launch (hard limit kMaxLoopIters)
    StepShape shape;
    odb_result* host_log;   // pinned host memory [kMaxLoopIters][batch]
    int32_t* host_iters;    // pinned host memory: copy of *iter
};
cudaError_t launch_accept_loop(const ControlBuffers& c, int batch, const odb_decode_params& p, int mask_id, int eos_id,
                               int dry, const LoopControl& lc, cudaStream_t st);

// ---------------------------------------------------------------------------------------
// Bounded mbarrier wait shared by every kernel that waits on one (GEMM, tensor-core attention): no wait on
// the device spins forever.  Returns false if the CTA has been aborted by another of its waits or the limit
// expired; on expiry the CTA's abort word is set and ODB_ERR_TIMEOUT recorded in the session's status word,
// the kernel then finishes normally (its roles stop, TMEM is released) and the host reads the status.
// ---------------------------------------------------------------------------------------
constexpr long long kWaitLimitCycles = 4000000000ll;   // ~2 s at the boost clock

__device__ __forceinline__ bool mbar_try_wait_parity(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(bar))), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* cta_abort, int* status,
                                                  long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait_parity(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait_parity(bar, parity)) {
        if (*cta_abort) return false;
        if (clock64() - t0 > limit_cycles) {
            *cta_abort = 1;
            atomicExch(status, ODB_ERR_TIMEOUT);
            return false;
        }
    }
    return true;
}
// Test entry: one CTA waits, with the given limit, on an mbarrier that nothing ever arrives at.
cudaError_t launch_expire_wait(long long limit_cycles, int* status, cudaStream_t st);

}  // namespace odb
