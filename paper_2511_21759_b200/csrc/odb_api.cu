// C ABI of the library: handles, argument validation, workspace carve-up and the host-side
// orchestration of one forward (refresh prefill or block decode step) over the kernels.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <string>
#include <vector>

#include "odb_internal.cuh"

using namespace odb;

namespace {

thread_local std::string g_cuda_error;

int32_t cuda_fail(cudaError_t e) {
    g_cuda_error = cudaGetErrorString(e);
    return ODB_ERR_CUDA;
}

#define ODB_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) return cuda_fail(e__);   \
    } while (0)

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

int32_t check_config(const odb_config* c) {
    if (!c) return ODB_ERR_ARG;
    if (c->n_layers < 1 || c->d_model < 16 || c->n_heads < 1 || c->vocab < 2) return ODB_ERR_SHAPE;
    if (c->head_dim != 64 && c->head_dim != 128) return ODB_ERR_SHAPE;
    if (c->d_model != c->n_heads * c->head_dim) return ODB_ERR_SHAPE;
    if (c->d_model % 16 || c->d_ffn % 16 || c->d_ffn < 16) return ODB_ERR_SHAPE;
    if (c->max_batch < 1 || c->max_batch > 64 || c->max_seq < 2) return ODB_ERR_SHAPE;
    if (c->max_block < 1 || c->max_block > kMaxBlock) return ODB_ERR_SHAPE;
    if (c->max_copies != 1 && c->max_copies != 4 && c->max_copies != 8) return ODB_ERR_SHAPE;
    if (c->mask_id < 0 || c->mask_id >= c->vocab || c->eos_id < 0 || c->eos_id >= c->vocab) return ODB_ERR_ARG;
    if (c->tp_world > 1) {
        const int R = c->tp_world;
        if (R != 2 && R != 4 && R != 8) return ODB_ERR_SHAPE;
        if (c->tp_rank < 0 || c->tp_rank >= R) return ODB_ERR_ARG;
        if (c->n_heads % R || c->d_ffn % (64 * R)) return ODB_ERR_SHAPE;
    } else if (c->tp_world < 0 || c->tp_rank != 0) {
        return ODB_ERR_ARG;
    }
    return ODB_OK;
}

// tensor-parallel shard sizes (the whole model when tp_world <= 1)
int tp_ranks(const odb_config& c) { return c.tp_world > 1 ? c.tp_world : 1; }
int heads_local(const odb_config& c) { return c.n_heads / tp_ranks(c); }
int ffn_local(const odb_config& c) { return c.d_ffn / tp_ranks(c); }
int vocab_tiles(const odb_config& c) { return (c.vocab + 127) / 128; }
void vocab_shard(const odb_config& c, int rank, int* tile0, int* rows) {
    const int T = vocab_tiles(c), R = tp_ranks(c), per = (T + R - 1) / R;
    int t0 = rank * per, t1 = t0 + per;
    if (t0 > T) t0 = T;
    if (t1 > T) t1 = T;
    const int first = t0 * 128;
    int last = t1 * 128;
    if (last > c.vocab) last = c.vocab;
    *tile0 = t0;
    *rows = last > first ? last - first : 0;
}

// Carve-up of the caller's workspace.  Offsets only; shared by odb_workspace_bytes and
// odb_session_create so that both always agree.
struct Layout {
    size_t rows, lm_chunk, tiles, partial_rows, attn_rows;
    size_t rope, state, results, status, loop, x, row_tok, row_pos, row_seq, row_copy, row_flags, lm_rows, tile_buf, big_tile_buf, step_tile_buf;
    size_t h, a, inv, q, k, v, o, g, partial, logits, conf, tok, conf_part, part_o, part_ml, ptable, pbars, noise;
    size_t tp_recv, tp_recv_slot, tp_flags, conf_part_bytes;   // tensor parallelism: two receive slots for partial sums, the flag words
    size_t total;
};

Layout make_layout(const odb_config& c) {
    Layout L{};
    const size_t step_rows = static_cast<size_t>(c.max_copies) * c.max_block;
    const size_t per_seq = step_rows > static_cast<size_t>(c.max_seq) ? step_rows : static_cast<size_t>(c.max_seq);
    L.rows = per_seq * c.max_batch;
    L.lm_chunk = L.rows < 2048 ? L.rows : 2048;
    const size_t refresh_tiles = static_cast<size_t>(c.max_batch) * ((c.max_seq + 63) / 64);
    const size_t step_tiles = static_cast<size_t>(c.max_batch) * c.max_copies;
    L.tiles = refresh_tiles > step_tiles ? refresh_tiles : step_tiles;
    L.partial_rows = L.rows > 4096 ? L.rows : 4096;
    L.attn_rows = L.rows > 2048 ? L.rows : 2048;
    const size_t d = c.d_model, F = ffn_local(c);
    const size_t nmax = 3 * d > 2 * F ? 3 * d : 2 * F;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.rope = take(static_cast<size_t>(c.max_seq) * (c.head_dim / 2) * sizeof(float2));
    L.state = take(sizeof(SeqState) * c.max_batch);
    L.results = take(sizeof(odb_result) * c.max_batch);
    L.status = take(sizeof(int));
    L.loop = take(4 * sizeof(int32_t));   // device-resident loop: iterations done, accept blocks arrived, iteration limit
    L.x = take(sizeof(int32_t) * c.max_batch * c.max_seq);
    L.row_tok = take(4 * L.rows);
    L.row_pos = take(4 * L.rows);
    L.row_seq = take(4 * L.rows);
    L.row_copy = take(4 * L.rows);
    L.row_flags = take(4 * L.rows);
    L.lm_rows = take(4 * L.rows);
    L.tile_buf = take(sizeof(QTile) * L.tiles);
    L.big_tile_buf = take(sizeof(QTile) * static_cast<size_t>(c.max_batch) * ((c.max_seq + 127) / 128));
    L.step_tile_buf = take(sizeof(StepTile) * static_cast<size_t>(c.max_batch) * c.max_copies);
    L.h = take(4 * L.rows * d);
    L.a = take(2 * L.rows * d);
    L.inv = take(4 * L.rows * ((d + kNormSliceCols - 1) / kNormSliceCols));   // sum-of-squares slices of the current RMSNorm
    L.q = take(2 * L.rows * d);
    L.k = take(2 * L.rows * d);
    L.v = take(2 * L.rows * d);
    L.o = take(2 * L.rows * d);
    L.g = take(2 * L.rows * F);
    L.partial = take(4 * L.partial_rows * nmax);
    L.logits = take(c.with_lm_head ? 4 * L.lm_chunk * c.vocab : 256);
    L.conf = take(4 * L.rows);
    L.tok = take(4 * L.rows);
    {
        const size_t lm_tiles = (static_cast<size_t>(c.vocab) + 127) / 128;
        L.conf_part_bytes = 12 * L.lm_chunk * (lm_tiles > static_cast<size_t>(kConfMaxChunks) ? lm_tiles : kConfMaxChunks);
        L.conf_part = take(L.conf_part_bytes);
    }
    L.part_o = take(4 * L.attn_rows * d);
    L.part_ml = take(4 * L.attn_rows * c.n_heads * 2);
    // persistent decode-step kernel: one table of projections per row-tile size (32, 64, 128), the grid barrier words
    L.ptable = take(3 * align_up(step_persistent_table_bytes(c.n_layers)));
    L.pbars = take(step_persistent_barrier_bytes(c.n_layers));
    L.noise = take(sizeof(float) * c.max_batch * kMaxLoopIters * kMaxBlock);   // deviates of the stochastic reverse step
    if (c.tp_world > 1) {
        // a slot holds the [rank][split][rows][d_model] fp32 partials of one O or down projection: up to 16 partials
        // of a decode step, fewer (whatever fits) of a refresh
        const size_t all_ranks = 4 * static_cast<size_t>(c.tp_world) * L.rows * d;   // one partial per rank of the largest forward
        L.tp_recv_slot = align_up(4 * L.partial_rows * nmax > all_ranks ? 4 * L.partial_rows * nmax : all_ranks);
        L.tp_recv = take(2 * L.tp_recv_slot);
        L.tp_flags = take(sizeof(unsigned int) * kTpFlagWords);   // flags, this rank's arrival and sequence counters
    }
    L.total = off;
    return L;
}

}  // namespace

struct odb_model {
    odb_config cfg;
    const __nv_bfloat16* embed;
    const float* final_norm;
    std::vector<const float*> norm1, norm2;
    std::vector<CUtensorMap> tm_qkv, tm_o, tm_gu, tm_d;
    CUtensorMap tm_lm;
    std::vector<const void*> p_qkv, p_o, p_gu;   // packed weight buffers (for L2 prefetch hints)
    const void* p_lm;
};

struct odb_session {
    odb_model* m;
    cudaStream_t st;
    uint8_t* ws;
    __nv_bfloat16* kv;
    Layout L;
    ControlBuffers cb;
    std::vector<SeqState> mirror;
    SeqState* pinned_state;
    odb_result* pinned_results;
    int* pinned_status;
    int phase;            // 0 idle, 1 refresh enqueued, 2 accepted, 3 step enqueued
    int last_rows, last_lm_rows;
    bool dump_logits;     // test mode: the LM head writes fp32 logits (odb_debug_read 0) instead of fusing the reduction
    // launch accounting: kernels launched per kind since the last read; with profiling on, a CUDA
    // event pair brackets every launch so that per-kind device time can be summed afterwards
    long long launches[ODB_PROFILE_KINDS];
    bool profiling;
    std::vector<cudaEvent_t> ev;        // pairs (start, stop)
    std::vector<int> ev_kind;
    size_t ev_used;
    // device-resident block loop: one instantiated graph per step shape and parameter set, recorded on a
    // stream of the session's own (the caller's stream may be the default stream, which cannot record)
    struct ResidentGraph {
        StepShape shape;
        odb_decode_params p;
        bool dump_logits;
        cudaGraph_t graph;
        cudaGraphExec_t exec;
        long long launches[ODB_PROFILE_KINDS];   // kernels of one pass of the loop body
    };
    std::vector<ResidentGraph> resident;
    cudaStream_t record_st;
    odb_result* pinned_log;   // [kMaxLoopIters][max_batch]
    int32_t* pinned_iters;    // [0] iterations run (written by the device); [1..3] the loop words of the next launch
    int pmaxp[4];             // persistent step kernel: most parts per output tile of the four projections of a layer
    bool persistent_off;      // the model is beyond the persistent step kernel's limits: steps run as separate kernels
    bool ptable_built[3];     // persistent step kernel: projection table for 32 / 64 / 128 rows per tile is on the device
    // tensor parallelism (model with tp_world > 1)
    struct Tp {
        bool attached = false;
        float* recv[kTpMaxWorld] = {};          // every rank's receive region (two slots), own at index rank
        ConfPartial* conf[kTpMaxWorld] = {};    // every rank's confidence-statistics buffer
        unsigned int* flags[kTpMaxWorld] = {};  // every rank's flag words
        bool alone = false;                     // measurement: all sources' flags are raised on this rank itself
        int seg_first = -1, seg_last = -1;      // test facility: segments of a forward to launch (-1: all)
        long long wait_limit = kWaitLimitCycles;
    } tp;
    template <class T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

extern "C" {

const char* odb_status_string(int32_t s) {
    switch (s) {
        case ODB_OK: return "ok";
        case ODB_ERR_ARG: return "invalid argument";
        case ODB_ERR_SHAPE: return "unsupported shape";
        case ODB_ERR_WORKSPACE: return "buffer too small";
        case ODB_ERR_STATE: return "call not valid in this state";
        case ODB_ERR_CUDA: return "CUDA error";
        case ODB_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

const char* odb_last_cuda_error(void) { return g_cuda_error.c_str(); }

size_t odb_packed_weight_bytes(int32_t N, int32_t K) {
    if (N < 1 || K < 8 || K % 8) return 0;
    return packed_weight_bytes(N, K);
}

int32_t odb_pack_weight(const void* src, void* dst, int32_t N, int32_t K, void* stream) {
    if (!src || !dst) return ODB_ERR_ARG;
    if (N < 1 || K < 8 || K % 8) return ODB_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) return ODB_ERR_ARG;
    ODB_CUDA(launch_pack_weight(src, dst, N, K, static_cast<cudaStream_t>(stream)));
    return ODB_OK;
}

size_t odb_packed_gate_up_bytes(int32_t F, int32_t K) {
    if (F < 1 || K < 8 || K % 8) return 0;
    return packed_gate_up_bytes(F, K);
}

int32_t odb_pack_gate_up(const void* src, void* dst, int32_t F, int32_t K, void* stream) {
    if (!src || !dst) return ODB_ERR_ARG;
    if (F < 1 || K < 8 || K % 8) return ODB_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) return ODB_ERR_ARG;
    ODB_CUDA(launch_pack_gate_up(src, dst, F, K, static_cast<cudaStream_t>(stream)));
    return ODB_OK;
}

int32_t odb_model_create(const odb_config* cfg, const odb_weights* w, odb_model** out) {
    int32_t rc = check_config(cfg);
    if (rc != ODB_OK) return rc;
    if (!w || !out || !w->embed || !w->final_norm || !w->norm1 || !w->norm2 || !w->wqkv || !w->wo || !w->wgu || !w->wd)
        return ODB_ERR_ARG;
    if ((cfg->with_lm_head != 0) != (w->lm_head != nullptr)) return ODB_ERR_ARG;
    odb_model* m = new (std::nothrow) odb_model();
    if (!m) return ODB_ERR_ARG;
    m->cfg = *cfg;
    m->embed = static_cast<const __nv_bfloat16*>(w->embed);
    m->final_norm = w->final_norm;
    m->p_lm = w->lm_head;
    const int d = cfg->d_model, F = ffn_local(*cfg), da = heads_local(*cfg) * cfg->head_dim, nl = cfg->n_layers;
    m->tm_qkv.resize(nl); m->tm_o.resize(nl); m->tm_gu.resize(nl); m->tm_d.resize(nl);
    cudaError_t e = cudaSuccess;
    for (int l = 0; l < nl && e == cudaSuccess; ++l) {
        if (!w->norm1[l] || !w->norm2[l] || !w->wqkv[l] || !w->wo[l] || !w->wgu[l] || !w->wd[l]) {
            delete m;
            return ODB_ERR_ARG;
        }
        m->norm1.push_back(w->norm1[l]);
        m->norm2.push_back(w->norm2[l]);
        m->p_qkv.push_back(w->wqkv[l]);
        m->p_o.push_back(w->wo[l]);
        m->p_gu.push_back(w->wgu[l]);
        e = make_weight_tmap(&m->tm_qkv[l], w->wqkv[l], 3 * da, d);
        if (e == cudaSuccess) e = make_weight_tmap(&m->tm_o[l], w->wo[l], d, da);
        if (e == cudaSuccess) e = make_gate_up_tmap(&m->tm_gu[l], w->wgu[l], F, d);
        if (e == cudaSuccess) e = make_weight_tmap(&m->tm_d[l], w->wd[l], d, F);
    }
    if (e == cudaSuccess && cfg->with_lm_head) {
        int tile0 = 0, rows = cfg->vocab;
        vocab_shard(*cfg, cfg->tp_rank, &tile0, &rows);
        if (rows < 1) {   // more ranks than vocabulary tiles
            delete m;
            return ODB_ERR_SHAPE;
        }
        e = make_weight_tmap(&m->tm_lm, w->lm_head, rows, d);
    }
    if (e != cudaSuccess) {
        delete m;
        return cuda_fail(e);
    }
    *out = m;
    return ODB_OK;
}

int32_t odb_model_destroy(odb_model* m) {
    delete m;
    return ODB_OK;
}

size_t odb_kv_bytes(const odb_config* c) {
    if (check_config(c) != ODB_OK) return 0;
    return static_cast<size_t>(c->max_batch) * c->n_layers * 2 * heads_local(*c) * c->max_seq * c->head_dim * 2;
}

size_t odb_workspace_bytes(const odb_config* c) {
    if (check_config(c) != ODB_OK) return 0;
    return make_layout(*c).total;
}

int32_t odb_session_create(odb_model* m, void* kv, size_t kv_bytes, void* workspace, size_t ws_bytes, void* stream,
                           odb_session** out) {
    if (!m || !kv || !workspace || !out) return ODB_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(kv) | reinterpret_cast<uintptr_t>(workspace)) & 255) return ODB_ERR_ARG;
    const odb_config& c = m->cfg;
    const Layout L = make_layout(c);
    if (kv_bytes < odb_kv_bytes(&c) || ws_bytes < L.total) return ODB_ERR_WORKSPACE;
    odb_session* s = new (std::nothrow) odb_session();
    if (!s) return ODB_ERR_ARG;
    s->m = m;
    s->st = static_cast<cudaStream_t>(stream);
    s->ws = static_cast<uint8_t*>(workspace);
    s->kv = static_cast<__nv_bfloat16*>(kv);
    s->L = L;
    s->phase = 0;
    s->last_rows = s->last_lm_rows = 0;
    s->dump_logits = false;
    memset(s->launches, 0, sizeof(s->launches));
    s->profiling = false;
    s->ev_used = 0;
    s->mirror.assign(c.max_batch, SeqState{});
    s->pinned_state = nullptr;
    s->pinned_results = nullptr;
    s->pinned_status = nullptr;
    s->record_st = nullptr;
    s->pinned_log = nullptr;
    s->pinned_iters = nullptr;
    s->ptable_built[0] = s->ptable_built[1] = s->ptable_built[2] = false;
    s->persistent_off = c.tp_world > 1;
    cudaError_t e = cudaMallocHost(&s->pinned_state, sizeof(SeqState) * c.max_batch);
    if (e == cudaSuccess) e = cudaMallocHost(&s->pinned_log, sizeof(odb_result) * kMaxLoopIters * c.max_batch);
    if (e == cudaSuccess) e = cudaMallocHost(&s->pinned_iters, 4 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s->record_st, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaMallocHost(&s->pinned_results, sizeof(odb_result) * c.max_batch);
    if (e == cudaSuccess) e = cudaMallocHost(&s->pinned_status, sizeof(int));
    // RoPE table: angle(pos, i) = pos * theta^(-2i/hd), evaluated in double, stored as fp32 (cos, sin)
    std::vector<float2> rope(static_cast<size_t>(c.max_seq) * (c.head_dim / 2));
    for (int i = 0; i < c.head_dim / 2; ++i) {
        const double inv = pow(static_cast<double>(c.rope_theta), -2.0 * i / c.head_dim);
        for (int p = 0; p < c.max_seq; ++p) {
            const double ang = p * inv;
            rope[static_cast<size_t>(p) * (c.head_dim / 2) + i] = make_float2(static_cast<float>(cos(ang)),
                                                                              static_cast<float>(sin(ang)));
        }
    }
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(s->ws + L.rope, rope.data(), rope.size() * sizeof(float2), cudaMemcpyHostToDevice, s->st);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->ws + L.state, 0, L.x - L.state, s->st);   // state, results, status
    // The tensor-core attention loads whole 64-row boxes: cache rows that are not keys of a work item are masked
    // in its softmax but still enter the P V product with weight zero, so they must hold finite values; the
    // q / k / v and output rows past a forward's last row are never read (the tensor maps end at that row).
    if (e == cudaSuccess) e = cudaMemsetAsync(kv, 0, odb_kv_bytes(&c), s->st);
    if (e == cudaSuccess && c.tp_world > 1)
        e = cudaMemsetAsync(s->ws + L.tp_flags, 0, sizeof(unsigned int) * kTpFlagWords, s->st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->st);
    if (e != cudaSuccess) {
        odb_session_destroy(s);
        return cuda_fail(e);
    }
    ControlBuffers& cb = s->cb;
    cb.state = s->at<SeqState>(L.state);
    cb.x = s->at<int32_t>(L.x);
    cb.max_seq = c.max_seq;
    cb.row_tok = s->at<int32_t>(L.row_tok);
    cb.row_pos = s->at<int32_t>(L.row_pos);
    cb.row_seq = s->at<int32_t>(L.row_seq);
    cb.row_copy = s->at<int32_t>(L.row_copy);
    cb.row_flags = s->at<int32_t>(L.row_flags);
    cb.lm_rows = s->at<int32_t>(L.lm_rows);
    cb.tiles = s->at<QTile>(L.tile_buf);
    cb.big_tiles = s->at<QTile>(L.big_tile_buf);
    cb.host_state = s->pinned_state; cb.host_results = s->pinned_results; cb.host_status = s->pinned_status;
    cb.status = s->at<int>(L.status);
    cb.step_tiles = s->at<StepTile>(L.step_tile_buf);
    cb.conf = s->at<float>(L.conf);
    cb.tok = s->at<int32_t>(L.tok);
    cb.results = s->at<odb_result>(L.results);
    cb.noise = s->at<float>(L.noise);
    *out = s;
    return ODB_OK;
}

int32_t odb_session_destroy(odb_session* s) {
    if (!s) return ODB_OK;
    if (s->pinned_state) cudaFreeHost(s->pinned_state);
    if (s->pinned_results) cudaFreeHost(s->pinned_results);
    if (s->pinned_status) cudaFreeHost(s->pinned_status);
    if (s->pinned_log) cudaFreeHost(s->pinned_log);
    if (s->pinned_iters) cudaFreeHost(s->pinned_iters);
    for (auto& g : s->resident) {
        if (g.exec) cudaGraphExecDestroy(g.exec);
        if (g.graph) cudaGraphDestroy(g.graph);
    }
    if (s->record_st) cudaStreamDestroy(s->record_st);
    for (cudaEvent_t e : s->ev) cudaEventDestroy(e);
    delete s;
    return ODB_OK;
}

static int32_t push_state(odb_session* s, int seq) {
    ODB_CUDA(cudaMemcpyAsync(s->cb.state + seq, &s->mirror[seq], sizeof(SeqState), cudaMemcpyHostToDevice, s->st));
    ODB_CUDA(cudaStreamSynchronize(s->st));
    return ODB_OK;
}

int32_t odb_session_set_sequence(odb_session* s, int32_t seq, const int32_t* ids, int32_t prompt_len, int32_t gen_len) {
    if (!s || !ids) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (seq < 0 || seq >= c.max_batch || prompt_len < 0 || gen_len < 1) return ODB_ERR_ARG;
    if (prompt_len + gen_len > c.max_seq) return ODB_ERR_SHAPE;
    for (int i = 0; i < prompt_len + gen_len; ++i)
        if (ids[i] < 0 || ids[i] >= c.vocab) return ODB_ERR_ARG;
    ODB_CUDA(cudaMemcpyAsync(s->cb.x + static_cast<size_t>(seq) * c.max_seq, ids, sizeof(int32_t) * (prompt_len + gen_len),
                             cudaMemcpyHostToDevice, s->st));
    SeqState st{};
    st.active = 1;
    st.P = prompt_len;
    st.T = prompt_len + gen_len;
    st.n_copies = 1;
    s->mirror[seq] = st;
    s->phase = 0;
    return push_state(s, seq);
}

int32_t odb_session_set_gen_len(odb_session* s, int32_t seq, int32_t new_gen_len) {
    if (!s) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (seq < 0 || seq >= c.max_batch) return ODB_ERR_ARG;
    if (s->phase != 1) return ODB_ERR_STATE;      // only between a refresh and its accept
    ODB_CUDA(cudaStreamSynchronize(s->st));
    // the refresh's row-table kernel has set the block; fetch it
    ODB_CUDA(cudaMemcpy(&s->mirror[seq], s->cb.state + seq, sizeof(SeqState), cudaMemcpyDeviceToHost));
    SeqState& st = s->mirror[seq];
    if (!st.active) return ODB_ERR_STATE;
    if (new_gen_len > st.T - st.P) return ODB_ERR_ARG;                 // never grows
    if (st.P + new_gen_len <= st.s) return ODB_ERR_ARG;                // keeps a position of the block
    st.T = st.P + new_gen_len;
    if (st.e > st.T) st.e = st.T;
    return push_state(s, seq);
}

int32_t odb_session_get_tokens(odb_session* s, int32_t seq, int32_t* ids, int32_t cap, int32_t* len) {
    if (!s || !ids || !len) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (seq < 0 || seq >= c.max_batch) return ODB_ERR_ARG;
    ODB_CUDA(cudaStreamSynchronize(s->st));
    ODB_CUDA(cudaMemcpy(&s->mirror[seq], s->cb.state + seq, sizeof(SeqState), cudaMemcpyDeviceToHost));
    const int T = s->mirror[seq].T;
    if (cap < T) return ODB_ERR_WORKSPACE;
    ODB_CUDA(cudaMemcpy(ids, s->cb.x + static_cast<size_t>(seq) * c.max_seq, sizeof(int32_t) * T, cudaMemcpyDeviceToHost));
    *len = T;
    return ODB_OK;
}

int32_t odb_session_set_sampling_noise(odb_session* s, int32_t seq, const float* u, int32_t n_iters, int32_t block_len) {
    if (!s || !u) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (seq < 0 || seq >= c.max_batch || n_iters < 1 || n_iters > kMaxLoopIters) return ODB_ERR_ARG;
    if (block_len < 1 || block_len > c.max_block) return ODB_ERR_SHAPE;
    float* dst = s->at<float>(s->L.noise) + static_cast<size_t>(seq) * kMaxLoopIters * kMaxBlock;
    ODB_CUDA(cudaMemcpy2DAsync(dst, sizeof(float) * kMaxBlock, u, sizeof(float) * block_len, sizeof(float) * block_len, n_iters,
                               cudaMemcpyHostToDevice, s->st));
    ODB_CUDA(cudaStreamSynchronize(s->st));
    return ODB_OK;
}

int32_t odb_session_set_active(odb_session* s, int32_t seq, int32_t active) {
    if (!s) return ODB_ERR_ARG;
    if (seq < 0 || seq >= s->m->cfg.max_batch) return ODB_ERR_ARG;
    ODB_CUDA(cudaStreamSynchronize(s->st));
    ODB_CUDA(cudaMemcpy(&s->mirror[seq], s->cb.state + seq, sizeof(SeqState), cudaMemcpyDeviceToHost));
    s->mirror[seq].active = active ? 1 : 0;
    return push_state(s, seq);
}

int32_t odb_session_status(odb_session* s) {
    if (!s) return ODB_ERR_ARG;
    int* dev = s->at<int>(s->L.status);
    ODB_CUDA(cudaMemcpyAsync(s->pinned_status, dev, sizeof(int), cudaMemcpyDeviceToHost, s->st));
    ODB_CUDA(cudaMemsetAsync(dev, 0, sizeof(int), s->st));
    ODB_CUDA(cudaStreamSynchronize(s->st));
    return *s->pinned_status;
}

}  // extern "C"

namespace {

// Brackets one kernel launch: counts it and, when profiling, records an event pair around it.
struct LaunchScope {
    odb_session* s;
    bool timed;
    size_t slot;
    LaunchScope(odb_session* s_, int kind) : s(s_), timed(false), slot(0) {
        ++s->launches[kind];
        if (!s->profiling) return;
        if (s->ev_used + 2 > s->ev.size()) {
            cudaEvent_t a = nullptr, b = nullptr;
            if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
            s->ev.push_back(a);
            s->ev.push_back(b);
            s->ev_kind.push_back(kind);
        }
        slot = s->ev_used;
        s->ev_kind[slot / 2] = kind;
        s->ev_used += 2;
        timed = cudaEventRecord(s->ev[slot], s->st) == cudaSuccess;
    }
    ~LaunchScope() {
        if (timed) cudaEventRecord(s->ev[slot + 1], s->st);
    }
};

int bn_index(int M) { return M <= 32 ? 0 : M <= 64 ? 1 : 2; }

// Whether a decode step of M rows runs as the persistent kernel (one cooperative launch for the whole forward).
bool use_persistent(const odb_session* s, int M) {
    const odb_config& c = s->m->cfg;
    return !s->persistent_off && step_persistent_supported(M, c.d_model, c.d_ffn, c.head_dim);
}

// The persistent kernel reads its projections (weight and operand tensor maps, split) from a table in the
// workspace; built on first use per row-tile size, outside any stream capture (it is a synchronous copy).
int32_t ensure_ptable(odb_session* s, int M) {
    const int bi = bn_index(M);
    if (s->ptable_built[bi]) return ODB_OK;
    const odb_model* m = s->m;
    const odb_config& c = m->cfg;
    const Layout& L = s->L;
    const int BN = 32 << bi, d = c.d_model, F = c.d_ffn, grid = step_persistent_grid();
    const int rows_cap = static_cast<int>(L.rows);
    CUtensorMap tx_a, tx_o, tx_g;
    ODB_CUDA(make_rows_tmap(&tx_a, s->ws + L.a, rows_cap, d, BN));
    ODB_CUDA(make_rows_tmap(&tx_o, s->ws + L.o, rows_cap, d, BN));
    ODB_CUDA(make_rows_tmap(&tx_g, s->ws + L.g, rows_cap, F, BN));
    std::vector<PGemmDesc> t(4 * c.n_layers + 1);
    const int kb_d = (d + 63) / 64, kb_F = (F + 63) / 64;
    for (int l = 0; l < c.n_layers; ++l) {
        step_persistent_fill_desc(t[4 * l + 0], m->tm_qkv[l], tx_a, m->norm1[l], (3 * d + 127) / 128, kb_d, 0, grid);
        step_persistent_fill_desc(t[4 * l + 1], m->tm_o[l], tx_o, nullptr, (d + 127) / 128, kb_d, 0, grid);
        step_persistent_fill_desc(t[4 * l + 2], m->tm_gu[l], tx_a, m->norm2[l], (F + 63) / 64, kb_d, 0, grid);
        step_persistent_fill_desc(t[4 * l + 3], m->tm_d[l], tx_g, nullptr, (d + 127) / 128, kb_F, 0, grid);
    }
    if (c.with_lm_head)
        step_persistent_fill_desc(t[4 * c.n_layers], m->tm_lm, tx_a, m->final_norm, (c.vocab + 127) / 128, kb_d, 1, grid);
    else
        step_persistent_fill_desc(t[4 * c.n_layers], m->tm_o[0], tx_a, m->final_norm, 1, 1, 0, grid);   // unused slot
    for (int j = 0; j < 4; ++j) {
        s->pmaxp[j] = step_persistent_max_parts(t[j]);
        if (s->pmaxp[j] > 8 || t[j].n_tiles > 256) t[j].g_use = 0;   // beyond the kernel's fixed tables
    }
    for (const PGemmDesc& pd : t)
        if (pd.g_use < 1) {   // a projection too large for the kernel's unit arithmetic: keep the separate kernels
            s->persistent_off = true;
            return ODB_OK;
        }
    uint8_t* dst = s->ws + L.ptable + bi * align_up(step_persistent_table_bytes(c.n_layers));
    ODB_CUDA(cudaStreamSynchronize(s->st));
    ODB_CUDA(cudaMemcpy(dst, t.data(), sizeof(PGemmDesc) * t.size(), cudaMemcpyHostToDevice));
    s->ptable_built[bi] = true;
    return ODB_OK;
}

// One forward over the M rows of the row table already built on the device.
int32_t forward(odb_session* s, int M, int n_lm, int n_tiles, bool write_cache, int n_step_tiles = 0, int n_big_tiles = 0,
                cudaStream_t st = nullptr) {
    const odb_model* m = s->m;
    const odb_config& c = m->cfg;
    const Layout& L = s->L;
    if (!st) st = s->st;
    // H, F, da: this rank's heads, FFN features and attention width (the whole model without tensor parallelism)
    const int d = c.d_model, F = ffn_local(c), H = heads_local(c), hd = c.head_dim, da = H * hd;
    const int R = tp_ranks(c);
    odb_session::Tp& tp = s->tp;
    // Tensor parallelism: a forward is a sequence of segments separated by its exchange points; `seg` counts them
    // as the launches below are walked, and a launch is issued only if its segment is in the requested range.
    int seg = 0;
    auto seg_on = [&]() { return tp.seg_first < 0 || (seg >= tp.seg_first && seg < tp.seg_last); };
    float* h = s->at<float>(L.h);
    __nv_bfloat16* a = s->at<__nv_bfloat16>(L.a);
    float* inv = s->at<float>(L.inv);   // sum(x^2) slices of the RMSNorm whose operand is in `a`
    RowScale inv_scale;
    inv_scale.ssq = inv;
    inv_scale.slots = (d + kNormSliceCols - 1) / kNormSliceCols;
    inv_scale.inv_d = 1.0f / static_cast<float>(d);
    inv_scale.eps = c.rms_eps;
    __nv_bfloat16* q = s->at<__nv_bfloat16>(L.q);
    __nv_bfloat16* k = s->at<__nv_bfloat16>(L.k);
    __nv_bfloat16* v = s->at<__nv_bfloat16>(L.v);
    __nv_bfloat16* o = s->at<__nv_bfloat16>(L.o);
    __nv_bfloat16* g = s->at<__nv_bfloat16>(L.g);
    float* partial = s->at<float>(L.partial);
    int* status = s->at<int>(L.status);
    const size_t nmax = 3 * static_cast<size_t>(d) > 2 * static_cast<size_t>(F) ? 3 * static_cast<size_t>(d)
                                                                                : 2 * static_cast<size_t>(F);
    // K splits of a projection with fp32 partial output; `exchanged`: the partials of all R ranks must fit a receive
    // slot and the consumer's 16-partial limit
    auto plan_splits = [&](int rows, int N, int K, bool exchanged) {
        int sp = gemm_pick_splits(rows, N, K);
        size_t cap = L.partial_rows * nmax / (static_cast<size_t>(rows) * N);
        if (exchanged) {   // R blocks of `sp` partials in a receive slot (sized for at least one partial per rank)
            cap = L.tp_recv_slot / sizeof(float) / (static_cast<size_t>(rows) * N * R);
            if (cap > static_cast<size_t>(16 / R)) cap = 16 / R;
        }
        if (static_cast<size_t>(sp) > cap) sp = static_cast<int>(cap < 1 ? 1 : cap);
        return sp;
    };
    // An exchange of kind `kind`: the projection that produces the data raises this rank's flags when its last CTA
    // has stored (fill_peers); the segment ends behind that launch; the consumer waits on the flags of all ranks
    // (end_exchange returns its argument).  Sequence numbers are counted on the device.
    auto fill_peers = [&](PeerOut& po, int kind) {
        po.n = R;
        po.rank = c.tp_rank;
        po.kind = kind;
        po.alone = tp.alone ? 1 : 0;
        for (int r = 0; r < R; ++r) po.flags[r] = tp.flags[r];
    };
    auto end_exchange = [&](int kind) {
        ++seg;
        TpWait tw;
        tw.region = tp.flags[c.tp_rank];
        tw.kind = kind;
        tw.world = R;
        tw.limit_cycles = tp.wait_limit;
        tw.status = status;
        return tw;
    };
    auto gemm = [&](const CUtensorMap& tw, const __nv_bfloat16* x, float* out, int rows, int N, int K, int sp,
                    const RowScale* row_scale = nullptr, int slot = -1) {
        GemmArgs ga;
        ga.tmap_w = tw;
        ga.x = x;
        ga.partial = out;
        ga.act_out = nullptr;
        if (row_scale) ga.row_scale = *row_scale;
        ga.M = rows; ga.N = N; ga.K = K;
        ga.splits = sp;
        ga.status = status;
        if (slot >= 0) {   // tensor-parallel partial sums: block `rank` of receive slot `slot` on every rank
            fill_peers(ga.peers, slot);
            for (int r = 0; r < R; ++r)
                ga.peers.partial[r] = tp.recv[r] + static_cast<size_t>(slot) * (L.tp_recv_slot / sizeof(float)) +
                                      static_cast<size_t>(c.tp_rank) * sp * rows * N;
        }
        return launch_gemm(ga, st);
    };
#define ODB_LAUNCH(kind, call)          \
    do {                                \
        LaunchScope scope__(s, kind);   \
        ODB_CUDA(call);                 \
    } while (0)
// a launch of the forward proper: only if its segment is requested (always, without tensor parallelism)
#define ODB_FWD(kind, call)             \
    do {                                \
        if (seg_on()) ODB_LAUNCH(kind, call); \
    } while (0)
    if (!write_cache && n_tiles > 0 && use_persistent(s, M) && s->ptable_built[bn_index(M)] && (!c.with_lm_head || n_lm == M)) {
        // decode step as ONE persistent kernel: every projection, the short phases between them and the LM head
        // with its confidence statistics; the per-row merge of the statistics follows as a second launch
        StepPersistentArgs pa{};
        pa.gemms = reinterpret_cast<const PGemmDesc*>(s->ws + L.ptable + bn_index(M) * align_up(step_persistent_table_bytes(c.n_layers)));
        pa.n_layers = c.n_layers; pa.M = M;
        pa.d = d; pa.F = F; pa.H = H; pa.hd = hd; pa.vocab = c.vocab; pa.mask_id = c.mask_id; pa.with_lm = (c.with_lm_head && !s->dump_logits) ? 1 : 0;
        pa.rms_eps = c.rms_eps;
        for (int j = 0; j < 4; ++j) pa.maxp[j] = s->pmaxp[j];
        pa.embed = m->embed;
        pa.row_tok = s->cb.row_tok; pa.row_pos = s->cb.row_pos; pa.row_flags = s->cb.row_flags;
        pa.h = h; pa.a = a; pa.ssq = inv;
        pa.q = q; pa.k = k; pa.v = v; pa.o = o; pa.g = g;
        pa.partial = partial;
        pa.rope = s->at<float2>(L.rope);
        pa.cache = s->kv; pa.max_seq = c.max_seq;
        pa.tiles = s->cb.tiles; pa.n_qtiles = n_tiles;
        int pks = step_persistent_grid() / (n_tiles * H);
        if (pks > 8) pks = 8;
        if (static_cast<size_t>(pks) * M > L.attn_rows) pks = static_cast<int>(L.attn_rows / M);
        if (pks < 1) pks = 1;
        pa.ksplit = pks;
        pa.part_o = s->at<float>(L.part_o); pa.part_ml = s->at<float>(L.part_ml);
        pa.conf_part = reinterpret_cast<ConfPartial*>(s->ws + L.conf_part);
        pa.bars = s->at<unsigned int>(L.pbars);
        pa.status = status;
        // measurement: per-CTA arrival / release times of every grid barrier, kept in the (unused) logits buffer
        static const bool ptiming = getenv("ODB_PERSISTENT_TIMING") && getenv("ODB_PERSISTENT_TIMING")[0] == '1';
        pa.timing = (ptiming && c.with_lm_head && !s->dump_logits) ? s->at<unsigned long long>(L.logits) : nullptr;
        ODB_CUDA(step_persistent_configure(pa));
        ODB_LAUNCH(ODB_KIND_GEMM, launch_step_persistent(pa, st));
        if (pa.with_lm) {
            ODB_LAUNCH(ODB_KIND_CONFIDENCE, launch_confidence_final(pa.conf_part, (c.vocab + 127) / 128, M, s->at<float>(L.conf),
                                                                       s->at<int32_t>(L.tok), st));
        } else if (c.with_lm_head) {
            // test mode: the kernel ended with the LM head's operand; the logits are materialised by a plain launch
            int sp = 1;
            ODB_LAUNCH(ODB_KIND_GEMM, gemm(m->tm_lm, a, s->at<float>(L.logits), M, c.vocab, d, sp, &inv_scale));
            ODB_LAUNCH(ODB_KIND_CONFIDENCE, launch_confidence(s->at<float>(L.logits), M, c.vocab, c.mask_id, s->at<float>(L.conf),
                                                                 s->at<int32_t>(L.tok), s->ws + L.conf_part, st));
        }
        return ODB_OK;
    }
    ODB_FWD(ODB_KIND_ELEMENTWISE, launch_embed(m->embed, s->cb.row_tok, h, M, d, st));
    const float* res = nullptr;   // split-K partials of the projection not yet added to the residual stream
    TpWait res_wait;              // tensor parallelism: the flags those partials are complete behind
    int res_splits = 0;
    size_t res_stride = 0;
    static const int ks_env = getenv("ODB_ATTN_KS") ? atoi(getenv("ODB_ATTN_KS")) : 0;
    static const bool tc_attention = !(getenv("ODB_ATTN_TC") && getenv("ODB_ATTN_TC")[0] == '0');
    int ks = (2 * 148 + n_tiles * H - 1) / (n_tiles * H);
    if (ks_env > 0 && !write_cache) ks = ks_env;
    if (ks > 8) ks = 8;
    if (static_cast<size_t>(ks) * M > L.attn_rows) ks = static_cast<int>(L.attn_rows / M);
    if (ks < 1) ks = 1;
    // L2 prefetch hints (decode steps only): while a short kernel runs between two GEMMs, HBM is
    // idle; the kernel asks L2 for the head of the next GEMM's weights.  Sizes in bytes.
    static const long long pf_mb = getenv("ODB_L2_PREFETCH_MB") ? atoll(getenv("ODB_L2_PREFETCH_MB")) : 8;   // measured: 8 MB helps, 24 MB and more lengthen the hinting kernel
    const bool hint = !write_cache && pdl_enabled() && pf_mb > 0;
    const unsigned long long pf_bytes = static_cast<unsigned long long>(pf_mb) << 20;
    auto hint_of = [&](const void* base, size_t total, size_t offset) {
        L2Prefetch pf{nullptr, 0};
        if (hint && offset < total) {
            pf.ptr = static_cast<const char*>(base) + offset;
            pf.bytes = total - offset < pf_bytes ? total - offset : pf_bytes;
        }
        return pf;
    };
    const size_t qkv_bytes = packed_weight_bytes(3 * da, d), o_bytes = packed_weight_bytes(d, da),
                 gu_bytes = packed_gate_up_bytes(F, d);
    for (int l = 0; l < c.n_layers; ++l) {
        ODB_FWD(ODB_KIND_ELEMENTWISE, launch_rmsnorm(h, res, res_splits, res_stride, m->norm1[l], a, inv, nullptr, M, d,
                                                        hint_of(m->p_qkv[l], qkv_bytes, 0), st, res_wait));
        int sp = plan_splits(M, 3 * da, d, false);
        ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_qkv[l], a, partial, M, 3 * da, d, sp));
        QkvRopeArgs qa;
        qa.partial = partial; qa.splits = sp; qa.pstride = static_cast<size_t>(M) * 3 * da;
        qa.scale = inv_scale;
        qa.rope = s->at<float2>(L.rope);
        qa.row_pos = s->cb.row_pos; qa.row_seq = s->cb.row_seq;
        qa.q = q; qa.k = k; qa.v = v;
        qa.cache = write_cache ? s->kv : nullptr;
        qa.layer = l; qa.n_layers = c.n_layers; qa.H = H; qa.hd = hd; qa.max_seq = c.max_seq; qa.M = M;
        qa.pf = hint_of(m->p_o[l], o_bytes, 0);
        ODB_FWD(ODB_KIND_ELEMENTWISE, launch_qkv_rope(qa, st));
        if (n_step_tiles > 0) {
            // several copies: one work item serves all copies of a block, cached K/V loaded once
            StepAttnArgs sa;
            sa.tiles = s->cb.step_tiles; sa.n_tiles = n_step_tiles;
            sa.q = q; sa.k = k; sa.v = v; sa.cache = s->kv; sa.row_flags = s->cb.row_flags; sa.o = o;
            sa.part_o = s->at<float>(L.part_o); sa.part_ml = s->at<float>(L.part_ml);
            sa.layer = l; sa.n_layers = c.n_layers; sa.H = H; sa.hd = hd; sa.max_seq = c.max_seq; sa.M = M;
            // one work item per SM at most (measured on 4 copies of a 32-token block, 32 heads: 4 key splits
            // beat 3, 6 and 8: every split writes and re-reads a full fp32 output tile)
            int sks = 148 / (n_step_tiles * H);
            if (ks_env > 0) sks = ks_env;
            if (sks > 8) sks = 8;
            if (static_cast<size_t>(sks) * M > L.attn_rows) sks = static_cast<int>(L.attn_rows / M);
            if (sks < 2) sks = 2;
            sa.ksplit = sks;
            sa.pf = hint_of(m->p_gu[l], gu_bytes, 0);
            // tensor-core work items for head dim 128 (batched steps: 33.5 -> 22.5 ms at 16 sequences x 256 rows with the
            // first, two-pass version of that kernel, when a single 128-row item per head still lost to mma.sync, 1.20
            // vs 1.12 ms per step at batch 1; in one pass it wins there too: 1.00 vs 1.13 ms, step 4.82 -> 4.63 ms)
            static const int tc_step_min = getenv("ODB_ATTN_TC_STEP_MIN") ? atoi(getenv("ODB_ATTN_TC_STEP_MIN")) : 1;
            if (hd == 128 && tc_attention && n_step_tiles * H >= tc_step_min) {
                const size_t cache_rows = static_cast<size_t>(c.max_batch) * c.n_layers * 2 * H * c.max_seq;
                // with a work item for every CTA slot there is nothing to gain from key splits: one CTA per item takes
                // the cached and the fresh keys and writes the final output (no partials, no merge kernel)
                if (ks_env == 1 || (ks_env <= 0 && n_step_tiles * H >= 2 * 148)) sa.ksplit = 1;
                ODB_FWD(ODB_KIND_ATTENTION, launch_step_attention_tc(sa, cache_rows, status, st));
                if (sa.ksplit > 1)
                    ODB_FWD(ODB_KIND_ATTENTION, launch_attention_combine(sa.part_o, sa.part_ml, o, M, H, hd, sa.ksplit, st));
            } else {
                ODB_FWD(ODB_KIND_ATTENTION, launch_step_attention(sa, st));
                if (seg_on()) ++s->launches[ODB_KIND_ATTENTION];
            }
        } else if (write_cache && hd == 128 && n_big_tiles > 0 && tc_attention) {
            // refresh with head dim 128: 128-row work items on the tcgen05 tensor cores, no key split
            AttnArgs aa;
            aa.tiles = s->cb.big_tiles; aa.n_tiles = n_big_tiles;
            aa.q = q; aa.k = k; aa.v = v; aa.cache = s->kv; aa.row_flags = s->cb.row_flags; aa.o = o;
            aa.part_o = nullptr; aa.part_ml = nullptr;
            aa.layer = l; aa.n_layers = c.n_layers; aa.H = H; aa.hd = hd; aa.max_seq = c.max_seq; aa.M = M; aa.ksplit = 1;
            aa.pf = L2Prefetch{nullptr, 0};
            ODB_FWD(ODB_KIND_ATTENTION, launch_attention_tc(aa, status, st));
        } else {
        AttnArgs aa;
        aa.tiles = s->cb.tiles; aa.n_tiles = n_tiles;
        aa.q = q; aa.k = k; aa.v = v; aa.cache = s->kv; aa.row_flags = s->cb.row_flags; aa.o = o;
        aa.part_o = s->at<float>(L.part_o); aa.part_ml = s->at<float>(L.part_ml);
        aa.layer = l; aa.n_layers = c.n_layers; aa.H = H; aa.hd = hd; aa.max_seq = c.max_seq; aa.M = M; aa.ksplit = ks;
        aa.early = write_cache ? 0 : 1;   // a refresh writes the cache it attends to: nothing may be read early
        aa.pf = hint_of(m->p_gu[l], gu_bytes, 0);
        ODB_FWD(ODB_KIND_ATTENTION, launch_attention(aa, st));
        if (ks > 1 && seg_on()) ++s->launches[ODB_KIND_ATTENTION];   // the split merge is a second kernel
        }
        sp = plan_splits(M, d, da, R > 1);
        const float* o_sum = partial;   // the partial sums the next RMSNorm adds to the residual stream
        int o_parts = sp;
        TpWait o_wait;
        if (R > 1) {
            // every rank's partial tiles land in slot 0 of every rank; all R * sp partials are added in (rank, split) order.
            // Reusing the slot every layer is safe: a peer stores its next O partials only after its wait on the down
            // exchange of this layer, i.e. after this rank's down projection has raised its flag, and that projection's
            // epilogue runs behind this rank's RMSNorm (the reader of slot 0) in the launch chain.  Slot 1 likewise,
            // with the roles of the two exchanges swapped; the statistics buffer: a peer reaches its next LM head only
            // through exchanges this rank signals after its merge of the current statistics.
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_o[l], o, nullptr, M, d, da, sp, nullptr, 0));
            o_wait = end_exchange(0);
            o_sum = tp.recv[c.tp_rank];
            o_parts = R * sp;
        } else {
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_o[l], o, partial, M, d, da, sp));
        }
        ODB_FWD(ODB_KIND_ELEMENTWISE, launch_rmsnorm(h, o_sum, o_parts, static_cast<size_t>(M) * d, m->norm2[l], a, inv, nullptr, M,
                                                        d, hint_of(m->p_gu[l], gu_bytes, pf_bytes), st, o_wait));
        // A tensor-parallel shard has few gate/up weight tiles (96 / 48 / 24 at 2 / 4 / 8 ranks of the 8B shape): one CTA
        // per tile would stream a megabyte each at a single CTA's rate, so the projection then runs with K splits like
        // the others and a small kernel forms SwiGLU from the split sums (one rank of 4 / 8, timed alone: 3.43 -> 2.74
        // and 4.07 -> 3.38 ms per step).
        const int gu_tiles = (F + 63) / 64;
        // (the whole model's 192 tiles on 148 SMs are unbalanced too, but there 2 or 3 K splits + the combine kernel
        // measured slower than the fused epilogue: 3.52 / 3.43 against 3.28 ms per step, 5.02 / 4.97 against 4.74 at 128 rows)
        const int gu_sp = (R > 1 && gu_tiles * ((M + 127) / 128) <= 128) ? plan_splits(M, gu_tiles * 128, d, false) : 1;
        if (gu_sp > 1) {
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_gu[l], a, partial, M, gu_tiles * 128, d, gu_sp));
            ODB_FWD(ODB_KIND_ELEMENTWISE, launch_swiglu_combine(partial, gu_sp, static_cast<size_t>(M) * gu_tiles * 128, inv_scale, g, M,
                                                               F, st));
        } else {   // gate/up projection with the SwiGLU epilogue: writes bf16 g directly
            GemmArgs ga;
            ga.tmap_w = m->tm_gu[l];
            ga.x = a;
            ga.partial = nullptr;
            ga.act_out = g;
            ga.row_scale = inv_scale;
            ga.M = M; ga.N = F; ga.K = d;
            ga.splits = 1;
            ga.status = status;
            ODB_FWD(ODB_KIND_GEMM, launch_gemm(ga, st));
        }
        sp = plan_splits(M, d, F, R > 1);
        if (R > 1) {
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_d[l], g, nullptr, M, d, F, sp, nullptr, 1));
            res_wait = end_exchange(1);
            res = tp.recv[c.tp_rank] + L.tp_recv_slot / sizeof(float);
            res_splits = R * sp;
        } else {
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_d[l], g, partial, M, d, F, sp));
            res = partial; res_splits = sp;
        }
        res_stride = static_cast<size_t>(M) * d;
    }
    if (!c.with_lm_head) {
        // fold the last projection into the residual stream (the normalised copy is not used)
        ODB_FWD(ODB_KIND_ELEMENTWISE, launch_rmsnorm(h, res, res_splits, res_stride, m->final_norm, a, inv, nullptr, M, d,
                                                        L2Prefetch{nullptr, 0}, st, res_wait));
        return ODB_OK;
    }
    float* logits = s->at<float>(L.logits);
    int lm_tile0_local = 0, lm_rows_local = c.vocab;
    vocab_shard(c, c.tp_rank, &lm_tile0_local, &lm_rows_local);
    for (int r0 = 0; r0 < n_lm; r0 += static_cast<int>(L.lm_chunk)) {
        const int rows = n_lm - r0 < static_cast<int>(L.lm_chunk) ? n_lm - r0 : static_cast<int>(L.lm_chunk);
        const __nv_bfloat16* x = a;
        const RowScale* scale = &inv_scale;
        ODB_FWD(ODB_KIND_ELEMENTWISE, launch_rmsnorm(h, res, res_splits, res_stride, m->final_norm, a, inv, s->cb.lm_rows + r0,
                                                        rows, d, hint_of(m->p_lm, packed_weight_bytes(lm_rows_local, d), 0), st, res_wait));
        if (s->dump_logits) {
            int sp = 1;
            ODB_FWD(ODB_KIND_GEMM, gemm(m->tm_lm, x, logits, rows, c.vocab, d, sp, scale));
            ODB_FWD(ODB_KIND_CONFIDENCE, launch_confidence(logits, rows, c.vocab, c.mask_id, s->at<float>(L.conf) + r0,
                                                                 s->at<int32_t>(L.tok) + r0, s->ws + L.conf_part, st));
        } else {
            // LM head fused with the confidence reduction: per (row, vocabulary tile) statistics instead
            // of logits, merged per row in tile order
            GemmArgs ga;
            ga.tmap_w = m->tm_lm;
            ga.x = x;
            ga.partial = nullptr;
            ga.act_out = nullptr;
            ga.row_scale = *scale;
            ga.conf.part = reinterpret_cast<ConfPartial*>(s->ws + L.conf_part);
            ga.conf.mask_id = c.mask_id;
            const int v_tile0 = lm_tile0_local, v_rows = lm_rows_local;
            ga.M = rows; ga.N = v_rows; ga.K = d;
            ga.splits = 1;
            ga.status = status;
            if (R > 1) {
                // this rank's vocabulary tiles: their statistics go to every rank, which then merges all tiles in order
                ga.conf.tile0 = v_tile0;
                ga.conf.tiles_total = vocab_tiles(c);
                fill_peers(ga.peers, 2);
                for (int r = 0; r < R; ++r) ga.peers.conf[r] = tp.conf[r];
            }
            ODB_FWD(ODB_KIND_GEMM, launch_gemm(ga, st));
            TpWait conf_wait;
            if (R > 1) conf_wait = end_exchange(2);
            ODB_FWD(ODB_KIND_CONFIDENCE, launch_confidence_final(ga.conf.part, vocab_tiles(c), rows, s->at<float>(L.conf) + r0,
                                                                       s->at<int32_t>(L.tok) + r0, st, conf_wait));
        }
    }
    return ODB_OK;
}

// Work items of the multi-copy step attention for a step of this shape (0: the per-copy kernel is used)
int step_items(const odb_session* s, const StepShape& sh) {
    return (!sh.multi || static_cast<size_t>(2) * sh.rows > s->L.attn_rows) ? 0 : sh.step_tiles;
}

}  // namespace

extern "C" {

int32_t odb_refresh_prefill(odb_session* s, const odb_decode_params* p, const int32_t* block_index) {
    if (!s || !p || !block_index) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (p->block_len < 1 || p->block_len > c.max_block) return ODB_ERR_SHAPE;
    const bool tp_on = c.tp_world > 1;
    const bool continuing = tp_on && s->tp.seg_first > 0;   // a later segment range of the refresh already begun
    if (tp_on && (!s->tp.attached || s->dump_logits)) return ODB_ERR_STATE;
    if (continuing ? s->phase != 1 : (s->phase == 1 || s->phase == 3)) return ODB_ERR_STATE;   // an accept is pending
    int M = 0, n_lm = 0, n_tiles = 0, n_big = 0;
    for (int i = 0; i < c.max_batch; ++i) {
        const SeqState& st = s->mirror[i];
        if (!st.active || block_index[i] < 0) continue;
        const int bs = st.P + block_index[i] * p->block_len;
        if (bs >= st.T) return ODB_ERR_ARG;
        M += st.T;
        n_lm += st.T - bs;
        n_tiles += (st.T + 63) / 64;
        n_big += (st.T + 127) / 128;
    }
    if (M == 0) return ODB_ERR_STATE;
    if (tp_on && static_cast<size_t>(n_lm) > s->L.lm_chunk) return ODB_ERR_SHAPE;   // one exchange of statistics per forward
    if (!continuing)
        ODB_LAUNCH(ODB_KIND_CONTROL, launch_build_refresh_rows(s->cb, c.max_batch, block_index, p->block_len, s->st));
    int32_t rc = forward(s, M, c.with_lm_head ? n_lm : 0, n_tiles, true, 0, n_big);
    if (rc != ODB_OK) return rc;
    s->last_rows = M;
    s->last_lm_rows = n_lm;
    s->phase = 1;
    return ODB_OK;
}

int32_t odb_block_decode_step(odb_session* s, const odb_decode_params* p) {
    if (!s || !p) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    const bool tp_on = c.tp_world > 1;
    const bool continuing = tp_on && s->tp.seg_first > 0;   // a later segment range of the step already begun
    if (tp_on && (!s->tp.attached || s->dump_logits)) return ODB_ERR_STATE;
    if (s->phase != (continuing ? 3 : 2)) return ODB_ERR_STATE;
    StepShape sh{0, 0, 0, 0};
    for (int i = 0; i < c.max_batch; ++i) step_shape_add(sh, s->mirror[i]);
    const int M = sh.rows;
    if (M == 0) return ODB_ERR_STATE;
    if (static_cast<size_t>(M) > s->L.rows) return ODB_ERR_SHAPE;
    if (use_persistent(s, M)) {
        const int32_t trc = ensure_ptable(s, M);
        if (trc != ODB_OK) return trc;
    }
    if (tp_on && static_cast<size_t>(M) > s->L.lm_chunk) return ODB_ERR_SHAPE;
    if (!continuing) ODB_LAUNCH(ODB_KIND_CONTROL, launch_build_step_rows(s->cb, c.max_batch, c.mask_id, s->st));
    int32_t rc = forward(s, M, c.with_lm_head ? M : 0, sh.tiles, false, step_items(s, sh));
    if (rc != ODB_OK) return rc;
    s->last_rows = M;
    s->last_lm_rows = M;
    s->phase = 3;
    return ODB_OK;
}

int32_t odb_unmask_accept(odb_session* s, const odb_decode_params* p, int32_t after_refresh, odb_result* results) {
    if (!s || !p || !results) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (p->block_len < 1 || p->block_len > c.max_block) return ODB_ERR_SHAPE;
    if (p->n_copies != 1 && p->n_copies != 4 && p->n_copies != 8) return ODB_ERR_ARG;
    if (p->sampling && (p->n_copies != 1 || p->sample_steps < 1 || p->sample_steps > kMaxLoopIters)) return ODB_ERR_ARG;
    if (p->n_copies > c.max_copies) return ODB_ERR_SHAPE;
    if (s->phase != (after_refresh ? 1 : 3)) return ODB_ERR_STATE;
    ODB_LAUNCH(ODB_KIND_CONTROL, launch_accept(s->cb, c.max_batch, *p, after_refresh, c.mask_id, c.eos_id,
                                           c.with_lm_head ? 0 : 1, s->st));
    int* dev_status = s->at<int>(s->L.status);
    // the kernel has written state, results and status into pinned host memory: one synchronisation, no copy
    ODB_CUDA(cudaStreamSynchronize(s->st));
    for (int i = 0; i < c.max_batch; ++i) s->mirror[i] = s->pinned_state[i];
    memcpy(results, s->pinned_results, sizeof(odb_result) * c.max_batch);
    s->phase = 2;
    if (*s->pinned_status != 0) {
        cudaMemsetAsync(dev_status, 0, sizeof(int), s->st);
        return *s->pinned_status;
    }
    return ODB_OK;
}

int32_t odb_decode_block_resident(odb_session* s, const odb_decode_params* p, int32_t max_iters, odb_result* log,
                                  int32_t log_cap, int32_t* n_iters) {
    if (!s || !p || !log || !n_iters || log_cap < 1) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (p->block_len < 1 || p->block_len > c.max_block) return ODB_ERR_SHAPE;
    if (p->n_copies != 1 && p->n_copies != 4 && p->n_copies != 8) return ODB_ERR_ARG;
    if (p->sampling && (p->n_copies != 1 || p->sample_steps < 1 || p->sample_steps > kMaxLoopIters)) return ODB_ERR_ARG;
    if (p->n_copies > c.max_copies) return ODB_ERR_SHAPE;
    if (s->phase != 2 || s->profiling) return ODB_ERR_STATE;   // event pairs cannot be recorded into the loop body
    if (c.tp_world > 1 && (!s->tp.attached || s->dump_logits || s->tp.seg_first >= 0)) return ODB_ERR_STATE;
    *n_iters = 0;
    if (max_iters <= 0 || max_iters > kMaxLoopIters) max_iters = kMaxLoopIters;
    if (max_iters > log_cap) max_iters = log_cap;
    StepShape sh{0, 0, 0, 0};
    for (int i = 0; i < c.max_batch; ++i) step_shape_add(sh, s->mirror[i]);
    if (sh.rows == 0) return ODB_ERR_STATE;
    if (static_cast<size_t>(sh.rows) > s->L.rows) return ODB_ERR_SHAPE;
    if (use_persistent(s, sh.rows)) {
        const int32_t trc = ensure_ptable(s, sh.rows);
        if (trc != ODB_OK) return trc;
    }

    odb_session::ResidentGraph* g = nullptr;
    for (auto& r : s->resident)
        if (memcmp(&r.shape, &sh, sizeof(sh)) == 0 && memcmp(&r.p, p, sizeof(*p)) == 0 && r.dump_logits == s->dump_logits)
            g = &r;
    int32_t* loop_words = s->at<int32_t>(s->L.loop);   // [0] iterations done, [1] arrivals, [2] iteration limit
    if (!g) {
        odb_session::ResidentGraph r{};
        r.shape = sh; r.p = *p; r.dump_logits = s->dump_logits;
        ODB_CUDA(cudaGraphCreate(&r.graph, 0));
        LoopControl lc;
        cudaError_t e = cudaGraphConditionalHandleCreate(&lc.handle, r.graph, 1, cudaGraphCondAssignDefault);
        cudaGraphNodeParams np = {cudaGraphNodeTypeConditional};
        np.conditional.handle = lc.handle;
        np.conditional.type = cudaGraphCondTypeWhile;
        np.conditional.size = 1;
        cudaGraphNode_t node;
        if (e == cudaSuccess) e = cudaGraphAddNode(&node, r.graph, nullptr, 0, &np);
        if (e == cudaSuccess)
            e = cudaStreamBeginCaptureToGraph(s->record_st, np.conditional.phGraph_out[0], nullptr, nullptr, 0,
                                              cudaStreamCaptureModeThreadLocal);
        if (e != cudaSuccess) {
            cudaGraphDestroy(r.graph);
            return cuda_fail(e);
        }
        lc.iter = loop_words;
        lc.arrivals = loop_words + 1;
        lc.max_iters = loop_words + 2;
        lc.shape = sh;
        lc.host_log = s->pinned_log;
        lc.host_iters = s->pinned_iters;
        long long before[ODB_PROFILE_KINDS];
        memcpy(before, s->launches, sizeof(before));
        // the body: row table, forward, accept.  Whatever a launch returns, the recording is closed before leaving.
        int32_t rc = [&]() -> int32_t {
            ODB_LAUNCH(ODB_KIND_CONTROL, launch_build_step_rows(s->cb, c.max_batch, c.mask_id, s->record_st));
            int32_t frc = forward(s, sh.rows, c.with_lm_head ? sh.rows : 0, sh.tiles, false, step_items(s, sh), 0, s->record_st);
            if (frc != ODB_OK) return frc;
            ODB_LAUNCH(ODB_KIND_CONTROL, launch_accept_loop(s->cb, c.max_batch, *p, c.mask_id, c.eos_id,
                                                            c.with_lm_head ? 0 : 1, lc, s->record_st));
            return ODB_OK;
        }();
        for (int k = 0; k < ODB_PROFILE_KINDS; ++k) r.launches[k] = s->launches[k] - before[k];
        memcpy(s->launches, before, sizeof(before));
        cudaGraph_t body = nullptr;
        e = cudaStreamEndCapture(s->record_st, &body);
        if (rc == ODB_OK && e == cudaSuccess) e = cudaGraphInstantiate(&r.exec, r.graph, 0);
        if (rc != ODB_OK || e != cudaSuccess) {
            if (r.exec) cudaGraphExecDestroy(r.exec);
            cudaGraphDestroy(r.graph);
            return rc != ODB_OK ? rc : cuda_fail(e);
        }
        // a ragged batch walks through many step shapes: keep the most recently recorded graphs only
        constexpr size_t kMaxResidentGraphs = 64;
        if (s->resident.size() >= kMaxResidentGraphs) {
            cudaGraphExecDestroy(s->resident.front().exec);
            cudaGraphDestroy(s->resident.front().graph);
            s->resident.erase(s->resident.begin());
        }
        s->resident.push_back(r);
        g = &s->resident.back();
    }
    s->pinned_iters[0] = 0;
    s->pinned_iters[1] = 0; s->pinned_iters[2] = 0; s->pinned_iters[3] = max_iters;
    ODB_CUDA(cudaMemcpyAsync(loop_words, s->pinned_iters + 1, 3 * sizeof(int32_t), cudaMemcpyHostToDevice, s->st));
    ODB_CUDA(cudaGraphLaunch(g->exec, s->st));
    ODB_CUDA(cudaStreamSynchronize(s->st));
    const int done = *s->pinned_iters;
    if (done < 1 || done > max_iters) return ODB_ERR_STATE;
    for (int k = 0; k < ODB_PROFILE_KINDS; ++k) s->launches[k] += g->launches[k] * done;
    for (int i = 0; i < c.max_batch; ++i) s->mirror[i] = s->pinned_state[i];
    memcpy(log, s->pinned_log, sizeof(odb_result) * static_cast<size_t>(done) * c.max_batch);
    *n_iters = done;
    s->last_rows = sh.rows;
    s->last_lm_rows = sh.rows;
    s->phase = 2;
    if (*s->pinned_status != 0) {
        cudaMemsetAsync(s->at<int>(s->L.status), 0, sizeof(int), s->st);
        return *s->pinned_status;
    }
    return ODB_OK;
}

int32_t odb_debug_read(odb_session* s, int32_t which, void* host, size_t cap, int32_t* rows) {
    if (!s || !host || !rows) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    const Layout& L = s->L;
    const size_t M = s->last_rows, nlm = s->last_lm_rows, d = c.d_model;
    const size_t da = static_cast<size_t>(heads_local(c)) * c.head_dim;   // row width of q / k / v / o (this rank's heads)
    size_t off = 0, bytes = 0, n = M;
    switch (which) {
        case 0: off = L.logits; n = nlm < L.lm_chunk ? nlm : L.lm_chunk; bytes = 4 * n * c.vocab; break;
        case 1: off = L.conf; n = nlm; bytes = 4 * n; break;
        case 2: off = L.tok; n = nlm; bytes = 4 * n; break;
        case 3: off = L.h; bytes = 4 * M * d; break;
        case 4: off = L.q; bytes = 2 * M * da; break;
        case 5: off = L.k; bytes = 2 * M * da; break;
        case 6: off = L.v; bytes = 2 * M * da; break;
        case 7: off = L.o; bytes = 2 * M * da; break;
        case 8: off = L.row_tok; bytes = 4 * M; break;
        case 9: off = L.row_pos; bytes = 4 * M; break;
        case 10: off = L.row_copy; bytes = 4 * M; break;
        case 11: off = L.logits; n = 1; bytes = cap < 4 * L.lm_chunk * c.vocab ? cap : 4 * L.lm_chunk * c.vocab; break;   // raw timing words
        default: return ODB_ERR_ARG;
    }
    if (which == 0 && (!c.with_lm_head || !s->dump_logits)) return ODB_ERR_STATE;
    if (which == 11 && !c.with_lm_head) return ODB_ERR_STATE;
    if (cap < bytes) return ODB_ERR_WORKSPACE;
    ODB_CUDA(cudaStreamSynchronize(s->st));
    ODB_CUDA(cudaMemcpy(host, s->ws + off, bytes, cudaMemcpyDeviceToHost));
    *rows = static_cast<int32_t>(n);
    return ODB_OK;
}

int32_t odb_debug_expire_wait(odb_session* s, int64_t limit_cycles) {
    if (!s || limit_cycles < 1 || limit_cycles > kWaitLimitCycles) return ODB_ERR_ARG;
    ODB_CUDA(launch_expire_wait(limit_cycles, s->at<int>(s->L.status), s->st));
    return ODB_OK;
}

int32_t odb_debug_set_logit_dump(odb_session* s, int32_t enable) {
    if (!s) return ODB_ERR_ARG;
    if (enable && s->m->cfg.tp_world > 1) return ODB_ERR_STATE;   // a rank holds a slice of the vocabulary only
    s->dump_logits = enable != 0;
    return ODB_OK;
}

int32_t odb_debug_gemm(const void* x, const void* w, float* out, void* scratch, size_t scratch_bytes, int32_t M,
                       int32_t N, int32_t K, int32_t k_splits, void* stream) {
    if (!x || !w || !out || !scratch) return ODB_ERR_ARG;
    if (M < 1 || N < 1 || K < 8 || K % 8) return ODB_ERR_SHAPE;
    int splits = k_splits > 0 ? k_splits : gemm_pick_splits(M, N, K);
    const int nkb = (K + 63) / 64;
    if (splits > nkb) splits = nkb;
    while (splits > 1 && ((nkb + splits - 1) / splits) * (splits - 1) >= nkb) --splits;
    const size_t part_bytes = align_up(static_cast<size_t>(splits) * M * N * 4);
    if (scratch_bytes < part_bytes + 256) return ODB_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status = reinterpret_cast<int*>(static_cast<uint8_t*>(scratch) + part_bytes);   // behind the partials
    ODB_CUDA(cudaMemsetAsync(status, 0, sizeof(int), st));
    GemmArgs ga;
    ODB_CUDA(make_weight_tmap(&ga.tmap_w, w, N, K));
    ga.x = x;
    ga.act_out = nullptr;
    ga.partial = static_cast<float*>(scratch);
    ga.M = M; ga.N = N; ga.K = K;
    ga.splits = splits;
    ga.status = status;
    ODB_CUDA(launch_gemm(ga, st));
    ODB_CUDA(launch_reduce_partials(ga.partial, splits, static_cast<size_t>(M) * N, out, static_cast<size_t>(M) * N, st));
    int host_status = 0;
    ODB_CUDA(cudaMemcpyAsync(&host_status, status, sizeof(int), cudaMemcpyDeviceToHost, st));
    ODB_CUDA(cudaStreamSynchronize(st));
    return host_status;
}

int32_t odb_session_profile(odb_session* s, int32_t enable) {
    if (!s) return ODB_ERR_ARG;
    ODB_CUDA(cudaStreamSynchronize(s->st));
    s->profiling = enable != 0;
    s->ev_used = 0;
    memset(s->launches, 0, sizeof(s->launches));
    return ODB_OK;
}

int32_t odb_session_profile_read(odb_session* s, double* ms_by_kind, int64_t* launches_by_kind) {
    if (!s || !ms_by_kind || !launches_by_kind) return ODB_ERR_ARG;
    ODB_CUDA(cudaStreamSynchronize(s->st));
    for (int k = 0; k < ODB_PROFILE_KINDS; ++k) {
        ms_by_kind[k] = 0.0;
        launches_by_kind[k] = s->launches[k];
        s->launches[k] = 0;
    }
    for (size_t i = 0; i + 1 < s->ev_used; i += 2) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s->ev[i], s->ev[i + 1]) == cudaSuccess) ms_by_kind[s->ev_kind[i / 2]] += ms;
    }
    s->ev_used = 0;
    return ODB_OK;
}

int32_t odb_session_tp_buffers(odb_session* s, void** recv, size_t* recv_bytes, void** flags, size_t* flags_bytes,
                               void** conf, size_t* conf_bytes) {
    if (!s || !recv || !recv_bytes || !flags || !flags_bytes || !conf || !conf_bytes) return ODB_ERR_ARG;
    if (s->m->cfg.tp_world < 2) return ODB_ERR_STATE;
    const Layout& L = s->L;
    *recv = s->ws + L.tp_recv;
    *recv_bytes = 2 * L.tp_recv_slot;
    *flags = s->ws + L.tp_flags;
    *flags_bytes = sizeof(unsigned int) * kTpFlagWords;   // peers write the flags; the counters behind them are this rank's own
    *conf = s->ws + L.conf_part;
    *conf_bytes = L.conf_part_bytes;
    return ODB_OK;
}

int32_t odb_session_tp_attach(odb_session* s, void* const* peer_recv, void* const* peer_flags, void* const* peer_conf) {
    if (!s || !peer_recv || !peer_flags || !peer_conf) return ODB_ERR_ARG;
    const odb_config& c = s->m->cfg;
    if (c.tp_world < 2) return ODB_ERR_STATE;
    if (s->phase == 1 || s->phase == 3) return ODB_ERR_STATE;   // a forward is in flight
    odb_session::Tp& tp = s->tp;
    for (int r = 0; r < c.tp_world; ++r) {
        const bool own = r == c.tp_rank;
        void* pr = own ? static_cast<void*>(s->ws + s->L.tp_recv) : peer_recv[r];
        void* pf = own ? static_cast<void*>(s->ws + s->L.tp_flags) : peer_flags[r];
        void* pc = own ? static_cast<void*>(s->ws + s->L.conf_part) : peer_conf[r];
        if (!pr || !pf || !pc) return ODB_ERR_ARG;
        if ((reinterpret_cast<uintptr_t>(pr) | reinterpret_cast<uintptr_t>(pc)) & 15 || reinterpret_cast<uintptr_t>(pf) & 3)
            return ODB_ERR_ARG;
        tp.recv[r] = static_cast<float*>(pr);
        tp.flags[r] = static_cast<unsigned int*>(pf);
        tp.conf[r] = static_cast<ConfPartial*>(pc);
    }
    tp.attached = true;
    return ODB_OK;
}

int32_t odb_tp_enable_peer_access(int32_t peer_device) {
    int dev = 0, n = 0;
    ODB_CUDA(cudaGetDevice(&dev));
    ODB_CUDA(cudaGetDeviceCount(&n));
    if (peer_device < 0 || peer_device >= n) return ODB_ERR_ARG;
    if (peer_device == dev) return ODB_OK;
    cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
    if (e == cudaErrorPeerAccessAlreadyEnabled) {
        cudaGetLastError();   // clear the sticky-less error state
        return ODB_OK;
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return ODB_OK;
}

int32_t odb_tp_vocab_range(const odb_config* cfg, int32_t rank, int32_t* first, int32_t* last) {
    if (!first || !last) return ODB_ERR_ARG;
    const int32_t rc = check_config(cfg);
    if (rc != ODB_OK) return rc;
    if (rank < 0 || rank >= tp_ranks(*cfg)) return ODB_ERR_ARG;
    int tile0 = 0, rows = 0;
    vocab_shard(*cfg, rank, &tile0, &rows);
    *first = tile0 * 128;
    *last = tile0 * 128 + rows;
    return ODB_OK;
}

int32_t odb_tp_segment_count(const odb_config* cfg) {
    if (check_config(cfg) != ODB_OK) return 0;
    if (cfg->tp_world < 2) return 1;
    return 2 * cfg->n_layers + (cfg->with_lm_head ? 1 : 0) + 1;
}

int32_t odb_debug_tp_segments(odb_session* s, int32_t first, int32_t last) {
    if (!s) return ODB_ERR_ARG;
    if (s->m->cfg.tp_world < 2) return ODB_ERR_STATE;
    if (first < 0) {
        if (s->phase == 1 || s->phase == 3) return ODB_ERR_STATE;   // finish the forward in progress first
        s->tp.seg_first = s->tp.seg_last = -1;
        return ODB_OK;
    }
    if (last <= first || last > odb_tp_segment_count(&s->m->cfg)) return ODB_ERR_ARG;
    s->tp.seg_first = first;
    s->tp.seg_last = last;
    return ODB_OK;
}

int32_t odb_debug_tp_alone(odb_session* s, int32_t enable) {
    if (!s) return ODB_ERR_ARG;
    if (s->m->cfg.tp_world < 2 || !s->tp.attached) return ODB_ERR_STATE;
    if (s->phase == 1 || s->phase == 3) return ODB_ERR_STATE;
    s->tp.alone = enable != 0;
    return ODB_OK;
}

int32_t odb_debug_tp_expire_wait(odb_session* s, int32_t kind, int64_t limit_cycles) {
    if (!s || kind < 0 || kind >= kTpKinds || limit_cycles < 1 || limit_cycles > kWaitLimitCycles) return ODB_ERR_ARG;
    if (s->m->cfg.tp_world < 2 || !s->tp.attached) return ODB_ERR_STATE;
    if (s->phase == 1 || s->phase == 3) return ODB_ERR_STATE;
    // a sequence number no rank has signalled: the flags stay below it, the wait runs into its limit
    TpWait tw;
    tw.region = s->tp.flags[s->m->cfg.tp_rank];
    tw.kind = kind;
    tw.bias = 1;   // one more exchange than this rank has completed: nobody has signalled it
    tw.world = s->m->cfg.tp_world;
    tw.limit_cycles = limit_cycles;
    tw.status = s->at<int>(s->L.status);
    ODB_CUDA(launch_tp_wait(tw, s->st));
    return ODB_OK;
}

namespace {

// kind 0: 16-byte loads from every thread; kind 1: a ring of bulk copies per SM (the projections' weight path)
int32_t measure_read(const void* buf, size_t bytes, int32_t reps, void* stream, double* gb_per_s, int kind) {
    if (!buf || !gb_per_s || reps < 1 || bytes < (1u << 20)) return ODB_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(buf) & 15) || (bytes & 15)) return ODB_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    ODB_CUDA(cudaGetDevice(&dev));
    ODB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    int* status = nullptr;
    if (kind == 1) {
        if (bytes < static_cast<size_t>(sms) * 16384) return ODB_ERR_ARG;
        ODB_CUDA(cudaMalloc(&status, sizeof(int)));
        cudaError_t z = cudaMemsetAsync(status, 0, sizeof(int), st);
        if (z != cudaSuccess) { cudaFree(status); return cuda_fail(z); }
    }
    size_t per_pass = bytes;
    auto pass = [&]() -> cudaError_t {
        return kind == 1 ? launch_bulk_read_stream(buf, bytes, sms, status, &per_pass, st)
                         : launch_read_stream(buf, bytes, nullptr, 4 * sms, st);
    };
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) e = pass();   // warm-up pass
    if (e == cudaSuccess) e = cudaEventRecord(e0, st);
    for (int i = 0; i < reps && e == cudaSuccess; ++i) e = pass();
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    int waited_out = 0;
    if (e == cudaSuccess && status) e = cudaMemcpy(&waited_out, status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (status) cudaFree(status);
    if (e != cudaSuccess) return cuda_fail(e);
    if (waited_out != 0) return ODB_ERR_TIMEOUT;
    *gb_per_s = static_cast<double>(per_pass) * reps / (static_cast<double>(ms) * 1e-3) / 1e9;
    return ODB_OK;
}

}  // namespace

int32_t odb_measure_read_bandwidth(const void* buf, size_t bytes, int32_t reps, void* stream, double* gb_per_s) {
    return measure_read(buf, bytes, reps, stream, gb_per_s, 0);
}

int32_t odb_measure_bulk_read_bandwidth(const void* buf, size_t bytes, int32_t reps, void* stream, double* gb_per_s) {
    return measure_read(buf, bytes, reps, stream, gb_per_s, 1);
}

double odb_step_algorithmic_bytes(const odb_config* c, int32_t keys) {
    if (check_config(c) != ODB_OK) return 0.0;
    const double d = c->d_model, F = c->d_ffn;
    const double per_layer = (3 * d * d + d * d + 2 * F * d + d * F) * 2.0 + 2.0 * keys * d * 2.0;
    return c->n_layers * per_layer + (c->with_lm_head ? 2.0 * c->vocab * d : 0.0);
}

}  // extern "C"
