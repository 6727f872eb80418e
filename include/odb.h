/*
 * odb.h - C ABI of the ODB-dLLM block-decoding hot path for NVIDIA B200 (sm_100a).
 *
 * What the library computes (paper: "Orchestrating Dual-Boundaries", arXiv 2511.21759):
 *   - odb_refresh_prefill   : the block-boundary cache refresh, a full bidirectional forward
 *                             that recomputes every response position and rewrites the K/V
 *                             cache of every position and layer (Sections 1, 2.1 and 4.1);
 *   - odb_block_decode_step : one decoding iteration of the current block over the main block
 *                             and its speculative copies, attending the cached K/V of every
 *                             token outside the block (DualCache, Section 2.1; copies and their
 *                             block-wise mask, Section 4.2; decoded-share layout, Section 4.2.2);
 *   - odb_unmask_accept     : the confidence-threshold accept rule (Section 3, Observation 3),
 *                             the accept-jump walk over the copies (Section 4.2.1) and, after a
 *                             refresh, adaptive length prediction (Section 4.1);
 *   - odb_decode_block_resident : step + accept repeated on the device until the block closes or
 *                             the step's shape changes (no host round trip per iteration).
 * Adaptive length prediction needs no call of its own: the [EOS] scan runs inside
 * odb_unmask_accept(after_refresh = 1), and the host can also shorten a response with
 * odb_session_set_gen_len, the same lever.
 *
 * Conventions
 *   - Every call returns an int32 status: ODB_OK (0) or a negative ODB_ERR_* code; nothing is
 *     printed, thrown or aborted.  odb_status_string() names a code.
 *   - The library allocates NO large device memory.  Weights, K/V cache and workspace are
 *     caller-owned device buffers passed as raw pointers with their byte sizes; the library
 *     borrows them until the handle that received them is destroyed.  (Handles themselves
 *     hold a few KB of device state: TMA descriptors are host objects; the RoPE table lives in
 *     the caller's workspace.)
 *   - All matrices are row-major with the reduction (input-feature) dimension contiguous,
 *     bf16.  RMSNorm gains are fp32.
 *   - Work is enqueued on the session's stream (a cudaStream_t passed as void*).
 *     odb_refresh_prefill and odb_block_decode_step are asynchronous.  odb_unmask_accept
 *     enqueues its kernel, waits for the stream and returns the per-sequence results in host
 *     memory, because the host control loop needs them to choose the next call.
 *   - Sessions are independent; one session is not thread-safe.
 *   - Device-side waits (TMA/MMA barriers) are bounded: a wait that expires records
 *     ODB_ERR_TIMEOUT in the session's device status word, the kernel finishes normally and the
 *     next odb_unmask_accept / odb_session_status reports it.
 */
#ifndef ODB_H_
#define ODB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    ODB_OK = 0,
    ODB_ERR_ARG = -1,       /* null pointer, bad enum, misaligned buffer */
    ODB_ERR_SHAPE = -2,     /* unsupported model shape or size beyond the configured maxima */
    ODB_ERR_WORKSPACE = -3, /* caller buffer too small */
    ODB_ERR_STATE = -4,     /* call not valid in the session's current state */
    ODB_ERR_CUDA = -5,      /* a CUDA runtime/driver call failed (odb_last_cuda_error) */
    ODB_ERR_TIMEOUT = -6    /* a bounded device-side wait expired */
};

/* kernel kinds of the launch accounting (odb_session_profile_read) */
enum {
    ODB_KIND_GEMM = 0,        /* tcgen05 weight-streaming GEMMs (QKV, O, gate/up, down, LM head) */
    ODB_KIND_ATTENTION = 1,   /* block-query attention (+ its split merge) */
    ODB_KIND_ELEMENTWISE = 2, /* embedding, RMSNorm, RoPE/cache scatter, SwiGLU */
    ODB_KIND_CONFIDENCE = 3,  /* vocab-wide max / sum / argmax */
    ODB_KIND_CONTROL = 4,     /* row tables, accept / jump / ALP */
    ODB_PROFILE_KINDS = 5
};

#define ODB_MAX_COPIES 8
#define ODB_MAX_RANKS 4
#define ODB_MAX_CHAIN 5

/* Model shape (the paper names LLaDA-Instruct / LLaDA-1.5 but states no internals; this is the
 * LLaDA-style pre-norm block: RMSNorm, MHA with rotate-half RoPE, SwiGLU, untied LM head).
 * Requirements: d_model == n_heads*head_dim; head_dim in {64,128}; d_model, d_ffn multiples of
 * 16; vocab >= 2. */
typedef struct odb_config {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t mask_id, eos_id;
    float rope_theta, rms_eps;
    int32_t max_batch;  /* sequences per session */
    int32_t max_seq;    /* prompt + response positions per sequence */
    int32_t max_block;  /* block length upper bound (<= 64) */
    int32_t max_copies; /* 1, 4 or 8 */
    int32_t with_lm_head; /* 0: single-layer microbench without LM head (no conf/tok outputs) */
    int32_t tp_world;   /* tensor-parallel ranks sharing this model: 0 or 1 = none; else 2, 4 or 8 (see below) */
    int32_t tp_rank;    /* this rank, 0 .. tp_world-1 */
} odb_config;

/* Tensor-parallel shards (tp_world = R > 1; beyond the paper, which runs on one GPU: the forward of Section 4.1
 * with its weights divided over R GPUs).  The shape fields above keep their GLOBAL values; requirements:
 * n_heads % R == 0, d_ffn % (64 R) == 0.  Rank r holds, and odb_weights describes, only its shard:
 *   wqkv  [3*Hl*head_dim][d_model]  rows = [Wq; Wk; Wv] of heads [r*Hl, (r+1)*Hl), Hl = n_heads / R
 *   wo    [d_model][Hl*head_dim]    the input columns of those heads
 *   wgu   gate/up-packed, the FFN features [r*Fl, (r+1)*Fl), Fl = d_ffn / R
 *   wd    [d_model][Fl]             the input columns of those features
 *   lm_head [Vl][d_model]           the vocabulary rows of tiles [r*Tl, min(T, (r+1)*Tl)), T = ceil(vocab / 128),
 *                                   Tl = ceil(T / R), a tile = 128 consecutive ids (odb_tp_vocab_range)
 * embedding, gains and the residual stream are replicated; the K/V cache holds the rank's own heads
 * (odb_kv_bytes shrinks accordingly).  The O and down projections produce partial sums of the full d_model
 * width: their epilogue stores every fp32 partial tile straight into the receive buffer of EVERY rank (plain
 * stores to peer memory, no bulk or multicast copy from a peer anywhere), the last CTA of the projection to have
 * stored its tiles raises this rank's flag on every rank, and the consuming RMSNorm kernel, which begins with a
 * bounded wait on the R flags, adds all partials in (rank, split) order - the same order on every rank, so the residual streams stay bit-identical.
 * The LM head's per-tile confidence statistics are exchanged the same way and merged in tile order.
 * The exchanges' sequence numbers are counted on the device, so a tensor-parallel step can be captured like any
 * other: odb_decode_block_resident works (every rank runs the same iterations: the accept decides from identical
 * confidences).  Not available under TP: the logits test mode, the persistent step kernel. */
#define ODB_TP_MAX_WORLD 8

/* Device pointers to the weights; per-layer arrays are HOST arrays of n_layers device pointers.
 * wqkv = [Wq; Wk; Wv] stacked on the output dimension, wgu = [Wgate; Wup] likewise.
 * Every projection matrix (wqkv, wo, wgu, wd, lm_head) is given in the library's PACKED layout,
 * produced from the row-major [out][in] matrix by odb_pack_weight: tiles of 128 output rows x 64
 * input columns, each tile 16 KB contiguous, tiles ordered [out_tile][in_block], zero padded to
 * whole tiles.  wgu uses the gate/up variant (odb_pack_gate_up): tile t holds gate rows
 * [64t, 64t+64) followed by up rows [64t, 64t+64), so that the GEMM epilogue can form
 * silu(gate) * up inside one tile.  The embedding table stays row-major. */
typedef struct odb_weights {
    const void* embed;          /* bf16 [vocab][d_model] */
    const void* lm_head;        /* packed bf16 [vocab][d_model], NULL iff with_lm_head == 0 */
    const float* final_norm;    /* fp32 [d_model] */
    const float* const* norm1;  /* fp32 [d_model] per layer */
    const void* const* wqkv;    /* packed bf16 [3*d_model][d_model] per layer */
    const void* const* wo;      /* packed bf16 [d_model][d_model] per layer */
    const float* const* norm2;  /* fp32 [d_model] per layer */
    const void* const* wgu;     /* gate/up-packed bf16 [2*d_ffn][d_model] per layer */
    const void* const* wd;      /* packed bf16 [d_model][d_ffn] per layer */
} odb_weights;

typedef struct odb_decode_params {
    int32_t block_len;          /* tokens per block (paper: 32) */
    int32_t n_copies;           /* 1 plain; 4 accept-jump (Section 4.2.1); 8 adds decoded-share (4.2.2) */
    float accept_threshold;     /* strict ">" */
    float truncate_threshold;   /* adaptive length prediction, strict ">" */
    int32_t stage2_min_decoded; /* decoded tokens in the block from which the 8-copy layout is used;
                                   -1 = ceil(4*block/7), where it fits the row budget of 4 full copies */
    int32_t alp;                /* 1: scan for [EOS] after a refresh and truncate */
    int32_t pick_best;          /* 0: accept-jump walk (Section 4.2.1).  1: the speculation the paper compares
                                   against (Fig. 7(a), Section 5.3): candidates are verified in the main block only,
                                   the copy filling the largest set of verified candidates is adopted and its fills
                                   and own accept set are the step's result (chain = that one copy) */
    int32_t sampling;           /* 1: instead of the threshold rule, the stochastic reverse step of the masked-diffusion
                                   process (Section 2.1, Eq. 1): iteration k = 0 .. sample_steps-1 of a block (the
                                   refresh is k = 0) leaves a masked position masked with probability
                                   (sample_steps-k-1)/(sample_steps-k) and otherwise commits its greedy token; the
                                   uniform deviates come from odb_session_set_sampling_noise.  One copy only. */
    int32_t sample_steps;       /* iterations a block is decoded in when sampling, 1 .. 64 */
} odb_decode_params;

/* Per-sequence result of odb_unmask_accept (host memory, valid on return). */
typedef struct odb_result {
    int32_t masks_left;    /* masked positions remaining in the current block */
    int32_t n_accepted;    /* tokens committed by this call */
    int32_t chain_len;     /* copies visited by the jump walk (>= 1) */
    int32_t chain[ODB_MAX_CHAIN];
    int32_t gen_len;       /* response length after this call (ALP may have shortened it) */
    int32_t block_start;   /* absolute position of the current block */
    int32_t block_end;
    int32_t accepted_pos[64]; /* first n_accepted entries: absolute positions, ascending link order */
    int32_t accepted_tok[64];
} odb_result;

typedef struct odb_model odb_model;
typedef struct odb_session odb_session;

const char* odb_status_string(int32_t status);
/* Text of the last CUDA error seen by this thread's library calls ("" if none). */
const char* odb_last_cuda_error(void);

/* Bytes of the packed form of a row-major bf16 matrix [N][K] (K a multiple of 8); 0 if invalid. */
size_t odb_packed_weight_bytes(int32_t N, int32_t K);
/* dst (packed, odb_packed_weight_bytes(N, K) bytes, device) <- src (row-major bf16 [N][K], device).
 * Both 16-byte aligned.  A pure permutation with zero padding; asynchronous on `stream`. */
int32_t odb_pack_weight(const void* src, void* dst, int32_t N, int32_t K, void* stream);

/* Gate/up variant: src is row-major bf16 [2F][K], gate rows first then up rows. */
size_t odb_packed_gate_up_bytes(int32_t F, int32_t K);
int32_t odb_pack_gate_up(const void* src, void* dst, int32_t F, int32_t K, void* stream);

/* Validates the shape, builds TMA descriptors for the weight matrices.  The weight buffers must
 * stay valid and unchanged while the model lives.  *out is set only on ODB_OK. */
int32_t odb_model_create(const odb_config* cfg, const odb_weights* w, odb_model** out);
int32_t odb_model_destroy(odb_model* m);

/* Bytes of the K/V cache: bf16 [max_batch][n_layers][2][n_heads][max_seq][head_dim]. */
size_t odb_kv_bytes(const odb_config* cfg);
/* Bytes of scratch the session needs for activations, split-K partials, logits, RoPE table,
 * row tables and control state, for the maxima in cfg. */
size_t odb_workspace_bytes(const odb_config* cfg);

/* kv and workspace are device buffers, 256-byte aligned, of at least odb_kv_bytes /
 * odb_workspace_bytes; stream is a cudaStream_t (NULL = default stream).  The call initialises
 * the workspace (RoPE table, state) and zeroes the K/V cache on the stream and waits for it (the
 * tensor-core attention loads whole 64-position boxes of the cache: positions that are not keys
 * are masked but must hold finite values). */
int32_t odb_session_create(odb_model* m, void* kv, size_t kv_bytes, void* workspace, size_t ws_bytes,
                           void* stream, odb_session** out);
int32_t odb_session_destroy(odb_session* s);

/* Sequence `seq` := ids_host[0 .. prompt_len+gen_len): the prompt followed by the response
 * allocation (normally all mask_id; already-decoded tokens are allowed, which is how a session
 * is resumed).  Resets the sequence to block 0.  Synchronous. */
int32_t odb_session_set_sequence(odb_session* s, int32_t seq, const int32_t* ids_host,
                                 int32_t prompt_len, int32_t gen_len);
/* Shortens the response of `seq` to new_gen_len tokens (never grows; must keep at least one
 * position of the current block).  Valid between a refresh and the accept that follows it. */
int32_t odb_session_set_gen_len(odb_session* s, int32_t seq, int32_t new_gen_len);
/* Copies the sequence's ids (prompt + current response length) to ids_host[0..cap); *len gets
 * the count.  Synchronous. */
int32_t odb_session_get_tokens(odb_session* s, int32_t seq, int32_t* ids_host, int32_t cap, int32_t* len);
/* Uniform [0, 1) deviates for the stochastic reverse step (odb_decode_params.sampling) of the block of `seq` that
 * the next refresh opens: u_host[k * block_len + i] decides position i of the block at iteration k (k = 0 is the
 * refresh's accept), n_iters <= 64 rows.  The deviates are data of the caller's (a counter-based stream, so that a
 * run can be reproduced); the library draws no random numbers.  Synchronous. */
int32_t odb_session_set_sampling_noise(odb_session* s, int32_t seq, const float* u_host, int32_t n_iters, int32_t block_len);
/* Marks a sequence inactive (finished) / active; inactive sequences take no part in later calls. */
int32_t odb_session_set_active(odb_session* s, int32_t seq, int32_t active);
/* Reads and clears the device status word (ODB_OK or ODB_ERR_TIMEOUT).  Synchronous. */
int32_t odb_session_status(odb_session* s);

/* Refresh prefill for every active sequence at the start of its block `block_index[seq]`
 * (host array [max_batch]; a negative entry leaves that sequence out of this refresh; entries
 * of inactive sequences are ignored; p supplies block_len): full forward over positions
 * [0, T), K/V of every position and layer written to the cache, confidence and greedy token of
 * response rows [block_start, T) left on the device for odb_unmask_accept.  Asynchronous. */
int32_t odb_refresh_prefill(odb_session* s, const odb_decode_params* p, const int32_t* block_index);

/* One decoding iteration of the current block of every active sequence, over the copies chosen
 * by the previous odb_unmask_accept.  Sequences whose block has no masked position left take no
 * part.  Leaves confidence and greedy token per copy and block position on the device.
 * Requires a preceding refresh + accept for the block.  Asynchronous. */
int32_t odb_block_decode_step(odb_session* s, const odb_decode_params* p);

/* Applies the accept rule and the jump walk to the outputs of the preceding refresh
 * (after_refresh = 1: copy 0 only, preceded by the [EOS] scan / truncation when p->alp) or
 * step (after_refresh = 0), commits tokens, ranks the next speculative candidates.
 * results: host array [max_batch].  Waits for the stream.
 * With a model built without LM head (layer microbenchmark) there are no confidences: the call
 * commits nothing and only lays out the copies of the next step (speculative fills: the first
 * masked positions with token id 0), so masks_left never decreases. */
int32_t odb_unmask_accept(odb_session* s, const odb_decode_params* p, int32_t after_refresh,
                          odb_result* results);

/* Device-resident block loop: the iterations of the open blocks, each an odb_block_decode_step
 * followed by the odb_unmask_accept of its outputs (Sections 2.1 and 4.2: a block is decoded by
 * repeated steps until none of its positions is masked), run on the device without returning to the
 * host in between.  The loop body is recorded once per step shape as a CUDA graph whose WHILE node
 * the accept kernel controls; it runs again while (a) fewer than max_iters iterations have run, (b) a
 * masked position is left in some open block, (c) the next step's row table has the shape of this one
 * (same number of rows, copies and attention work items: it changes when a sequence closes its block,
 * when fewer candidates than copies are left, and at the switch to the decoded-share layout), and
 * (d) no device-side wait has expired.  The results are the ones the two calls would have produced,
 * bit for bit.
 * Requires the state after an odb_unmask_accept (a refresh + accept for the block came before).
 * max_iters: upper bound on iterations, <= 0 or > 64 means 64, never more than log_cap.
 * log: host array [log_cap][max_batch]; entry [i][seq] is the odb_result of iteration i.
 * *n_iters: iterations run (>= 1 on success).  Waits for the stream.  When the loop stops with masked
 * positions left (a shape change or max_iters), call again or continue with the two single calls.
 * Not available while odb_session_profile is on (ODB_ERR_STATE). */
int32_t odb_decode_block_resident(odb_session* s, const odb_decode_params* p, int32_t max_iters,
                                  odb_result* log, int32_t log_cap, int32_t* n_iters);

/* ---- test / measurement entry points --------------------------------------------------- */

/* Test mode.  By default the LM-head GEMM never writes logits: its epilogue reduces each 128-entry
 * vocabulary tile to (max, sum of exp, argmax) per row and a small kernel merges the tiles.  With the
 * dump enabled the LM head writes fp32 logits to the workspace (readable with odb_debug_read 0) and a
 * separate reduction produces confidence and token; greedy tokens are identical in both modes,
 * confidences agree to fp32 rounding of a differently ordered sum. */
int32_t odb_debug_set_logit_dump(odb_session* s, int32_t enable);

/* Test of the timeout path without a fault.  Every device-side wait of the library (TMA / MMA barriers) is the same
 * bounded wait; this call enqueues one small kernel whose single wait cannot be satisfied (an mbarrier nothing
 * arrives at) with a limit of limit_cycles SM clock cycles (1 .. the library's own limit).  The wait runs out, the
 * kernel records ODB_ERR_TIMEOUT in the session's status word and returns normally; the next odb_session_status
 * (or odb_unmask_accept / odb_decode_block_resident) reports it and clears it, and the session stays usable.
 * Asynchronous. */
int32_t odb_debug_expire_wait(odb_session* s, int64_t limit_cycles);

/* Copies a device buffer of the last forward to the host.  which: 0 logits fp32 [rows][vocab]
 * (needs the logit dump);
 * 1 conf fp32 [rows]; 2 tok int32 [rows]; 3 residual stream fp32 [rows][d_model]; 4 q, 5 k,
 * 6 v bf16 [rows][d_model] of the LAST layer; 7 attention output bf16 [rows][d_model];
 * 8 row tokens int32 [rows]; 9 row positions int32 [rows]; 10 row copy ids int32 [rows];
 * 11 the raw timing words of the persistent step kernel (see ODB_PERSISTENT_TIMING below; up to cap_bytes).
 * *rows gets the row count of that buffer.  Synchronous.
 *
 * Environment switches of the decode step, read once per process: ODB_PERSISTENT=1 runs a step of up to 128 rows
 * as ONE cooperative launch (all projections, the short phases between them and the LM head's statistics; same
 * results to rounding order, measured slower than the separate kernels, off by default); with it,
 * ODB_PERSISTENT_TIMING=1 records per CTA the global-timer value at which it arrived at and was released from
 * every grid barrier of the step: uint64 [CTAs][barriers][2] in the logits buffer, 10 barriers per layer (9
 * without key splits) and one before the LM head. */
int32_t odb_debug_read(odb_session* s, int32_t which, void* host, size_t cap_bytes, int32_t* rows);

/* out[M][N] (fp32, device) = x[M][K] (bf16, device) * w[N][K]^T (PACKED bf16, device) with the
 * weight-streaming tcgen05 GEMM, K split k_splits ways and reduced in fixed order.  scratch:
 * device buffer of >= k_splits*M*N*4 + 512 bytes.  k_splits = 0 picks the library's heuristic.
 * Runs on `stream` and waits for it; returns ODB_ERR_TIMEOUT if a device-side wait expired. */
int32_t odb_debug_gemm(const void* x, const void* w, float* out, void* scratch, size_t scratch_bytes,
                       int32_t M, int32_t N, int32_t K, int32_t k_splits, void* stream);

/* The same GEMM as odb_debug_gemm, for callers that may not allocate device memory.  (The paper
 * has no counterpart to this call; it exists for integration only.)
 *
 * Who needs it: code that runs after the process has handed every remaining byte of device memory
 * to a pool of its own (a serving engine that sized its K/V cache to fill the GPU), a plug-in inside
 * a host application that owns the device allocator, or a latency-critical path that cannot accept
 * the implicit device synchronisation and the late failure modes of cudaMalloc.  Such a caller still
 * passes x, w_packed and out, but has no buffer to lend for the split-K partial sums, so this entry
 * point keeps them in a fixed array that is part of the library's device image:
 * ODB_STATIC_SCRATCH_BYTES of partial sums plus a 256-byte status slot.  Every GPU that loads the
 * library holds that array from load until the process exits.
 *
 * Limit: k_splits * M * N * 4 bytes must fit ODB_STATIC_SCRATCH_BYTES (k_splits after the library's
 * heuristic when 0 is passed), otherwise ODB_ERR_WORKSPACE is returned and nothing is launched.
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 * The first call on a device looks up the array's device address (with that device current).  Every
 * call ends by waiting for `stream` and reading the status word back to the host, so it cannot be
 * issued on a stream that is being captured.
 * All calls on a device share the one array: two calls whose kernels overlap on the GPU (different
 * streams, or different host threads) race on it; serialise them.  The array keeps the previous
 * call's contents; the call itself clears the one word that has to start at zero.
 * Otherwise identical to odb_debug_gemm: out[M][N] fp32 = x[M][K] bf16 * w[N][K]^T (packed bf16);
 * runs on `stream`, waits for it, returns ODB_OK or ODB_ERR_TIMEOUT / ODB_ERR_CUDA. */
#define ODB_STATIC_SCRATCH_BYTES (8u << 20)
int32_t odb_gemm_static_scratch(const void* x, const void* w_packed, float* out, int32_t M, int32_t N, int32_t K,
                                int32_t k_splits, void* stream);

/* Launch accounting.  odb_session_profile(s, 1) waits for the stream, clears the counters and
 * from then on brackets every kernel launch of the session with a CUDA event pair (this
 * serialises nothing but costs two event records per launch; leave it off when timing whole
 * steps).  odb_session_profile_read waits for the stream, returns per kind the launches counted
 * since the last read and (profiling on) the summed device time in ms, and clears both.
 * Launches are counted whether profiling is on or off. */
int32_t odb_session_profile(odb_session* s, int32_t enable);
int32_t odb_session_profile_read(odb_session* s, double* ms_by_kind, int64_t* launches_by_kind);

/* ---- tensor parallelism (sessions of a model created with tp_world > 1) ----
 * odb_session_tp_buffers: device pointers (inside this session's workspace) of the three regions its peers
 * write into - receive slots for the partial sums, flag words (followed by this rank's own arrival and sequence
 * counters, which peers never touch), confidence statistics - and their sizes.  The
 * caller carries them to the other ranks (same process: as they are; other processes: as offsets into an
 * inter-process mapping of the workspace allocation) and hands every rank the R pointers of each kind with
 * odb_session_tp_attach (entry tp_rank is this session's own).  Until attached, refresh / step calls return
 * ODB_ERR_STATE.  Every rank must issue the same sequence of refresh / step / accept calls.
 * The library never waits on the host for a peer: a rank that never arrives makes the bounded device-side wait
 * expire, which the next odb_unmask_accept or odb_session_status reports as ODB_ERR_TIMEOUT. */
int32_t odb_session_tp_buffers(odb_session* s, void** recv, size_t* recv_bytes, void** flags, size_t* flags_bytes,
                               void** conf, size_t* conf_bytes);
int32_t odb_session_tp_attach(odb_session* s, void* const* peer_recv, void* const* peer_flags, void* const* peer_conf);
/* Lets kernels on the calling thread's current device store into memory of `peer_device` (cudaDeviceEnablePeerAccess;
 * already enabled, or peer_device being the current device, is success).  ODB_ERR_CUDA if the two cannot be peers. */
int32_t odb_tp_enable_peer_access(int32_t peer_device);
/* first and one-past-last vocabulary id of rank `rank`'s LM-head shard; ODB_ERR_ARG for a bad rank, the
 * configuration's own error for a configuration odb_model_create would refuse */
int32_t odb_tp_vocab_range(const odb_config* cfg, int32_t rank, int32_t* first, int32_t* last);
/* Test facility for running all ranks of a group on ONE GPU without kernels that wait on one another: a forward
 * is cut into odb_tp_segment_count segments at its exchange points (after a flag is raised, before it is waited
 * for).  With a range set, a refresh / step call launches only the kernels of segments [first, last) of the
 * forward; the caller issues segment k on every rank before segment k+1 on any, on one stream, so that every
 * flag is up before the kernel that waits for it starts.  first = 0 begins a forward, later ranges continue it; the accept
 * follows the last segment.  first < 0 restores whole forwards. */
int32_t odb_tp_segment_count(const odb_config* cfg);
int32_t odb_debug_tp_segments(odb_session* s, int32_t first, int32_t last);
/* Measurement facility: a rank timed WITHOUT its peers.  With enable != 0 the session raises, on itself, the flags
 * of all sources at every exchange, so its waits pass although no peer runs; the partial sums and statistics of the
 * absent ranks are whatever their blocks of the receive buffers hold (results are meaningless, device time is that
 * of one rank's kernels).  Attach the session to its own three regions for every rank first. */
int32_t odb_debug_tp_alone(odb_session* s, int32_t enable);
/* Test facility: one launch of the flag wait for exchange `kind` (0, 1: partial-sum slots, 2: statistics) for one exchange
 * more than this rank has completed, with the given cycle limit; nothing raises the flags, so the wait expires and the status
 * word reports ODB_ERR_TIMEOUT (read and cleared by odb_session_status). */
int32_t odb_debug_tp_expire_wait(odb_session* s, int32_t kind, int64_t limit_cycles);

/* Measurement: the rate at which this GPU streams `bytes` (a multiple of 16, 16-byte aligned, at least 1 MiB; use
 * far more than the L2 holds) of device memory with a read-only kernel of 16-byte loads, `reps` passes after one
 * warm-up pass, timed with CUDA events on `stream`.  The decode step is a read stream (weights and K/V are read
 * once, almost nothing is written), so this is the ceiling it is measured against beside the copy bandwidth.
 * Synchronous. */
int32_t odb_measure_read_bandwidth(const void* buf, size_t bytes, int32_t reps, void* stream, double* gb_per_s);

/* The same measurement through the path the projections' weights take: one thread per SM keeps a ring of seven
 * 16 KiB bulk copies (global to shared memory, completion on an mbarrier) in flight over its contiguous share of
 * the buffer; the bytes are not consumed.  Same arguments (bytes at least 16 KiB per SM); the whole 16 KiB chunks
 * of every SM's share are what is read and counted.  Waits are bounded: ODB_ERR_TIMEOUT if a copy never
 * completed.  Allocates and frees one status word (synchronous, not for use inside a capture). */
int32_t odb_measure_bulk_read_bandwidth(const void* buf, size_t bytes, int32_t reps, void* stream, double* gb_per_s);

/* Algorithmic bytes one odb_block_decode_step must move for `rows` query rows and `keys`
 * visible cached positions per sequence (weights once + K/V once); used by the benchmark. */
double odb_step_algorithmic_bytes(const odb_config* cfg, int32_t keys);

#ifdef __cplusplus
}
#endif
#endif /* ODB_H_ */
