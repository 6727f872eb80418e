// Control kernels: row tables of a refresh / a block step, and the unmask/accept kernel
// (threshold accept rule, accept-jump walk over the block copies, adaptive length prediction,
// choice of the next speculative candidates).  A few hundred scalars per sequence: one small
// block per sequence, the sequential parts on thread 0.
#include "odb_internal.cuh"

namespace odb {

namespace {

struct BlockIndexParam {
    int32_t block_index[64];
    int32_t block_len;
};

// Rows of a refresh: every position of every active sequence, in sequence order.
__global__ void build_refresh_rows_kernel(ControlBuffers c, int batch, BlockIndexParam bp) {
    const int seq = blockIdx.x;
    SeqState* st = c.state + seq;
    if (!st->active || bp.block_index[seq] < 0) {
        if (threadIdx.x == 0) st->in_fwd = 0;
        return;
    }
    __shared__ int row0, lm0, tile0, big0;
    if (threadIdx.x == 0) {
        int r = 0, l = 0, t = 0, tb = 0;
        for (int j = 0; j < seq; ++j) {
            const SeqState* o = c.state + j;
            if (!o->active || bp.block_index[j] < 0) continue;
            const int sj = o->P + bp.block_index[j] * bp.block_len;
            r += o->T;
            l += o->T - sj;
            t += (o->T + 63) / 64;
            tb += (o->T + 127) / 128;
        }
        row0 = r; lm0 = l; tile0 = t; big0 = tb;
        const int s = st->P + bp.block_index[seq] * bp.block_len;
        st->in_fwd = 1;
        st->block_idx = bp.block_index[seq];
        st->s = s;
        st->e = min(s + bp.block_len, st->T);
        st->row0 = r;
        st->n_rows = st->T;
        st->lm_row0 = l;
        st->lm_s = s;
        st->lm_n = st->T - s;
        st->n_ranks = 0;
        st->n_copies = 1;
        st->copy_mask[0] = 0;
        st->stage2 = 0;
    }
    __syncthreads();
    const int T = st->T;
    const int s = st->P + bp.block_index[seq] * bp.block_len;
    const int32_t* x = c.x + static_cast<size_t>(seq) * c.max_seq;
    for (int p = threadIdx.x; p < T; p += blockDim.x) {
        const int row = row0 + p;
        c.row_tok[row] = x[p];
        c.row_pos[row] = p;
        c.row_seq[row] = seq;
        c.row_copy[row] = 0;
        c.row_flags[row] = 0;
        if (p >= s) c.lm_rows[lm0 + (p - s)] = row;
    }
    for (int j = threadIdx.x; j < (T + 63) / 64; j += blockDim.x) {
        QTile q;
        q.q_row0 = row0 + 64 * j;
        q.nq = min(64, T - 64 * j);
        q.seq = seq;
        q.cA = 0; q.cB0 = 0; q.cB1 = 0;
        q.f0 = row0; q.n0 = T;
        q.f1 = 0; q.n1 = 0;
        c.tiles[tile0 + j] = q;
    }
    for (int j = threadIdx.x; j < (T + 127) / 128; j += blockDim.x) {
        QTile q;
        q.q_row0 = row0 + 128 * j;
        q.nq = min(128, T - 128 * j);
        q.seq = seq;
        q.cA = 0; q.cB0 = 0; q.cB1 = 0;
        q.f0 = row0; q.n0 = T;
        q.f1 = 0; q.n1 = 0;
        c.big_tiles[big0 + j] = q;
    }
}

// Rows of a block step (Section 4.2; decoded-share layout: Section 4.2.2, caption of Fig. 8):
// copy 0 holds the whole block; a speculative copy holds the whole block (stage 1) or only the
// positions still masked in the committed state (stage 2).  Position ids are the true positions.
__device__ int step_rows_of(const SeqState* st) {
    const int B = st->e - st->s;
    return st->stage2 ? B + (st->n_copies - 1) * st->n_masked : st->n_copies * B;
}

__device__ int step_tiles_of(const SeqState* st) {
    const int B = st->e - st->s;
    return step_tiles_of_counts(st->n_copies, B, st->stage2 ? st->n_masked : B);
}

__global__ void build_step_rows_kernel(ControlBuffers c, int batch, int mask_id) {
    const int seq = blockIdx.x;
    SeqState* st = c.state + seq;
    if (!st->active || st->n_masked <= 0) {
        if (threadIdx.x == 0) st->in_fwd = 0;
        return;
    }
    __shared__ int xs[kMaxBlock];      // the block's committed tokens
    __shared__ int mpre[kMaxBlock];    // masked positions before position i of the block
    __shared__ int row_base, tile_base;
    const int32_t* x = c.x + static_cast<size_t>(seq) * c.max_seq;
    const int s = st->s, e = st->e, B = e - s;
    for (int i = threadIdx.x; i < B; i += blockDim.x) xs[i] = x[s + i];
    __syncthreads();
    if (threadIdx.x == 0) {
        st->in_fwd = 1;
        int row = 0, tile = 0;
        for (int j = 0; j < seq; ++j) {
            const SeqState* o = c.state + j;
            if (!o->active || o->n_masked <= 0) continue;
            row += step_rows_of(o);
            tile += o->n_copies;
        }
        int nm = 0;
        for (int i = 0; i < B; ++i) {
            mpre[i] = nm;
            nm += xs[i] == mask_id;
        }
        row_base = row; tile_base = tile;
        st->row0 = row;
        // copy 0 holds the whole block; a speculative copy the whole block or, in the decoded-share layout, the
        // positions still masked
        for (int cp = 0; cp < st->n_copies; ++cp) {
            st->copy_row0[cp] = row;
            st->copy_nrows[cp] = (st->stage2 && cp > 0) ? nm : B;
            row += st->copy_nrows[cp];
        }
    }
    __syncthreads();
    // one thread per (copy, position): the rows of the copies, copy after copy
    for (int it = threadIdx.x; it < st->n_copies * B; it += blockDim.x) {
        const int cp = it / B, i = it % B;
        const bool decoded = xs[i] != mask_id;
        const bool shared = st->stage2 && cp > 0;
        if (shared && decoded) continue;
        const int row = st->copy_row0[cp] + (shared ? mpre[i] : i);
        int tok = xs[i];
        for (int r = 0; r < st->n_ranks; ++r)
            if (((st->copy_mask[cp] >> r) & 1) && st->rank_off[r] == i) tok = st->rank_tok[r];
        c.row_tok[row] = tok;
        c.row_pos[row] = s + i;
        c.row_seq[row] = seq;
        c.row_copy[row] = cp;
        c.row_flags[row] = decoded ? kRowDecoded : 0;
        c.lm_rows[row] = row;
    }
    if (threadIdx.x != 0) return;
    int row = row_base;
    const int tile = tile_base;
    for (int cp = 0; cp < st->n_copies; ++cp) {
        row += st->copy_nrows[cp];
        QTile q;
        q.q_row0 = st->copy_row0[cp];
        q.nq = st->copy_nrows[cp];
        q.seq = seq;
        q.cA = s; q.cB0 = e; q.cB1 = st->T;
        q.f0 = q.q_row0; q.n0 = q.nq;
        const bool shared = st->stage2 && cp > 0;
        q.f1 = shared ? st->copy_row0[0] : 0;
        q.n1 = shared ? st->copy_nrows[0] : 0;
        c.tiles[tile + cp] = q;
    }
    st->n_rows = row - st->row0;
    st->lm_row0 = st->row0;
    // attention work items that share the cached K/V among copies: copies are packed, in order, into
    // items of at most 8 slabs of 16 rows (the host counts them with the same rule, step_tiles_of)
    int stile = 0;
    for (int j = 0; j < seq; ++j) {
        const SeqState* o = c.state + j;
        if (!o->active || o->n_masked <= 0) continue;
        stile += step_tiles_of(o);
    }
    StepTile cur{};
    int have = 0;
    auto add_src = [&](int cp) {
        for (int i = 0; i < cur.n_src; ++i)
            if (cur.src_copy[i] == cp) return;
        cur.src_copy[cur.n_src] = cp;
        cur.src_row0[cur.n_src] = st->copy_row0[cp];
        cur.src_n[cur.n_src] = st->copy_nrows[cp];
        ++cur.n_src;
    };
    auto flush = [&]() {
        if (st->stage2) add_src(0);   // copy 0's decoded rows are visible to every speculative copy
        c.step_tiles[stile++] = cur;
        have = 0;
    };
    for (int cp = 0; cp < st->n_copies; ++cp) {
        const int slabs = (st->copy_nrows[cp] + 15) / 16;
        if (have && cur.n_slabs + slabs > 8) flush();
        if (!have) {
            cur.seq = seq; cur.cA = s; cur.cB0 = e; cur.cB1 = st->T;
            cur.n_slabs = 0; cur.n_src = 0; cur.stage2 = st->stage2;
            have = 1;
        }
        for (int k = 0; k < slabs; ++k) {
            cur.slab_copy[cur.n_slabs] = cp;
            cur.slab_row0[cur.n_slabs] = st->copy_row0[cp] + 16 * k;
            cur.slab_n[cur.n_slabs] = min(16, st->copy_nrows[cp] - 16 * k);
            ++cur.n_slabs;
        }
        add_src(cp);
    }
    if (have) flush();
}

// Accept rule (Section 3, Observation 3): every masked position whose confidence exceeds tau
// (strict); if none, the single most confident one (lowest position on a tie).
__device__ int accept_set(const float* conf, const bool* masked, int B, float tau, bool* acc) {
    int n = 0, best = -1;
    for (int i = 0; i < B; ++i) {
        acc[i] = masked[i] && conf[i] > tau;
        n += acc[i];
        if (masked[i] && (best < 0 || conf[i] > conf[best])) best = i;
    }
    if (n == 0 && best >= 0) { acc[best] = true; n = 1; }
    return n;
}

// Stochastic reverse step (Section 2.1, Eq. 1) at iteration k of the n_steps a block is decoded in: a masked
// position stays masked with probability s / t = (n_steps - k - 1) / (n_steps - k), decided by its uniform
// deviate u (unmask iff u >= s / t, in fp32); the last iteration unmasks everything left.
__device__ int sample_set(const float* u, const bool* masked, int B, int k, int n_steps, bool* acc) {
    const bool all = k >= n_steps - 1;
    const float stay = all ? 0.f : static_cast<float>(n_steps - k - 1) / static_cast<float>(n_steps - k);
    int n = 0;
    for (int i = 0; i < B; ++i) {
        acc[i] = masked[i] && (all || u[i] >= stay);
        n += acc[i];
    }
    return n;
}

// st / res: the block's shared-memory copies of the sequence's state and result (the decisions are one thread's
// serial walk: every field it touches would otherwise be a dependent global load)
__device__ void accept_body(const ControlBuffers& c, const odb_decode_params& p, int after_refresh, int mask_id, int eos_id,
                            int dry, SeqState* st, odb_result* res) {
    const int seq = blockIdx.x;
    if (!st->active || !st->in_fwd) {
        if (threadIdx.x == 0) {
            res->masks_left = st->active ? st->n_masked : 0;
            res->n_accepted = 0;
            res->chain_len = 0;
            res->gen_len = st->T - st->P;
            res->block_start = st->s;
            res->block_end = st->e;
        }
        return;
    }
    __shared__ float conf[ODB_MAX_COPIES][kMaxBlock];
    __shared__ int tok[ODB_MAX_COPIES][kMaxBlock];
    __shared__ int xs[kMaxBlock];          // the block's committed tokens (step only)
    int32_t* x = c.x + static_cast<size_t>(seq) * c.max_seq;
    const int s = st->s;
    int n_copies = 1;
    // After a step the whole block gathers the copies' confidences and tokens and the block's tokens (the
    // decisions below are taken by thread 0 alone, in the order the method states them)
    const bool gathered = !dry && !after_refresh;
    if (gathered) {
        n_copies = st->n_copies;
        for (int i = threadIdx.x; i < n_copies * kMaxBlock; i += blockDim.x) {
            conf[i / kMaxBlock][i % kMaxBlock] = -1.f;
            tok[i / kMaxBlock][i % kMaxBlock] = -1;
        }
        for (int i = threadIdx.x; i < st->e - s; i += blockDim.x) xs[i] = x[s + i];
        __syncthreads();
        for (int cp = 0; cp < n_copies; ++cp) {
            const int r0 = st->copy_row0[cp], r1 = r0 + st->copy_nrows[cp];
            for (int r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
                const int i = c.row_pos[r] - s;
                conf[cp][i] = c.conf[r];
                tok[cp][i] = c.tok[r];
            }
        }
        __syncthreads();
    }
    if (threadIdx.x != 0) return;

    if (dry) {
        // model without LM head (layer microbenchmark): there is nothing to decide on, so commit
        // nothing and lay out the next step as if no position had been accepted; the speculative
        // fills are the first masked positions with token id 0
        if (after_refresh) st->e = min(s + p.block_len, st->T);
        const int B = st->e - s;
        int n_masked = 0, n_ranks = 0;
        const int k_ranks = p.n_copies >= 8 ? 4 : p.n_copies >= 4 ? 2 : 0;
        for (int i = 0; i < B; ++i) {
            if (x[s + i] != mask_id) continue;
            if (n_ranks < k_ranks) { st->rank_off[n_ranks] = i; st->rank_tok[n_ranks] = 0; ++n_ranks; }
            ++n_masked;
        }
        st->n_ranks = n_ranks;
        st->n_masked = n_masked;
        const int thr = p.stage2_min_decoded >= 0 ? p.stage2_min_decoded : (4 * B + 6) / 7;
        const int stage2 = (p.n_copies >= 8 && (B - n_masked) >= thr) ? 1 : 0;
        const int want = p.n_copies >= 8 ? (stage2 ? 8 : 4) : p.n_copies >= 4 ? 4 : 1;
        const int all_masks[ODB_MAX_COPIES] = {0, 1, 2, 3, 4, 7, 8, 15};
        int nc = 0;
        for (int i = 0; i < want; ++i)
            if ((all_masks[i] >> n_ranks) == 0) st->copy_mask[nc++] = all_masks[i];
        st->n_copies = nc;
        st->stage2 = stage2;
        res->masks_left = n_masked;
        res->n_accepted = 0;
        res->chain_len = 1;
        res->chain[0] = 0;
        res->gen_len = st->T - st->P;
        res->block_start = s;
        res->block_end = st->e;
        return;
    }
    if (after_refresh) {
        // adaptive length prediction (Section 4.1): first [EOS] of the whole predicted response
        // whose confidence exceeds the truncate threshold cuts the response there (slot kept)
        if (p.alp) {
            for (int q = s; q < st->T; ++q) {
                const int r = st->lm_row0 + (q - st->lm_s);
                if (c.tok[r] == eos_id && c.conf[r] > p.truncate_threshold) { st->T = q + 1; break; }
            }
        }
        st->e = min(s + p.block_len, st->T);
        for (int i = 0; i < st->e - s; ++i) {
            const int r = st->lm_row0 + (s + i - st->lm_s);
            conf[0][i] = c.conf[r];
            tok[0][i] = c.tok[r];
        }
    }
    const int B = st->e - s;
    if (after_refresh) st->block_iter = 0;
    const int k_iter = st->block_iter < kMaxLoopIters ? st->block_iter : kMaxLoopIters - 1;
    const float* noise = c.noise + (static_cast<size_t>(seq) * kMaxLoopIters + k_iter) * kMaxBlock;
    ++st->block_iter;
    bool masked0[kMaxBlock], masked[kMaxBlock], acc[kMaxBlock], taken[kMaxBlock];
    for (int i = 0; i < B; ++i) { masked0[i] = (gathered ? xs[i] : x[s + i]) == mask_id; taken[i] = false; }

    // accept-jump walk (Section 4.2.1): start in the main block; a candidate is hit if its
    // position was accepted with the token it had been filled with; jump to the largest copy
    // whose extra candidates are all hit; the accepted sets along the chain are committed,
    // an earlier link winning at a shared position
    int cur = 0, chain_len = 0, n_acc = 0;
    const bool pick = p.pick_best && !after_refresh;
    if (pick) {
        // the compared speculation (Fig. 7(a), Section 5.3): candidates verified in the main block only; the copy
        // filling the largest set of hits is adopted, and its fills and own accept set are the whole result
        accept_set(conf[0], masked0, B, p.accept_threshold, acc);
        int hit = 0;
        for (int r = 0; r < st->n_ranks; ++r) {
            const int o = st->rank_off[r];
            if (acc[o] && tok[0][o] == st->rank_tok[r]) hit |= 1 << r;
        }
        for (int cp = 1; cp < n_copies; ++cp) {
            const int Y = st->copy_mask[cp];
            if (Y & ~hit) continue;
            if (cur == 0 || __popc(Y) > __popc(st->copy_mask[cur]) ||
                (__popc(Y) == __popc(st->copy_mask[cur]) && Y < st->copy_mask[cur]))
                cur = cp;
        }
        auto commit = [&](int i, int t) {
            taken[i] = true;
            x[s + i] = t;
            if (n_acc < 64) { res->accepted_pos[n_acc] = s + i; res->accepted_tok[n_acc] = t; }
            ++n_acc;
        };
        if (cur != 0) {
            const int Y = st->copy_mask[cur];
            bool any = false;
            for (int i = 0; i < B; ++i) masked[i] = masked0[i];
            for (int r = 0; r < st->n_ranks; ++r)
                if ((Y >> r) & 1) { masked[st->rank_off[r]] = false; commit(st->rank_off[r], st->rank_tok[r]); }
            for (int i = 0; i < B; ++i) any |= masked[i];
            if (any) accept_set(conf[cur], masked, B, p.accept_threshold, acc);
            else for (int i = 0; i < B; ++i) acc[i] = false;
        }
        for (int i = 0; i < B; ++i)
            if (acc[i] && !taken[i]) commit(i, tok[cur][i]);
        res->chain[0] = cur;
        chain_len = 1;
    }
    while (!pick) {
        res->chain[chain_len < ODB_MAX_CHAIN ? chain_len : ODB_MAX_CHAIN - 1] = cur;
        ++chain_len;
        const int X = after_refresh ? 0 : st->copy_mask[cur];
        bool any = false;
        for (int i = 0; i < B; ++i) masked[i] = masked0[i];
        for (int r = 0; r < st->n_ranks; ++r)
            if ((X >> r) & 1) masked[st->rank_off[r]] = false;
        for (int i = 0; i < B; ++i) any |= masked[i];
        if (!any) break;
        if (p.sampling) sample_set(noise, masked, B, k_iter, p.sample_steps, acc);
        else accept_set(conf[cur], masked, B, p.accept_threshold, acc);
        for (int i = 0; i < B; ++i) {
            if (acc[i] && !taken[i]) {
                taken[i] = true;
                x[s + i] = tok[cur][i];
                if (n_acc < 64) { res->accepted_pos[n_acc] = s + i; res->accepted_tok[n_acc] = tok[cur][i]; }
                ++n_acc;
            }
        }
        if (after_refresh) break;
        int hit = 0;
        for (int r = 0; r < st->n_ranks; ++r) {
            const int o = st->rank_off[r];
            if (!((X >> r) & 1) && acc[o] && tok[cur][o] == st->rank_tok[r]) hit |= 1 << r;
        }
        int best = -1;
        for (int cp = 0; cp < n_copies; ++cp) {
            const int Y = st->copy_mask[cp];
            if ((Y & X) != X || Y == X || ((Y & ~X) & ~hit)) continue;
            if (best < 0 || __popc(Y) > __popc(st->copy_mask[best]) ||
                (__popc(Y) == __popc(st->copy_mask[best]) && Y < st->copy_mask[best]))
                best = cp;
        }
        if (best < 0) break;
        cur = best;
    }

    // state after the walk; next candidates: the most confident still-masked positions of the
    // adopted copy (Section 4.2), ties to the lower position
    int n_masked = 0;
    for (int i = 0; i < B; ++i) {
        masked[i] = masked0[i] && !taken[i];
        n_masked += masked[i];
    }
    const int k_ranks = p.n_copies >= 8 ? 4 : p.n_copies >= 4 ? 2 : 0;
    int n_ranks = 0;
    for (int r = 0; r < k_ranks; ++r) {
        int best = -1;
        for (int i = 0; i < B; ++i)
            if (masked[i] && (best < 0 || conf[cur][i] > conf[cur][best])) best = i;
        if (best < 0) break;
        masked[best] = false;
        st->rank_off[n_ranks] = best;
        st->rank_tok[n_ranks] = tok[cur][best];
        ++n_ranks;
    }
    st->n_ranks = n_ranks;
    st->n_masked = n_masked;
    // stage switch (Section 4.2.2 gives no number): decoded-share once eight copies fit the row
    // budget of four full copies, B + 7 (B - n_dec) <= 4 B
    const int thr = p.stage2_min_decoded >= 0 ? p.stage2_min_decoded : (4 * B + 6) / 7;
    const int stage2 = (p.n_copies >= 8 && (B - n_masked) >= thr) ? 1 : 0;
    const int want = p.n_copies >= 8 ? (stage2 ? 8 : 4) : p.n_copies >= 4 ? 4 : 1;
    const int all_masks[ODB_MAX_COPIES] = {0, 1, 2, 3, 4, 7, 8, 15};
    int nc = 0;
    for (int i = 0; i < want; ++i)
        if ((all_masks[i] >> n_ranks) == 0) st->copy_mask[nc++] = all_masks[i];
    st->n_copies = nc;
    st->stage2 = stage2;

    res->masks_left = n_masked;
    res->n_accepted = n_acc;
    res->chain_len = chain_len;
    res->gen_len = st->T - st->P;
    res->block_start = s;
    res->block_end = st->e;
}

// One block per sequence.  After the decisions, the block writes the sequence's state and result (and block 0
// the status word) straight into pinned host memory.
struct AcceptShared {
    SeqState st;
    odb_result res;
};
__device__ __forceinline__ void accept_load(const ControlBuffers& c, AcceptShared* sh) {
    const int seq = blockIdx.x;
    const int* gs = reinterpret_cast<const int*>(c.state + seq);
    const int* gr = reinterpret_cast<const int*>(c.results + seq);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(SeqState) / 4); i += blockDim.x) reinterpret_cast<int*>(&sh->st)[i] = gs[i];
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(odb_result) / 4); i += blockDim.x) reinterpret_cast<int*>(&sh->res)[i] = gr[i];
    __syncthreads();
}
// state and result back to the device copies and out to pinned host memory (host_res: where this call's results go)
__device__ __forceinline__ void accept_store(const ControlBuffers& c, const AcceptShared* sh, odb_result* host_res) {
    const int seq = blockIdx.x;
    const int* ss = reinterpret_cast<const int*>(&sh->st);
    const int* sr = reinterpret_cast<const int*>(&sh->res);
    int* gs = reinterpret_cast<int*>(c.state + seq);
    int* hs = reinterpret_cast<int*>(c.host_state + seq);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(SeqState) / 4); i += blockDim.x) { gs[i] = ss[i]; hs[i] = ss[i]; }
    int* gr = reinterpret_cast<int*>(c.results + seq);
    int* hr = reinterpret_cast<int*>(host_res);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(odb_result) / 4); i += blockDim.x) { gr[i] = sr[i]; hr[i] = sr[i]; }
}

__global__ void accept_kernel(ControlBuffers c, odb_decode_params p, int after_refresh, int mask_id, int eos_id, int dry) {
    __shared__ AcceptShared sh;
    accept_load(c, &sh);
    accept_body(c, p, after_refresh, mask_id, eos_id, dry, &sh.st, &sh.res);
    __syncthreads();
    accept_store(c, &sh, c.host_results + blockIdx.x);
    if (blockIdx.x == 0 && threadIdx.x == 0) *c.host_status = *c.status;
    __threadfence_system();
}

// The accept of the device-resident loop: the same decisions, then the hand-over to the next iteration.
__global__ void accept_loop_kernel(ControlBuffers c, odb_decode_params p, int mask_id, int eos_id, int dry, LoopControl lc) {
    __shared__ AcceptShared sh;
    accept_load(c, &sh);
    accept_body(c, p, 0, mask_id, eos_id, dry, &sh.st, &sh.res);
    __syncthreads();
    const int seq = blockIdx.x, batch = gridDim.x;
    const int it = *lc.iter;      // stable until every block has arrived below
    accept_store(c, &sh, lc.host_log + static_cast<size_t>(it) * batch + seq);
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x != 0) return;
    // fail-safe: the loop ends unless the last block below asks for another pass (block 0 writes this before it
    // arrives, the last block writes after every arrival, so the last block's word stands)
    if (seq == 0) {
        cudaGraphSetConditional(lc.handle, 0u);
        __threadfence();
    }
    if (atomicAdd(lc.arrivals, 1) != batch - 1) return;
    // last block of the iteration: every sequence's state is final
    __threadfence();
    StepShape next{0, 0, 0, 0};
    for (int i = 0; i < batch; ++i) {
        const volatile SeqState* vs = c.state + i;
        SeqState st{};
        st.active = vs->active; st.n_masked = vs->n_masked; st.s = vs->s; st.e = vs->e;
        st.n_copies = vs->n_copies; st.stage2 = vs->stage2;
        step_shape_add(next, st);
    }
    const int err = *reinterpret_cast<const volatile int*>(c.status);
    const bool same = next.rows == lc.shape.rows && next.tiles == lc.shape.tiles &&
                      next.step_tiles == lc.shape.step_tiles && next.multi == lc.shape.multi;
    const int limit = min(*lc.max_iters, kMaxLoopIters);
    const bool again = it + 1 < limit && err == 0 && next.rows > 0 && same;
    *lc.arrivals = 0;
    *lc.iter = it + 1;
    *lc.host_iters = it + 1;
    *c.host_status = err;
    __threadfence_system();
    cudaGraphSetConditional(lc.handle, again ? 1u : 0u);
}

// A wait that runs out by design: the barrier is initialised for one arrival that never comes.
__global__ void expire_wait_kernel(long long limit_cycles, int* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(&bar))));
        abort_word = 0;
    }
    __syncthreads();
    mbar_wait_bounded(&bar, 0, &abort_word, status, limit_cycles);
}

}  // namespace

cudaError_t launch_expire_wait(long long limit_cycles, int* status, cudaStream_t st) {
    expire_wait_kernel<<<1, 32, 0, st>>>(limit_cycles, status);
    return cudaGetLastError();
}

cudaError_t launch_accept_loop(const ControlBuffers& c, int batch, const odb_decode_params& p, int mask_id, int eos_id,
                               int dry, const LoopControl& lc, cudaStream_t st) {
    accept_loop_kernel<<<batch, 64, 0, st>>>(c, p, mask_id, eos_id, dry, lc);
    return cudaGetLastError();
}

cudaError_t launch_build_step_rows(const ControlBuffers& c, int batch, int mask_id, cudaStream_t st) {
    build_step_rows_kernel<<<batch, 64, 0, st>>>(c, batch, mask_id);
    return cudaGetLastError();
}

cudaError_t launch_accept(const ControlBuffers& c, int batch, const odb_decode_params& p, int after_refresh,
                          int mask_id, int eos_id, int dry, cudaStream_t st) {
    accept_kernel<<<batch, 64, 0, st>>>(c, p, after_refresh, mask_id, eos_id, dry);
    return cudaGetLastError();
}

cudaError_t launch_build_refresh_rows(const ControlBuffers& c, int batch, const int32_t* block_index,
                                           int block_len, cudaStream_t st) {
    BlockIndexParam bp;
    for (int i = 0; i < 64; ++i) bp.block_index[i] = i < batch ? block_index[i] : 0;
    bp.block_len = block_len;
    build_refresh_rows_kernel<<<batch, 256, 0, st>>>(c, batch, bp);
    return cudaGetLastError();
}

}  // namespace odb
