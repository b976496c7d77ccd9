// Episode scheduler: continuous batching of multi-turn games on top of spiral_prefill and the decode
// step (part of spiral_api.cu's translation unit).
//
// Algorithm 1 plays many games at once; each turn appends an observation to a game's context and
// generates a response of unknown length, so games start, finish and change turns at different
// times.  The scheduler keeps the decode batch full from a FIFO of waiting turns:
//   * a turn is admitted when the batch has a free slot and the page pool can hold its worst case
//     (context + observation + response budget) beside what the running turns may still claim;
//   * the observations admitted in one tick go through one spiral_prefill call (all but each one's
//     last token, which is the input of that game's first decode step);
//   * every tick decodes one token for all running turns; the sampled tokens stay on the device as
//     the next inputs (indexed by game), and reach the host one tick late through a pinned ring, so
//     the host never waits for the step it has just launched;
//   * a response ends with the end-of-sequence token or when its budget is used up.  The budget is
//     counted at launch; an end-of-sequence token is seen one tick late, by which time the game has
//     run one more step -- that step's sample is dropped, and its only effect is that the final
//     token's key/value is already cached (remembered per game, see tail_cached).
// Host bookkeeping only; all device work goes through the library's own entry points.
namespace {

__global__ void scatter_tokens_kernel(const int32_t* __restrict__ tok_out, const int32_t* __restrict__ game, int n,
                                      int32_t* __restrict__ last_tok) {
    grid_dependency_sync();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) last_tok[game[i]] = tok_out[i];
}

enum GameState { G_FREE = 0, G_IDLE, G_QUEUED, G_RUNNING };
constexpr int SCHED_RING = 4;           // in-flight steps whose tokens have not been read yet (2 are ever used)

struct SchedGame {
    GameState state = G_FREE;
    std::vector<int32_t> obs;           // observation of the queued turn
    std::vector<int32_t> response;      // tokens of the current / last turn
    std::vector<float> response_lp;     // their log-probabilities under the sampling policy (when collected)
    int max_new = 0;
    int launched = 0;                   // decode steps launched for this turn
    int reserved = 0;                   // pages this turn may still claim beyond those the game owns
    int last_token = -1;                // final token of the last response when its key/value is not cached yet
    bool tail_cached = true;
    bool stop_seen = false;             // end-of-sequence read: later samples of the turn are dropped
    int finish_reason = 0;
};
struct SchedStep {
    int n = 0;
    std::vector<int32_t> games;
    std::vector<int> turns;             // turn number of each game when the step was launched
    int32_t* tok_host = nullptr;        // pinned [max_batch]
    float* lp_host = nullptr;           // pinned [max_batch]
    cudaEvent_t ev = nullptr;
    bool pending = false;
};
}  // namespace

struct spiral_sched {
    spiral_ctx* ctx;
    spiral_kv* kv;
    int eos;
    std::vector<SchedGame> games;
    std::vector<int> turn_no;           // per cache row: turns ever queued on it (tells a late sample of an old turn apart)
    std::vector<int> queue;             // FIFO of games with a waiting turn
    std::vector<int> running;           // games decoding, in slot order
    std::vector<int> finished;          // games whose turn is complete and not polled yet
    SchedStep steps[SCHED_RING];
    int step_next = 0;
    int reserved_total = 0;
    int32_t* last_tok = nullptr;        // device [max_games]: next input token of every game
    int32_t* tok_out = nullptr;         // device [max_batch]
    float* lp_out = nullptr;            // device [max_batch] log-probabilities of the step's tokens
    bool collect_lp = false;
    int32_t* obs_dev = nullptr;         // device staging of the observations admitted in a tick
    int32_t* obs_host = nullptr;        // pinned
    size_t obs_cap = 0;
    cudaEvent_t obs_ev = nullptr;
    bool obs_ev_used = false;
    int64_t ticks = 0, decoded = 0, dropped = 0, appended = 0;
    // admission in batches: a small append costs a pass over all weights, so waiting turns are held until
    // they bring admit_tokens observation tokens together, or the batch has drained to low_water running turns
    int admit_tokens = 1024;
    int low_water = 0;                  // set at creation: half the batch
};

static void sched_destroy(spiral_sched* s) {
    if (!s) return;
    cudaSetDevice(s->ctx->device);
    cudaDeviceSynchronize();
    for (auto& st : s->steps) {
        if (st.tok_host) cudaFreeHost(st.tok_host);
        if (st.lp_host) cudaFreeHost(st.lp_host);
        if (st.ev) cudaEventDestroy(st.ev);
    }
    cudaFree(s->last_tok); cudaFree(s->tok_out); cudaFree(s->lp_out); cudaFree(s->obs_dev);
    if (s->obs_host) cudaFreeHost(s->obs_host);
    if (s->obs_ev) cudaEventDestroy(s->obs_ev);
    delete s;
}

extern "C" int spiral_sched_create(spiral_ctx* ctx, spiral_kv* kv, int eos_token, spiral_sched** out) {
    if (!ctx || !kv || kv->ctx != ctx || !out) return SPIRAL_ERR_INVALID;
    if (eos_token >= ctx->d.vocab) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(ctx->device));
    spiral_sched* s = new (std::nothrow) spiral_sched();
    if (!s) return SPIRAL_ERR_OOM;
    s->ctx = ctx; s->kv = kv; s->eos = eos_token;
    s->low_water = ctx->max_batch / 2;
    s->games.resize(kv->max_games);
    s->turn_no.assign(kv->max_games, 0);
    for (int g = 0; g < kv->max_games; ++g)          // rows already holding a context stay with their owner
        if (kv->seq_len[g] > 0) s->games[g].state = G_IDLE;
    cudaError_t e = cudaMalloc((void**)&s->last_tok, (size_t)kv->max_games * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc((void**)&s->tok_out, (size_t)ctx->max_batch * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc((void**)&s->lp_out, (size_t)ctx->max_batch * sizeof(float));
    if (e == cudaSuccess) e = cudaMemset(s->last_tok, 0, (size_t)kv->max_games * sizeof(int32_t));
    for (auto& st : s->steps) {
        if (e == cudaSuccess) e = cudaMallocHost((void**)&st.tok_host, (size_t)ctx->max_batch * sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMallocHost((void**)&st.lp_host, (size_t)ctx->max_batch * sizeof(float));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&st.ev, cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s->obs_ev, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        g_cuda_error = std::string("scheduler allocation: ") + cudaGetErrorString(e);
        cudaGetLastError();
        sched_destroy(s);
        return e == cudaErrorMemoryAllocation ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;
    }
    *out = s;
    return SPIRAL_OK;
}

extern "C" void spiral_sched_free(spiral_sched* s) { sched_destroy(s); }

extern "C" int spiral_sched_open(spiral_sched* s, int32_t* game_out) {
    if (!s || !game_out) return SPIRAL_ERR_INVALID;
    for (int g = 0; g < (int)s->games.size(); ++g)
        if (s->games[g].state == G_FREE) {
            s->games[g] = SchedGame{};
            s->games[g].state = G_IDLE;
            *game_out = g;
            return SPIRAL_OK;
        }
    return SPIRAL_ERR_OOM;
}

// A new game that starts from the cached context of an idle one (a system prompt common to many games is
// appended once and shared page by page).
extern "C" int spiral_sched_fork(spiral_sched* s, int src_game, int32_t* game_out, void* stream) {
    if (!s || !game_out || src_game < 0 || src_game >= (int)s->games.size()) return SPIRAL_ERR_INVALID;
    const SchedGame& S = s->games[src_game];
    if (S.state != G_IDLE || s->kv->seq_len[src_game] < 1) return SPIRAL_ERR_INVALID;
    int g = -1;
    for (int i = 0; i < (int)s->games.size() && g < 0; ++i)
        if (s->games[i].state == G_FREE) g = i;
    if (g < 0) return SPIRAL_ERR_OOM;
    // the partly filled last page is copied: it must not eat into what running turns have reserved
    if (s->kv->seq_len[src_game] % s->kv->page_size != 0 && (int)s->kv->free_list.size() - s->reserved_total < 1)
        return SPIRAL_ERR_OOM;
    int rc = spiral_kv_fork(s->ctx, s->kv, src_game, g, s->kv->seq_len[src_game], stream);
    if (rc) return rc;
    s->games[g] = SchedGame{};
    s->games[g].state = G_IDLE;
    s->games[g].tail_cached = S.tail_cached;
    s->games[g].last_token = S.last_token;
    *game_out = g;
    return SPIRAL_OK;
}

extern "C" int spiral_sched_close(spiral_sched* s, int game) {
    if (!s || game < 0 || game >= (int)s->games.size()) return SPIRAL_ERR_INVALID;
    SchedGame& G = s->games[game];
    if (G.state != G_IDLE) return SPIRAL_ERR_INVALID;          // free already, or a turn is waiting / running
    for (size_t i = 0; i < s->finished.size(); ++i)
        if (s->finished[i] == game) { s->finished.erase(s->finished.begin() + i); break; }
    const int32_t id = game;
    int rc = spiral_kv_release(s->kv, 1, &id);
    if (rc) return rc;
    G = SchedGame{};
    return SPIRAL_OK;
}

extern "C" int spiral_sched_turn(spiral_sched* s, int game, int n_obs, const int32_t* obs_host, int max_new_tokens) {
    if (!s || game < 0 || game >= (int)s->games.size() || n_obs < 1 || !obs_host || max_new_tokens < 1)
        return SPIRAL_ERR_INVALID;
    SchedGame& G = s->games[game];
    if (G.state != G_IDLE) return SPIRAL_ERR_INVALID;
    for (size_t i = 0; i < s->finished.size(); ++i)            // an unread response is given up by starting a new turn
        if (s->finished[i] == game) { s->finished.erase(s->finished.begin() + i); break; }
    for (int i = 0; i < n_obs; ++i)
        if (obs_host[i] < 0 || obs_host[i] >= s->ctx->d.vocab) return SPIRAL_ERR_INVALID;
    const int tail = G.tail_cached ? 0 : 1;
    // the whole turn must fit the game's context and, on an empty pool, the pool
    const long long final_len = (long long)s->kv->seq_len[game] + tail + n_obs + max_new_tokens;
    if (final_len > s->kv->max_ctx) return SPIRAL_ERR_INVALID;
    if ((final_len + s->kv->page_size - 1) / s->kv->page_size > s->kv->n_pages) return SPIRAL_ERR_OOM;
    G.obs.clear();
    if (tail) G.obs.push_back(G.last_token);                  // the last response's final token enters the context now
    G.obs.insert(G.obs.end(), obs_host, obs_host + n_obs);
    G.tail_cached = true;
    G.max_new = max_new_tokens;
    G.launched = 0; G.response.clear(); G.response_lp.clear(); G.stop_seen = false; G.finish_reason = 0;
    G.state = G_QUEUED;
    ++s->turn_no[game];
    s->queue.push_back(game);
    return SPIRAL_OK;
}

// tokens of the oldest in-flight step(s) -- all but the `keep` most recent -- into the games' responses
static int sched_drain(spiral_sched* s, int keep) {
    for (;;) {
        int pending = 0, oldest = -1;
        for (int k = 0; k < SCHED_RING; ++k) {
            const int idx = (s->step_next + k) % SCHED_RING;          // from the oldest slot on
            if (s->steps[idx].pending) { if (oldest < 0) oldest = idx; ++pending; }
        }
        if (pending <= keep) return SPIRAL_OK;
        SchedStep& st = s->steps[oldest];
        CU_TRY(cudaEventSynchronize(st.ev));
        for (int i = 0; i < st.n; ++i) {
            SchedGame& G = s->games[st.games[i]];
            if (st.turns[i] != s->turn_no[st.games[i]] || G.state != G_RUNNING || G.stop_seen ||
                (int)G.response.size() >= G.max_new) {
                ++s->dropped;               // the step after an end-of-sequence token: its sample belongs to no response
                continue;
            }
            const int tok = st.tok_host[i];
            G.response.push_back(tok);
            if (s->collect_lp) G.response_lp.push_back(st.lp_host[i]);
            if (s->eos >= 0 && tok == s->eos) { G.stop_seen = true; G.finish_reason = 1; }
            else if ((int)G.response.size() == G.max_new) G.finish_reason = 2;
        }
        st.pending = false;
    }
}

// games whose turn is over leave the batch; their reservation returns to the pool
static void sched_retire(spiral_sched* s) {
    size_t w = 0;
    for (size_t i = 0; i < s->running.size(); ++i) {
        const int g = s->running[i];
        SchedGame& G = s->games[g];
        // all samples of a budget-limited turn have been read, or the end-of-sequence token has been seen
        const bool over = G.stop_seen || ((int)G.response.size() >= G.max_new);
        if (!over) { s->running[w++] = g; continue; }
        // steps launched = tokens fed = response tokens whose key/value is cached (+1: the observation's last token)
        const int n_resp = (int)G.response.size();
        G.tail_cached = G.launched > n_resp;          // the step after the final token ran (end-of-sequence, seen late)
        G.last_token = n_resp ? G.response.back() : -1;
        s->reserved_total -= G.reserved;
        G.reserved = 0;
        G.state = G_IDLE;
        s->finished.push_back(g);
    }
    s->running.resize(w);
}

extern "C" int spiral_sched_tick(spiral_sched* s, const float* gumbel_dev, float temperature, void* stream) {
    if (!s || !gumbel_dev || !(temperature > 0.f)) return SPIRAL_ERR_INVALID;
    spiral_ctx* ctx = s->ctx;
    spiral_kv* kv = s->kv;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    ++s->ticks;
    // 1. read the tokens of every step but the one launched last tick; retire finished turns.  When nothing
    //    could be launched otherwise (all running turns are at their budget), read that last step too.
    int rc = sched_drain(s, 1);
    if (rc) return rc;
    sched_retire(s);
    // (waiting turns do not count: this tick may admit none of them -- the head may not fit, the gate may be
    // shut -- and the pages or the drained batch they wait for come from exactly the turns retired here)
    bool any_launchable = false;
    for (int g : s->running) any_launchable = any_launchable || s->games[g].launched < s->games[g].max_new;
    if (!any_launchable) {
        rc = sched_drain(s, 0);
        if (rc) return rc;
        sched_retire(s);
    }
    // 2. admit waiting turns, first come first served
    std::vector<int> admitted;
    size_t obs_tokens = 0;
    size_t waiting_tokens = 0;
    for (int g : s->queue) waiting_tokens += s->games[g].obs.size();
    const bool open_gate = (int)s->running.size() <= s->low_water || waiting_tokens >= (size_t)s->admit_tokens;
    while (open_gate && !s->queue.empty() && (int)s->running.size() < ctx->max_batch) {
        const int g = s->queue.front();
        SchedGame& G = s->games[g];
        const int final_len = kv->seq_len[g] + (int)G.obs.size() + G.max_new;
        const int need = pages_missing(kv, g, final_len);
        if (need > (int)kv->free_list.size() - s->reserved_total) break;       // the head waits; so does everyone behind it
        s->queue.erase(s->queue.begin());
        G.reserved = need;
        s->reserved_total += need;
        G.state = G_RUNNING;
        s->running.push_back(g);
        admitted.push_back(g);
        obs_tokens += G.obs.size();
    }
    if (!admitted.empty()) {
        // observations minus their last tokens -> one append; the last tokens -> the games' next inputs
        if (obs_tokens > s->obs_cap) {
            if (s->obs_ev_used) CU_TRY(cudaEventSynchronize(s->obs_ev));
            cudaFree(s->obs_dev);
            if (s->obs_host) cudaFreeHost(s->obs_host);
            s->obs_dev = nullptr; s->obs_host = nullptr; s->obs_cap = 0;
            const size_t cap = std::max<size_t>(4096, 2 * obs_tokens);
            CU_TRY(cudaMalloc((void**)&s->obs_dev, cap * sizeof(int32_t)));
            CU_TRY(cudaMallocHost((void**)&s->obs_host, cap * sizeof(int32_t)));
            s->obs_cap = cap;
        }
        if (s->obs_ev_used) CU_TRY(cudaEventSynchronize(s->obs_ev));
        std::vector<int32_t> ids, offs(1, 0);
        size_t at = 0;
        const size_t firsts_at = obs_tokens - admitted.size();      // the staging's tail holds the first decode inputs
        for (size_t k = 0; k < admitted.size(); ++k) {
            SchedGame& G = s->games[admitted[k]];
            const size_t body = G.obs.size() - 1;
            if (body > 0) {
                std::memcpy(s->obs_host + at, G.obs.data(), body * sizeof(int32_t));
                at += body;
                ids.push_back(admitted[k]);
                offs.push_back((int32_t)at);
            }
            s->obs_host[firsts_at + k] = G.obs.back();
        }
        CU_TRY(cudaMemcpyAsync(s->obs_dev, s->obs_host, obs_tokens * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        CU_TRY(cudaEventRecord(s->obs_ev, st));
        s->obs_ev_used = true;
        for (size_t k = 0; k < admitted.size(); ++k)
            CU_TRY(cudaMemcpyAsync(s->last_tok + admitted[k], s->obs_dev + firsts_at + k, sizeof(int32_t),
                                   cudaMemcpyDeviceToDevice, st));
        // spiral_prefill takes at most max_batch games per call
        for (size_t b = 0; b < ids.size(); b += ctx->max_batch) {
            const int nb = (int)std::min<size_t>(ctx->max_batch, ids.size() - b);
            std::vector<int32_t> o(offs.begin() + b, offs.begin() + b + nb + 1);
            rc = spiral_prefill(ctx, kv, nb, ids.data() + b, s->obs_dev, o.data(), nullptr, stream);
            if (rc) return rc;
        }
        for (int g : admitted) {
            SchedGame& G = s->games[g];
            s->appended += (int64_t)G.obs.size() - 1;
            const int left = pages_missing(kv, g, kv->seq_len[g] + 1 + G.max_new);     // what the turn may still claim
            s->reserved_total += left - G.reserved;
            G.reserved = left;
            G.obs.clear();
        }
    }
    // 3. one token for every running turn that has budget left
    std::vector<int32_t> batch;
    for (int g : s->running)
        if (s->games[g].launched < s->games[g].max_new && !s->games[g].stop_seen) batch.push_back(g);
    if (batch.empty()) return 0;
    const int n = (int)batch.size();
    int pages_before = 0;
    for (int g : batch) pages_before += kv->n_game_pages[g];
    rc = decode_step_impl(ctx, kv, n, batch.data(), s->last_tok, gumbel_dev, temperature, 1.f, s->tok_out,
                          s->collect_lp ? s->lp_out : nullptr, nullptr, stream, true);
    if (rc) return rc;
    for (int g : batch) {
        SchedGame& G = s->games[g];
        ++G.launched;
        const int left = pages_missing(kv, g, kv->seq_len[g] + (G.max_new - G.launched));
        s->reserved_total += left - G.reserved;
        G.reserved = left;
    }
    LAUNCH(ctx, scatter_tokens_kernel, (n + 127) / 128, 128, 0, st, (const int32_t*)s->tok_out,
           (const int32_t*)meta_i32(ctx), n, s->last_tok);
    SchedStep& rec = s->steps[s->step_next];
    s->step_next = (s->step_next + 1) % SCHED_RING;
    if (rec.pending) return SPIRAL_ERR_CUDA;           // cannot happen: at most two steps are ever unread
    rec.n = n;
    rec.games.assign(batch.begin(), batch.end());
    rec.turns.resize(n);
    for (int i = 0; i < n; ++i) rec.turns[i] = s->turn_no[batch[i]];
    CU_TRY(cudaMemcpyAsync(rec.tok_host, s->tok_out, (size_t)n * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    if (s->collect_lp)
        CU_TRY(cudaMemcpyAsync(rec.lp_host, s->lp_out, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaEventRecord(rec.ev, st));
    rec.pending = true;
    s->decoded += n;
    return n;
}

// Log-probabilities of the sampled tokens (what the learner's update of Algorithm 1 needs beside the
// tokens) are collected from the next tick on; spiral_sched_poll_logprob hands them back with the tokens.
extern "C" int spiral_sched_collect_logprob(spiral_sched* s, int on) {
    if (!s) return SPIRAL_ERR_INVALID;
    for (const SchedGame& G : s->games)
        if (G.state == G_RUNNING) return SPIRAL_ERR_INVALID;           // not in the middle of responses
    s->collect_lp = on != 0;
    return SPIRAL_OK;
}

extern "C" int spiral_sched_policy(spiral_sched* s, int admit_tokens, int low_water) {
    if (!s || admit_tokens < 1 || low_water < 0) return SPIRAL_ERR_INVALID;
    s->admit_tokens = admit_tokens;
    s->low_water = low_water;
    return SPIRAL_OK;
}

extern "C" int spiral_sched_poll(spiral_sched* s, int32_t* game_out, int32_t* tokens_out, int max_tokens,
                                 int32_t* n_tokens_out, int32_t* reason_out) {
    if (!s || !game_out || !n_tokens_out || max_tokens < 0 || (max_tokens > 0 && !tokens_out)) return SPIRAL_ERR_INVALID;
    if (s->finished.empty()) return 0;
    const int g = s->finished.front();
    SchedGame& G = s->games[g];
    if ((int)G.response.size() > max_tokens) return SPIRAL_ERR_TOO_LARGE;
    s->finished.erase(s->finished.begin());
    *game_out = g;
    *n_tokens_out = (int32_t)G.response.size();
    if (reason_out) *reason_out = G.finish_reason;
    if (!G.response.empty()) std::memcpy(tokens_out, G.response.data(), G.response.size() * sizeof(int32_t));
    return 1;
}

extern "C" int spiral_sched_poll_logprob(spiral_sched* s, int32_t* game_out, int32_t* tokens_out, float* logprob_out,
                                         int max_tokens, int32_t* n_tokens_out, int32_t* reason_out) {
    if (!s || !logprob_out || !s->collect_lp) return SPIRAL_ERR_INVALID;
    if (s->finished.empty()) return 0;
    const SchedGame& G = s->games[s->finished.front()];
    if ((int)G.response.size() > max_tokens) return SPIRAL_ERR_TOO_LARGE;
    if (G.response_lp.size() != G.response.size()) return SPIRAL_ERR_INVALID;      // the turn began before collection
    if (!G.response_lp.empty()) std::memcpy(logprob_out, G.response_lp.data(), G.response_lp.size() * sizeof(float));
    return spiral_sched_poll(s, game_out, tokens_out, max_tokens, n_tokens_out, reason_out);
}

extern "C" int spiral_sched_stats(const spiral_sched* s, int64_t* out, int n_out) {
    if (!s || !out || n_out < 1) return SPIRAL_ERR_INVALID;
    const int64_t v[8] = {(int64_t)s->queue.size(), (int64_t)s->running.size(), (int64_t)s->finished.size(),
                          (int64_t)s->kv->free_list.size(), (int64_t)s->reserved_total, s->decoded, s->dropped, s->appended};
    for (int i = 0; i < n_out && i < 8; ++i) out[i] = v[i];
    return SPIRAL_OK;
}
