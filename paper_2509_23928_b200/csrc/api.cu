// Host layer of libhivis: argument checking, per-slot state, launch sequencing.
// Every step of the path runs in the CUDA kernels; nothing here computes on the CPU.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "hivis_internal.cuh"

struct hivis_ctx {
    hivis_config cfg;
    int dtype;
    size_t esize;
    int qw, kvw, qkvw;
    int rows_cap;                 // batch rows the workspaces hold: max(max_batch, 16)
    int device;
    // weights (library-owned copies)
    void *embed, *lm_head, *fc, *norm1, *wqkv, *bqkv, *wo, *norm2, *wgu, *wdown, *resid_proj;
    void *Kc, *Vc;
    double* inv_freq;
    // per-slot state
    int* kv_len;
    int* pend_id;
    float* pend_feat;
    // per-call work
    int *d_slots, *d_pos0, *cur_id;
    float *feat, *u, *qkv, *attn, *y, *act, *rho_raw, *rho, *ssq1, *ssq2;
    bf16 *feat_h, *xq, *attn_h, *xm, *act_h;
    u64* keys;
    int key_stride;
    float2* vstats;               // sampled verification: (max, sum exp) of every piece of every logits row
    u64* vkeys;                   // verification: argmax keys [max_batch][max_k + 1] and arrival counters
    int* varrive;                 // [max_batch]; both zero between calls
    float *part_acc, *part_ml;
    int* counters;
    int chunk, nsplit_cap;
    // persistent chain kernel
    int num_sms;
    bool chain_ok;                // cooperative launch available and the kernel fits
    bool chain_ok_coop;           // cooperative launch available
    bool opt_chain;               // option HIVIS_OPT_CHAIN_KERNEL
    u64* bar_counter;
    u64 bar_count_host;           // value of *bar_counter once everything enqueued has run
    int* error_flag;              // [0]: a device-side wait ran out; [1] (= id_flag): a token id was out of range
    int* id_flag;
    // tensor-core chain kernel (bf16, up to 16 sequences)
    bool tc_ok;                   // cooperative launch available, shapes supported, tensor maps built
    long long wait_cycles;        // option HIVIS_OPT_WAIT_LIMIT_US, in cycles
    bool debug_skew;              // option HIVIS_OPT_DEBUG_MISS_BARRIER: the next draft's grid barriers cannot complete
    int opt_tc;                   // option HIVIS_OPT_TC_KERNEL: 0 off, 1 for two or more sequences, 2 always
    bool opt_phase_times;         // option HIVIS_OPT_PHASE_TIMES
    int opt_l2_keep;              // option HIVIS_OPT_L2_KEEP: phases whose weights are asked to stay in L2
    int opt_tc_prefill;           // option HIVIS_OPT_TC_PREFILL: 0 = never, else the smallest call (pairs) that takes the tensor-core path
    bool pf_ok;                   // the tensor-core prefill can run (bf16, shapes, buffers)
    bf16 *pf_xe, *pf_xq;          // [map_cap][d] pair-major operands of the tensor-core prefill
    float* pf_ssq;                // [ceil(d / 128)][map_cap]
    float2* pf_rope;              // [map_cap][head_dim / 2]
    u64* phase_t;                 // [HIVIS_MAX_K][HIVIS_PHASE_EVENTS][num_sms]
    int phase_k;                  // draft steps of the last recorded launch (0: none)
    TcMaps tc_maps;
    float* tc_partial;
    int* tile_ctr;
    int tc_tiles;
    bf16* xe_h;
    float2* rope_tab;
    int *slot_of, *row_of;
    long long map_cap;
    // tree drafting
    TreeBufs tree;
    float* tree_logits;           // [TREE_MAX_TOPK][vocab] logits of the level's nodes
    float* tree_g;                // [TREE_MAX_TOPK][d] layer outputs of the previous level
    int tree_depth[HIVIS_MAX_BATCH];    // depth of the tree drafted last on the slot and not verified yet, else 0
    int tree_count[HIVIS_MAX_BATCH];    // its number of kept nodes
    // host mirrors
    int kv_upper[HIVIS_MAX_BATCH];      // upper bound of the slot's row count
    bool kv_exact[HIVIS_MAX_BATCH];
    bool pending[HIVIS_MAX_BATCH];
    bool have_pair[HIVIS_MAX_BATCH];
    int last_k[HIVIS_MAX_BATCH];        // k of the draft that has not been verified yet, else 0
    int tap_B;
    bool tap_mma;
    int64_t launches;
    char err[256];
    std::vector<void*> allocs;
    // optional per-kernel-class timing of hivis_draft (events around every launch)
    bool prof_on;
    std::vector<cudaEvent_t> prof_ev;
    std::vector<int> prof_cls;
    size_t prof_n;
};

enum { CLS_FUSE = 0, CLS_QKV, CLS_ATTN, CLS_OPROJ, CLS_GATEUP, CLS_DOWN, CLS_LM, CLS_OTHER, CLS_CHAIN, CLS_COUNT };
static_assert(CLS_COUNT == HIVIS_PROFILE_CLASSES, "profile classes");

static void prof_mark(hivis_ctx* c, int cls, cudaStream_t st, bool begin) {
    if (!c->prof_on) return;
    const size_t i = c->prof_n * 2 + (begin ? 0 : 1);
    while (c->prof_ev.size() <= i) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) { c->prof_on = false; return; }
        c->prof_ev.push_back(e);
    }
    cudaEventRecord(c->prof_ev[i], st);
    if (begin) {
        if (c->prof_cls.size() <= c->prof_n) c->prof_cls.resize(c->prof_n + 1);
        c->prof_cls[c->prof_n] = cls;
    } else {
        c->prof_n += 1;
    }
}

static int fail(hivis_ctx* c, int code, const char* fmt, ...) {
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof(c->err), fmt, ap);
        va_end(ap);
    }
    return code;
}
static char g_init_err[256] = "";
// text for failures of calls that have no context; hivis_last_error(NULL) returns it
void hivis_set_global_error(const char* msg) { snprintf(g_init_err, sizeof(g_init_err), "%s", msg); }

#define CK(c, call)                                                                            \
    do {                                                                                       \
        cudaError_t e_ = (call);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return fail(c, HIVIS_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));    \
    } while (0)
#define CKL(c, call)            \
    do {                        \
        CK(c, call);            \
        (c)->launches += 1;     \
    } while (0)
// a launch of the draft chain, timed per kernel class when profiling is on
#define CKP(c, cls, st, call)               \
    do {                                    \
        prof_mark(c, cls, st, true);        \
        CK(c, call);                        \
        (c)->launches += 1;                 \
        prof_mark(c, cls, st, false);       \
    } while (0)

extern "C" {
static void fill_chain_args(hivis_ctx* c, ChainArgs* a);
}

static bool misaligned(const void* p) { return (((uintptr_t)p) & 15u) != 0; }

template <typename T>
static bool dalloc(hivis_ctx* c, T** p, size_t count) {
    void* q = nullptr;
    const size_t bytes = (count * sizeof(T) + 255) & ~(size_t)255;
    if (cudaMalloc(&q, bytes ? bytes : 256) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    c->allocs.push_back(q);
    *p = (T*)q;
    return true;
}

static void free_all(hivis_ctx* c) {
    for (void* p : c->allocs) cudaFree(p);
    c->allocs.clear();
}

static int check_slots(hivis_ctx* c, int B, const int* slots_host, SlotList* sl) {
    if (B < 1 || B > c->cfg.max_batch) return fail(c, HIVIS_ERR_CAPACITY, "B=%d outside [1,%d]", B, c->cfg.max_batch);
    bool seen[HIVIS_MAX_BATCH] = {false};
    sl->n = B;
    for (int b = 0; b < B; ++b) {
        const int s = slots_host ? slots_host[b] : b;
        if (s < 0 || s >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", s);
        if (seen[s]) return fail(c, HIVIS_ERR_ARG, "slot %d listed twice", s);
        seen[s] = true;
        sl->slot[b] = s;
    }
    return HIVIS_OK;
}

extern "C" {

const char* hivis_last_error(const hivis_ctx* ctx) { return ctx ? ctx->err : g_init_err; }

int64_t hivis_launch_count(const hivis_ctx* ctx) { return ctx ? ctx->launches : 0; }

int64_t hivis_step_bytes(const hivis_ctx* c, int B, const int* kv_rows_host) {
    if (!c) return 0;
    const hivis_config& g = c->cfg;
    const int64_t d = g.d, F = g.ffn, V = g.vocab;
    int64_t params = 2 * d * d + (int64_t)c->qkvw * d + d * c->qw + 3 * d * F + V * d;
    int64_t bytes = params * (int64_t)c->esize;
    for (int b = 0; b < B; ++b) {
        const int64_t rows = kv_rows_host ? kv_rows_host[b] : 0;
        bytes += 2 * (rows + 1) * c->kvw * (int64_t)c->esize;
    }
    return bytes;
}

int hivis_destroy(hivis_ctx* c) {
    if (!c) return HIVIS_OK;
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    free_all(c);
    delete c;
    return HIVIS_OK;
}

int hivis_init(hivis_ctx** out, const hivis_config* cfg, const hivis_weights* w, void* stream) {
    auto bad = [&](int code, const char* msg) {
        snprintf(g_init_err, sizeof(g_init_err), "%s", msg);
        return code;
    };
    if (!out || !cfg || !w) return bad(HIVIS_ERR_ARG, "null argument");
    *out = nullptr;
    if (cfg->struct_size != sizeof(hivis_config)) return bad(HIVIS_ERR_ARG, "struct_size mismatch");
    if (cfg->dtype != HIVIS_F32 && cfg->dtype != HIVIS_BF16) return bad(HIVIS_ERR_DTYPE, "unknown dtype");
    if (cfg->d < 8 || cfg->d % 8) return bad(HIVIS_ERR_SHAPE, "d must be a positive multiple of 8");
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return bad(HIVIS_ERR_SHAPE, "head_dim must be 64 or 128");
    if (cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads)
        return bad(HIVIS_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
    if (cfg->ffn < 8 || cfg->ffn % 8) return bad(HIVIS_ERR_SHAPE, "ffn must be a positive multiple of 8");
    if (cfg->vocab < 1) return bad(HIVIS_ERR_SHAPE, "vocab must be positive");
    if (cfg->max_batch < 1 || cfg->max_batch > HIVIS_MAX_BATCH) return bad(HIVIS_ERR_CAPACITY, "max_batch out of range");
    if (cfg->max_k < 1 || cfg->max_k > HIVIS_MAX_K) return bad(HIVIS_ERR_CAPACITY, "max_k out of range");
    if (cfg->max_len < 1) return bad(HIVIS_ERR_CAPACITY, "max_len must be positive");
    if (!(cfg->rms_eps >= 0.f) || !(cfg->rope_base > 0.f)) return bad(HIVIS_ERR_ARG, "bad rms_eps / rope_base");
    const void* req[] = {w->embed, w->lm_head, w->fc, w->norm1, w->wq, w->wk, w->wv, w->wo, w->norm2,
                         w->w_gate, w->w_up, w->w_down};
    for (const void* p : req)
        if (!p || misaligned(p)) return bad(HIVIS_ERR_ARG, "a required weight pointer is null or not 16-byte aligned");
    const void* opt[] = {w->bq, w->bk, w->bv, w->resid_proj};
    for (const void* p : opt)
        if (p && misaligned(p)) return bad(HIVIS_ERR_ARG, "an optional weight pointer is not 16-byte aligned");
    const int nb = (w->bq != nullptr) + (w->bk != nullptr) + (w->bv != nullptr);
    if (nb != 0 && nb != 3) return bad(HIVIS_ERR_ARG, "bq, bk, bv must be given together");

    hivis_ctx* c = new (std::nothrow) hivis_ctx();
    if (!c) return bad(HIVIS_ERR_NOMEM, "host allocation failed");
    c->cfg = *cfg;
    c->dtype = cfg->dtype;
    c->esize = cfg->dtype == HIVIS_BF16 ? 2 : 4;
    c->qw = cfg->n_q_heads * cfg->head_dim;
    c->kvw = cfg->n_kv_heads * cfg->head_dim;
    c->qkvw = c->qw + 2 * c->kvw;
    c->rows_cap = cfg->max_batch > TC_OP_ROWS ? cfg->max_batch : TC_OP_ROWS;
    c->launches = 0;
    c->err[0] = 0;
    c->tap_B = 0;
    c->tap_mma = false;
    c->prof_on = false;
    c->prof_n = 0;
    if (cudaGetDevice(&c->device) != cudaSuccess) {
        delete c;
        return bad(HIVIS_ERR_CUDA, "cudaGetDevice failed");
    }
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = c->esize;
    const long long d = cfg->d, F = cfg->ffn, V = cfg->vocab, R = c->rows_cap, MB = cfg->max_batch;
    c->chunk = 128;
    c->nsplit_cap = (cfg->max_len + 31) / 32 + 1;       // blocks of 32 rows, and the rows of the running call
    if (c->nsplit_cap > 513) c->nsplit_cap = 513;
    c->opt_chain = true;
    c->chain_ok = false;
    c->opt_tc = 1;
    c->wait_cycles = 2000000000ll;
    c->debug_skew = false;
    c->tc_ok = false;
    c->tc_partial = nullptr;
    c->opt_phase_times = false;
    c->opt_l2_keep = 0;
    c->opt_tc_prefill = HIVIS_TC_PREFILL_MIN_PAIRS;
    c->pf_ok = false;
    c->pf_xe = c->pf_xq = nullptr;
    c->pf_ssq = nullptr;
    c->phase_t = nullptr;
    c->phase_k = 0;
    c->tile_ctr = nullptr;
    c->tc_tiles = 0;
    c->bar_count_host = 0;
    {
        int coop = 0;
        c->num_sms = 0;
        if (cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess ||
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) != cudaSuccess) {
            cudaGetLastError();
            coop = 0;
        }
        c->chain_ok = coop != 0 && c->num_sms > 0;
        c->chain_ok_coop = c->chain_ok;
    }
    c->key_stride = cfg->max_k + 1;
    c->map_cap = MB * (long long)cfg->max_len;
    const long long tiles1 = (d + HIVIS_MMA_TILE_ROWS - 1) / HIVIS_MMA_TILE_ROWS;

    char *embed, *lm, *fc, *n1, *wqkv, *bqkv = nullptr, *wo, *n2, *wgu, *wdown, *rp = nullptr, *Kc, *Vc;
    bool ok = dalloc(c, &embed, V * d * es) && dalloc(c, &lm, V * d * es) && dalloc(c, &fc, 2 * d * d * es) &&
              dalloc(c, &n1, d * es) && dalloc(c, &wqkv, (long long)c->qkvw * d * es) &&
              dalloc(c, &wo, d * c->qw * es) && dalloc(c, &n2, d * es) && dalloc(c, &wgu, 2 * F * d * es) &&
              dalloc(c, &wdown, d * F * es) &&
              dalloc(c, &Kc, MB * c->kvw * (long long)cfg->max_len * es) &&
              dalloc(c, &Vc, MB * c->kvw * (long long)cfg->max_len * es);
    if (ok && nb) ok = dalloc(c, &bqkv, (long long)c->qkvw * es);
    if (ok && w->resid_proj) ok = dalloc(c, &rp, d * d * es);
    ok = ok && dalloc(c, &c->inv_freq, cfg->head_dim / 2) && dalloc(c, &c->kv_len, MB) &&
         dalloc(c, &c->pend_id, MB) && dalloc(c, &c->pend_feat, MB * d) && dalloc(c, &c->d_slots, R) &&
         dalloc(c, &c->d_pos0, R) && dalloc(c, &c->cur_id, R) && dalloc(c, &c->feat, R * d) &&
         dalloc(c, &c->feat_h, R * d) && dalloc(c, &c->u, R * d) && dalloc(c, &c->xq, R * d) &&
         dalloc(c, &c->qkv, R * c->qkvw) && dalloc(c, &c->attn, R * c->qw) && dalloc(c, &c->attn_h, R * c->qw) &&
         dalloc(c, &c->y, R * d) && dalloc(c, &c->xm, R * d) && dalloc(c, &c->act, R * F) &&
         dalloc(c, &c->act_h, R * F) && dalloc(c, &c->rho_raw, (long long)HIVIS_MAX_K * d) &&
         dalloc(c, &c->rho, (long long)HIVIS_MAX_K * d) && dalloc(c, &c->ssq1, tiles1 * R) &&
         dalloc(c, &c->ssq2, tiles1 * R) && dalloc(c, &c->keys, R * c->key_stride) &&
         dalloc(c, &c->vkeys, MB * (cfg->max_k + 1)) && dalloc(c, &c->varrive, MB) &&
         dalloc(c, &c->vstats, (long long)sampled_stats_entries(cfg->max_batch, cfg->max_k, cfg->vocab)) &&
         dalloc(c, &c->part_acc, R * cfg->n_q_heads * (long long)c->nsplit_cap * cfg->head_dim) &&
         dalloc(c, &c->part_ml, R * cfg->n_q_heads * (long long)c->nsplit_cap * 2) &&
         dalloc(c, &c->counters, R * cfg->n_q_heads) && dalloc(c, &c->bar_counter, 1) &&
         dalloc(c, &c->error_flag, 2) && dalloc(c, &c->slot_of, c->map_cap) &&
         dalloc(c, &c->row_of, c->map_cap) && dalloc(c, &c->xe_h, R * d) &&
         dalloc(c, &c->rope_tab, 2 * 16 * (cfg->head_dim / 2));
    {
        TreeBufs& T = c->tree;
        ok = ok && dalloc(c, &T.P, 1) && dalloc(c, &T.fr_cand, TREE_MAX_TOPK) && dalloc(c, &T.fr_tok, TREE_MAX_TOPK) &&
             dalloc(c, &T.fr_pslot, TREE_MAX_TOPK) && dalloc(c, &T.fr_store, TREE_MAX_TOPK) &&
             dalloc(c, &T.fr_anc, TREE_MAX_TOPK * TREE_MAX_DEPTH) && dalloc(c, &T.fr_score, TREE_MAX_TOPK) &&
             dalloc(c, &T.top_tok, TREE_MAX_TOPK * TREE_MAX_TOPK) && dalloc(c, &T.top_lp, TREE_MAX_TOPK * TREE_MAX_TOPK) &&
             dalloc(c, &T.cand_n, 1) && dalloc(c, &T.cand_tok, TREE_MAX_CAND) && dalloc(c, &T.cand_par, TREE_MAX_CAND) &&
             dalloc(c, &T.cand_depth, TREE_MAX_CAND) && dalloc(c, &T.cand_store, TREE_MAX_CAND) &&
             dalloc(c, &T.cand_keep, TREE_MAX_CAND) && dalloc(c, &T.cand_pos, TREE_MAX_CAND) &&
             dalloc(c, &T.cand_score, TREE_MAX_CAND) && dalloc(c, &T.kept_n, 1) && dalloc(c, &T.kept_tok, HIVIS_TREE_MAX_KEEP) &&
             dalloc(c, &T.kept_par, HIVIS_TREE_MAX_KEEP) && dalloc(c, &T.kept_store, HIVIS_TREE_MAX_KEEP) &&
             dalloc(c, &T.row_keys, HIVIS_TREE_MAX_KEEP + 1) && dalloc(c, &T.piece_stats, (long long)TREE_MAX_TOPK * tree_topk_pieces((int)V)) &&
             dalloc(c, &T.piece_keys, (long long)TREE_MAX_TOPK * tree_topk_pieces((int)V) * TREE_MAX_TOPK) && dalloc(c, &c->tree_logits, (long long)TREE_MAX_TOPK * V) &&
             dalloc(c, &c->tree_g, (long long)TREE_MAX_TOPK * d);
    }
    if (!ok) {
        free_all(c);
        delete c;
        return bad(HIVIS_ERR_NOMEM, "device allocation failed");
    }
    c->embed = embed; c->lm_head = lm; c->fc = fc; c->norm1 = n1; c->wqkv = wqkv; c->bqkv = bqkv;
    c->wo = wo; c->norm2 = n2; c->wgu = wgu; c->wdown = wdown; c->resid_proj = rp; c->Kc = Kc; c->Vc = Vc;
    c->id_flag = c->error_flag + 1;

    int rc = HIVIS_OK;
    auto run = [&]() -> int {
        CK(c, cudaMemcpyAsync(embed, w->embed, V * d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(lm, w->lm_head, V * d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(fc, w->fc, 2 * d * d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(n1, w->norm1, d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(n2, w->norm2, d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(wo, w->wo, d * c->qw * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(wdown, w->w_down, d * F * es, cudaMemcpyDeviceToDevice, st));
        // q | k | v rows stacked into one matrix
        CK(c, cudaMemcpyAsync(wqkv, w->wq, (long long)c->qw * d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(wqkv + (long long)c->qw * d * es, w->wk, (long long)c->kvw * d * es, cudaMemcpyDeviceToDevice, st));
        CK(c, cudaMemcpyAsync(wqkv + (long long)(c->qw + c->kvw) * d * es, w->wv, (long long)c->kvw * d * es, cudaMemcpyDeviceToDevice, st));
        if (nb) {
            CK(c, cudaMemcpyAsync(bqkv, w->bq, c->qw * es, cudaMemcpyDeviceToDevice, st));
            CK(c, cudaMemcpyAsync(bqkv + c->qw * es, w->bk, c->kvw * es, cudaMemcpyDeviceToDevice, st));
            CK(c, cudaMemcpyAsync(bqkv + (c->qw + c->kvw) * es, w->bv, c->kvw * es, cudaMemcpyDeviceToDevice, st));
        }
        if (rp) CK(c, cudaMemcpyAsync(rp, w->resid_proj, d * d * es, cudaMemcpyDeviceToDevice, st));
        // gate and up rows interleaved: row 2i = gate_i, row 2i+1 = up_i
        CKL(c, launch_copy_rows(w->w_gate, wgu, F, d * es, 0, 2, st));
        CKL(c, launch_copy_rows(w->w_up, wgu, F, d * es, 1, 2, st));
        std::vector<double> inv(cfg->head_dim / 2);
        for (int i = 0; i < cfg->head_dim / 2; ++i)
            inv[i] = std::pow((double)cfg->rope_base, -2.0 * i / cfg->head_dim);
        CK(c, cudaMemcpyAsync(c->inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice, st));
        CK(c, cudaStreamSynchronize(st));          // inv lives on this stack frame
        CK(c, cudaMemsetAsync(c->kv_len, 0, MB * sizeof(int), st));
        CK(c, cudaMemsetAsync(c->pend_id, 0, MB * sizeof(int), st));
        CK(c, cudaMemsetAsync(c->counters, 0, R * cfg->n_q_heads * sizeof(int), st));
        CK(c, cudaMemsetAsync(c->bar_counter, 0, sizeof(u64), st));
        CK(c, cudaMemsetAsync(c->error_flag, 0, 2 * sizeof(int), st));
        CK(c, cudaMemsetAsync(c->vkeys, 0, MB * (cfg->max_k + 1) * sizeof(u64), st));
        CK(c, cudaMemsetAsync(c->varrive, 0, MB * sizeof(int), st));
        CK(c, cudaMemsetAsync(c->xe_h, 0, R * d * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->feat_h, 0, R * d * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->xq, 0, R * d * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->attn_h, 0, R * c->qw * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->xm, 0, R * d * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->act_h, 0, R * F * sizeof(bf16), st));
        CK(c, cudaMemsetAsync(c->Kc, 0, MB * c->kvw * (long long)cfg->max_len * es, st));
        CK(c, cudaMemsetAsync(c->Vc, 0, MB * c->kvw * (long long)cfg->max_len * es, st));
        return HIVIS_OK;
    };
    rc = run();
    if (rc != HIVIS_OK) {
        snprintf(g_init_err, sizeof(g_init_err), "%s", c->err);
        free_all(c);
        delete c;
        return rc;
    }
    if (c->chain_ok) {
        ChainArgs ca;
        fill_chain_args(c, &ca);
        c->chain_ok = chain_smem_bytes(ca, c->dtype, c->num_sms) != 0;
    }
    if (c->dtype == HIVIS_BF16 && c->num_sms > 0 && c->chain_ok_coop && (cfg->max_len + 31) / 32 + 1 <= c->nsplit_cap &&
        tc_supported(cfg->d, cfg->head_dim, cfg->n_q_heads, cfg->n_kv_heads, cfg->ffn)) {
        ChainArgs ca;
        fill_chain_args(c, &ca);
        c->tc_tiles = tc_max_tiles(ca.ph);
        bool ok2 = dalloc(c, &c->tc_partial, (size_t)c->num_sms * 2 * 16 * 128) && dalloc(c, &c->tile_ctr, c->tc_tiles) &&
                   dalloc(c, &c->phase_t, (size_t)HIVIS_MAX_K * HIVIS_PHASE_EVENTS * c->num_sms);
        if (ok2) ok2 = cudaMemsetAsync(c->tile_ctr, 0, c->tc_tiles * sizeof(int), st) == cudaSuccess;
        if (ok2)
            ok2 = tc_build_maps(&c->tc_maps, ca.ph, cfg->d, c->qw, cfg->ffn, c->feat_h, c->xq, c->attn_h, c->xm, c->act_h,
                                c->xe_h, c->Kc, c->Vc, MB * (long long)cfg->n_kv_heads * cfg->max_len,
                                cfg->head_dim) == cudaSuccess;
        if (!ok2) cudaGetLastError();
        c->tc_ok = ok2;
    }
    if (c->dtype == HIVIS_BF16 && prefill_tc_supported(cfg->d, c->kvw)) {
        c->pf_ok = dalloc(c, &c->pf_xe, (size_t)c->map_cap * d) && dalloc(c, &c->pf_xq, (size_t)c->map_cap * d) &&
                   dalloc(c, &c->pf_ssq, (size_t)((d + 127) / 128) * c->map_cap) &&
                   dalloc(c, &c->pf_rope, (size_t)c->map_cap * (cfg->head_dim / 2));
    }
    for (int s = 0; s < HIVIS_MAX_BATCH; ++s) {
        c->kv_upper[s] = 0;
        c->kv_exact[s] = true;
        c->pending[s] = false;
        c->have_pair[s] = false;
        c->last_k[s] = 0;
        c->tree_depth[s] = 0;
        c->tree_count[s] = 0;
    }
    *out = c;
    return HIVIS_OK;
}

// residual rows in the context dtype -> fp32 rho rows (projected by resid_proj when present)
static int prepare_rho(hivis_ctx* c, const void* resid, int R, cudaStream_t st) {
    const int d = c->cfg.d;
    float* dst = c->resid_proj ? c->rho_raw : c->rho;
    CKL(c, launch_convert_rows(c->dtype, resid, dst, (long long)R * d, st));
    if (c->resid_proj) {
        LinArgs a;
        memset(&a, 0, sizeof(a));
        a.W = c->resid_proj; a.N = d; a.K = d; a.B = R; a.ldb = c->rows_cap;
        a.xin = c->rho_raw; a.out = c->rho;
        CKL(c, launch_gemv_alu(c->dtype, PRO_PLAIN, EPI_QKV, a, st));
    }
    return HIVIS_OK;
}

// Split the cache rows of the longest listed sequence: `want` splits if possible, at least 32 rows
// per split, never more splits than the partial buffers hold.
static void plan_attention(const hivis_ctx* c, int max_rows, int want, int* chunk, int* nsplit) {
    if (want > c->nsplit_cap) want = c->nsplit_cap;
    if (want < 1) want = 1;
    int ch = (max_rows + want - 1) / want;
    ch = (ch + 31) / 32 * 32;
    if (ch < 32) ch = 32;
    *chunk = ch;
    *nsplit = (max_rows + ch - 1) / ch;
}

static void fill_chain_args(hivis_ctx* c, ChainArgs* a) {
    const hivis_config& g = c->cfg;
    memset(a, 0, sizeof(*a));
    a->ph[PH_FC] = {c->fc, g.d, 2 * g.d};
    a->ph[PH_QKV] = {c->wqkv, c->qkvw, g.d};
    a->ph[PH_O] = {c->wo, g.d, c->qw};
    a->ph[PH_GU] = {c->wgu, 2 * g.ffn, g.d};
    a->ph[PH_DOWN] = {c->wdown, g.d, g.ffn};
    a->ph[PH_LM] = {c->lm_head, g.vocab, g.d};
    a->d = g.d; a->qw = c->qw; a->kvw = c->kvw; a->F = g.ffn; a->V = g.vocab; a->Hq = g.n_q_heads;
    a->Hkv = g.n_kv_heads; a->dh = g.head_dim; a->max_len = g.max_len; a->eps = g.rms_eps;
    a->scale = 1.0f / sqrtf((float)g.head_dim);
    a->norm1 = c->norm1; a->norm2 = c->norm2; a->bqkv = c->bqkv; a->embed = c->embed;
    a->kv_len = c->kv_len; a->pend_feat = c->pend_feat; a->pend_id = c->pend_id;
    a->u = c->u; a->qkv = c->qkv; a->attn = c->attn; a->y = c->y; a->act = c->act; a->feat = c->feat;
    a->keys = c->keys; a->Kc = c->Kc; a->Vc = c->Vc; a->inv_freq = c->inv_freq;
    a->part_acc = c->part_acc; a->part_ml = c->part_ml; a->counters = c->counters;
    a->bar_counter = c->bar_counter; a->error_flag = c->error_flag; a->id_flag = c->id_flag;
}

static bool use_mma(const hivis_ctx* c, int B, bool prefill) {
    return c->dtype == HIVIS_BF16 && (prefill || B >= 2);
}

// fusion FC for rows [b0, b0+nb): u, gamma1*u (bf16), partial sums of squares
static int run_fuse(hivis_ctx* c, bool mma, int b0, int nb, const float* feat, const void* feat_h,
                    const int* ids, int id_stride, const u64* keys, const float* rho, cudaStream_t st) {
    const int d = c->cfg.d;
    LinArgs a;
    memset(&a, 0, sizeof(a));
    a.W = c->fc; a.N = d; a.K = 2 * d; a.B = nb; a.ldb = c->rows_cap; a.d = d;
    a.feat = feat; a.feat_h = feat_h; a.embed = c->embed; a.vocab = c->cfg.vocab; a.id_flag = c->id_flag;
    a.ids = ids; a.id_stride = id_stride; a.keys = keys; a.key_stride = c->key_stride;
    a.rho = rho;
    a.out = c->u + (long long)b0 * d;
    if (mma) {
        a.out_h = c->xq + (long long)b0 * d;
        a.gamma_out = c->norm1;
        a.ssq_out = c->ssq1 + b0;
        CKP(c, CLS_FUSE, st, launch_gemm_mma(PRO_FUSE, EPI_FUSE, a, st));
    } else {
        CKP(c, CLS_FUSE, st, launch_gemv_alu(c->dtype, PRO_FUSE, EPI_FUSE, a, st));
    }
    return HIVIS_OK;
}

// RMSNorm + projection rows [row0, row0+N) of the stacked QKV matrix
static int run_qkv(hivis_ctx* c, bool mma, int b0, int nb, int row0, int N, float* out, cudaStream_t st) {
    const int d = c->cfg.d;
    LinArgs a;
    memset(&a, 0, sizeof(a));
    a.W = (const char*)c->wqkv + (long long)row0 * d * c->esize;
    a.N = N; a.K = d; a.B = nb; a.ldb = c->rows_cap; a.eps = c->cfg.rms_eps;
    a.bias = c->bqkv ? (const char*)c->bqkv + (long long)row0 * c->esize : nullptr;
    a.out = out;
    if (mma) {
        a.xin_h = c->xq + (long long)b0 * d;
        a.ssq_in = c->ssq1 + b0;
        a.ssq_tiles = (d + HIVIS_MMA_TILE_ROWS - 1) / HIVIS_MMA_TILE_ROWS;
        CKP(c, CLS_QKV, st, launch_gemm_mma(PRO_PLAIN, EPI_QKV, a, st));
    } else {
        a.xin = c->u + (long long)b0 * d;
        a.gamma = c->norm1;
        CKP(c, CLS_QKV, st, launch_gemv_alu(c->dtype, PRO_NORM, EPI_QKV, a, st));
    }
    return HIVIS_OK;
}

// Rows [b0, b0+nb) after the attention: O projection + residual, RMSNorm + gate/up + SiLU * up, down projection +
// residual (-> feat, the layer output), LM head + argmax keys (logits written too when asked for).
static int run_after_attention(hivis_ctx* c, bool mma, int b0, int nb, u64* keys_out, int keys_out_stride,
                               float* logits_out, long long logits_ld, cudaStream_t st) {
    const hivis_config& g = c->cfg;
    const int d = g.d, F = g.ffn, V = g.vocab;
    const int tiles1 = (d + HIVIS_MMA_TILE_ROWS - 1) / HIVIS_MMA_TILE_ROWS;
    LinArgs a;
    // ---- O projection + residual
    memset(&a, 0, sizeof(a));
    a.W = c->wo; a.N = d; a.K = c->qw; a.B = nb; a.ldb = c->rows_cap;
    a.addend = c->u + (long long)b0 * d; a.out = c->y + (long long)b0 * d;
    if (mma) {
        a.xin_h = c->attn_h + (long long)b0 * c->qw;
        a.out_h = c->xm + (long long)b0 * d; a.gamma_out = c->norm2; a.ssq_out = c->ssq2 + b0;
        CKP(c, CLS_OPROJ, st, launch_gemm_mma(PRO_PLAIN, EPI_OPROJ, a, st));
    } else {
        a.xin = c->attn + (long long)b0 * c->qw;
        CKP(c, CLS_OPROJ, st, launch_gemv_alu(c->dtype, PRO_PLAIN, EPI_OPROJ, a, st));
    }
    // ---- RMSNorm + gate/up + SiLU * up
    memset(&a, 0, sizeof(a));
    a.W = c->wgu; a.N = 2 * F; a.K = d; a.B = nb; a.ldb = c->rows_cap; a.eps = g.rms_eps;
    if (mma) {
        a.xin_h = c->xm + (long long)b0 * d; a.ssq_in = c->ssq2 + b0; a.ssq_tiles = tiles1;
        a.out_h = c->act_h + (long long)b0 * F;
        CKP(c, CLS_GATEUP, st, launch_gemm_mma(PRO_PLAIN, EPI_GATEUP, a, st));
    } else {
        a.xin = c->y + (long long)b0 * d; a.gamma = c->norm2; a.out = c->act + (long long)b0 * F;
        CKP(c, CLS_GATEUP, st, launch_gemv_alu(c->dtype, PRO_NORM, EPI_GATEUP, a, st));
    }
    // ---- down projection + residual -> g, carried to the next step as its feature
    memset(&a, 0, sizeof(a));
    a.W = c->wdown; a.N = d; a.K = F; a.B = nb; a.ldb = c->rows_cap;
    a.addend = c->y + (long long)b0 * d; a.out = c->feat + (long long)b0 * d;
    a.out_h = c->feat_h + (long long)b0 * d;
    if (mma) {
        a.xin_h = c->act_h + (long long)b0 * F;
        CKP(c, CLS_DOWN, st, launch_gemm_mma(PRO_PLAIN, EPI_DOWN, a, st));
    } else {
        a.xin = c->act + (long long)b0 * F;
        CKP(c, CLS_DOWN, st, launch_gemv_alu(c->dtype, PRO_PLAIN, EPI_DOWN, a, st));
    }
    // ---- LM head + argmax
    memset(&a, 0, sizeof(a));
    a.W = c->lm_head; a.N = V; a.K = d; a.B = nb; a.ldb = c->rows_cap;
    a.keys_out = keys_out; a.keys_out_stride = keys_out_stride;
    a.logits_out = logits_out;
    a.logits_ld = logits_ld;
    if (mma) {
        a.xin_h = c->feat_h + (long long)b0 * d;
        CKP(c, CLS_LM, st, launch_gemm_mma(PRO_PLAIN, EPI_LM, a, st));
    } else {
        a.xin = c->feat + (long long)b0 * d;
        CKP(c, CLS_LM, st, launch_gemv_alu(c->dtype, PRO_PLAIN, EPI_LM, a, st));
    }
    return HIVIS_OK;
}

int hivis_prefill(hivis_ctx* c, int B, const int* seq_slots_host, const int32_t* ids, const void* hidden,
                  const int32_t* cu_seqlens_host, const int32_t* start_pos_host, const void* resid0,
                  void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    SlotList sl, start;
    int rc = check_slots(c, B, seq_slots_host, &sl);
    if (rc) return rc;
    if (!ids || !hidden || !cu_seqlens_host) return fail(c, HIVIS_ERR_ARG, "null argument");
    if (misaligned(ids) || misaligned(hidden) || (resid0 && misaligned(resid0)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (cu_seqlens_host[0] != 0) return fail(c, HIVIS_ERR_ARG, "cu_seqlens must start at 0");
    CuSeqlens cu;
    start.n = B;
    int new_upper[HIVIS_MAX_BATCH];
    for (int b = 0; b < B; ++b) {
        const int T = cu_seqlens_host[b + 1] - cu_seqlens_host[b];
        if (T < 1) return fail(c, HIVIS_ERR_ARG, "sequence %d has no entries", b);
        const int s = sl.slot[b];
        int base = c->kv_upper[s];
        start.slot[b] = -1;
        if (!start_pos_host && c->pending[s])
            return fail(c, HIVIS_ERR_STATE, "slot %d still holds a pending pair whose K/V row was never cached: draft it "
                        "first, or pass start_pos to rebuild the rows from there", s);
        if (start_pos_host) {
            if (start_pos_host[b] < 0 || start_pos_host[b] > c->kv_upper[s])
                return fail(c, HIVIS_ERR_ARG, "start_pos %d outside [0,%d]", start_pos_host[b], c->kv_upper[s]);
            base = start_pos_host[b];
            start.slot[b] = base;
        }
        if (base + T - 1 > c->cfg.max_len)
            return fail(c, HIVIS_ERR_CAPACITY, "slot %d would hold %d rows > max_len %d", s, base + T - 1, c->cfg.max_len);
        new_upper[b] = base + T - 1;
        cu.v[b] = cu_seqlens_host[b];
    }
    cu.v[B] = cu_seqlens_host[B];
    const long long total = cu.v[B];
    if (total > c->map_cap) return fail(c, HIVIS_ERR_CAPACITY, "packed batch too long");
    cudaStream_t st = (cudaStream_t)stream;
    const int d = c->cfg.d;
    const float* rho0 = nullptr;
    if (resid0) {
        rc = prepare_rho(c, resid0, 1, st);
        if (rc) return rc;
        rho0 = c->rho;
    }
    CKL(c, launch_prefill_setup(c->dtype, sl, cu, start, d, ids, hidden, c->kv_len, c->pend_feat, c->pend_id,
                                c->slot_of, c->row_of, st));
    if (c->pf_ok && c->opt_tc_prefill > 0 && total >= c->opt_tc_prefill) {
        // many pairs: the two GEMMs of the prefix build on the tensor cores, all pairs in one pass
        PrefillTcArgs a;
        memset(&a, 0, sizeof(a));
        a.n_pairs = (int)total; a.pair_cap = (int)c->map_cap;
        a.d = d; a.kvw = c->kvw; a.Hkv = c->cfg.n_kv_heads; a.dh = c->cfg.head_dim; a.max_len = c->cfg.max_len;
        a.vocab = c->cfg.vocab; a.eps = c->cfg.rms_eps;
        a.ids = ids; a.hidden = (const bf16*)hidden; a.embed = (const bf16*)c->embed; a.fc = (const bf16*)c->fc;
        a.wkv = (const bf16*)c->wqkv + (long long)c->qw * d;
        a.bkv = c->bqkv ? (const bf16*)c->bqkv + c->qw : nullptr;
        a.norm1 = (const bf16*)c->norm1; a.rho0 = rho0;
        a.xe = c->pf_xe; a.xq = c->pf_xq; a.ssq = c->pf_ssq; a.rope = c->pf_rope;
        a.slot_of = c->slot_of; a.row_of = c->row_of; a.inv_freq = c->inv_freq;
        a.Kc = (bf16*)c->Kc; a.Vc = (bf16*)c->Vc;
        a.wait_cycles = c->wait_cycles; a.error_flag = c->error_flag; a.id_flag = c->id_flag;
        CK(c, launch_prefill_tc(a, st));
        c->launches += 4;
    } else {
    const bool mma = use_mma(c, 16, true);
    for (long long j0 = 0; j0 < total; j0 += 16) {
        const int P = (int)(total - j0 < 16 ? total - j0 : 16);
        const char* hid = (const char*)hidden + j0 * d * c->esize;
        rc = run_fuse(c, mma, 0, P, mma ? nullptr : (const float*)hid, mma ? hid : nullptr, ids + j0, 1, nullptr,
                      rho0, st);
        if (rc) return rc;
        rc = run_qkv(c, mma, 0, P, c->qw, 2 * c->kvw, c->qkv, st);   // K and V rows only
        if (rc) return rc;
        CKL(c, launch_kv_append(c->dtype, c->qkv, P, c->slot_of + j0, c->row_of + j0, c->inv_freq,
                                c->cfg.n_kv_heads, c->cfg.head_dim, c->cfg.max_len, c->Kc, c->Vc, st));
    }
    }
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        c->kv_exact[s] = c->kv_exact[s] || start_pos_host != nullptr;
        c->kv_upper[s] = new_upper[b];
        c->pending[s] = true;
        c->have_pair[s] = true;
        c->last_k[s] = 0;
    }
    return HIVIS_OK;
}

// Arguments of the tensor-core chain kernel for B columns and k steps (the whole step; callers narrow seq_first /
// seq_last and bar_base when they run a part of it).
static void fill_tc_args(hivis_ctx* c, TcArgs* out, int B, int k, int lo, const float* rho, int n_resid,
                         const int32_t* forced_ids, float* out_logits) {
    const hivis_config& g = c->cfg;
    ChainArgs ca;
    fill_chain_args(c, &ca);
    TcArgs& a = *out;
    memset(&a, 0, sizeof(a));
    for (int p = 0; p < PH_COUNT; ++p) a.ph[p] = ca.ph[p];
    a.k = k; a.B = B; a.lo = lo;
    a.d = g.d; a.qw = c->qw; a.kvw = c->kvw; a.F = g.ffn; a.V = g.vocab; a.Hq = g.n_q_heads; a.Hkv = g.n_kv_heads;
    a.dh = g.head_dim; a.max_len = g.max_len; a.eps = g.rms_eps; a.scale = 1.0f / sqrtf((float)g.head_dim);
    a.norm1 = (const bf16*)c->norm1; a.norm2 = (const bf16*)c->norm2; a.bqkv = (const bf16*)c->bqkv;
    a.rho = rho; a.n_resid = n_resid;
    a.slots = c->d_slots; a.pos0 = c->d_pos0; a.cur_id = c->cur_id; a.forced = forced_ids;
    a.keys = c->keys; a.key_stride = c->key_stride;
    a.u = c->u; a.qkv = c->qkv; a.attn = c->attn; a.y = c->y; a.feat = c->feat;
    a.feat_h = c->feat_h; a.xq_h = c->xq; a.attn_h = c->attn_h; a.xm_h = c->xm; a.act_h = c->act_h;
    a.xe_h = c->xe_h; a.embed = (const bf16*)c->embed; a.rope_tab = c->rope_tab;
    a.ssq1 = c->ssq1; a.ssq2 = c->ssq2; a.logits_out = out_logits;
    a.partial = c->tc_partial; a.tile_ctr = c->tile_ctr;
    a.Kc = c->Kc; a.Vc = c->Vc; a.inv_freq = c->inv_freq; a.part_acc = c->part_acc; a.part_ml = c->part_ml;
    a.counters = c->counters;
    a.attn_nslot = c->nsplit_cap;
    a.bar_counter = c->bar_counter; a.bar_base = c->bar_count_host + (c->debug_skew ? (1ull << 40) : 0ull);
    a.wait_cycles = c->wait_cycles; a.error_flag = c->error_flag; a.id_flag = c->id_flag;
    a.l2_keep = c->opt_l2_keep;
    a.phase_t = nullptr;
    a.seq_first = 0; a.seq_last = 7;
}

// hivis_draft and hivis_draft_sampled (uniforms != nullptr: every step's token is drawn with the Gumbel-max rule)
static int draft_impl(hivis_ctx* c, int B, const int* seq_slots_host, int k, const void* resid, int n_resid,
                      int32_t* out_ids, const int32_t* forced_ids, float* out_logits, float inv_t, const float* uniforms,
                      void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    SlotList sl;
    int rc = check_slots(c, B, seq_slots_host, &sl);
    if (rc) return rc;
    if (!out_ids) return fail(c, HIVIS_ERR_ARG, "out_ids is null");
    if (misaligned(out_ids) || (forced_ids && misaligned(forced_ids)) || (out_logits && misaligned(out_logits)) ||
        (resid && misaligned(resid)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (k < 1 || k > c->cfg.max_k) return fail(c, HIVIS_ERR_CAPACITY, "k=%d outside [1,%d]", k, c->cfg.max_k);
    if (resid && (n_resid < 1 || n_resid > HIVIS_MAX_K)) return fail(c, HIVIS_ERR_ARG, "n_resid=%d outside [1,%d]", n_resid, HIVIS_MAX_K);
    int max_rows = 0;
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        if (!c->pending[s]) return fail(c, HIVIS_ERR_STATE, "slot %d has no pending pair", s);
        if (c->kv_upper[s] + k > c->cfg.max_len)
            return fail(c, HIVIS_ERR_CAPACITY, "slot %d: %d rows + k=%d > max_len %d", s, c->kv_upper[s], k, c->cfg.max_len);
        if (c->kv_upper[s] + k > max_rows) max_rows = c->kv_upper[s] + k;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const hivis_config& g = c->cfg;
    const int d = g.d, F = g.ffn, V = g.vocab;
    if (resid) {
        rc = prepare_rho(c, resid, n_resid, st);
        if (rc) return rc;
    }
    if (B == 1 && c->opt_chain && c->chain_ok && !(c->tc_ok && c->opt_tc == 2)) {
        // one sequence: all k steps in one persistent cooperative kernel
        ChainArgs a;
        fill_chain_args(c, &a);
        a.k = k;
        a.rho = resid ? c->rho : nullptr;
        a.n_resid = resid ? n_resid : 1;
        a.slot = sl.slot[0];
        a.forced = forced_ids;
        a.logits_out = out_logits;
        a.gumbel_u = uniforms;
        a.inv_t = inv_t;
        a.out_ids = out_ids;
        plan_attention(c, max_rows, c->num_sms / g.n_q_heads, &a.attn_chunk, &a.attn_nsplit);
        a.bar_base = c->bar_count_host + (c->debug_skew ? (1ull << 40) : 0ull);
        a.wait_cycles = c->wait_cycles;
        c->debug_skew = false;
        CKP(c, CLS_CHAIN, st, launch_draft_chain(a, c->dtype, c->num_sms, st));
        c->bar_count_host += (u64)c->num_sms * (u64)(chain_barriers_per_step() * k);
        const int s0 = sl.slot[0];
        c->kv_upper[s0] += k;
        c->pending[s0] = false;
        c->last_k[s0] = k;
        c->tap_B = 1;
        c->tap_mma = false;
        return HIVIS_OK;
    }
    if (c->tc_ok && c->opt_tc != 0 && B <= 16) {
        // bf16, up to 16 sequences: all k steps in one cooperative tensor-core kernel
        const int lo = tc_lo_offset(B);
        CKP(c, CLS_OTHER, st, launch_tc_setup(sl, k, d, lo, c->d_slots, c->d_pos0, c->kv_len, c->pend_feat, c->pend_id,
                                              c->feat, c->feat_h, c->cur_id, c->keys, c->key_stride, (const bf16*)c->embed,
                                              V, c->xe_h, c->id_flag, st));
        TcArgs a;
        fill_tc_args(c, &a, B, k, lo, resid ? c->rho : nullptr, resid ? n_resid : 1, forced_ids, out_logits);
        a.gumbel_u = uniforms;
        a.inv_t = inv_t;
        if (c->opt_phase_times) {
            CK(c, cudaMemsetAsync(c->phase_t, 0, (size_t)k * HIVIS_PHASE_EVENTS * c->num_sms * sizeof(u64), st));
            a.phase_t = c->phase_t;
            c->phase_k = k;
        }
        c->debug_skew = false;
        CKP(c, CLS_CHAIN, st, launch_tc_chain(c->tc_maps, a, c->num_sms, st));
        c->bar_count_host += (u64)c->num_sms * (u64)(tc_barriers_per_step() * k);
        CKP(c, CLS_OTHER, st, launch_draft_finish(B, k, c->keys, c->key_stride, out_ids, st));
        for (int b = 0; b < B; ++b) {
            const int s = sl.slot[b];
            c->kv_upper[s] += k;
            c->pending[s] = false;
            c->last_k[s] = k;
        }
        c->tap_B = B;
        c->tap_mma = true;
        return HIVIS_OK;
    }
    if (uniforms)
        return fail(c, HIVIS_ERR_SHAPE, "drawing the drafted tokens runs in the chain kernels only: one sequence, or up to 16 "
                    "sequences of a bf16 context with the kernels switched on");
    CKP(c, CLS_OTHER, st, launch_draft_setup(sl, k, d, c->d_slots, c->d_pos0, c->kv_len, c->pend_feat, c->pend_id, c->feat,
                              c->feat_h, c->cur_id, c->keys, c->key_stride, st));
    const bool mma = use_mma(c, B, false);
    int chunk = 0, nsplit = 0;
    plan_attention(c, max_rows, (max_rows + c->chunk - 1) / c->chunk, &chunk, &nsplit);
    const int tiles1 = (d + HIVIS_MMA_TILE_ROWS - 1) / HIVIS_MMA_TILE_ROWS;
    const int bstep = mma ? 16 : B;
    for (int s = 0; s < k; ++s) {
        const float* rho = resid ? c->rho + (long long)(s < n_resid - 1 ? s : n_resid - 1) * d : nullptr;
        // ---- fuse + residual
        for (int b0 = 0; b0 < B; b0 += bstep) {
            const int nb = B - b0 < bstep ? B - b0 : bstep;
            const int* idp = nullptr;
            int idst = 1;
            const u64* keyp = nullptr;
            if (s == 0) idp = c->cur_id + b0;
            else if (forced_ids) { idp = forced_ids + (long long)b0 * k + (s - 1); idst = k; }
            else keyp = c->keys + (long long)b0 * c->key_stride + (s - 1);
            rc = run_fuse(c, mma, b0, nb, c->feat + (long long)b0 * d, c->feat_h + (long long)b0 * d, idp, idst,
                          keyp, rho, st);
            if (rc) return rc;
            // ---- RMSNorm + QKV
            rc = run_qkv(c, mma, b0, nb, 0, c->qkvw, c->qkv + (long long)b0 * c->qkvw, st);
            if (rc) return rc;
        }
        // ---- RoPE, KV append, attention over the text-only cache
        {
            AttnArgs a;
            memset(&a, 0, sizeof(a));
            a.qkv = c->qkv; a.ld = c->qkvw; a.Kc = c->Kc; a.Vc = c->Vc; a.slots = c->d_slots; a.pos0 = c->d_pos0;
            a.step = s; a.inv_freq = c->inv_freq; a.Hq = g.n_q_heads; a.Hkv = g.n_kv_heads; a.dh = g.head_dim;
            a.max_len = g.max_len; a.B = B; a.scale = 1.0f / sqrtf((float)g.head_dim); a.chunk = chunk;
            a.nsplit = nsplit; a.part_acc = c->part_acc; a.part_ml = c->part_ml; a.counters = c->counters;
            a.attn = c->attn; a.attn_h = c->attn_h;
            CKP(c, CLS_ATTN, st, launch_attention(c->dtype, a, st));
        }
        for (int b0 = 0; b0 < B; b0 += bstep) {
            const int nb = B - b0 < bstep ? B - b0 : bstep;
            rc = run_after_attention(c, mma, b0, nb, c->keys + (long long)b0 * c->key_stride + s, c->key_stride,
                                     out_logits ? out_logits + ((long long)b0 * k + s) * V : nullptr, (long long)k * V, st);
            if (rc) return rc;
        }
    }
    CKP(c, CLS_OTHER, st, launch_draft_finish(B, k, c->keys, c->key_stride, out_ids, st));
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        c->kv_upper[s] += k;
        c->pending[s] = false;
        c->last_k[s] = k;
    }
    c->tap_B = B;
    c->tap_mma = mma;
    return HIVIS_OK;
}

int hivis_draft(hivis_ctx* c, int B, const int* seq_slots_host, int k, const void* resid, int n_resid,
                int32_t* out_ids, const int32_t* forced_ids, float* out_logits, void* stream) {
    return draft_impl(c, B, seq_slots_host, k, resid, n_resid, out_ids, forced_ids, out_logits, 0.f, nullptr, stream);
}

int hivis_draft_sampled(hivis_ctx* c, int B, const int* seq_slots_host, int k, const void* resid, int n_resid,
                        float temperature, const float* uniforms, int32_t* out_ids, float* out_logits, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (!uniforms || misaligned(uniforms)) return fail(c, HIVIS_ERR_ARG, "uniforms is null or not 16-byte aligned");
    if (!(temperature > 0.f)) return fail(c, HIVIS_ERR_ARG, "temperature must be positive");
    return draft_impl(c, B, seq_slots_host, k, resid, n_resid, out_ids, nullptr, out_logits, 1.0f / temperature, uniforms,
                      stream);
}

int hivis_verify(hivis_ctx* c, int B, const int* seq_slots_host, int k, const int32_t* draft_ids,
                 const void* target_logits, int logits_dtype, int32_t* out_accept, int32_t* out_next,
                 int32_t* out_kv_len, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    SlotList sl;
    int rc = check_slots(c, B, seq_slots_host, &sl);
    if (rc) return rc;
    if (!draft_ids || !target_logits || !out_accept || !out_next) return fail(c, HIVIS_ERR_ARG, "null argument");
    if (misaligned(draft_ids) || misaligned(target_logits) || misaligned(out_accept) || misaligned(out_next) ||
        (out_kv_len && misaligned(out_kv_len)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (logits_dtype != HIVIS_F32 && logits_dtype != HIVIS_BF16) return fail(c, HIVIS_ERR_DTYPE, "unknown logits dtype");
    if (k < 1 || k > c->cfg.max_k) return fail(c, HIVIS_ERR_CAPACITY, "k=%d outside [1,%d]", k, c->cfg.max_k);
    for (int b = 0; b < B; ++b)
        if (c->last_k[sl.slot[b]] != k)
            return fail(c, HIVIS_ERR_STATE, "slot %d: verify(k=%d) must follow a draft of the same k", sl.slot[b], k);
    cudaStream_t st = (cudaStream_t)stream;
    int nl = 0;
    CK(c, launch_verify(logits_dtype, sl, k, c->cfg.vocab, draft_ids, target_logits, c->vkeys, c->varrive, c->kv_len,
                        out_accept, out_next, out_kv_len, st, &nl));
    c->launches += nl;
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        c->last_k[s] = 0;
        c->kv_exact[s] = false;          // between pairs and pairs + k - 1 until read back
    }
    return HIVIS_OK;
}

int hivis_verify_sampled(hivis_ctx* c, int B, const int* seq_slots_host, int k, const int32_t* draft_ids,
                         const float* draft_logits, const void* target_logits, int logits_dtype, float temperature,
                         const float* u_accept, const float* u_sample, int32_t* out_accept, int32_t* out_next,
                         int32_t* out_kv_len, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    SlotList sl;
    int rc = check_slots(c, B, seq_slots_host, &sl);
    if (rc) return rc;
    if (!draft_ids || !draft_logits || !target_logits || !u_accept || !u_sample || !out_accept || !out_next)
        return fail(c, HIVIS_ERR_ARG, "null argument");
    if (misaligned(draft_ids) || misaligned(draft_logits) || misaligned(target_logits) || misaligned(u_accept) ||
        misaligned(u_sample) || misaligned(out_accept) || misaligned(out_next) || (out_kv_len && misaligned(out_kv_len)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (logits_dtype != HIVIS_F32 && logits_dtype != HIVIS_BF16) return fail(c, HIVIS_ERR_DTYPE, "unknown logits dtype");
    if (!(temperature > 0.f)) return fail(c, HIVIS_ERR_ARG, "temperature must be positive");
    if (k < 1 || k > c->cfg.max_k) return fail(c, HIVIS_ERR_CAPACITY, "k=%d outside [1,%d]", k, c->cfg.max_k);
    for (int b = 0; b < B; ++b)
        if (c->last_k[sl.slot[b]] != k)
            return fail(c, HIVIS_ERR_STATE, "slot %d: verification (k=%d) must follow a draft of the same k", sl.slot[b], k);
    CK(c, launch_verify_sampled(logits_dtype, sl, k, c->cfg.vocab, temperature, draft_ids, draft_logits, target_logits,
                                c->vstats, u_accept, u_sample, c->kv_len, out_accept, out_next, out_kv_len,
                                (cudaStream_t)stream));
    c->launches += 2;
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        c->last_k[s] = 0;
        c->kv_exact[s] = false;
    }
    return HIVIS_OK;
}

int hivis_draft_tree(hivis_ctx* c, int slot, int topk, int depth, int keep, const void* resid, int n_resid,
                     int32_t* out_tokens, int32_t* out_parents, float* out_scores, int32_t* out_count, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    if (!out_tokens || !out_parents || !out_scores || !out_count) return fail(c, HIVIS_ERR_ARG, "null output pointer");
    if (misaligned(out_tokens) || misaligned(out_parents) || misaligned(out_scores) || misaligned(out_count) ||
        (resid && misaligned(resid)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (topk < 1 || topk > HIVIS_TREE_MAX_TOPK || topk > c->cfg.vocab)
        return fail(c, HIVIS_ERR_CAPACITY, "topk=%d outside [1,%d]", topk, HIVIS_TREE_MAX_TOPK);
    if (depth < 1 || depth > c->cfg.max_k) return fail(c, HIVIS_ERR_CAPACITY, "depth=%d outside [1,%d]", depth, c->cfg.max_k);
    if (keep < 1 || keep > HIVIS_TREE_MAX_KEEP) return fail(c, HIVIS_ERR_CAPACITY, "keep=%d outside [1,%d]", keep, HIVIS_TREE_MAX_KEEP);
    if (resid && (n_resid < 1 || n_resid > HIVIS_MAX_K)) return fail(c, HIVIS_ERR_ARG, "n_resid=%d outside [1,%d]", n_resid, HIVIS_MAX_K);
    if (!c->pending[slot]) return fail(c, HIVIS_ERR_STATE, "slot %d has no pending pair", slot);
    const int tree_rows = 1 + (depth - 1) * topk;
    if (c->kv_upper[slot] + tree_rows > c->cfg.max_len)
        return fail(c, HIVIS_ERR_CAPACITY, "slot %d: %d rows + %d tree rows > max_len %d", slot, c->kv_upper[slot], tree_rows,
                    c->cfg.max_len);
    cudaStream_t st = (cudaStream_t)stream;
    const hivis_config& g = c->cfg;
    const int d = g.d, V = g.vocab;
    int rc;
    if (resid) {
        rc = prepare_rho(c, resid, n_resid, st);
        if (rc) return rc;
    }
    const TreeBufs& T = c->tree;
    CKL(c, launch_tree_begin(slot, d, c->kv_len, c->pend_feat, c->pend_id, c->feat, c->feat_h, c->cur_id, c->d_slots, T, st));
    // bf16 drafters with up to 16 nodes per level (always, by the limit on topk) run the levels' GEMMs in the
    // tensor-core chain kernel, one step long and in two parts around the tree's own attention
    const bool tc = c->tc_ok && c->opt_tc != 0;
    for (int level = 0; level < depth; ++level) {
        const int nb = level == 0 ? 1 : topk;
        if (level > 0 && !tc) CKL(c, launch_tree_gather(nb, d, c->tree_g, T, c->feat, c->feat_h, c->cur_id, st));
        const int row = level < n_resid - 1 ? level : n_resid - 1;
        const float* rho = resid ? c->rho + (long long)row * d : nullptr;
        if (tc) {
            const int lo = tc_lo_offset(nb);
            const u64 G = (u64)c->num_sms;
            CKL(c, launch_tree_operands_tc(nb, TC_OP_ROWS, d, lo, c->feat, c->cur_id, level > 0 ? c->feat : nullptr, T,
                                           (const bf16*)c->embed, V, c->feat_h, c->xe_h, c->d_pos0, c->id_flag, st));
            TcArgs a;
            fill_tc_args(c, &a, nb, 1, lo, rho, 1, nullptr, c->tree_logits);
            a.seq_first = 0; a.seq_last = 2;                         // gather, fusion FC, QKV
            c->debug_skew = false;
            CKL(c, launch_tc_chain(c->tc_maps, a, c->num_sms, st));
            c->bar_count_host += G * 3;
            CK(c, launch_tree_attention(c->dtype, nb, c->qkv, c->qkvw, g.n_q_heads, g.n_kv_heads, g.head_dim, g.max_len, slot,
                                        level, T, c->inv_freq, c->Kc, c->Vc, c->attn, c->attn_h, lo, st));
            c->launches += 2;
            a.seq_first = 4; a.seq_last = 7;                         // O, gate/up, down, LM head (logits of every node)
            a.bar_base = c->bar_count_host - G * 4;                  // as if gather .. attention had been arrived on
            CKL(c, launch_tc_chain(c->tc_maps, a, c->num_sms, st));
            c->bar_count_host += G * 4;
        } else {
            const bool mma = use_mma(c, nb, false);
            rc = run_fuse(c, mma, 0, nb, c->feat, c->feat_h, c->cur_id, 1, nullptr, rho, st);
            if (rc) return rc;
            rc = run_qkv(c, mma, 0, nb, 0, c->qkvw, c->qkv, st);
            if (rc) return rc;
            CK(c, launch_tree_attention(c->dtype, nb, c->qkv, c->qkvw, g.n_q_heads, g.n_kv_heads, g.head_dim, g.max_len, slot,
                                        level, T, c->inv_freq, c->Kc, c->Vc, c->attn, c->attn_h, 0, st));
            c->launches += 2;
            rc = run_after_attention(c, mma, 0, nb, c->keys, c->key_stride, c->tree_logits, V, st);
            if (rc) return rc;
        }
        CKL(c, launch_tree_topk(nb, c->tree_logits, V, topk, T, st));
        c->launches += 1;                                            // (two kernels)
        // (the tensor-core path reads the level's outputs where the down projection left them: they are overwritten only
        // by the next level's own down projection, after its operands were prepared)
        if (!tc) CK(c, cudaMemcpyAsync(c->tree_g, c->feat, (size_t)nb * d * sizeof(float), cudaMemcpyDeviceToDevice, st));
        CKL(c, launch_tree_select(level, depth, nb, topk, T, st));
    }
    CKL(c, launch_tree_finalize(keep, T, out_tokens, out_parents, out_scores, out_count, st));
    const int total = topk + (depth - 1) * topk * topk;
    c->pending[slot] = false;
    c->last_k[slot] = 0;
    c->tree_depth[slot] = depth;
    c->tree_count[slot] = keep < total ? keep : total;
    c->tap_B = 0;
    return HIVIS_OK;
}

int hivis_verify_tree(hivis_ctx* c, int slot, const void* target_logits, int logits_dtype, int32_t* out_accept,
                      int32_t* out_path, int32_t* out_next, int32_t* out_kv_len, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    if (!target_logits || !out_accept || !out_path || !out_next) return fail(c, HIVIS_ERR_ARG, "null argument");
    if (misaligned(target_logits) || misaligned(out_accept) || misaligned(out_path) || misaligned(out_next) ||
        (out_kv_len && misaligned(out_kv_len)))
        return fail(c, HIVIS_ERR_ARG, "device pointer not 16-byte aligned");
    if (logits_dtype != HIVIS_F32 && logits_dtype != HIVIS_BF16) return fail(c, HIVIS_ERR_DTYPE, "unknown logits dtype");
    if (c->tree_depth[slot] == 0) return fail(c, HIVIS_ERR_STATE, "slot %d: no draft tree waits for verification", slot);
    const hivis_config& g = c->cfg;
    CK(c, launch_tree_verify(c->dtype, logits_dtype, slot, c->tree_depth[slot], c->tree_count[slot] + 1, g.vocab, g.n_kv_heads,
                             g.head_dim, g.max_len, c->tree, target_logits, c->Kc, c->Vc, c->kv_len, out_accept, out_path,
                             out_next, out_kv_len, (cudaStream_t)stream));
    c->launches += 2;
    c->kv_upper[slot] += c->tree_depth[slot];        // at most: the root's row and depth - 1 accepted rows
    if (c->kv_upper[slot] > g.max_len) c->kv_upper[slot] = g.max_len;
    c->kv_exact[slot] = false;
    c->tree_depth[slot] = 0;
    c->tree_count[slot] = 0;
    return HIVIS_OK;
}

int hivis_reset(hivis_ctx* c, int slot, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    CKL(c, launch_set_int(c->kv_len + slot, 0, (cudaStream_t)stream));
    c->kv_upper[slot] = 0;
    c->kv_exact[slot] = true;
    c->pending[slot] = false;
    c->have_pair[slot] = false;
    c->last_k[slot] = 0;
    c->tree_depth[slot] = 0;
    return HIVIS_OK;
}

int hivis_get_kv_len(hivis_ctx* c, int slot, int* n_rows_host, int* pending_host, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    int rows = 0;
    CK(c, cudaMemcpyAsync(&rows, c->kv_len + slot, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CK(c, cudaStreamSynchronize((cudaStream_t)stream));
    c->kv_upper[slot] = rows;
    c->kv_exact[slot] = true;
    if (n_rows_host) *n_rows_host = rows;
    if (pending_host) *pending_host = c->pending[slot] ? 1 : 0;
    return HIVIS_OK;
}

int hivis_set_kv_len(hivis_ctx* c, int slot, int n_rows, int restore_pending, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    if (n_rows < 0 || n_rows > c->cfg.max_len) return fail(c, HIVIS_ERR_CAPACITY, "n_rows %d outside [0,%d]", n_rows, c->cfg.max_len);
    if (restore_pending && !c->have_pair[slot]) return fail(c, HIVIS_ERR_STATE, "slot %d never held a pair", slot);
    CKL(c, launch_set_int(c->kv_len + slot, n_rows, (cudaStream_t)stream));
    c->kv_upper[slot] = n_rows;
    c->kv_exact[slot] = true;
    if (restore_pending) c->pending[slot] = true;
    c->last_k[slot] = 0;
    c->tree_depth[slot] = 0;
    return HIVIS_OK;
}

int hivis_set_kv_len_batch(hivis_ctx* c, int B, const int* slots_host, const int* n_rows_host, int restore_pending,
                           void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (!n_rows_host) return fail(c, HIVIS_ERR_ARG, "n_rows_host is null");
    SlotList sl;
    int rc = check_slots(c, B, slots_host, &sl);
    if (rc) return rc;
    CuSeqlens rows;
    for (int b = 0; b < B; ++b) {
        if (n_rows_host[b] < 0 || n_rows_host[b] > c->cfg.max_len)
            return fail(c, HIVIS_ERR_CAPACITY, "n_rows %d outside [0,%d]", n_rows_host[b], c->cfg.max_len);
        if (restore_pending && !c->have_pair[sl.slot[b]]) return fail(c, HIVIS_ERR_STATE, "slot %d never held a pair", sl.slot[b]);
        rows.v[b] = n_rows_host[b];
    }
    CKL(c, launch_set_rows(sl, rows, c->kv_len, (cudaStream_t)stream));
    for (int b = 0; b < B; ++b) {
        const int s = sl.slot[b];
        c->kv_upper[s] = n_rows_host[b];
        c->kv_exact[s] = true;
        if (restore_pending) c->pending[s] = true;
        c->last_k[s] = 0;
        c->tree_depth[s] = 0;
    }
    return HIVIS_OK;
}

int hivis_read_kv(hivis_ctx* c, int slot, int row0, int n, float* out_k, float* out_v, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (slot < 0 || slot >= c->cfg.max_batch) return fail(c, HIVIS_ERR_ARG, "slot %d out of range", slot);
    if (!out_k || !out_v || misaligned(out_k) || misaligned(out_v)) return fail(c, HIVIS_ERR_ARG, "bad output pointer");
    if (row0 < 0 || n < 0 || row0 + n > c->cfg.max_len) return fail(c, HIVIS_ERR_CAPACITY, "rows [%d,%d) outside the cache", row0, row0 + n);
    CKL(c, launch_read_kv(c->dtype, c->Kc, c->Vc, slot, row0, n, c->cfg.n_kv_heads, c->cfg.head_dim,
                          c->cfg.max_len, out_k, out_v, (cudaStream_t)stream));
    return HIVIS_OK;
}

int hivis_set_option(hivis_ctx* c, int option, int value) {
    if (!c) return HIVIS_ERR_ARG;
    if (option == HIVIS_OPT_CHAIN_KERNEL) {
        c->opt_chain = value != 0;
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_TC_KERNEL) {
        if (value < 0 || value > 2) return fail(c, HIVIS_ERR_ARG, "HIVIS_OPT_TC_KERNEL takes 0, 1 or 2");
        c->opt_tc = value;
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_WAIT_LIMIT_US) {
        if (value < 100 || value > 10000000) return fail(c, HIVIS_ERR_ARG, "wait limit %d us outside [100, 10000000]", value);
        c->wait_cycles = (long long)value * 2000ll;          // at most ~2 GHz
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_DEBUG_MISS_BARRIER) {
        c->debug_skew = value != 0;
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_PHASE_TIMES) {
        c->opt_phase_times = value != 0;
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_TC_PREFILL) {
        c->opt_tc_prefill = value == 1 ? HIVIS_TC_PREFILL_MIN_PAIRS : (value < 0 ? 0 : value);
        return HIVIS_OK;
    }
    if (option == HIVIS_OPT_L2_KEEP) {
        if (value < 0 || value >= (1 << PH_COUNT)) return fail(c, HIVIS_ERR_ARG, "HIVIS_OPT_L2_KEEP takes a mask of %d bits", PH_COUNT);
        c->opt_l2_keep = value;
        return HIVIS_OK;
    }
    return fail(c, HIVIS_ERR_ARG, "unknown option %d", option);
}

int hivis_status(hivis_ctx* c, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int flags[2] = {0, 0};
    CK(c, cudaMemcpyAsync(flags, c->error_flag, 2 * sizeof(int), cudaMemcpyDeviceToHost, st));
    CK(c, cudaStreamSynchronize(st));
    const int flag = flags[0];
    if (flag == 0 && flags[1] == 0) return HIVIS_OK;
    if (flag == 0) {
        CK(c, cudaMemsetAsync(c->id_flag, 0, sizeof(int), st));
        CK(c, cudaStreamSynchronize(st));
        return fail(c, HIVIS_ERR_ARG, "a token id outside [0, vocab) reached the embedding lookup and was read as token 0");
    }
    // a kernel gave up on a wait: bring the barrier bookkeeping back to a known state
    CK(c, cudaMemsetAsync(c->bar_counter, 0, sizeof(u64), st));
    CK(c, cudaMemsetAsync(c->error_flag, 0, 2 * sizeof(int), st));
    CK(c, cudaMemsetAsync(c->counters, 0, (size_t)c->rows_cap * c->cfg.n_q_heads * sizeof(int), st));
    if (c->tile_ctr) CK(c, cudaMemsetAsync(c->tile_ctr, 0, (size_t)c->tc_tiles * sizeof(int), st));
    CK(c, cudaStreamSynchronize(st));
    c->bar_count_host = 0;
    return fail(c, HIVIS_ERR_TIMEOUT, "a device-side wait ran out (code %d); results of that call are invalid", flag);
}

int hivis_read_phase_times(hivis_ctx* c, uint64_t* out_host, long long capacity, int* k_host, int* grid_host,
                           void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (!k_host || !grid_host) return fail(c, HIVIS_ERR_ARG, "null argument");
    if (c->phase_k == 0 || !c->phase_t) return fail(c, HIVIS_ERR_STATE, "no draft has recorded phase times");
    *k_host = c->phase_k;
    *grid_host = c->num_sms;
    const long long n = (long long)c->phase_k * HIVIS_PHASE_EVENTS * c->num_sms;
    if (!out_host || capacity < n) return fail(c, HIVIS_ERR_CAPACITY, "phase times need room for %lld entries", n);
    cudaStream_t st = (cudaStream_t)stream;
    CK(c, cudaMemcpyAsync(out_host, c->phase_t, (size_t)n * sizeof(u64), cudaMemcpyDeviceToHost, st));
    CK(c, cudaStreamSynchronize(st));
    return HIVIS_OK;
}

int hivis_profile_begin(hivis_ctx* c) {
    if (!c) return HIVIS_ERR_ARG;
    c->prof_on = true;
    c->prof_n = 0;
    return HIVIS_OK;
}

int hivis_profile_end(hivis_ctx* c, float* ms_host, int64_t* launches_host) {
    if (!c) return HIVIS_ERR_ARG;
    if (!ms_host || !launches_host) return fail(c, HIVIS_ERR_ARG, "null argument");
    for (int i = 0; i < HIVIS_PROFILE_CLASSES; ++i) { ms_host[i] = 0.f; launches_host[i] = 0; }
    c->prof_on = false;
    if (c->prof_n) CK(c, cudaEventSynchronize(c->prof_ev[c->prof_n * 2 - 1]));
    for (size_t i = 0; i < c->prof_n; ++i) {
        float ms = 0.f;
        CK(c, cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
        ms_host[c->prof_cls[i]] += ms;
        launches_host[c->prof_cls[i]] += 1;
    }
    c->prof_n = 0;
    return HIVIS_OK;
}

int hivis_debug_tap(hivis_ctx* c, int which, float* out, void* stream) {
    if (!c) return HIVIS_ERR_ARG;
    if (!out || misaligned(out)) return fail(c, HIVIS_ERR_ARG, "bad output pointer");
    if (c->tap_B < 1) return fail(c, HIVIS_ERR_STATE, "no draft has run yet");
    cudaStream_t st = (cudaStream_t)stream;
    const long long B = c->tap_B, d = c->cfg.d, F = c->cfg.ffn;
    const float* src = nullptr;
    long long n = 0;
    switch (which) {
        case HIVIS_TAP_U: src = c->u; n = B * d; break;
        case HIVIS_TAP_ATTN: src = c->attn; n = B * c->qw; break;
        case HIVIS_TAP_Y: src = c->y; n = B * d; break;
        case HIVIS_TAP_G: src = c->feat; n = B * d; break;
        case HIVIS_TAP_Q:
            // q sits at the start of every row of the stacked q | k | v buffer
            CK(c, cudaMemcpy2DAsync(out, (size_t)c->qw * sizeof(float), c->qkv, (size_t)c->qkvw * sizeof(float),
                                    (size_t)c->qw * sizeof(float), (size_t)B, cudaMemcpyDeviceToDevice, st));
            return HIVIS_OK;
        case HIVIS_TAP_ACT:
            n = B * F;
            if (c->tap_mma) {
                CKL(c, launch_bf16_to_f32(c->act_h, out, n, st));
                return HIVIS_OK;
            }
            src = c->act;
            break;
        default: return fail(c, HIVIS_ERR_ARG, "unknown tap %d", which);
    }
    CK(c, cudaMemcpyAsync(out, src, n * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return HIVIS_OK;
}

}  // extern "C"
