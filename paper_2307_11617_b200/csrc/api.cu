// C ABI of librfast: handle life cycle, uploads, per-round launches, state read-back.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <memory>
#include <new>
#include <string>
#include <vector>

#include "kernels.cuh"
#include "logit_fused.cuh"
#include "persist.cuh"
#include "rfast_internal.h"

using namespace rfast;

namespace rfast {
// MLP gradient (tensor-core path), defined in grad_mlp.cu
struct MlpPlan;
int  mlp_plan_create(int n, int rows, int F, int H, int C, int B, int64_t stride, int max_events,
                     const float* d_feat, const __nv_bfloat16* xb, const float* x, float* gbuf, cudaStream_t st,
                     MlpPlan** out, size_t* dev_bytes, std::string& err);
int  mlp_plan_status(MlpPlan* plan, cudaStream_t st);
void mlp_plan_clear_status(MlpPlan* plan, cudaStream_t st);
void mlp_plan_destroy(MlpPlan* plan);
int  mlp_grad_launch(MlpPlan* plan, const GradArgs& g, const __nv_bfloat16* xb, const int* label,
                     int n_events, cudaStream_t st, int64_t* launches, std::string& err);
}  // namespace rfast

static std::string g_create_error;

// Host copy of the raw arrays of an open-ended schedule (what rfast_append_schedule extends).
struct RawSchedule {
    std::vector<int32_t> act_ptr, act_node, batch_idx;
    std::vector<int8_t> send_r, send_c;
    std::vector<float> alpha_round;
    bool has_alpha = false;
    rfast_schedule view() const {
        rfast_schedule v{};
        v.K = (int32_t)act_ptr.size() - 1;
        v.act_ptr = act_ptr.data();  v.act_node = act_node.data();
        v.send_r = send_r.data();  v.n_send_r = (int64_t)send_r.size();
        v.send_c = send_c.data();  v.n_send_c = (int64_t)send_c.size();
        v.batch_idx = batch_idx.empty() ? nullptr : batch_idx.data();  v.n_batch_idx = (int64_t)batch_idx.size();
        v.alpha_round = has_alpha ? alpha_round.data() : nullptr;
        return v;
    }
};

// raw arrays of a schedule that compile_schedule has accepted
static std::unique_ptr<RawSchedule> raw_of(const rfast_schedule* s, int batch) {
    auto raw = std::make_unique<RawSchedule>();
    const int64_t nE = s->act_ptr[s->K];
    raw->act_ptr.assign(s->act_ptr, s->act_ptr + s->K + 1);
    if (nE > 0) raw->act_node.assign(s->act_node, s->act_node + nE);
    if (s->n_send_r > 0) raw->send_r.assign(s->send_r, s->send_r + s->n_send_r);
    if (s->n_send_c > 0) raw->send_c.assign(s->send_c, s->send_c + s->n_send_c);
    if (batch > 0) raw->batch_idx.assign(s->batch_idx, s->batch_idx + s->n_batch_idx);
    raw->has_alpha = s->alpha_round != nullptr;
    if (raw->has_alpha) raw->alpha_round.assign(s->alpha_round, s->alpha_round + s->K);
    return raw;
}

// raw := raw followed by the rounds of `more` (events and rounds of `more` count from 0; its copy of
// zeta^0 is dropped).  Returns an error text, or nullptr.
static const char* append_raw(RawSchedule& raw, const rfast_schedule* more, int n, int batch, float alpha) {
    if (!more || more->K < 0 || !more->act_ptr) return "schedule: null or K < 0";
    if (more->act_ptr[0] != 0) return "schedule: act_ptr[0] != 0";
    for (int r = 0; r < more->K; ++r)
        if (more->act_ptr[r + 1] < more->act_ptr[r]) return "schedule: act_ptr decreases";
    const int64_t nE2 = more->act_ptr[more->K];
    if (nE2 > 0 && !more->act_node) return "schedule: act_node is null";
    if ((more->n_send_r > 0 && !more->send_r) || (more->n_send_c > 0 && !more->send_c) || more->n_send_r < 0 || more->n_send_c < 0)
        return "schedule: send codes are null";
    const int64_t lead = (int64_t)n * batch;
    if (batch > 0 && (!more->batch_idx || more->n_batch_idx != lead + nE2 * batch))
        return "schedule: batch_idx must hold (n + events) * B entries";
    const int K1 = (int)raw.act_ptr.size() - 1;
    if ((int64_t)K1 + more->K > INT32_MAX / 2 || (int64_t)raw.act_ptr.back() + nE2 > INT32_MAX / 2) return "schedule: too many rounds or events";
    const int32_t ev0 = raw.act_ptr.back();
    for (int r = 1; r <= more->K; ++r) raw.act_ptr.push_back(ev0 + more->act_ptr[r]);
    if (nE2 > 0) raw.act_node.insert(raw.act_node.end(), more->act_node, more->act_node + nE2);
    if (more->n_send_r > 0) raw.send_r.insert(raw.send_r.end(), more->send_r, more->send_r + more->n_send_r);
    if (more->n_send_c > 0) raw.send_c.insert(raw.send_c.end(), more->send_c, more->send_c + more->n_send_c);
    if (batch > 0) raw.batch_idx.insert(raw.batch_idx.end(), more->batch_idx + lead, more->batch_idx + more->n_batch_idx);
    if (raw.has_alpha || more->alpha_round) {                  // a part without its own step sizes runs at the problem's alpha
        if (!raw.has_alpha) raw.alpha_round.assign(K1, alpha);
        raw.has_alpha = true;
        for (int r = 0; r < more->K; ++r) raw.alpha_round.push_back(more->alpha_round ? more->alpha_round[r] : alpha);
    }
    return nullptr;
}

// Has nothing of the rounds compiled in `o` moved in `c` (the same rounds, more appended)?
static bool prefix_same(const Compiled& o, const Compiled& c) {
    const int64_t nE1 = o.n_events;
    return c.n_events >= nE1 && c.n_v_slots >= o.n_v_slots && c.n_rho_slots >= o.n_rho_slots &&
           std::equal(o.v_slot.begin(), o.v_slot.end(), c.v_slot.begin()) &&
           std::equal(o.rho_slot.begin(), o.rho_slot.end(), c.rho_slot.begin()) &&
           std::equal(o.used_tau_v.begin(), o.used_tau_v.end(), c.used_tau_v.begin()) &&
           std::equal(o.used_tau_rho.begin(), o.used_tau_rho.end(), c.used_tau_rho.begin()) &&
           std::equal(o.mix_slot.begin(), o.mix_slot.end(), c.mix_slot.begin()) &&
           std::equal(o.news_new.begin(), o.news_new.end(), c.news_new.begin()) &&
           std::equal(o.news_prev.begin(), o.news_prev.end(), c.news_prev.begin()) &&
           std::equal(o.out_cur.begin(), o.out_cur.end(), c.out_cur.begin()) &&
           std::equal(o.out_new.begin(), o.out_new.end(), c.out_new.begin()) &&
           (nE1 == 0 || std::memcmp(o.ev.data(), c.ev.data(), (size_t)nE1 * sizeof(EvDesc)) == 0);
}

struct rfast_ctx {
    cudaStream_t stream = nullptr;
    int n = 0, root = 0, model = 0, batch = 0, rows = 0, F = 0, C = 0, H = 0;
    int64_t p = 0, stride = 0;
    float alpha = 0, l2 = 0;
    HostGraph R, Cg;
    // device state
    float *x = nullptr, *z = nullptr, *zc = nullptr, *gbuf = nullptr, *x0 = nullptr;
    bool compensated = false;
    bool rho2 = false;                // compensation level 2: two-float running sums
    bool buckets = false;             // mass on the G_C edges kept per consumption instead of as running sums
    int64_t rlo_off() const { return rho2 ? (int64_t)comp.n_rho_slots * stride : 0; }
    float *quad_d = nullptr, *quad_b = nullptr, *feat = nullptr, *target = nullptr;
    int* label = nullptr;
    int64_t* sp_ptr = nullptr;
    int64_t* sp_tile_ptr = nullptr;   // [n*rows][ranges+1] first entry of each shard row in each range of 512 coordinates
    int sp_tiles = 0, sp_ranges = 0;
    int* sp_col = nullptr;
    float* sp_val = nullptr;
    __nv_bfloat16* xb = nullptr;
    float *vbuf = nullptr, *rbuf = nullptr, *scratch = nullptr;
    float* row_tmp = nullptr;         // one row (element-wise objective: a recomputed gradient row on its way out)
    // diagnostics scratch, sized with the schedule: row selectors, per-block partial results,
    // mean iterate, per-row residuals of the full least-squares gradient
    int* d_diag_idx = nullptr;  int64_t diag_idx_cap = 0;
    double* d_diag_part = nullptr;
    float* d_xbar = nullptr;  float* d_diag_res = nullptr;
    // sampled objectives, full gradient at the mean iterate (allocated at the first call that asks
    // for it, kept for the life of the handle): a copy of x, a double per coordinate, descriptors and a batch table over whole shards
    double* d_diag_rowloss = nullptr;
    float* d_diag_x = nullptr;  double* d_diag_acc = nullptr;  EvDesc* d_diag_ev = nullptr;  int* d_diag_bidx = nullptr;
    MlpPlan* mlp = nullptr;
    // compiled schedule
    bool has_sched = false;
    Compiled comp;
    EvDesc *d_ev = nullptr, *d_init_ev = nullptr;
    int *d_mix_slot = nullptr, *d_news_new = nullptr, *d_news_prev = nullptr, *d_out_cur = nullptr,
        *d_out_new = nullptr, *d_batch_idx = nullptr;
    float *d_mix_w = nullptr, *d_out_a = nullptr;
    struct Block { void* p; size_t bytes; };
    std::vector<Block> sched_allocs;        // device blocks owned by the loaded schedule
    std::vector<Block> spare;               // blocks of the schedule being replaced, handed out again while the
                                            // next one is put in place (a re-load then allocates nothing)
    std::vector<float> alpha_round;         // per-round step size, empty: constant alpha
    uint64_t sched_hash = 0;                // identity of the loaded schedule (checkpoints)
    // persistent multi-round kernel (L2-resident problems)
    bool opt_persistent = false, opt_graphs = true, persist_ok = false;
    int64_t opt_wait_limit_ms = 2000, opt_phantom = 0;
    int persist_grid = 0;
    int* d_act_ptr = nullptr;
    float* d_alpha_round = nullptr;
    unsigned int* d_bar = nullptr;
    int* d_pstatus = nullptr;
    int max_round_events = 0;
    // sparse logistic: one cluster per activation, one pass over HBM (logit_fused.cuh)
    bool opt_fused = true;
    int fused_cluster = 0, fused_ranges = 0;      // cluster size (0: the path is not available), ranges per CTA
    int fused_threads = 512, fused_stash = 0;
    size_t fused_smem = 0;
    // open-ended schedules: rounds may be appended (rfast_append_schedule)
    bool opt_open_end = false;
    std::vector<int> holds;                 // rounds at which the loaded schedule was held open (its end, earlier ends)
    std::unique_ptr<RawSchedule> raw;       // the raw arrays loaded so far (kept only when open-ended)
    // snapshot of x and y whose transfer to the host runs under the work that follows (rfast_snapshot)
    float *snap_x = nullptr, *snap_y = nullptr;
    cudaStream_t snap_stream = nullptr;
    cudaEvent_t snap_ready = nullptr, snap_done = nullptr;
    int round = 0;
    int64_t launches = 0;
    // recorded span of rounds [graph_r0, graph_r1): a sequence of graphs of about a thousand kernels each
    struct GraphChunk { cudaGraphExec_t exec; int64_t launches; };
    std::vector<GraphChunk> graph_chunks;
    int graph_r0 = -1, graph_r1 = -1;
    size_t dev_bytes = 0, sched_bytes = 0;
    std::string err;
};

namespace {

int set_err(rfast_ctx* c, int code, const std::string& msg) {
    if (c) c->err = msg; else g_create_error = msg;
    return code;
}

#define CK(call)                                                                               \
    do {                                                                                       \
        cudaError_t e_ = (call);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return set_err(ctx, e_ == cudaErrorMemoryAllocation ? RFAST_ENOMEM : RFAST_ECUDA, \
                           std::string(#call) + ": " + cudaGetErrorString(e_));                \
    } while (0)

template <class T>
cudaError_t dev_alloc(rfast_ctx* c, T** ptr, size_t count, bool sched = false) {
    *ptr = nullptr;
    if (count == 0) count = 1;
    const size_t want = count * sizeof(T);
    if (sched) {                                   // a block of the replaced schedule that fits (not more than twice the size)
        int best = -1;
        for (int k = 0; k < (int)c->spare.size(); ++k)
            if (c->spare[k].bytes >= want && c->spare[k].bytes <= 2 * want + 256 &&
                (best < 0 || c->spare[k].bytes < c->spare[best].bytes)) best = k;
        if (best >= 0) {
            const rfast_ctx::Block b = c->spare[best];
            c->spare.erase(c->spare.begin() + best);
            *ptr = (T*)b.p;
            c->dev_bytes += b.bytes;  c->sched_bytes += b.bytes;
            c->sched_allocs.push_back(b);
            return cudaSuccess;
        }
    }
    cudaError_t e = cudaMalloc((void**)ptr, want);
    if (e == cudaSuccess) {
        c->dev_bytes += want;
        if (sched) { c->sched_allocs.push_back({*ptr, want}); c->sched_bytes += want; }
    }
    return e;
}

template <class T>
int upload(rfast_ctx* ctx, T** dptr, const std::vector<T>& h) {
    CK(dev_alloc(ctx, dptr, h.size(), true));
    if (!h.empty())
        CK(cudaMemcpyAsync(*dptr, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice, ctx->stream));
    return RFAST_OK;
}

// host [rows][p] -> device [rows][stride], padding zeroed
int upload_rows(rfast_ctx* ctx, float* dst, const float* src, int64_t rows) {
    CK(cudaMemsetAsync(dst, 0, (size_t)rows * ctx->stride * sizeof(float), ctx->stream));
    CK(cudaMemcpy2DAsync(dst, ctx->stride * sizeof(float), src, ctx->p * sizeof(float),
                         ctx->p * sizeof(float), rows, cudaMemcpyHostToDevice, ctx->stream));
    return RFAST_OK;
}

void drop_spare(rfast_ctx* c) {
    for (auto& b : c->spare) cudaFree(b.p);
    c->spare.clear();
}

// recycle: the blocks are kept aside for the schedule that is about to be put in place
void free_schedule(rfast_ctx* c, bool recycle = false) {
    for (auto& gc : c->graph_chunks) cudaGraphExecDestroy(gc.exec);
    c->graph_chunks.clear();
    c->graph_r0 = c->graph_r1 = -1;
    if (recycle) c->spare.insert(c->spare.end(), c->sched_allocs.begin(), c->sched_allocs.end());
    else for (auto& b : c->sched_allocs) cudaFree(b.p);
    c->sched_allocs.clear();
    c->dev_bytes -= c->sched_bytes;
    c->sched_bytes = 0;
    c->d_ev = c->d_init_ev = nullptr;
    c->vbuf = c->rbuf = c->scratch = nullptr;
    c->d_diag_idx = nullptr; c->d_diag_part = nullptr; c->d_xbar = nullptr; c->d_diag_res = nullptr;
    c->d_act_ptr = nullptr; c->d_alpha_round = nullptr; c->d_bar = nullptr; c->d_pstatus = nullptr;
    c->persist_ok = false;
    c->has_sched = false;
}

ModelTraffic traffic_of(int model, bool compensated, bool one_pass = false) {
    ModelTraffic mt;
    mt.elementwise = (model == RFAST_MODEL_QUAD_DIAG);
    mt.data_streams = (mt.elementwise ? 2 : 0) + (compensated ? 2 : 0);
    // sparse logistic: the fused gradient+tracking pass reads x, z, g_old and writes g (4);
    // the others: gradient reads x (the MLP: a bf16 copy written by the mix pass), writes g,
    // tracking reads z, g_old, g_new (5).  z's write and the packets are counted elsewhere.
    mt.grad_track_streams = (model == RFAST_MODEL_LOGISTIC_SPARSE ? 4 : 5) + (mt.elementwise ? 0 : (compensated ? 2 : 0));
    mt.method_streams = 2;    // element-wise: d and b, the remembered gradient recomputed; others: g_old read, g_new written
    if (one_pass) mt.grad_track_streams = 2 + (compensated ? 2 : 0);   // nothing is read twice
    return mt;
}

int validate_problem(const rfast_problem* p, std::string& err) {
    auto bad = [&](const char* m) { err = m; return RFAST_EINVAL; };
    if (!p) return bad("problem is null");
    if (p->n <= 0 || p->n > 65535) return bad("n must be in [1, 65535]");
    if (p->p <= 0) return bad("p must be positive");
    if (!(p->alpha == p->alpha)) return bad("alpha is NaN");
    switch (p->model) {
        case RFAST_MODEL_QUAD_DIAG:
            if (!p->quad_d || !p->quad_b) return bad("QUAD_DIAG needs quad_d and quad_b");
            if (p->batch != 0) return bad("QUAD_DIAG takes batch = 0");
            break;
        case RFAST_MODEL_LEAST_SQUARES:
            if (!p->feat || !p->target || p->rows <= 0) return bad("LEAST_SQUARES needs feat, target, rows");
            if (p->n_features != p->p) return bad("LEAST_SQUARES needs n_features = p");
            if (p->batch < 0 || p->batch > 4096 || p->rows > (p->batch ? 1 << 30 : 4096))
                return bad("LEAST_SQUARES: batch (or the whole shard when batch = 0) is limited to 4096 rows");
            break;
        case RFAST_MODEL_SOFTMAX:
            if (!p->feat || !p->label || p->rows <= 0 || p->batch <= 0) return bad("SOFTMAX needs feat, label, rows, batch");
            if (p->n_classes < 2 || p->n_features <= 0 || p->p != (int64_t)p->n_classes * p->n_features + p->n_classes)
                return bad("SOFTMAX needs p = C*F + C");
            if ((int64_t)p->batch * p->n_classes > 8192) return bad("SOFTMAX: batch * classes limited to 8192");
            break;
        case RFAST_MODEL_MLP:
            if (!p->feat || !p->label || p->rows <= 0 || p->batch <= 0) return bad("MLP needs feat, label, rows, batch");
            if (p->p != (int64_t)p->n_hidden * p->n_features + p->n_hidden + (int64_t)p->n_classes * p->n_hidden + p->n_classes)
                return bad("MLP needs p = H*F + H + C*H + C");
            break;
        case RFAST_MODEL_LOGISTIC_SPARSE:
            if (!p->sp_rowptr || !p->sp_col || !p->sp_val || !p->label || p->rows <= 0 || p->batch <= 0)
                return bad("LOGISTIC_SPARSE needs sp_rowptr, sp_col, sp_val, label, rows, batch");
            if (p->p > 0x7fffffff) return bad("LOGISTIC_SPARSE: p limited to 2^31 - 1");
            break;
        default:
            return bad("unknown model");
    }
    return RFAST_OK;
}

dim3 tile_grid(int n4, int U, int events) { return dim3((n4 + kThreads * U - 1) / (kThreads * U), events); }

GradArgs grad_args(rfast_ctx* ctx, const EvDesc* d_ev) {
    GradArgs g{};
    g.ev = d_ev; g.x = ctx->x; g.gbuf = ctx->gbuf; g.stride = ctx->stride;
    g.gplane = (int64_t)ctx->n * ctx->stride;
    g.batch_idx = ctx->d_batch_idx; g.rows = ctx->rows; g.F = ctx->F; g.C = ctx->C; g.H = ctx->H;
    g.p = ctx->p; g.l2 = ctx->l2; g.B = ctx->batch;
    return g;
}

// sparse logistic: gradient tile + tracking in one pass (or the gradient alone for the initial trackers)
int launch_logit_track(rfast_ctx* ctx, const RoundArgs& a, const EvDesc* d_ev, int nev, int init_only) {
    GradArgs g = grad_args(ctx, d_ev);
    const dim3 grid(ctx->sp_tiles, nev);
    if (ctx->compensated)
        k_logit_track<true><<<grid, kThreads, 0, ctx->stream>>>(a, g, ctx->sp_tile_ptr, ctx->sp_ranges, ctx->sp_col, ctx->sp_val, ctx->scratch, init_only);
    else
        k_logit_track<false><<<grid, kThreads, 0, ctx->stream>>>(a, g, ctx->sp_tile_ptr, ctx->sp_ranges, ctx->sp_col, ctx->sp_val, ctx->scratch, init_only);
    ctx->launches += 1;
    CK(cudaGetLastError());
    return RFAST_OK;
}

const void* logit_fused_fn(bool comp, int threads) {
    if (threads == 512) return comp ? (const void*)k_logit_fused<true, 512> : (const void*)k_logit_fused<false, 512>;
    return comp ? (const void*)k_logit_fused<true, 1024> : (const void*)k_logit_fused<false, 1024>;
}

// Sparse logistic, one pass: the smallest cluster (1, 2, 4, 8 CTAs) whose CTAs can each keep
// their slice of x and z in shared memory, first with 512 threads per CTA and half of an SM's
// shared memory (two CTAs of different activations share an SM, one streams while the other
// computes), else with 1024 threads and the whole of it.  want > 0 asks for that cluster size.
bool plan_logit_fused(rfast_ctx* ctx, int want) {
    ctx->fused_cluster = 0;
    if (ctx->model != RFAST_MODEL_LOGISTIC_SPARSE || ctx->batch > kFusedMaxBatch || ctx->batch < 1) return false;
    int dev = 0, max_smem = 0, sm_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    cudaDeviceGetAttribute(&sm_smem, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
    int64_t rows_nnz = 0;
    cudaMemcpy(&rows_nnz, ctx->sp_ptr + (size_t)ctx->n * ctx->rows, sizeof(int64_t), cudaMemcpyDeviceToHost);
    const double nnz_per_batch = (double)rows_nnz / std::max<int64_t>(1, (int64_t)ctx->n * ctx->rows) * ctx->batch;
    for (int threads : {512, 1024}) {
        const int64_t budget = threads == 512 ? std::min<int64_t>(max_smem, sm_smem / 2 - 1024) : max_smem;
        for (int cs = 1; cs <= 8; cs *= 2) {
            if (want > 0 && cs != want) continue;
            const int R = (ctx->sp_ranges + cs - 1) / cs;
            if (R * (kLogitRange / 4) > kFusedPerThread * threads) continue;           // float4 of a slice per thread
            const int64_t fixed = (int64_t)2 * R * kLogitRange * sizeof(float) + 4096;   // slices + the kernel's static arrays
            if (fixed > budget) continue;
            // the sampled rows' entries of a slice are kept on chip as far as they fit: room for 1.5 x the mean
            const int64_t want_stash = (int64_t)(1.5 * nnz_per_batch / cs) + 64;
            const int stash = (int)(std::max<int64_t>(0, std::min<int64_t>(want_stash, (budget - fixed) / 6)) / 8 * 8);
            const size_t smem = (size_t)2 * R * kLogitRange * sizeof(float) + (size_t)stash * 6;
            const void* fn = logit_fused_fn(ctx->compensated, threads);
            if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) { cudaGetLastError(); continue; }
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3(cs, 1, 1); cfg.blockDim = dim3(threads, 1, 1); cfg.dynamicSmemBytes = smem;
            cudaLaunchAttribute at{};
            at.id = cudaLaunchAttributeClusterDimension;
            at.val.clusterDim.x = cs; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
            cfg.attrs = &at; cfg.numAttrs = 1;
            int nclusters = 0;
            if (cudaOccupancyMaxActiveClusters(&nclusters, fn, &cfg) != cudaSuccess || nclusters < 1) { cudaGetLastError(); continue; }
            ctx->fused_cluster = cs; ctx->fused_ranges = R; ctx->fused_smem = smem; ctx->fused_stash = stash;
            ctx->fused_threads = threads;
            return true;
        }
    }
    return false;
}

int launch_logit_fused(rfast_ctx* ctx, const RoundArgs& a, const EvDesc* d_ev, int nev) {
    LogitFusedArgs P{};
    P.a = a; P.a.ev = d_ev;
    P.g = grad_args(ctx, d_ev);
    P.range_ptr = ctx->sp_tile_ptr; P.nranges = ctx->sp_ranges;
    P.sp_col = ctx->sp_col; P.sp_val = ctx->sp_val; P.label = ctx->label;
    P.ranges_per_cta = ctx->fused_ranges;
    P.stash_cap = ctx->fused_stash;
    P.status = ctx->d_pstatus; P.limit_ns = (unsigned long long)ctx->opt_wait_limit_ms * 1000000ull;
    P.phantom_bytes = (unsigned int)ctx->opt_phantom * 16u;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(ctx->fused_cluster, nev, 1); cfg.blockDim = dim3(ctx->fused_threads, 1, 1);
    cfg.dynamicSmemBytes = ctx->fused_smem; cfg.stream = ctx->stream;
    cudaLaunchAttribute at{};
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = ctx->fused_cluster; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    cfg.attrs = &at; cfg.numAttrs = 1;
    if (ctx->fused_threads == 512) {
        if (ctx->compensated) CK(cudaLaunchKernelEx(&cfg, k_logit_fused<true, 512>, P));
        else CK(cudaLaunchKernelEx(&cfg, k_logit_fused<false, 512>, P));
    } else {
        if (ctx->compensated) CK(cudaLaunchKernelEx(&cfg, k_logit_fused<true, 1024>, P));
        else CK(cudaLaunchKernelEx(&cfg, k_logit_fused<false, 1024>, P));
    }
    ctx->launches += 1;
    return RFAST_OK;
}

// sample gradients of `nev` events (descriptors on the device) into gbuf[par^1]
int launch_gradients(rfast_ctx* ctx, const EvDesc* d_ev, int nev) {
    GradArgs g = grad_args(ctx, d_ev);
    cudaStream_t st = ctx->stream;
    switch (ctx->model) {
        case RFAST_MODEL_LEAST_SQUARES: {
            const int use_all = ctx->batch == 0;
            g.B = use_all ? ctx->rows : ctx->batch;
            k_ls_residual<<<dim3((g.B + 7) / 8, nev), 256, 0, st>>>(g, ctx->feat, ctx->target, ctx->scratch, use_all);
            k_ls_grad<<<dim3((g.F + 255) / 256, nev), 256, 0, st>>>(g, ctx->feat, ctx->scratch, use_all);
            ctx->launches += 2;
            break;
        }
        case RFAST_MODEL_SOFTMAX: {
            g.B = ctx->batch;
            k_softmax_logits<<<dim3(g.B, nev), 256, 0, st>>>(g, ctx->feat, ctx->scratch);
            const size_t sm = (size_t)g.B * g.C * sizeof(float) + (size_t)g.B * sizeof(int);
            k_softmax_grad<<<dim3((unsigned)((g.p + 255) / 256), nev), 256, sm, st>>>(g, ctx->feat, ctx->label, ctx->scratch);
            ctx->launches += 2;
            break;
        }
        case RFAST_MODEL_LOGISTIC_SPARSE: {
            k_logit_coef<<<dim3((g.B + 7) / 8, nev), 256, 0, st>>>(g, ctx->sp_ptr, ctx->sp_col, ctx->sp_val, ctx->label, ctx->scratch);
            ctx->launches += 1;       // the second phase is fused with the tracking pass (k_logit_track)
            break;
        }
        case RFAST_MODEL_MLP: {
            g.B = ctx->batch;
            int rc = mlp_grad_launch(ctx->mlp, g, ctx->xb, ctx->label, nev, st, &ctx->launches, ctx->err);
            if (rc != RFAST_OK) return rc;
            break;
        }
        default:
            break;
    }
    CK(cudaGetLastError());
    return RFAST_OK;
}

// floats in front of the x staging area: delta [B][C] + row ids [B] (softmax), residuals [B] (least squares)
int persist_xs_off(rfast_ctx* ctx) {
    const int B = ctx->batch ? ctx->batch : ctx->rows;
    const int head = ctx->model == RFAST_MODEL_SOFTMAX ? B * ctx->C + B : B;
    return (head + 3) / 4 * 4;
}
size_t persist_smem(rfast_ctx* ctx) { return ((size_t)persist_xs_off(ctx) + ctx->stride) * sizeof(float); }
const void* persist_kernel(rfast_ctx* ctx) {
    if (ctx->model == RFAST_MODEL_LEAST_SQUARES)
        return ctx->compensated ? (const void*)k_persist_rounds<RFAST_MODEL_LEAST_SQUARES, true>
                                : (const void*)k_persist_rounds<RFAST_MODEL_LEAST_SQUARES, false>;
    if (ctx->model == RFAST_MODEL_SOFTMAX)
        return ctx->compensated ? (const void*)k_persist_rounds<RFAST_MODEL_SOFTMAX, true>
                                : (const void*)k_persist_rounds<RFAST_MODEL_SOFTMAX, false>;
    return nullptr;
}

// after a synchronisation: did a bounded device-side wait run out?
int check_device_status(rfast_ctx* ctx) {
    if (ctx->d_pstatus) {
        int st = 0;
        CK(cudaMemcpyAsync(&st, ctx->d_pstatus, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
        CK(cudaStreamSynchronize(ctx->stream));
        if (st != 0) return set_err(ctx, RFAST_ETIMEOUT, st == kFusedTimeout ? "the bulk copies of the one-pass kernel did not land in time"
                                                                              : "a grid barrier of the persistent kernel ran out of time");
    }
    if (ctx->mlp) {
        const int st = mlp_plan_status(ctx->mlp, ctx->stream);
        if (st < 0) return set_err(ctx, RFAST_ECUDA, "reading the device status word failed");
        if (st > 0) return set_err(ctx, RFAST_ETIMEOUT, "a bounded wait in the MLP gradient kernels ran out (role " + std::to_string(st) + ")");
    }
    return RFAST_OK;
}

int reset_state(rfast_ctx* ctx) {
    const size_t plane = (size_t)ctx->n * ctx->stride * sizeof(float);
    // a bounded wait that ran out earlier is forgotten: the state starts over
    if (ctx->d_pstatus) CK(cudaMemsetAsync(ctx->d_pstatus, 0, sizeof(int), ctx->stream));
    if (ctx->mlp) mlp_plan_clear_status(ctx->mlp, ctx->stream);
    if (ctx->x0) CK(cudaMemcpyAsync(ctx->x, ctx->x0, plane, cudaMemcpyDeviceToDevice, ctx->stream));
    else CK(cudaMemsetAsync(ctx->x, 0, plane, ctx->stream));
    const int n4 = (int)(ctx->stride / 4);
    if (ctx->zc) CK(cudaMemsetAsync(ctx->zc, 0, plane, ctx->stream));
    if (ctx->model == RFAST_MODEL_QUAD_DIAG) {
        k_quad_grad<<<dim3((n4 + kThreads - 1) / kThreads, ctx->n), kThreads, 0, ctx->stream>>>(
            ctx->x, ctx->quad_d, ctx->quad_b, ctx->z, ctx->stride, n4);
        CK(cudaGetLastError());
    } else {
        CK(cudaMemsetAsync(ctx->gbuf, 0, 2 * plane, ctx->stream));
        if (ctx->model == RFAST_MODEL_MLP) {      // bf16 copy of x0 for the matrix products
            k_rows_to_bf16<<<dim3((n4 + kThreads - 1) / kThreads, ctx->n), kThreads, 0, ctx->stream>>>(
                ctx->x, ctx->xb, ctx->stride, n4);
            CK(cudaGetLastError());
        }
        // z_i^0 = g_i^0 = grad f_i(x_i^0; zeta_i^0)  (initialisation line of Algorithm 1)
        int rc = launch_gradients(ctx, ctx->d_init_ev, ctx->n);
        if (rc != RFAST_OK) return rc;
        if (ctx->model == RFAST_MODEL_LOGISTIC_SPARSE) {
            RoundArgs a{};
            a.stride = ctx->stride; a.n4 = n4;
            if ((rc = launch_logit_track(ctx, a, ctx->d_init_ev, ctx->n, 1)) != RFAST_OK) return rc;
        }
        CK(cudaMemcpyAsync(ctx->z, ctx->gbuf, plane, cudaMemcpyDeviceToDevice, ctx->stream));
    }
    ctx->round = 0;
    return RFAST_OK;
}

}  // namespace

extern "C" {

const char* rfast_version(void) { return "rfast-b200 0.1 (sm_100a)"; }

const char* rfast_last_error(const rfast_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

void rfast_destroy(rfast_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    free_schedule(c);
    drop_spare(c);
    if (c->snap_stream) { cudaStreamSynchronize(c->snap_stream); cudaStreamDestroy(c->snap_stream); }
    if (c->snap_ready) cudaEventDestroy(c->snap_ready);
    if (c->snap_done) cudaEventDestroy(c->snap_done);
    if (c->mlp) mlp_plan_destroy(c->mlp);
    void* ptrs[] = {c->x, c->z, c->zc, c->gbuf, c->x0, c->quad_d, c->quad_b, c->feat, c->target, c->label,
                    c->sp_ptr, c->sp_tile_ptr, c->sp_col, c->sp_val, c->xb, c->row_tmp,
                    c->d_diag_rowloss, c->d_diag_x, c->d_diag_acc, c->d_diag_ev, c->d_diag_bidx, c->snap_x, c->snap_y};
    for (void* q : ptrs) if (q) cudaFree(q);
    delete c;
}

int rfast_create(const rfast_problem* prob, void* cuda_stream, rfast_ctx** out) try {
    if (!out) return set_err(nullptr, RFAST_EINVAL, "out is null");
    *out = nullptr;
    std::string err;
    int rc = validate_problem(prob, err);
    if (rc != RFAST_OK) return set_err(nullptr, rc, err);
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        cudaGetLastError();
        return set_err(nullptr, RFAST_ECUDA, "no CUDA device: this library has no CPU path");
    }
    rfast_ctx* ctx = new rfast_ctx();
    struct Guard { rfast_ctx* c; ~Guard() { if (c) { g_create_error = c->err; rfast_destroy(c); } } } guard{ctx};
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->n = prob->n; ctx->root = prob->root; ctx->p = prob->p; ctx->alpha = prob->alpha; ctx->l2 = prob->l2;
    ctx->model = prob->model; ctx->batch = prob->batch; ctx->rows = prob->rows;
    ctx->F = prob->n_features; ctx->C = prob->n_classes; ctx->H = prob->n_hidden;
    ctx->compensated = prob->compensated != 0;
    ctx->rho2 = prob->compensated >= 2;
    ctx->buckets = prob->tracker == RFAST_TRACKER_BUCKETS;
    ctx->stride = (prob->p + 31) / 32 * 32;
    if (ctx->stride / 4 > 0x7fffffff) return set_err(ctx, RFAST_EINVAL, "p too large");
    if ((rc = build_host_graph(prob->G_R, ctx->n, true, ctx->R, err)) != RFAST_OK) return set_err(ctx, rc, "G_R: " + err);
    if ((rc = build_host_graph(prob->G_C, ctx->n, false, ctx->Cg, err)) != RFAST_OK) return set_err(ctx, rc, "G_C: " + err);
    if ((rc = check_roots(ctx->R, ctx->Cg, ctx->root, err)) != RFAST_OK) return set_err(ctx, rc, err);

    const size_t plane = (size_t)ctx->n * ctx->stride;
    CK(dev_alloc(ctx, &ctx->x, plane));
    CK(dev_alloc(ctx, &ctx->z, plane));
    if (ctx->compensated) CK(dev_alloc(ctx, &ctx->zc, plane));
    if (prob->x0) {
        CK(dev_alloc(ctx, &ctx->x0, plane));
        if ((rc = upload_rows(ctx, ctx->x0, prob->x0, ctx->n)) != RFAST_OK) return rc;
    }
    const size_t nrows = (size_t)ctx->n * ctx->rows;
    switch (ctx->model) {
        case RFAST_MODEL_QUAD_DIAG:
            CK(dev_alloc(ctx, &ctx->quad_d, plane));
            CK(dev_alloc(ctx, &ctx->quad_b, plane));
            if ((rc = upload_rows(ctx, ctx->quad_d, prob->quad_d, ctx->n)) != RFAST_OK) return rc;
            if ((rc = upload_rows(ctx, ctx->quad_b, prob->quad_b, ctx->n)) != RFAST_OK) return rc;
            CK(dev_alloc(ctx, &ctx->row_tmp, (size_t)ctx->stride));
            break;
        case RFAST_MODEL_LEAST_SQUARES:
        case RFAST_MODEL_SOFTMAX:
        case RFAST_MODEL_MLP:
            CK(dev_alloc(ctx, &ctx->feat, nrows * ctx->F));
            CK(cudaMemcpyAsync(ctx->feat, prob->feat, nrows * ctx->F * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
            if (ctx->model == RFAST_MODEL_LEAST_SQUARES) {
                CK(dev_alloc(ctx, &ctx->target, nrows));
                CK(cudaMemcpyAsync(ctx->target, prob->target, nrows * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
            } else {
                for (size_t k = 0; k < nrows; ++k)
                    if (prob->label[k] < 0 || prob->label[k] >= ctx->C) return set_err(ctx, RFAST_EINVAL, "label out of range");
                CK(dev_alloc(ctx, &ctx->label, nrows));
                CK(cudaMemcpyAsync(ctx->label, prob->label, nrows * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
            }
            break;
        case RFAST_MODEL_LOGISTIC_SPARSE: {
            const int64_t nnz = prob->sp_rowptr[nrows];
            if (prob->sp_rowptr[0] != 0 || nnz < 0) return set_err(ctx, RFAST_EINVAL, "sp_rowptr must start at 0");
            for (size_t r = 0; r < nrows; ++r) {
                if (prob->sp_rowptr[r + 1] < prob->sp_rowptr[r]) return set_err(ctx, RFAST_EINVAL, "sp_rowptr decreases");
                for (int64_t q = prob->sp_rowptr[r]; q < prob->sp_rowptr[r + 1]; ++q) {
                    if (prob->sp_col[q] < 0 || prob->sp_col[q] >= ctx->p ||
                        (q > prob->sp_rowptr[r] && prob->sp_col[q - 1] >= prob->sp_col[q]))
                        return set_err(ctx, RFAST_EINVAL, "sp_col must be strictly ascending inside a row and below p");
                }
                if (prob->label[r] != 1 && prob->label[r] != -1) return set_err(ctx, RFAST_EINVAL, "labels must be -1 or +1");
            }
            {   // per shard row, where each range of kLogitRange coordinates starts (one walk over the entries)
                ctx->sp_tiles = (int)((ctx->p + kLogitTile - 1) / kLogitTile);
                ctx->sp_ranges = (int)((ctx->p + kLogitRange - 1) / kLogitRange);
                std::vector<int64_t> tp((size_t)nrows * (ctx->sp_ranges + 1));
                for (size_t r = 0; r < nrows; ++r) {
                    int64_t q = prob->sp_rowptr[r];
                    const int64_t qe = prob->sp_rowptr[r + 1];
                    int64_t* dst = tp.data() + r * (ctx->sp_ranges + 1);
                    for (int t = 0; t <= ctx->sp_ranges; ++t) {
                        const int64_t bound = (int64_t)t * kLogitRange;
                        while (q < qe && prob->sp_col[q] < bound) ++q;
                        dst[t] = q;
                    }
                }
                CK(dev_alloc(ctx, &ctx->sp_tile_ptr, tp.size()));
                CK(cudaMemcpyAsync(ctx->sp_tile_ptr, tp.data(), tp.size() * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream));
                CK(cudaStreamSynchronize(ctx->stream));       // tp goes out of scope
            }
            CK(dev_alloc(ctx, &ctx->sp_ptr, nrows + 1));
            CK(dev_alloc(ctx, &ctx->sp_col, (size_t)nnz));
            CK(dev_alloc(ctx, &ctx->sp_val, (size_t)nnz));
            CK(dev_alloc(ctx, &ctx->label, nrows));
            CK(cudaMemcpyAsync(ctx->sp_ptr, prob->sp_rowptr, (nrows + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream));
            CK(cudaMemcpyAsync(ctx->sp_col, prob->sp_col, (size_t)nnz * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
            CK(cudaMemcpyAsync(ctx->sp_val, prob->sp_val, (size_t)nnz * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
            CK(cudaMemcpyAsync(ctx->label, prob->label, nrows * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
            break;
        }
    }
    if (ctx->model != RFAST_MODEL_QUAD_DIAG) CK(dev_alloc(ctx, &ctx->gbuf, 2 * plane));
    if (ctx->model == RFAST_MODEL_MLP) {
        CK(dev_alloc(ctx, &ctx->xb, plane));
        CK(cudaMemsetAsync(ctx->xb, 0, plane * sizeof(__nv_bfloat16), ctx->stream));
        size_t mb = 0;
        rc = mlp_plan_create(ctx->n, ctx->rows, ctx->F, ctx->H, ctx->C, ctx->batch, ctx->stride, ctx->n,
                             ctx->feat, ctx->xb, ctx->x, ctx->gbuf, ctx->stream, &ctx->mlp, &mb, err);
        if (rc != RFAST_OK) return set_err(ctx, rc, err);
        ctx->dev_bytes += mb;
    }
    CK(cudaStreamSynchronize(ctx->stream));    // the caller's arrays may go away now
    plan_logit_fused(ctx, 0);
    guard.c = nullptr;
    *out = ctx;
    return RFAST_OK;
} catch (const std::bad_alloc&) {
    return set_err(nullptr, RFAST_ENOMEM, "host allocation failed");
} catch (...) {
    return set_err(nullptr, RFAST_EINVAL, "unexpected failure in rfast_create");
}

// Puts a compiled schedule in place: descriptors up, version-row pools, scratch.  `s` holds the raw
// arrays `comp` was compiled from.  keep_state: rounds were appended to the schedule in place; the
// rows written so far and the round counter carry over instead of the state starting at round 0.
static int install_schedule(rfast_ctx* ctx, const rfast_schedule* s, Compiled&& comp, bool keep_state) {
    int rc;
    // rounds appended: the version rows written so far carry over into the (possibly larger) pools
    float *old_v = nullptr, *old_r = nullptr;
    const int64_t old_nv = ctx->comp.n_v_slots, old_nr = ctx->comp.n_rho_slots;
    if (keep_state) {
        old_v = ctx->vbuf;  old_r = ctx->rbuf;
        auto& al = ctx->sched_allocs;
        al.erase(std::remove_if(al.begin(), al.end(), [&](const rfast_ctx::Block& b) { return b.p == (void*)old_v || b.p == (void*)old_r; }), al.end());
    }
    struct OldRows {                                   // freed on every way out
        float *v, *r;
        ~OldRows() { if (v) cudaFree(v); if (r) cudaFree(r); }
    } old_rows{old_v, old_r};
    struct Spare {                                     // what the new schedule did not take over is freed on every way out
        rfast_ctx* c;
        ~Spare() { drop_spare(c); }
    } spare{ctx};
    free_schedule(ctx, true);
    ctx->alpha_round.clear();
    if (s->alpha_round) {
        for (int r = 0; r < s->K; ++r)
            if (!(s->alpha_round[r] == s->alpha_round[r])) return set_err(ctx, RFAST_ESCHED, "schedule: alpha_round holds a NaN");
        ctx->alpha_round.assign(s->alpha_round, s->alpha_round + s->K);
    }
    {   // hash of the raw arrays: a checkpoint is only valid for this very schedule.  Eight bytes
        // per step (multiply and fold), the tail byte by byte: the arrays run to tens of megabytes
        // and this sits in every rfast_load_schedule
        uint64_t hsh = 1469598103934665603ull;
        auto mix = [&](const void* ptr, size_t bytes) {
            const unsigned char* q = (const unsigned char*)ptr;
            size_t k = 0;
            for (; k + 8 <= bytes; k += 8) {
                uint64_t w;
                std::memcpy(&w, q + k, 8);
                hsh = (hsh ^ w) * 0x9E3779B97F4A7C15ull;
                hsh ^= hsh >> 29;
            }
            for (; k < bytes; ++k) { hsh ^= q[k]; hsh *= 1099511628211ull; }
            hsh ^= bytes;
            hsh *= 1099511628211ull;
        };
        mix(&s->K, sizeof s->K);
        mix(s->act_ptr, (size_t)(s->K + 1) * sizeof(int32_t));
        if (s->act_ptr[s->K] > 0) mix(s->act_node, (size_t)s->act_ptr[s->K] * sizeof(int32_t));
        if (s->n_send_r > 0) mix(s->send_r, (size_t)s->n_send_r);
        if (s->n_send_c > 0) mix(s->send_c, (size_t)s->n_send_c);
        if (ctx->batch > 0) mix(s->batch_idx, (size_t)s->n_batch_idx * sizeof(int32_t));
        if (s->alpha_round) mix(s->alpha_round, (size_t)s->K * sizeof(float));
        for (int b : ctx->holds) mix(&b, sizeof b);     // where rounds were appended: the rows depend on it
        ctx->sched_hash = hsh;
    }
    ctx->comp = std::move(comp);
    Compiled& c = ctx->comp;
    ctx->max_round_events = 0;
    for (int r = 0; r < c.K; ++r) ctx->max_round_events = std::max(ctx->max_round_events, c.act_ptr[r + 1] - c.act_ptr[r]);
    if ((rc = upload(ctx, &ctx->d_ev, c.ev))) return rc;
    if ((rc = upload(ctx, &ctx->d_mix_slot, c.mix_slot))) return rc;
    if ((rc = upload(ctx, &ctx->d_mix_w, c.mix_w))) return rc;
    if ((rc = upload(ctx, &ctx->d_news_new, c.news_new))) return rc;
    if ((rc = upload(ctx, &ctx->d_news_prev, c.news_prev))) return rc;
    if ((rc = upload(ctx, &ctx->d_out_cur, c.out_cur))) return rc;
    if ((rc = upload(ctx, &ctx->d_out_new, c.out_new))) return rc;
    if ((rc = upload(ctx, &ctx->d_out_a, c.out_a))) return rc;
    std::vector<int> bidx;
    if (ctx->batch > 0) bidx.assign(s->batch_idx, s->batch_idx + s->n_batch_idx);
    if ((rc = upload(ctx, &ctx->d_batch_idx, bidx))) return rc;
    std::vector<EvDesc> init(ctx->n);
    for (int i = 0; i < ctx->n; ++i) {
        EvDesc d{};
        d.node = i; d.v_out = -1; d.g_par = 1; d.sample = i;     // result lands in gradient buffer 0
        init[i] = d;
    }
    if ((rc = upload(ctx, &ctx->d_init_ev, init))) return rc;
    CK(dev_alloc(ctx, &ctx->vbuf, (size_t)c.n_v_slots * ctx->stride, true));
    CK(dev_alloc(ctx, &ctx->rbuf, (size_t)c.n_rho_slots * ctx->stride * (ctx->rho2 ? 2 : 1), true));
    CK(cudaMemsetAsync(ctx->vbuf, 0, std::max<size_t>(1, (size_t)c.n_v_slots * ctx->stride) * sizeof(float), ctx->stream));
    CK(cudaMemsetAsync(ctx->rbuf, 0, std::max<size_t>(1, (size_t)c.n_rho_slots * ctx->stride * (ctx->rho2 ? 2 : 1)) * sizeof(float), ctx->stream));
    if (keep_state) {
        const size_t row = (size_t)ctx->stride * sizeof(float);
        if (old_v && old_nv > 0) CK(cudaMemcpyAsync(ctx->vbuf, old_v, old_nv * row, cudaMemcpyDeviceToDevice, ctx->stream));
        if (old_r && old_nr > 0) {
            CK(cudaMemcpyAsync(ctx->rbuf, old_r, old_nr * row, cudaMemcpyDeviceToDevice, ctx->stream));
            if (ctx->rho2)                              // the low-order words sit one pool further on
                CK(cudaMemcpyAsync(ctx->rbuf + (size_t)c.n_rho_slots * ctx->stride, old_r + (size_t)old_nr * ctx->stride,
                                   old_nr * row, cudaMemcpyDeviceToDevice, ctx->stream));
        }
    }
    // scratch of the two-phase gradients: residuals / logits / coefficients per (event, row[, class])
    size_t per_ev = 0;
    if (ctx->model == RFAST_MODEL_LEAST_SQUARES) per_ev = ctx->batch ? ctx->batch : ctx->rows;
    if (ctx->model == RFAST_MODEL_SOFTMAX) per_ev = (size_t)ctx->batch * ctx->C;
    if (ctx->model == RFAST_MODEL_LOGISTIC_SPARSE) per_ev = ctx->batch;
    CK(dev_alloc(ctx, &ctx->scratch, per_ev * std::max(ctx->n, ctx->max_round_events), true));
    // persistent path: act_ptr / step sizes on the device, barrier counter, status word
    if ((rc = upload(ctx, &ctx->d_act_ptr, c.act_ptr))) return rc;
    if (!ctx->alpha_round.empty() && (rc = upload(ctx, &ctx->d_alpha_round, ctx->alpha_round))) return rc;
    CK(dev_alloc(ctx, &ctx->d_bar, 1, true));
    CK(dev_alloc(ctx, &ctx->d_pstatus, 1, true));
    CK(cudaMemsetAsync(ctx->d_pstatus, 0, sizeof(int), ctx->stream));
    ctx->persist_ok = false;
    if ((ctx->model == RFAST_MODEL_LEAST_SQUARES || ctx->model == RFAST_MODEL_SOFTMAX) &&
        (size_t)ctx->n * ctx->stride * sizeof(float) <= ((size_t)8 << 20) && persist_smem(ctx) <= 200 * 1024) {
        int dev = 0, coop = 0, sms = 0, occ = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const size_t smem = persist_smem(ctx);
        const void* fn = persist_kernel(ctx);
        if (fn) cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (coop && fn && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, kThreads, smem) == cudaSuccess && occ > 0) {
            const int tiles = (int)((ctx->stride / 4 + kThreads - 1) / kThreads);
            const int B = ctx->batch ? ctx->batch : ctx->rows;
            const int per_ev = std::max(tiles, ctx->model == RFAST_MODEL_SOFTMAX ? (B + 3) / 4 : (B + 7) / 8);
            const int want = std::max(1, ctx->max_round_events * per_ev);
            ctx->persist_grid = std::min(want, sms);          // one CTA per SM keeps the barrier short
            ctx->persist_ok = true;
        }
    }
    {   // diagnostics scratch (nothing is allocated when the diagnostics run)
        ctx->diag_idx_cap = (int64_t)ctx->n + 2 * (int64_t)std::max(std::max(ctx->Cg.E, c.n_rho_slots), 1);
        CK(dev_alloc(ctx, &ctx->d_diag_idx, (size_t)ctx->diag_idx_cap, true));
        CK(dev_alloc(ctx, &ctx->d_diag_part, (size_t)((ctx->p + kThreads - 1) / kThreads) * kDiagSlots, true));
        if (ctx->model == RFAST_MODEL_LEAST_SQUARES) {
            CK(dev_alloc(ctx, &ctx->d_xbar, (size_t)ctx->stride, true));
            CK(dev_alloc(ctx, &ctx->d_diag_res, (size_t)ctx->n * ctx->rows, true));
        }
    }
    ctx->has_sched = true;
    if (!keep_state && (rc = reset_state(ctx)) != RFAST_OK) return rc;
    CK(cudaStreamSynchronize(ctx->stream));
    return RFAST_OK;
}

int rfast_load_schedule(rfast_ctx* ctx, const rfast_schedule* s) try {
    if (!ctx) return RFAST_EINVAL;
    CK(cudaStreamSynchronize(ctx->stream));
    Compiled comp;
    std::string err;
    const bool one_pass = ctx->model == RFAST_MODEL_LOGISTIC_SPARSE && ctx->opt_fused && ctx->fused_cluster > 0;
    std::vector<int> holds;
    if (ctx->opt_open_end && s && s->K >= 0) holds.push_back(s->K);
    int rc = compile_schedule(ctx->R, ctx->Cg, s, ctx->batch, ctx->rows, traffic_of(ctx->model, ctx->compensated, one_pass), ctx->buckets, comp, err, &holds);
    if (rc != RFAST_OK) return set_err(ctx, rc, err);
    ctx->holds = holds;
    ctx->raw.reset();
    if (ctx->opt_open_end) ctx->raw = raw_of(s, ctx->batch);   // the raw arrays are what an append extends
    return install_schedule(ctx, s, std::move(comp), false);
} catch (const std::bad_alloc&) {
    return set_err(ctx, RFAST_ENOMEM, "host allocation failed");
} catch (...) {
    return set_err(ctx, RFAST_EINVAL, "unexpected failure in rfast_load_schedule");
}

int rfast_append_schedule(rfast_ctx* ctx, const rfast_schedule* more) try {
    if (!ctx) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (!ctx->opt_open_end || !ctx->raw)
        return set_err(ctx, RFAST_ESTATE, "rounds can only be appended to a schedule loaded with RFAST_OPT_OPEN_END set");
    CK(cudaStreamSynchronize(ctx->stream));
    // the loaded rounds followed by the new ones, as one raw schedule
    auto raw = std::make_unique<RawSchedule>(*ctx->raw);
    if (const char* bad = append_raw(*raw, more, ctx->n, ctx->batch, ctx->alpha)) return set_err(ctx, RFAST_ESCHED, bad);
    const rfast_schedule all = raw->view();
    std::vector<int> holds = ctx->holds;                       // every earlier end stays a hold, the new end is open
    if (holds.empty() || holds.back() != all.K) holds.push_back(all.K);
    Compiled comp;
    std::string err;
    const bool one_pass = ctx->model == RFAST_MODEL_LOGISTIC_SPARSE && ctx->opt_fused && ctx->fused_cluster > 0;
    int rc = compile_schedule(ctx->R, ctx->Cg, &all, ctx->batch, ctx->rows, traffic_of(ctx->model, ctx->compensated, one_pass), ctx->buckets, comp, err, &holds);
    if (rc != RFAST_OK) return set_err(ctx, rc, err);
    // nothing of the rounds already loaded may have moved: same rows, same descriptors
    if (!prefix_same(ctx->comp, comp))
        return set_err(ctx, RFAST_ESCHED, "internal: appending rounds would move a version row of the rounds already loaded");
    const int round = ctx->round;
    ctx->holds = holds;
    ctx->raw = std::move(raw);
    rc = install_schedule(ctx, &all, std::move(comp), true);
    if (rc != RFAST_OK) return rc;
    ctx->round = round;
    return RFAST_OK;
} catch (const std::bad_alloc&) {
    return set_err(ctx, RFAST_ENOMEM, "host allocation failed");
} catch (...) {
    return set_err(ctx, RFAST_EINVAL, "unexpected failure in rfast_append_schedule");
}

int rfast_reset(rfast_ctx* ctx) {
    if (!ctx) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    return reset_state(ctx);
}

// Enqueues the kernels of rounds [r0, r1) on the handle's stream.
static int issue_rounds(rfast_ctx* ctx, int r0, int r1) {
    const Compiled& c = ctx->comp;
    RoundArgs a{};
    a.mix_slot = ctx->d_mix_slot; a.mix_w = ctx->d_mix_w;
    a.news_new = ctx->d_news_new; a.news_prev = ctx->d_news_prev;
    a.out_cur = ctx->d_out_cur; a.out_new = ctx->d_out_new; a.out_a = ctx->d_out_a;
    a.x = ctx->x; a.z = ctx->z; a.zc = ctx->zc; a.vbuf = ctx->vbuf; a.rbuf = ctx->rbuf; a.rlo_off = ctx->rlo_off();
    a.stride = ctx->stride; a.n4 = (int)(ctx->stride / 4); a.alpha = ctx->alpha;
    const bool pf = (size_t)ctx->n * ctx->stride * sizeof(float) > ((size_t)64 << 20);   // one state array against half of L2
    for (int r = r0; r < r1; ++r) {
        const int nev = c.act_ptr[r + 1] - c.act_ptr[r];
        if (nev == 0) continue;
        a.ev = ctx->d_ev + c.act_ptr[r];
        if (!ctx->alpha_round.empty()) a.alpha = ctx->alpha_round[r];
        if (ctx->model == RFAST_MODEL_QUAD_DIAG) {
            if (ctx->compensated) k_fused_quad<1, true><<<tile_grid(a.n4, 1, nev), kThreads, 0, ctx->stream>>>(a, ctx->quad_d, ctx->quad_b);
            else k_fused_quad<1, false><<<tile_grid(a.n4, 1, nev), kThreads, 0, ctx->stream>>>(a, ctx->quad_d, ctx->quad_b);
            ctx->launches += 1;
        } else if (ctx->model == RFAST_MODEL_LOGISTIC_SPARSE && ctx->opt_fused && ctx->fused_cluster > 0) {
            int rc = launch_logit_fused(ctx, a, a.ev, nev);
            if (rc != RFAST_OK) return rc;
        } else {
            const int64_t gplane = (int64_t)ctx->n * ctx->stride;
            const dim3 tg = tile_grid(a.n4, 1, nev);
            if (ctx->model == RFAST_MODEL_MLP) {
                if (pf) k_mix<1, true, true><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->xb);
                else k_mix<1, true, false><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->xb);
            } else {
                if (pf) k_mix<1, false, true><<<tg, kThreads, 0, ctx->stream>>>(a, nullptr);
                else k_mix<1, false, false><<<tg, kThreads, 0, ctx->stream>>>(a, nullptr);
            }
            ctx->launches += 1;
            int rc = launch_gradients(ctx, a.ev, nev);
            if (rc != RFAST_OK) return rc;
            if (ctx->model == RFAST_MODEL_LOGISTIC_SPARSE) {
                if ((rc = launch_logit_track(ctx, a, a.ev, nev, 0)) != RFAST_OK) return rc;
            } else {
                if (ctx->compensated) {
                    if (pf) k_track<1, true, true><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->gbuf, gplane);
                    else k_track<1, true, false><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->gbuf, gplane);
                } else {
                    if (pf) k_track<1, false, true><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->gbuf, gplane);
                    else k_track<1, false, false><<<tg, kThreads, 0, ctx->stream>>>(a, ctx->gbuf, gplane);
                }
                ctx->launches += 1;
            }
        }
    }
    CK(cudaGetLastError());
    return RFAST_OK;
}

int rfast_run(rfast_ctx* ctx, int32_t rounds, int sync) {
    if (!ctx) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (rounds < 0 || ctx->round + (int64_t)rounds > ctx->comp.K)
        return set_err(ctx, RFAST_ESTATE, "run would pass the end of the schedule");
    const int r0 = ctx->round, r1 = ctx->round + rounds;
    // Many short kernels per round make the launch path the bottleneck of the small problems:
    // the rounds of one call are recorded once into CUDA graphs and replayed when the same
    // span is run again (after a reset).  The legacy default stream cannot be captured; there
    // the kernels are launched directly.
    const bool graph_ok = ctx->opt_graphs && ctx->stream != nullptr && rounds >= 2;
    if (ctx->persist_ok && ctx->opt_persistent && rounds >= 1) {
        PersistArgs P{};
        P.a.mix_slot = ctx->d_mix_slot; P.a.mix_w = ctx->d_mix_w;
        P.a.news_new = ctx->d_news_new; P.a.news_prev = ctx->d_news_prev;
        P.a.out_cur = ctx->d_out_cur; P.a.out_new = ctx->d_out_new; P.a.out_a = ctx->d_out_a;
        P.a.x = ctx->x; P.a.z = ctx->z; P.a.zc = ctx->zc; P.a.vbuf = ctx->vbuf; P.a.rbuf = ctx->rbuf; P.a.rlo_off = ctx->rlo_off();
        P.a.stride = ctx->stride; P.a.n4 = (int)(ctx->stride / 4); P.a.alpha = ctx->alpha;
        P.a.ev = ctx->d_ev;
        P.g = grad_args(ctx, ctx->d_ev);
        P.use_all = (ctx->model == RFAST_MODEL_LEAST_SQUARES && ctx->batch == 0) ? 1 : 0;
        if (P.use_all) P.g.B = ctx->rows;
        P.act_ptr = ctx->d_act_ptr; P.alpha_round = ctx->d_alpha_round; P.r0 = r0; P.r1 = r1;
        P.feat = ctx->feat; P.target = ctx->target; P.label = ctx->label; P.scratch = ctx->scratch;
        P.bar = ctx->d_bar; P.status = ctx->d_pstatus;
        P.xs_off = persist_xs_off(ctx); P.rows_per_item = 4;
        P.phantom = (unsigned int)ctx->opt_phantom; P.limit_ns = (unsigned long long)ctx->opt_wait_limit_ms * 1000000ull;
        CK(cudaMemsetAsync(ctx->d_pstatus, 0, sizeof(int), ctx->stream));
        CK(cudaMemsetAsync(ctx->d_bar, 0, sizeof(unsigned int), ctx->stream));
        void* args[] = {&P};
        CK(cudaLaunchCooperativeKernel(persist_kernel(ctx), dim3(ctx->persist_grid), dim3(kThreads), args,
                                       persist_smem(ctx), ctx->stream));
        ctx->launches += 1;
    } else if (graph_ok && !ctx->graph_chunks.empty() && ctx->graph_r0 == r0 && ctx->graph_r1 == r1) {
        for (const auto& gc : ctx->graph_chunks) {
            CK(cudaGraphLaunch(gc.exec, ctx->stream));
            ctx->launches += gc.launches;
        }
    } else if (graph_ok) {
        // The span is recorded as a sequence of graphs of about kChunkLaunches kernels, each
        // launched as soon as it is instantiated: the device works on one chunk while the host
        // records the next, so a first run does not wait for the whole span to be captured.
        constexpr int64_t kChunkLaunches = 1024;
        for (auto& gc : ctx->graph_chunks) cudaGraphExecDestroy(gc.exec);
        ctx->graph_chunks.clear();
        ctx->graph_r0 = ctx->graph_r1 = -1;
        const int per_round = ctx->model == RFAST_MODEL_QUAD_DIAG ? 1 : ctx->model == RFAST_MODEL_MLP ? 6 : 4;
        const int chunk_rounds = (int)std::max<int64_t>(2, kChunkLaunches / per_round);
        for (int ra = r0; ra < r1; ra += chunk_rounds) {
            const int rb = std::min(r1, ra + chunk_rounds);
            const int64_t l0 = ctx->launches;
            CK(cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
            int rc = issue_rounds(ctx, ra, rb);
            cudaGraph_t graph = nullptr;
            cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph);
            if (rc != RFAST_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
            if (e != cudaSuccess) return set_err(ctx, RFAST_ECUDA, std::string("cudaStreamEndCapture: ") + cudaGetErrorString(e));
            cudaGraphExec_t exec = nullptr;
            e = cudaGraphInstantiate(&exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) return set_err(ctx, RFAST_ECUDA, std::string("cudaGraphInstantiate: ") + cudaGetErrorString(e));
            ctx->graph_chunks.push_back({exec, ctx->launches - l0});
            CK(cudaGraphLaunch(exec, ctx->stream));
        }
        ctx->graph_r0 = r0; ctx->graph_r1 = r1;
    } else {
        int rc = issue_rounds(ctx, r0, r1);
        if (rc != RFAST_OK) return rc;
    }
    ctx->round = r1;
    if (sync) {
        CK(cudaStreamSynchronize(ctx->stream));
        return check_device_status(ctx);
    }
    return RFAST_OK;
}

int rfast_set_option(rfast_ctx* ctx, int option, int64_t value) {
    if (!ctx) return RFAST_EINVAL;
    switch (option) {
        case RFAST_OPT_PERSISTENT: ctx->opt_persistent = value != 0; return RFAST_OK;
        case RFAST_OPT_GRAPHS: ctx->opt_graphs = value != 0; return RFAST_OK;
        case RFAST_OPT_WAIT_LIMIT_MS:
            if (value < 1 || value > 60000) return set_err(ctx, RFAST_EINVAL, "wait limit must be 1..60000 ms");
            ctx->opt_wait_limit_ms = value; return RFAST_OK;
        case RFAST_OPT_ONE_PASS:
        case RFAST_OPT_CLUSTER_SIZE:
            if (ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "this option must be set before a schedule is loaded (the byte accounting follows it)");
            if (option == RFAST_OPT_ONE_PASS) { ctx->opt_fused = value != 0; return RFAST_OK; }
            if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return set_err(ctx, RFAST_EINVAL, "cluster size must be 0 (automatic), 1, 2, 4 or 8");
            if (!plan_logit_fused(ctx, (int)value)) {
                plan_logit_fused(ctx, 0);
                if (value != 0) return set_err(ctx, RFAST_EINVAL, "the problem does not fit a cluster of that size");
            }
            return RFAST_OK;
        case RFAST_OPT_OPEN_END:
            if (ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "this option must be set before a schedule is loaded (the version rows follow it)");
            if (value != 0 && ctx->buckets) return set_err(ctx, RFAST_EINVAL, "rounds can be appended to running sums only, not to mass buckets");
            ctx->opt_open_end = value != 0; return RFAST_OK;
        case RFAST_OPT_PHANTOM_ARRIVALS:
            if (value < 0 || value > 1024) return set_err(ctx, RFAST_EINVAL, "phantom arrivals must be 0..1024");
            ctx->opt_phantom = value; return RFAST_OK;
        default: return set_err(ctx, RFAST_EINVAL, "unknown option");
    }
}

int rfast_sync(rfast_ctx* ctx) {
    if (!ctx) return RFAST_EINVAL;
    CK(cudaStreamSynchronize(ctx->stream));
    return check_device_status(ctx);
}

int64_t rfast_query(rfast_ctx* ctx, int what) {
    if (!ctx) return RFAST_EINVAL;
    const Compiled& c = ctx->comp;
    const bool hs = ctx->has_sched;
    switch (what) {
        case RFAST_Q_ROUND: return ctx->round;
        case RFAST_Q_EVENTS_TOTAL: return hs ? c.n_events : 0;
        case RFAST_Q_EVENTS_RUN: return hs ? c.act_ptr[ctx->round] : 0;
        case RFAST_Q_LAUNCHES: return ctx->launches;
        case RFAST_Q_BYTES_RUN: return hs ? c.round_streams[ctx->round] * 4 * ctx->p : 0;
        case RFAST_Q_BYTES_TOTAL: return hs ? c.round_streams[c.K] * 4 * ctx->p : 0;
        case RFAST_Q_METHOD_BYTES_RUN: return hs ? c.round_streams_method[ctx->round] * 4 * ctx->p : 0;
        case RFAST_Q_METHOD_BYTES_TOTAL: return hs ? c.round_streams_method[c.K] * 4 * ctx->p : 0;
        case RFAST_Q_V_SLOTS: return hs ? c.n_v_slots : 0;
        case RFAST_Q_RHO_SLOTS: return hs ? c.n_rho_slots : 0;
        case RFAST_Q_DEVICE_BYTES: return (int64_t)ctx->dev_bytes;
        case RFAST_Q_N_USED_TAU_V: return hs ? (int64_t)c.used_tau_v.size() : 0;
        case RFAST_Q_N_USED_TAU_RHO: return hs ? (int64_t)c.used_tau_rho.size() : 0;
        default: return set_err(ctx, RFAST_EINVAL, "unknown counter");
    }
}

}  // extern "C"

namespace {

// Integer state of Algorithm 1 as of the handle's current round, replayed from the compiled
// schedule: local counters, the row of every edge's latest and buffered running sum, the stamp
// and row of every node's last v packet.
struct RoundView {
    std::vector<int> t;                       // [n]   t_i
    std::vector<int> rho_latest, rho_buf;     // [E_C] row ids, -1: nothing stored (stamp 0)
    std::vector<int> tau_v, tau_rho;          // [E_R], [E_C] stamps as of the receiver's last activation
    std::vector<int> v_row, v_stamp;          // [n]   row of the last v packet if the engine holds it, else -1 / 0
};

// is a version written in round `write` and last read in round `last` held at round `round`?
inline bool version_live(int write, int last, int round) { return write < round && last >= round; }

RoundView round_view(const rfast_ctx* ctx) {
    const Compiled& c = ctx->comp;
    const int n = ctx->n;
    RoundView v;
    v.t.assign(n, 0);
    v.rho_latest.assign(ctx->Cg.E, -1);
    v.rho_buf.assign(ctx->Cg.E, -1);
    v.tau_v.assign(ctx->R.E, 0);
    v.tau_rho.assign(ctx->Cg.E, 0);
    v.v_row.assign(n, -1);
    v.v_stamp.assign(n, 0);
    const int ev_end = c.act_ptr[ctx->round];
    std::vector<int> last_ev(n, -1);
    for (int ev = 0; ev < ev_end; ++ev) {
        const EvDesc& d = c.ev[ev];
        const int i = d.node;
        v.t[i]++;
        last_ev[i] = ev;
        for (int e = ctx->R.rowptr[i], k = 0; e < ctx->R.rowptr[i + 1]; ++e, ++k) v.tau_v[e] = c.used_tau_v[c.in_r_off[ev] + k];
        for (int e = ctx->Cg.rowptr[i], k = 0; e < ctx->Cg.rowptr[i + 1]; ++e, ++k) v.tau_rho[e] = c.used_tau_rho[c.in_c_off[ev] + k];
        if (ctx->buckets) continue;
        for (int k = 0; k < d.out_cnt; ++k) v.rho_latest[c.out_edge[d.out_beg + k]] = c.out_new[d.out_beg + k];
        for (int k = 0; k < d.news_cnt; ++k) v.rho_buf[c.news_edge[d.news_beg + k]] = c.news_new[d.news_beg + k];
    }
    for (int i = 0; i < n; ++i) {
        const int ev = last_ev[i];
        if (ev >= 0 && c.v_slot[ev] >= 0 && version_live(c.v_write[ev], c.v_last[ev], ctx->round)) {
            v.v_row[i] = c.v_slot[ev];
            v.v_stamp[i] = v.t[i];
        }
    }
    return v;
}

// Rows of a pool, picked by index, straight out of / into the caller's unpadded buffer: one
// copy per row, nothing staged and nothing allocated.  A negative index reads as a zero row
// and is skipped on a write.  lo_off > 0: the pool keeps a low-order word per value that far
// behind; a write clears it.
int rows_by_index(rfast_ctx* ctx, float* pool, const std::vector<int>& idx, void* host, bool write, int64_t lo_off = 0) {
    const size_t rowb = (size_t)ctx->p * sizeof(float);
    char* h = (char*)host;
    for (size_t r = 0; r < idx.size(); ++r, h += rowb) {
        if (idx[r] < 0) {
            if (!write) std::memset(h, 0, rowb);
            continue;
        }
        float* d = pool + (int64_t)idx[r] * ctx->stride;
        if (write) {
            CK(cudaMemcpyAsync(d, h, rowb, cudaMemcpyHostToDevice, ctx->stream));
            if (lo_off > 0) CK(cudaMemsetAsync(d + lo_off, 0, rowb, ctx->stream));
        } else {
            CK(cudaMemcpyAsync(h, d, rowb, cudaMemcpyDeviceToHost, ctx->stream));
        }
    }
    CK(cudaStreamSynchronize(ctx->stream));
    return RFAST_OK;
}

// Where the engine keeps packet version (graph, id, stamp) at the current round: row id, or -1.
int packet_row(rfast_ctx* ctx, int graph, int id, int stamp, int* row, std::string& err) {
    const Compiled& c = ctx->comp;
    *row = -1;
    if (graph == 0) {
        if (id < 0 || id >= ctx->n) { err = "packet: node id out of range"; return RFAST_EINVAL; }
        if (stamp < 1 || stamp > (int)c.ev_of[id].size()) return RFAST_OK;
        const int ev = c.ev_of[id][stamp - 1];
        if (c.v_slot[ev] >= 0 && version_live(c.v_write[ev], c.v_last[ev], ctx->round)) *row = c.v_slot[ev];
        return RFAST_OK;
    }
    if (graph != 1) { err = "packet: graph must be 0 (v over G_R) or 1 (rho over G_C)"; return RFAST_EINVAL; }
    if (ctx->buckets) { err = "packet: the bucket tracker keeps no running sums"; return RFAST_ESTATE; }
    if (id < 0 || id >= ctx->Cg.E) { err = "packet: edge id out of range"; return RFAST_EINVAL; }
    const int j = ctx->Cg.col[id];
    if (stamp < 1 || stamp > (int)c.ev_of[j].size()) return RFAST_OK;
    const int64_t vid = c.out_c_off[c.ev_of[j][stamp - 1]] + ctx->Cg.opos[id];
    if (c.rho_slot[vid] >= 0 && version_live(c.rho_write[vid], c.rho_last[vid], ctx->round)) *row = c.rho_slot[vid];
    return RFAST_OK;
}

}  // namespace

extern "C" {

int rfast_snapshot(rfast_ctx* ctx, float* x_dst, float* y_dst) {
    if (!ctx || !x_dst || !y_dst) return ctx ? set_err(ctx, RFAST_EINVAL, "snapshot: null destination") : RFAST_EINVAL;
    const size_t plane = (size_t)ctx->n * ctx->stride * sizeof(float);
    if (!ctx->snap_stream) {
        CK(dev_alloc(ctx, &ctx->snap_x, (size_t)ctx->n * ctx->stride, false));
        CK(dev_alloc(ctx, &ctx->snap_y, (size_t)ctx->n * ctx->stride, false));
        CK(cudaEventCreateWithFlags(&ctx->snap_ready, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&ctx->snap_done, cudaEventDisableTiming));
        CK(cudaStreamCreateWithFlags(&ctx->snap_stream, cudaStreamNonBlocking));
        CK(cudaEventRecord(ctx->snap_done, ctx->snap_stream));
    }
    // the copy on the device waits for the previous snapshot's transfer (it reads the same buffers),
    // the transfer for the copy; the handle's stream is free again after the copy
    CK(cudaStreamWaitEvent(ctx->stream, ctx->snap_done, 0));
    CK(cudaMemcpyAsync(ctx->snap_x, ctx->x, plane, cudaMemcpyDeviceToDevice, ctx->stream));
    CK(cudaMemcpyAsync(ctx->snap_y, ctx->z, plane, cudaMemcpyDeviceToDevice, ctx->stream));
    CK(cudaEventRecord(ctx->snap_ready, ctx->stream));
    CK(cudaStreamWaitEvent(ctx->snap_stream, ctx->snap_ready, 0));
    const size_t rowb = (size_t)ctx->p * sizeof(float);
    CK(cudaMemcpy2DAsync(x_dst, rowb, ctx->snap_x, ctx->stride * sizeof(float), rowb, ctx->n, cudaMemcpyDeviceToHost, ctx->snap_stream));
    CK(cudaMemcpy2DAsync(y_dst, rowb, ctx->snap_y, ctx->stride * sizeof(float), rowb, ctx->n, cudaMemcpyDeviceToHost, ctx->snap_stream));
    CK(cudaEventRecord(ctx->snap_done, ctx->snap_stream));
    return RFAST_OK;
}

int rfast_snapshot_wait(rfast_ctx* ctx) {
    if (!ctx) return RFAST_EINVAL;
    if (ctx->snap_stream) CK(cudaStreamSynchronize(ctx->snap_stream));
    return RFAST_OK;
}

int rfast_seek(rfast_ctx* ctx, int32_t round) {
    if (!ctx) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (round < 0 || round > ctx->comp.K) return set_err(ctx, RFAST_EINVAL, "seek: round outside 0 .. K");
    CK(cudaStreamSynchronize(ctx->stream));
    ctx->round = round;
    return RFAST_OK;
}

int rfast_read_packet(rfast_ctx* ctx, int graph, int32_t id, int32_t stamp, float* dst, size_t bytes) {
    if (!ctx || !dst) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (bytes != (size_t)ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "packet: size mismatch");
    int row = -1;
    std::string err;
    const int rc = packet_row(ctx, graph, id, stamp, &row, err);
    if (rc != RFAST_OK) return set_err(ctx, rc, err);
    if (row < 0) return RFAST_NOT_HELD;
    const float* src = (graph == 0 ? ctx->vbuf : ctx->rbuf) + (int64_t)row * ctx->stride;
    CK(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return RFAST_OK;
}

int rfast_write_packet(rfast_ctx* ctx, int graph, int32_t id, int32_t stamp, const float* src, size_t bytes) {
    if (!ctx || !src) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (bytes != (size_t)ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "packet: size mismatch");
    int row = -1;
    std::string err;
    const int rc = packet_row(ctx, graph, id, stamp, &row, err);
    if (rc != RFAST_OK) return set_err(ctx, rc, err);
    if (row < 0) return RFAST_NOT_HELD;
    float* dst = (graph == 0 ? ctx->vbuf : ctx->rbuf) + (int64_t)row * ctx->stride;
    CK(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, ctx->stream));
    if (graph == 1 && ctx->rho2) CK(cudaMemsetAsync(dst + ctx->rlo_off(), 0, bytes, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return RFAST_OK;
}

int rfast_read_state(rfast_ctx* ctx, int which, void* dst, size_t bytes) try {
    if (!ctx || !dst) return RFAST_EINVAL;
    const Compiled& c = ctx->comp;
    auto ints = [&](const int* src, size_t cnt) {
        if (bytes != cnt * sizeof(int)) return set_err(ctx, RFAST_EINVAL, "read_state: size mismatch");
        if (bytes) std::memcpy(dst, src, bytes);
        return RFAST_OK;
    };
    const int n = ctx->n, n4 = (int)(ctx->stride / 4);
    auto rows_out = [&](const float* dev, int64_t rows) -> int {
        if (bytes != (size_t)rows * ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "read_state: size mismatch");
        if (rows == 0) return RFAST_OK;
        CK(cudaMemcpy2DAsync(dst, ctx->p * sizeof(float), dev, ctx->stride * sizeof(float), ctx->p * sizeof(float),
                             rows, cudaMemcpyDeviceToHost, ctx->stream));
        CK(cudaStreamSynchronize(ctx->stream));
        return RFAST_OK;
    };
    auto picked = [&](float* pool, const std::vector<int>& idx) -> int {
        if (bytes != idx.size() * (size_t)ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "read_state: size mismatch");
        return rows_by_index(ctx, pool, idx, dst, false);
    };
    const bool is_float = which <= RFAST_STATE_RHO_BUF || which == RFAST_STATE_V_LATEST;
    if (is_float) {
        int rc = check_device_status(ctx);
        if (rc != RFAST_OK) return rc;
    }
    switch (which) {
        case RFAST_STATE_X: return rows_out(ctx->x, n);
        case RFAST_STATE_Y: return rows_out(ctx->z, n);
        case RFAST_STATE_ROUND: return ints(&ctx->round, 1);
        default: break;
    }
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    switch (which) {
        case RFAST_STATE_USED_TAU_V: return ints(c.used_tau_v.data(), c.used_tau_v.size());
        case RFAST_STATE_USED_TAU_RHO: return ints(c.used_tau_rho.data(), c.used_tau_rho.size());
        case RFAST_STATE_TAU_V_END: return ints(c.tau_v_end.data(), c.tau_v_end.size());
        case RFAST_STATE_TAU_RHO_END: return ints(c.tau_rho_end.data(), c.tau_rho_end.size());
        default: break;
    }
    const RoundView rv = round_view(ctx);
    switch (which) {
        case RFAST_STATE_T_LOCAL: return ints(rv.t.data(), n);
        case RFAST_STATE_TAU_V: return ints(rv.tau_v.data(), rv.tau_v.size());
        case RFAST_STATE_TAU_RHO: return ints(rv.tau_rho.data(), rv.tau_rho.size());
        case RFAST_STATE_V_HELD: return ints(rv.v_stamp.data(), n);
        case RFAST_STATE_V_LATEST: return picked(ctx->vbuf, rv.v_row);
        case RFAST_STATE_G_LAST: {
            if (ctx->model == RFAST_MODEL_QUAD_DIAG) {
                // not stored for the element-wise objective: recomputed from x, a row at a time
                if (bytes != (size_t)n * ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "read_state: size mismatch");
                for (int i = 0; i < n; ++i) {
                    const int64_t row = (int64_t)i * ctx->stride;
                    k_quad_grad<<<dim3((n4 + kThreads - 1) / kThreads, 1), kThreads, 0, ctx->stream>>>(
                        ctx->x + row, ctx->quad_d + row, ctx->quad_b + row, ctx->row_tmp, ctx->stride, n4);
                    CK(cudaMemcpyAsync((char*)dst + (size_t)i * ctx->p * sizeof(float), ctx->row_tmp,
                                       (size_t)ctx->p * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
                }
                CK(cudaStreamSynchronize(ctx->stream));
                return RFAST_OK;
            }
            std::vector<int> idx(n);
            for (int i = 0; i < n; ++i) idx[i] = (rv.t[i] & 1) * n + i;
            return picked(ctx->gbuf, idx);
        }
        case RFAST_STATE_RHO_LATEST:
        case RFAST_STATE_RHO_BUF:
            if (ctx->buckets)
                return set_err(ctx, RFAST_ESTATE, "read_state: the bucket tracker keeps no running sums (rho, rho~ views do not exist)");
            return picked(ctx->rbuf, which == RFAST_STATE_RHO_LATEST ? rv.rho_latest : rv.rho_buf);
        default: return set_err(ctx, RFAST_EINVAL, "read_state: unknown view");
    }
} catch (...) {
    return set_err(ctx, RFAST_ENOMEM, "read_state: host allocation failed");
}

int rfast_write_state(rfast_ctx* ctx, int which, const void* src, size_t bytes) try {
    if (!ctx || !src) return RFAST_EINVAL;
    const int n = ctx->n, n4 = (int)(ctx->stride / 4);
    auto rows_in = [&](float* dev) -> int {
        if (bytes != (size_t)n * ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "write_state: size mismatch");
        CK(cudaMemcpy2DAsync(dev, ctx->stride * sizeof(float), src, ctx->p * sizeof(float), ctx->p * sizeof(float),
                             n, cudaMemcpyHostToDevice, ctx->stream));     // the padding stays zero
        return RFAST_OK;
    };
    auto picked = [&](float* pool, const std::vector<int>& idx, int64_t lo_off) -> int {
        if (bytes != idx.size() * (size_t)ctx->p * sizeof(float)) return set_err(ctx, RFAST_EINVAL, "write_state: size mismatch");
        return rows_by_index(ctx, pool, idx, const_cast<void*>(src), true, lo_off);
    };
    int rc;
    switch (which) {
        case RFAST_STATE_X:
            if ((rc = rows_in(ctx->x)) != RFAST_OK) return rc;
            if (ctx->model == RFAST_MODEL_MLP) {           // the matrix products read a bf16 copy of x
                k_rows_to_bf16<<<dim3((n4 + kThreads - 1) / kThreads, n), kThreads, 0, ctx->stream>>>(ctx->x, ctx->xb, ctx->stride, n4);
                CK(cudaGetLastError());
            }
            CK(cudaStreamSynchronize(ctx->stream));
            return RFAST_OK;
        case RFAST_STATE_Y:
            if ((rc = rows_in(ctx->z)) != RFAST_OK) return rc;
            if (ctx->zc) CK(cudaMemsetAsync(ctx->zc, 0, (size_t)n * ctx->stride * sizeof(float), ctx->stream));
            CK(cudaStreamSynchronize(ctx->stream));
            return RFAST_OK;
        default: break;
    }
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    if (which != RFAST_STATE_G_LAST && which != RFAST_STATE_RHO_LATEST && which != RFAST_STATE_RHO_BUF &&
        which != RFAST_STATE_V_LATEST)
        return set_err(ctx, RFAST_EINVAL, "write_state: only the float views can be written (integer state follows from the schedule and the round)");
    const RoundView rv = round_view(ctx);
    switch (which) {
        case RFAST_STATE_G_LAST: {
            if (ctx->model == RFAST_MODEL_QUAD_DIAG)
                return set_err(ctx, RFAST_ESTATE, "write_state: the element-wise objective keeps no gradient (it is recomputed from x)");
            std::vector<int> idx(n);
            for (int i = 0; i < n; ++i) idx[i] = (rv.t[i] & 1) * n + i;
            return picked(ctx->gbuf, idx, 0);
        }
        case RFAST_STATE_V_LATEST: return picked(ctx->vbuf, rv.v_row, 0);
        default:
            if (ctx->buckets)
                return set_err(ctx, RFAST_ESTATE, "write_state: the bucket tracker keeps no running sums (rho, rho~ views do not exist)");
            return picked(ctx->rbuf, which == RFAST_STATE_RHO_LATEST ? rv.rho_latest : rv.rho_buf, ctx->rlo_off());
    }
} catch (...) {
    return set_err(ctx, RFAST_ENOMEM, "write_state: host allocation failed");
}

static int compile_host_impl(const rfast_problem* prob, const rfast_schedule* s, int32_t* used_tau_v,
                             int32_t* used_tau_rho, int32_t* v_ver, int32_t* rho_ver, int64_t* counts,
                             uint64_t* digest, char* errbuf, size_t err_len) try {
    std::string err;
    auto done = [&](int rc) {
        if (errbuf && err_len) { std::snprintf(errbuf, err_len, "%s", err.c_str()); }
        return rc;
    };
    if (!prob || prob->n <= 0) { err = "problem is null or n <= 0"; return done(RFAST_EINVAL); }
    HostGraph R, C;
    int rc;
    if ((rc = build_host_graph(prob->G_R, prob->n, true, R, err)) != RFAST_OK) return done(rc);
    if ((rc = build_host_graph(prob->G_C, prob->n, false, C, err)) != RFAST_OK) return done(rc);
    if ((rc = check_roots(R, C, prob->root, err)) != RFAST_OK) return done(rc);
    Compiled c;
    if ((rc = compile_schedule(R, C, s, prob->batch, prob->rows, traffic_of(prob->model, prob->compensated != 0),
                               prob->tracker == RFAST_TRACKER_BUCKETS, c, err)) != RFAST_OK) return done(rc);
    if (used_tau_v) std::copy(c.used_tau_v.begin(), c.used_tau_v.end(), used_tau_v);
    if (used_tau_rho) std::copy(c.used_tau_rho.begin(), c.used_tau_rho.end(), used_tau_rho);
    if (v_ver)
        for (int64_t ev = 0; ev < c.n_events; ++ev) {
            v_ver[3 * ev] = c.v_slot[ev]; v_ver[3 * ev + 1] = c.v_write[ev]; v_ver[3 * ev + 2] = c.v_last[ev];
        }
    if (rho_ver)
        for (size_t v = 0; v < c.rho_slot.size(); ++v) {
            rho_ver[3 * v] = c.rho_slot[v]; rho_ver[3 * v + 1] = c.rho_write[v]; rho_ver[3 * v + 2] = c.rho_last[v];
        }
    if (counts) {
        counts[0] = c.n_v_slots; counts[1] = c.n_rho_slots; counts[2] = c.n_events; counts[3] = c.round_streams[c.K];
    }
    if (digest) {          // everything the kernels are driven by, folded into one number
        uint64_t h = 1469598103934665603ull;
        auto mix = [&](const void* ptr, size_t bytes) {
            const unsigned char* q = (const unsigned char*)ptr;
            for (size_t k = 0; k < bytes; ++k) { h ^= q[k]; h *= 1099511628211ull; }
        };
        auto vec = [&](const auto& v) { if (!v.empty()) mix(v.data(), v.size() * sizeof(v[0])); };
        vec(c.ev); vec(c.mix_slot); vec(c.mix_w); vec(c.news_new); vec(c.news_prev); vec(c.news_edge);
        vec(c.out_cur); vec(c.out_new); vec(c.out_a); vec(c.out_edge); vec(c.round_streams); vec(c.round_streams_method);
        *digest = h;
    }
    return done(RFAST_OK);
} catch (...) {
    if (errbuf && err_len) std::snprintf(errbuf, err_len, "host allocation failed");
    return RFAST_ENOMEM;
}

int rfast_compile_host(const rfast_problem* prob, const rfast_schedule* s, int32_t* used_tau_v,
                       int32_t* used_tau_rho, int32_t* v_ver, int32_t* rho_ver, int64_t* counts,
                       char* errbuf, size_t err_len) {
    return compile_host_impl(prob, s, used_tau_v, used_tau_rho, v_ver, rho_ver, counts, nullptr, errbuf, err_len);
}

int rfast_compile_append_check(const rfast_problem* prob, const rfast_schedule* first, const rfast_schedule* more,
                               int64_t* counts, char* errbuf, size_t err_len) try {
    std::string err;
    auto done = [&](int rc) {
        if (errbuf && err_len) { std::snprintf(errbuf, err_len, "%s", err.c_str()); }
        return rc;
    };
    if (!prob || prob->n <= 0) { err = "problem is null or n <= 0"; return done(RFAST_EINVAL); }
    HostGraph R, C;
    int rc;
    if ((rc = build_host_graph(prob->G_R, prob->n, true, R, err)) != RFAST_OK) return done(rc);
    if ((rc = build_host_graph(prob->G_C, prob->n, false, C, err)) != RFAST_OK) return done(rc);
    if ((rc = check_roots(R, C, prob->root, err)) != RFAST_OK) return done(rc);
    const ModelTraffic mt = traffic_of(prob->model, prob->compensated != 0);
    const bool buckets = prob->tracker == RFAST_TRACKER_BUCKETS;
    Compiled c1, c2, whole;
    std::vector<int> holds;
    if (first && first->K >= 0) holds.push_back(first->K);
    if ((rc = compile_schedule(R, C, first, prob->batch, prob->rows, mt, buckets, c1, err, &holds)) != RFAST_OK) return done(rc);
    auto raw = raw_of(first, prob->batch);
    if (const char* bad = append_raw(*raw, more, prob->n, prob->batch, prob->alpha)) { err = bad; return done(RFAST_ESCHED); }
    const rfast_schedule all = raw->view();
    if (holds.back() != all.K) holds.push_back(all.K);
    if ((rc = compile_schedule(R, C, &all, prob->batch, prob->rows, mt, buckets, c2, err, &holds)) != RFAST_OK) return done(rc);
    if (!prefix_same(c1, c2)) { err = "appending rounds moved a version row of the rounds already loaded"; return done(RFAST_ESCHED); }
    // the stamps consumed are those of the whole schedule compiled at once
    if ((rc = compile_schedule(R, C, &all, prob->batch, prob->rows, mt, buckets, whole, err)) != RFAST_OK) return done(rc);
    if (whole.used_tau_v != c2.used_tau_v || whole.used_tau_rho != c2.used_tau_rho || whole.t_end != c2.t_end) {
        err = "the appended schedule consumes other stamps than the whole schedule compiled at once";
        return done(RFAST_ESCHED);
    }
    if (counts) {
        counts[0] = c1.n_v_slots; counts[1] = c1.n_rho_slots; counts[2] = c2.n_v_slots; counts[3] = c2.n_rho_slots;
        counts[4] = whole.n_v_slots; counts[5] = whole.n_rho_slots;
    }
    return done(RFAST_OK);
} catch (const std::bad_alloc&) {
    if (errbuf && err_len) std::snprintf(errbuf, err_len, "host allocation failed");
    return RFAST_ENOMEM;
}

int rfast_compile_digest(const rfast_problem* prob, const rfast_schedule* s, uint64_t* digest, char* errbuf, size_t err_len) {
    if (!digest) return RFAST_EINVAL;
    return compile_host_impl(prob, s, nullptr, nullptr, nullptr, nullptr, nullptr, digest, errbuf, err_len);
}

}  // extern "C"

namespace {

struct CkptHeader {
    uint64_t magic, sched_hash;
    int64_t  p, stride, n_events;
    int32_t  n, model, compensated, K, n_v_slots, n_rho_slots, round, pad;
};
constexpr uint64_t kCkptMagic = 0x5246415354434B31ull;   // "RFASTCK1"

// the device buffers that make up the state, in blob order
std::vector<std::pair<void*, size_t>> state_buffers(rfast_ctx* c) {
    const size_t plane = (size_t)c->n * c->stride * sizeof(float);
    std::vector<std::pair<void*, size_t>> v;
    v.push_back({c->x, plane});
    v.push_back({c->z, plane});
    if (c->zc) v.push_back({c->zc, plane});
    if (c->gbuf) v.push_back({c->gbuf, 2 * plane});
    if (c->xb) v.push_back({c->xb, plane / 2});
    v.push_back({c->vbuf, (size_t)c->comp.n_v_slots * c->stride * sizeof(float)});
    v.push_back({c->rbuf, (size_t)c->comp.n_rho_slots * c->stride * sizeof(float) * (c->rho2 ? 2 : 1)});
    return v;
}

CkptHeader make_header(rfast_ctx* c) {
    CkptHeader h{};
    h.magic = kCkptMagic; h.sched_hash = c->sched_hash;
    h.p = c->p; h.stride = c->stride; h.n_events = c->comp.n_events;
    h.n = c->n; h.model = c->model; h.compensated = c->compensated + (c->rho2 ? 1 : 0); h.K = c->comp.K;
    h.n_v_slots = c->comp.n_v_slots; h.n_rho_slots = c->comp.n_rho_slots; h.round = c->round;
    h.pad = c->buckets ? 1 : 0;
    return h;
}

}  // namespace

extern "C" {

int64_t rfast_checkpoint_size(rfast_ctx* ctx) {
    if (!ctx) return RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    size_t total = sizeof(CkptHeader);
    for (auto& b : state_buffers(ctx)) total += b.second;
    return (int64_t)total;
}

int rfast_checkpoint_save(rfast_ctx* ctx, void* dst, size_t bytes) {
    if (!ctx || !dst) return RFAST_EINVAL;
    const int64_t need = rfast_checkpoint_size(ctx);
    if (need < 0) return (int)need;
    if ((size_t)need != bytes) return set_err(ctx, RFAST_EINVAL, "checkpoint_save: size mismatch");
    int rc = check_device_status(ctx);
    if (rc != RFAST_OK) return rc;
    CkptHeader h = make_header(ctx);
    std::memcpy(dst, &h, sizeof h);
    char* q = (char*)dst + sizeof h;
    for (auto& b : state_buffers(ctx)) {
        if (b.second) CK(cudaMemcpyAsync(q, b.first, b.second, cudaMemcpyDeviceToHost, ctx->stream));
        q += b.second;
    }
    CK(cudaStreamSynchronize(ctx->stream));
    return RFAST_OK;
}

int rfast_checkpoint_load(rfast_ctx* ctx, const void* src, size_t bytes) {
    if (!ctx || !src) return RFAST_EINVAL;
    const int64_t need = rfast_checkpoint_size(ctx);
    if (need < 0) return (int)need;
    if ((size_t)need != bytes) return set_err(ctx, RFAST_EINVAL, "checkpoint_load: size mismatch");
    CkptHeader h;
    std::memcpy(&h, src, sizeof h);
    CkptHeader mine = make_header(ctx);
    mine.round = h.round;
    if (std::memcmp(&h, &mine, sizeof h) != 0 || h.round < 0 || h.round > ctx->comp.K)
        return set_err(ctx, RFAST_EINVAL, "checkpoint_load: blob belongs to another problem or schedule");
    const char* q = (const char*)src + sizeof h;
    for (auto& b : state_buffers(ctx)) {
        if (b.second) CK(cudaMemcpyAsync(b.first, q, b.second, cudaMemcpyHostToDevice, ctx->stream));
        q += b.second;
    }
    CK(cudaStreamSynchronize(ctx->stream));
    ctx->round = h.round;
    return RFAST_OK;
}

// Full gradient of F = sum_i f_i at the mean iterate for the objectives that sample minibatches,
// out of the very kernels the activations use: the shard of every node is walked in chunks of B
// rows (a minibatch that is rows [cB, (c+1)B) of the shard), all nodes at once, from a state whose
// rows all hold xbar; the mean over the chunks of a node's minibatch gradients is its full
// gradient (the L2 term is in each of them).  x (and its bf16 copy) is moved aside and put back,
// bit for bit; the gradients land in the rows of the gradient pool that hold no remembered
// gradient.  Leaves sum_c (grad F(xbar))_c^2 per block in part[block][5].
static int sampled_full_gradient(rfast_ctx* ctx, const RoundView& rv, int blocks) {
    const int n = ctx->n, B = ctx->batch, chunks = ctx->rows / B;
    const size_t plane = (size_t)n * ctx->stride;
    const int n4 = (int)(ctx->stride / 4);
    if (!ctx->d_diag_x) {
        // sizes follow the problem, not the schedule: kept for the life of the handle
        CK(dev_alloc(ctx, &ctx->d_diag_x, plane, false));
        CK(dev_alloc(ctx, &ctx->d_diag_acc, (size_t)ctx->stride, false));
        CK(dev_alloc(ctx, &ctx->d_diag_ev, (size_t)chunks * n, false));
        CK(dev_alloc(ctx, &ctx->d_diag_bidx, (size_t)chunks * n * B, false));
        if (!ctx->d_xbar) {
            CK(dev_alloc(ctx, &ctx->d_xbar, (size_t)ctx->stride, true));
            CK(cudaMemsetAsync(ctx->d_xbar, 0, ctx->stride * sizeof(float), ctx->stream));
        }
        std::vector<int> bidx((size_t)chunks * n * B);
        for (int c = 0; c < chunks; ++c)
            for (int i = 0; i < n; ++i)
                for (int k = 0; k < B; ++k) bidx[((size_t)c * n + i) * B + k] = c * B + k;
        CK(cudaMemcpy(ctx->d_diag_bidx, bidx.data(), bidx.size() * sizeof(int), cudaMemcpyHostToDevice));
    }
    std::vector<EvDesc> evs((size_t)chunks * n);
    std::vector<int> sel(n);
    for (int i = 0; i < n; ++i) sel[i] = ((rv.t[i] & 1) ^ 1) * n + i;          // the row that holds no remembered gradient
    for (int c = 0; c < chunks; ++c)
        for (int i = 0; i < n; ++i) {
            EvDesc d{};
            d.node = i; d.v_out = -1; d.g_par = rv.t[i] & 1; d.sample = c * n + i;
            evs[(size_t)c * n + i] = d;
        }
    CK(cudaMemcpy(ctx->d_diag_ev, evs.data(), evs.size() * sizeof(EvDesc), cudaMemcpyHostToDevice));
    int* d_sel = ctx->d_diag_idx;                                                // n ints, free again by now
    CK(cudaMemcpyAsync(d_sel, sel.data(), n * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
    CK(cudaMemcpyAsync(ctx->d_diag_x, ctx->x, plane * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
    k_diag_fill_rows<<<dim3((n4 + kThreads - 1) / kThreads, n), kThreads, 0, ctx->stream>>>(ctx->x, ctx->d_xbar, ctx->stride, n4);
    if (ctx->xb) k_rows_to_bf16<<<dim3((n4 + kThreads - 1) / kThreads, n), kThreads, 0, ctx->stream>>>(ctx->x, ctx->xb, ctx->stride, n4);
    CK(cudaMemsetAsync(ctx->d_diag_acc, 0, ctx->stride * sizeof(double), ctx->stream));
    int* const sched_bidx = ctx->d_batch_idx;
    const int64_t launches = ctx->launches;                                      // counts what rfast_run launches only
    ctx->d_batch_idx = ctx->d_diag_bidx;
    int rc = RFAST_OK;
    for (int c = 0; c < chunks && rc == RFAST_OK; ++c) {
        const EvDesc* ev = ctx->d_diag_ev + (size_t)c * n;
        rc = launch_gradients(ctx, ev, n);
        if (rc == RFAST_OK && ctx->model == RFAST_MODEL_LOGISTIC_SPARSE) {
            RoundArgs a{};
            a.stride = ctx->stride; a.n4 = n4;
            rc = launch_logit_track(ctx, a, ev, n, 1);
        }
        if (rc == RFAST_OK)
            k_diag_accumulate<<<blocks, kThreads, 0, ctx->stream>>>(ctx->gbuf, d_sel, n, ctx->stride, ctx->p, ctx->d_diag_acc);
    }
    ctx->d_batch_idx = sched_bidx;
    ctx->launches = launches;
    // x back in place whatever happened above
    cudaMemcpyAsync(ctx->x, ctx->d_diag_x, plane * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream);
    if (ctx->xb) k_rows_to_bf16<<<dim3((n4 + kThreads - 1) / kThreads, n), kThreads, 0, ctx->stream>>>(ctx->x, ctx->xb, ctx->stride, n4);
    if (rc != RFAST_OK) return rc;
    k_diag_norm2<<<blocks, kThreads, 0, ctx->stream>>>(ctx->d_diag_acc, ctx->p, 1.0 / chunks, ctx->d_diag_part);
    CK(cudaGetLastError());
    return RFAST_OK;
}

int rfast_diagnostics(rfast_ctx* ctx, double* out, int32_t n_out) try {
    if (!ctx || !out || (n_out != 5 && n_out != 7 && n_out != 8))
        return ctx ? set_err(ctx, RFAST_EINVAL, "diagnostics: n_out must be 5, 7 or 8") : RFAST_EINVAL;
    if (!ctx->has_sched) return set_err(ctx, RFAST_ESTATE, "no schedule loaded");
    const Compiled& c = ctx->comp;
    const int n = ctx->n;
    // which rows hold the current g, the latest rho and the buffered rho of every edge
    const RoundView rv = round_view(ctx);
    std::vector<int> gsel(n), latest = rv.rho_latest, buf = rv.rho_buf;
    int E = ctx->Cg.E;
    if (ctx->buckets) {
        // the mass in transit is the content of the buckets begun and not yet consumed
        latest.clear();
        for (size_t v = 0; v < c.rho_leader.size(); ++v)
            if (c.rho_leader[v] == (int64_t)v && c.rho_write[v] < ctx->round && c.rho_last[v] >= ctx->round)
                latest.push_back(c.rho_slot[v]);
        E = (int)latest.size();
        buf.assign(latest.size(), -1);
    }
    for (int i = 0; i < n; ++i) gsel[i] = (rv.t[i] & 1) * n + i;
    if ((int64_t)n + 2 * (int64_t)E > ctx->diag_idx_cap) return set_err(ctx, RFAST_ESTATE, "diagnostics: scratch too small");
    const int blocks = (int)((ctx->p + kThreads - 1) / kThreads);
    int *d_gsel = ctx->d_diag_idx, *d_latest = d_gsel + n, *d_buf = d_latest + E;
    CK(cudaMemcpyAsync(d_gsel, gsel.data(), n * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
    if (E > 0) {
        CK(cudaMemcpyAsync(d_latest, latest.data(), E * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
        CK(cudaMemcpyAsync(d_buf, buf.data(), E * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
    }
    const bool want_mf = n_out >= 7;
    const bool ls = ctx->model == RFAST_MODEL_LEAST_SQUARES;
    const bool sampled = want_mf && ctx->batch > 0 && ctx->rows % ctx->batch == 0 &&
                         (ctx->model == RFAST_MODEL_SOFTMAX || ctx->model == RFAST_MODEL_MLP || ctx->model == RFAST_MODEL_LOGISTIC_SPARSE);
    const bool sampled_model = ctx->model == RFAST_MODEL_SOFTMAX || ctx->model == RFAST_MODEL_MLP || ctx->model == RFAST_MODEL_LOGISTIC_SPARSE;
    const bool lossy = n_out == 8 && sampled_model && (ctx->model == RFAST_MODEL_LOGISTIC_SPARSE || ctx->C <= 32);
    if (lossy && !ctx->d_diag_rowloss) CK(dev_alloc(ctx, &ctx->d_diag_rowloss, (size_t)n * ctx->rows, false));
    if ((sampled || lossy) && !ctx->d_xbar) {          // the mean iterate is wanted on the device
        CK(dev_alloc(ctx, &ctx->d_xbar, (size_t)ctx->stride, true));
        CK(cudaMemsetAsync(ctx->d_xbar, 0, ctx->stride * sizeof(float), ctx->stream));
    }
    k_diagnostics<<<blocks, kThreads, 0, ctx->stream>>>(ctx->x, ctx->z, ctx->zc, ctx->gbuf, d_gsel, ctx->quad_d,
                                                          ctx->quad_b, ctx->rbuf, ctx->rlo_off(), d_latest, d_buf, n, E,
                                                          ctx->stride, ctx->p, want_mf && (ls || sampled || lossy) ? ctx->d_xbar : nullptr,
                                                          ctx->d_diag_part);
    if (want_mf && ls) {
        k_diag_ls_residual<<<dim3((ctx->rows + 7) / 8, n), 256, 0, ctx->stream>>>(ctx->feat, ctx->target, ctx->d_xbar,
                                                                                    ctx->d_diag_res, ctx->rows, ctx->F);
        k_diag_ls_grad<<<blocks, kThreads, 0, ctx->stream>>>(ctx->feat, ctx->d_xbar, ctx->d_diag_res, n, ctx->rows,
                                                               ctx->F, ctx->l2, ctx->d_diag_part);
    }
    CK(cudaGetLastError());
    if (sampled) {
        int rc = sampled_full_gradient(ctx, rv, blocks);
        if (rc != RFAST_OK) return rc;
    }
    std::vector<double> rowloss;
    if (lossy) {                                           // F(xbar): every row of every shard, a warp per row
        const dim3 grid((ctx->rows + 7) / 8, n);
        if (ctx->model == RFAST_MODEL_SOFTMAX)
            k_diag_loss_softmax<<<grid, 256, 0, ctx->stream>>>(ctx->feat, ctx->label, ctx->d_xbar, ctx->d_diag_rowloss, ctx->rows, ctx->F, ctx->C);
        else if (ctx->model == RFAST_MODEL_MLP)
            k_diag_loss_mlp<<<grid, 256, 8 * (size_t)ctx->H * sizeof(double), ctx->stream>>>(ctx->feat, ctx->label, ctx->d_xbar, ctx->d_diag_rowloss,
                                                                                             ctx->rows, ctx->F, ctx->H, ctx->C);
        else
            k_diag_loss_logistic<<<grid, 256, 0, ctx->stream>>>(ctx->sp_ptr, ctx->sp_col, ctx->sp_val, ctx->label, ctx->d_xbar, ctx->d_diag_rowloss, ctx->rows);
        CK(cudaGetLastError());
        rowloss.resize((size_t)n * ctx->rows);
        CK(cudaMemcpyAsync(rowloss.data(), ctx->d_diag_rowloss, rowloss.size() * sizeof(double), cudaMemcpyDeviceToHost, ctx->stream));
    }
    std::vector<double> part((size_t)blocks * kDiagSlots);
    CK(cudaMemcpyAsync(part.data(), ctx->d_diag_part, part.size() * sizeof(double), cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));       // the host vectors above may go now
    double cons = 0, xb2 = 0, res = 0, gs = 0, z2 = 0, gf2 = 0, fl = 0;
    for (int b = 0; b < blocks; ++b) {          // fixed order: the same bits on every run
        const double* q = part.data() + (size_t)b * kDiagSlots;
        cons += q[0]; xb2 += q[1];
        res = std::max(res, q[2]); gs = std::max(gs, q[3]);
        z2 += q[4]; gf2 += q[5]; fl += q[6];
    }
    out[0] = std::sqrt(std::max(cons, 0.0)); out[1] = std::sqrt(xb2); out[2] = res; out[3] = gs; out[4] = std::sqrt(z2);
    if (want_mf) {
        const bool have = ls || sampled || ctx->model == RFAST_MODEL_QUAD_DIAG;
        out[5] = have ? std::sqrt(gf2) : std::nan("");
        out[6] = have ? gf2 + std::max(cons, 0.0) : std::nan("");
        if (n_out == 8) {
            out[7] = have && !sampled_model ? fl : std::nan("");
            if (lossy) {                                   // mean loss per shard + the L2 term of every node, fixed order
                double tot = 0;
                for (int i = 0; i < n; ++i) {
                    double si = 0;
                    for (int k = 0; k < ctx->rows; ++k) si += rowloss[(size_t)i * ctx->rows + k];
                    tot += si / ctx->rows;
                }
                out[7] = tot + 0.5 * n * (double)ctx->l2 * xb2;
            }
        }
    }
    return RFAST_OK;
} catch (...) {
    return set_err(ctx, RFAST_ENOMEM, "diagnostics: host allocation failed");
}

}  // extern "C"
