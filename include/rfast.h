/*
 * rfast.h -- C ABI of the R-FAST activation engine (one CUDA device, sm_100a).
 *
 * The engine simulates n workers running R-FAST (Robust Fully-Asynchronous Stochastic
 * Gradient Tracking) on one GPU.  The problem is the paper's eq. (1): min_x sum_i f_i(x)
 * over n workers that exchange packets over two graphs, G_R = G(W) with W row-stochastic
 * (consensus, "pull") and G_C = G(A) with A column-stochastic (tracking, "push"), sharing a
 * root (Assumptions 1-2).  Asynchrony is data: a schedule says which nodes are active in
 * each round and, for every packet, whether it is lost or how late it becomes usable
 * (Algorithm 2, step S.0; Assumption 3).
 *
 * Conventions
 *   - Every call returns an int status: RFAST_OK or a negative RFAST_E* code.  Nothing
 *     throws, aborts or prints.  rfast_last_error() returns a text for the last failure.
 *   - All pointers in rfast_problem / rfast_schedule are HOST pointers owned by the caller;
 *     the library copies what it needs before the call returns.  Output buffers of
 *     rfast_read_state are HOST pointers owned by the caller.
 *   - The handle owns all device memory; rfast_destroy frees it.
 *   - All device work is enqueued on the CUDA stream given at create time (a cudaStream_t
 *     passed as void*; NULL = the legacy default stream).  One handle is not thread-safe.
 *   - Node ids are 0-based.  Edge (j, i) of G(M) exists iff M_ij > 0; then j sends to i
 *     (Section III-A).  Graphs are given by receiver (CSR over receivers).
 *   - There is no CPU fallback: without a CUDA device rfast_create fails with RFAST_ECUDA.
 */
#ifndef RFAST_H
#define RFAST_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RFAST_OK         0
#define RFAST_EINVAL   (-1)  /* bad argument / size mismatch */
#define RFAST_EGRAPH   (-2)  /* Assumption 1 or 2 violated */
#define RFAST_ESCHED   (-3)  /* inconsistent schedule arrays */
#define RFAST_ENOMEM   (-4)  /* host or device allocation failed */
#define RFAST_ECUDA    (-5)  /* CUDA runtime error (text in rfast_last_error) */
#define RFAST_ETIMEOUT (-6)  /* a bounded device-side wait ran out */
#define RFAST_ESTATE   (-7)  /* call not valid in this state (e.g. run past the schedule) */

typedef struct rfast_ctx rfast_ctx;

/* Weight matrix M (W or A) by receiver.  Row i lists the in-neighbours of i:
 * col[rowptr[i] .. rowptr[i+1]) are sender ids j in strictly ascending order, j != i, and
 * w[e] = M[i][col[e]] > 0.  diag[i] = M[i][i] > 0 (Assumption 1 i). */
typedef struct rfast_graph {
    int32_t        n_edges;
    const int32_t* rowptr;   /* [n+1] */
    const int32_t* col;      /* [n_edges] */
    const float*   w;        /* [n_edges] */
    const float*   diag;     /* [n] */
} rfast_graph;

/* Local objectives f_i.  A minibatch gradient is the mean over the B sampled rows of node i's
 * shard; each f_i carries its own (l2/2)||x||^2.  Parameter layouts (x is one flat vector):
 *   QUAD_DIAG        f_i(x) = 0.5 || d_i .* (x - b_i) ||^2, deterministic, element-wise
 *   LEAST_SQUARES    f_i(x) = 1/(2B) sum_k (a_k.x - y_k)^2;  batch = 0 means the whole shard
 *   SOFTMAX          x = [W (C x F, row c = class c) | bias (C)], cross-entropy
 *   MLP              x = [W1 (H x F) | b1 (H) | W2 (C x H) | b2 (C)], hidden = relu(W1 a + b1),
 *                    cross-entropy; operands of the matrix products are rounded to bf16
 *                    (round-to-nearest-even from fp32), accumulation in fp32
 *   LOGISTIC_SPARSE  f_i(x) = 1/B sum_k log(1 + exp(-y_k a_k.x)), y in {-1,+1}, a_k sparse */
enum {
    RFAST_MODEL_QUAD_DIAG       = 0,
    RFAST_MODEL_LEAST_SQUARES   = 1,
    RFAST_MODEL_SOFTMAX         = 2,
    RFAST_MODEL_MLP             = 3,
    RFAST_MODEL_LOGISTIC_SPARSE = 4
};

typedef struct rfast_problem {
    int32_t     n;            /* workers */
    int32_t     root;         /* a common root of G(W) and G(A^T) (Assumption 2) */
    int64_t     p;            /* dimension of x */
    float       alpha;        /* constant step size gamma (Algorithm 1, S1) */
    float       l2;           /* coefficient of the (l2/2)||x||^2 term in every f_i */
    rfast_graph G_R;          /* W, row-stochastic    */
    rfast_graph G_C;          /* A, column-stochastic */
    int32_t     model;        /* RFAST_MODEL_* */
    int32_t     batch;        /* B rows per activation (0: QUAD_DIAG, or whole shard for LEAST_SQUARES) */
    int32_t     rows;         /* rows in every node's shard (0 for QUAD_DIAG) */
    int32_t     n_features;   /* F (LEAST_SQUARES: F = p; LOGISTIC_SPARSE: F = p) */
    int32_t     n_classes;    /* C (SOFTMAX, MLP) */
    int32_t     n_hidden;     /* H (MLP) */
    const float*   quad_d;    /* [n][p]            QUAD_DIAG */
    const float*   quad_b;    /* [n][p]            QUAD_DIAG */
    const float*   feat;      /* [n][rows][F]      dense features */
    const float*   target;    /* [n][rows]         LEAST_SQUARES */
    const int32_t* label;     /* [n][rows]         class id (SOFTMAX, MLP) or -1/+1 (LOGISTIC_SPARSE) */
    const int64_t* sp_rowptr; /* [n*rows+1]        LOGISTIC_SPARSE, CSR over all shards, */
    const int32_t* sp_col;    /*                   columns strictly ascending inside a row */
    const float*   sp_val;
    const float*   x0;        /* [n][p] initial iterates, or NULL for zeros */
    int32_t     compensated;  /* tracker arithmetic of S2b/S2c: 0 = plain fp32; 1 = the tracker is  */
                              /* carried as a sum of two floats and the rounding errors of the      */
                              /* mass-moving operations are fed back (keeps the conservation of      */
                              /* Lemma 3 over long horizons; one more fp32 stream read and written); */
                              /* 2 = the running sums rho are two floats as well (their fp32         */
                              /* resolution otherwise limits what a receiver sees once they have     */
                              /* grown; doubles the rho traffic)                                     */
    int32_t     tracker;      /* how the mass in transit over G_C is kept (same mathematics):         */
                              /* RFAST_TRACKER_RUNNING_SUMS: rho_ji and rho~_ij as Algorithm 1 prints  */
                              /* them; RFAST_TRACKER_BUCKETS: the edge masses of the augmented system   */
                              /* (Appendix F), see below                                               */
} rfast_problem;

/* RFAST_TRACKER_BUCKETS.  S2b consumes rho_ij^{tau_new} - rho~_ij = the sum of a_ij z^{t+1/2}_j over
 * the sender's local iterations tau_prev < t <= tau_new: the mass that is on the edge, the quantity
 * the augmented system of Appendix F carries instead of ever-growing running sums.  The schedule is
 * known in full before the run, so the host knows for every sender activation which receiver
 * activation will consume its contribution; with this option the sender adds it to a row that
 * holds exactly the contributions of one such consumption ("bucket") and the receiver adds that
 * row.  Same result as the running sums in exact arithmetic; in fp32 the subtraction of two
 * large running sums falls away (no loss of resolution over long horizons), a consumption reads
 * one row instead of two and a sender reads a row only when the bucket is not empty.  The views
 * RFAST_STATE_RHO_LATEST and RFAST_STATE_RHO_BUF do not exist with this option (RFAST_ESTATE). */
enum { RFAST_TRACKER_RUNNING_SUMS = 0, RFAST_TRACKER_BUCKETS = 1 };

/* Raw schedule (value independent).  Round r activates the nodes
 * act_node[act_ptr[r] .. act_ptr[r+1]) (strictly ascending).  Every activation is an
 * "event"; events are numbered in array order.  All members of a round read the state and
 * packets as of the start of the round.
 * send_r / send_c hold one code per (event, out-edge of its node) for G_R / G_C, events in
 * order, the out-edges of a node by ascending receiver id:  -1 = packet lost;  d >= 0 = the
 * packet sent in round r is usable from round r + 1 + d on.  A receiver always uses, per
 * in-edge, the packet with the largest sender stamp among those usable (Algorithm 1, S2).
 * batch_idx: minibatch row indices into the node's shard, B per sample: first the initial
 * samples zeta_i^0 of nodes 0..n-1 (used for z_i^0 = grad f_i(x_i^0; zeta_i^0)), then one
 * sample per event.  Ignored (may be NULL) when the problem's batch is 0. */
typedef struct rfast_schedule {
    int32_t        K;
    const int32_t* act_ptr;     /* [K+1] */
    const int32_t* act_node;    /* [act_ptr[K]] */
    int64_t        n_send_r;
    const int8_t*  send_r;      /* [n_send_r] */
    int64_t        n_send_c;
    const int8_t*  send_c;      /* [n_send_c] */
    int64_t        n_batch_idx;
    const int32_t* batch_idx;   /* [(n + events) * B] */
    const float*   alpha_round; /* [K] step size gamma^r of every activation of round r (the paper    */
                                /* allows a time-varying gamma^t, Algorithm 1 S1 / Algorithm 2 S.1),  */
                                /* or NULL: the problem's constant alpha                              */
} rfast_schedule;

/* Views for rfast_read_state.  Float views are fp32 row-major, unpadded. */
enum {
    RFAST_STATE_X            = 0,  /* float [n][p]     x_i                                        */
    RFAST_STATE_Y            = 1,  /* float [n][p]     tracker z_i (the "y" of push-pull methods)  */
    RFAST_STATE_G_LAST       = 2,  /* float [n][p]     remembered sample gradient                  */
    RFAST_STATE_RHO_LATEST   = 3,  /* float [|E_C|][p] sender running sums rho, G_C edge order      */
    RFAST_STATE_RHO_BUF      = 4,  /* float [|E_C|][p] receiver buffers rho~, G_C edge order        */
    RFAST_STATE_T_LOCAL      = 5,  /* int32 [n]        local counters t_i after the rounds run      */
    RFAST_STATE_USED_TAU_V   = 6,  /* int32 per (event, in-edge of G_R): stamp mixed in at S2a,     */
                                   /*       whole loaded schedule, events in order                  */
    RFAST_STATE_USED_TAU_RHO = 7,  /* int32 per (event, in-edge of G_C): stamp consumed at S2b      */
    RFAST_STATE_TAU_V_END    = 8,  /* int32 [|E_R|]    tau_v at the end of the loaded schedule      */
    RFAST_STATE_TAU_RHO_END  = 9,  /* int32 [|E_C|]    tau_rho at the end of the loaded schedule    */
    RFAST_STATE_ROUND        = 10, /* int32 [1]        rounds run so far                            */
    RFAST_STATE_V_LATEST     = 11, /* float [n][p]     v_i of node i's last activation (the payload of  */
                                   /*       its packet with stamp t_i, Algorithm 1 S1/S3) where the     */
                                   /*       engine holds it; a zero row where it does not: t_i = 0,     */
                                   /*       every copy was lost, or no receiver will mix it in again    */
    RFAST_STATE_V_HELD       = 12, /* int32 [n]        the stamp t_i where V_LATEST holds node i's row, */
                                   /*       0 where the row is zero                                     */
    RFAST_STATE_TAU_V        = 13, /* int32 [|E_R|]    tau_v per G_R edge after the rounds run so far   */
                                   /*       (the stamp the receiver mixed in at its last activation)    */
    RFAST_STATE_TAU_RHO      = 14, /* int32 [|E_C|]    tau_rho per G_C edge after the rounds run so far */
    /* other names for the same views */
    RFAST_STATE_ACT_COUNTS           = RFAST_STATE_T_LOCAL,      /* activations per node = t_i          */
    RFAST_STATE_COMPILED_STAMPS_V    = RFAST_STATE_USED_TAU_V,
    RFAST_STATE_COMPILED_STAMPS_RHO  = RFAST_STATE_USED_TAU_RHO
};

/* Counters for rfast_query. */
enum {
    RFAST_Q_ROUND          = 0,  /* rounds run so far */
    RFAST_Q_EVENTS_TOTAL   = 1,  /* activation events in the loaded schedule */
    RFAST_Q_EVENTS_RUN     = 2,  /* activation events run so far */
    RFAST_Q_LAUNCHES       = 3,  /* kernels launched by rfast_run since create */
    RFAST_Q_BYTES_RUN      = 4,  /* algorithmic bytes of the rounds run since the last reset:     */
                                 /* every fp32 stream the compiled schedule makes a kernel read  */
                                 /* or write, 4 bytes per coordinate                             */
    RFAST_Q_V_SLOTS        = 5,  /* version rows allocated for v packets   */
    RFAST_Q_RHO_SLOTS      = 6,  /* version rows allocated for rho packets */
    RFAST_Q_DEVICE_BYTES   = 7,  /* device memory held by the handle */
    RFAST_Q_N_USED_TAU_V   = 8,  /* element count of RFAST_STATE_USED_TAU_V   */
    RFAST_Q_N_USED_TAU_RHO = 9,  /* element count of RFAST_STATE_USED_TAU_RHO */
    RFAST_Q_BYTES_TOTAL    = 10, /* the same count for the whole loaded schedule */
    RFAST_Q_METHOD_BYTES_RUN   = 11, /* bytes the method itself must move (rounds run since the last  */
                                     /* reset): per activation x and z read once, v written if a packet */
                                     /* leaves, the neighbours' v read, x written, the remembered        */
                                     /* gradient read and the new one written (element-wise objective:   */
                                     /* its two data streams instead), the news rows read, z written, the */
                                     /* running sums read and written.  RFAST_Q_BYTES_* also count what   */
                                     /* only the implementation moves: re-reads between the kernels a     */
                                     /* step is split into, the low-order tracker words of compensated    */
                                     /* arithmetic                                                        */
    RFAST_Q_METHOD_BYTES_TOTAL = 12  /* the same count for the whole loaded schedule */
};

/* Problem statement -> device (eq. (1), Assumptions 1-2).  Validates Assumption 1
 * (positive diagonal, W rows and A columns sum to 1 within 1e-5) and Assumption 2 (root
 * reaches every node along G(W) and along G(A^T)); RFAST_EGRAPH otherwise.  Copies the
 * shards to the device and sets x = x0, v = rho = rho~ = 0, t = 0 (initialisation line of
 * Algorithm 1).  The trackers z_i^0 = grad f_i(x_i^0; zeta_i^0) need the initial samples
 * and are set by rfast_load_schedule.  *out is NULL on failure. */
int rfast_create(const rfast_problem* prob, void* cuda_stream, rfast_ctx** out);

/* Compiles a schedule (Algorithm 2, S.0) for the handle and resets the state to the
 * initial one (round 0).  A second call replaces the schedule and starts over at round 0 as
 * well; rounds are appended with rfast_append_schedule.  Host side, integers only: for every event and in-edge the stamp
 * that is consumed (tau_v, tau_rho of Algorithm 1, i.e. the delays d_v, d_rho of
 * Algorithm 2), then the lifetime of every packet version and a version row for each.
 * Uploads the per-round descriptors.  RFAST_ESCHED if the arrays are inconsistent (sizes,
 * order, ids, codes < -1). */
int rfast_load_schedule(rfast_ctx* ctx, const rfast_schedule* s);

/* Appends the rounds of `more` to the loaded schedule (Algorithm 2 goes on: k keeps counting).
 * The state, the packets on their way and the round counter stay as they are; afterwards
 * rfast_run can go on through the new rounds, and the result equals, bit for bit, that of the
 * whole schedule loaded at once.  Needs RFAST_OPT_OPEN_END set before the first
 * rfast_load_schedule: only then does the engine keep, past the end of what is loaded, what a
 * later activation may still read (per edge the version its receiver holds and every packet
 * that is on its way or waiting in an inbox, every sender's latest running sums); the rows
 * of the rounds already loaded never move.  RFAST_ESTATE without that option or without a
 * schedule; running sums only (not RFAST_TRACKER_BUCKETS, whose last bucket per edge lumps
 * together what a later round would consume apart).
 *   more: as for rfast_load_schedule, its rounds and events numbered from 0: act_ptr[0] = 0,
 *   send codes per (event of `more`, out-edge), delays counted from the event's own round;
 *   batch_idx holds (n + events of `more`) * B entries of which the first n * B (zeta^0) are
 *   ignored; alpha_round (optional) has more->K entries -- where only one of the parts gives
 *   step sizes, the other runs at the problem's alpha.
 * May be called at any round counter (the rounds not yet run stay as compiled).  The host
 * cost is that of compiling the whole schedule loaded so far; device pools that have to grow
 * are copied once.  RFAST_ESCHED as for rfast_load_schedule (nothing is changed then); on
 * RFAST_ENOMEM / RFAST_ECUDA while the pools are being replaced the handle is left without a
 * schedule.  Checkpoints are tied to the sequence of loads: a blob saved after an append
 * restores only into a handle that went through the same load and appends. */
int rfast_append_schedule(rfast_ctx* ctx, const rfast_schedule* more);

/* Runs the next `rounds` rounds: for every active node S1 (v = x - alpha z), S2a (mix over
 * G_R), the sample gradient at the new x, S2b/S2c (tracking over G_C with the running sums
 * rho and the buffers rho~), S3/S4/S5 as compiled (Algorithm 1).  Asynchronous unless
 * sync != 0.  RFAST_ESTATE without a schedule or past its end. */
int rfast_run(rfast_ctx* ctx, int32_t rounds, int sync);

/* Stream-ordered copy of one view into a caller-owned HOST buffer of exactly `bytes` bytes
 * (RFAST_EINVAL on mismatch); returns after the copy has completed.  Allocates nothing. */
int rfast_read_state(rfast_ctx* ctx, int which, void* dst, size_t bytes);

/* Back to the initial state of the loaded schedule (x0, z^0, zero packets, round 0).  Also
 * clears the status of a bounded device-side wait that ran out (RFAST_ETIMEOUT). */
int rfast_reset(rfast_ctx* ctx);

/* Sets the round counter to `round` (0 .. K) without running anything.  Everything integer in
 * Algorithm 1 -- the counters t_i, the stamps tau_v, tau_rho, which packet versions are in
 * flight -- is a function of the schedule and the round, so it follows; the float state is
 * left as it is and is meant to be loaded next with rfast_write_state / rfast_write_packet
 * (state of another run of the same schedule, e.g. a reference implementation's, or a
 * perturbed one).  RFAST_ESTATE without a schedule, RFAST_EINVAL outside 0 .. K. */
int rfast_seek(rfast_ctx* ctx, int32_t round);

/* Mirror of rfast_read_state for the float views: copies a caller-owned HOST buffer of exactly
 * `bytes` bytes (fp32 row-major, unpadded) into the view, as of the handle's current round;
 * returns after the copy has completed.
 *   X, Y            all n rows (Y: the tracker z_i; a two-float tracker's low word is cleared)
 *   G_LAST          the remembered sample gradients (RFAST_ESTATE for the element-wise
 *                   objective, which recomputes it from x)
 *   RHO_LATEST      rho of every G_C edge whose sender has been active (t_j >= 1); rows of
 *                   other edges are ignored (rho^0 = 0 is not stored)
 *   RHO_BUF         rho~ of every G_C edge with tau_rho >= 1; other rows are ignored.  rho~ is
 *                   the consumed version kept alive: where tau_rho = t_j it is the same row as
 *                   RHO_LATEST, so write RHO_BUF before RHO_LATEST
 *   V_LATEST        rows flagged by RFAST_STATE_V_HELD; other rows are ignored
 * Packets in flight that are neither the latest nor the buffered version of their edge are
 * written with rfast_write_packet.  Integer views cannot be written (RFAST_EINVAL): they
 * follow from the schedule and the round, see rfast_seek. */
int rfast_write_state(rfast_ctx* ctx, int which, const void* src, size_t bytes);

/* One packet version, addressed the way Algorithm 1 S3 stamps it.
 *   graph = 0: the v packet of node `id` with local stamp `stamp` (v_id^stamp);
 *   graph = 1: the running sum rho of G_C edge `id` (receiver-CSR edge id) with its sender's
 *              local stamp `stamp`.
 * The engine holds a version only from the round after it was produced until the last round
 * in which the schedule makes some activation read it.  Returns RFAST_OK and copies p floats
 * from / to the caller-owned HOST buffer (`bytes` = p * 4, RFAST_EINVAL otherwise), or
 * RFAST_NOT_HELD (a positive code, nothing copied) when that version has no row at the
 * handle's current round: it was never sent or is never read, it is yet to be produced, or its
 * last reader has run.  RFAST_ESTATE for graph = 1 with RFAST_TRACKER_BUCKETS. */
#define RFAST_NOT_HELD 1
int rfast_read_packet(rfast_ctx* ctx, int graph, int32_t id, int32_t stamp, float* dst, size_t bytes);
int rfast_write_packet(rfast_ctx* ctx, int graph, int32_t id, int32_t stamp, const float* src, size_t bytes);

/* A counter (>= 0), or a negative status for an unknown id / NULL handle. */
int64_t rfast_query(rfast_ctx* ctx, int what);

/* Execution options.  The first two never change results: every path produces the same bits.
 *   RFAST_OPT_PERSISTENT  0 (default): one kernel per phase of a round.  1: problems whose state
 *                         fits L2 (least squares, softmax regression) run a span of rounds as
 *                         ONE cooperative persistent kernel with grid barriers between the
 *                         phases of a round.  Every barrier wait is bounded; if one runs out
 *                         the kernel returns and the next synchronising call reports
 *                         RFAST_ETIMEOUT (the state is then undefined, the device healthy:
 *                         rfast_reset starts over).
 *   RFAST_OPT_GRAPHS      1 (default): spans of rounds are recorded into CUDA graphs (chunks of
 *                         about a thousand kernels, each launched as soon as it is instantiated)
 *                         and replayed (non-default streams only); 0: direct launches.
 *   RFAST_OPT_WAIT_LIMIT_MS     bound of every device-side barrier wait, 1..60000 (default 2000).
 *   RFAST_OPT_PHANTOM_ARRIVALS  failure injection for tests, made on the host: the grid barrier
 *                         expects this many arrivals that nobody makes, so its bounded wait runs
 *                         out and the timeout path is exercised (default 0).  The one-pass
 *                         sparse-logistic kernel takes the same option: its copy barrier then
 *                         expects 16 bytes per unit that nobody delivers.
 *   RFAST_OPT_ONE_PASS    sparse-logistic objective.  1 (default): an activation runs as one
 *                         thread-block cluster whose CTAs keep their slices of the new x and of z
 *                         in shared memory between the mixing step, the sparse dot products and
 *                         the tracking step, so every vector crosses HBM once (taken when a
 *                         cluster of at most 8 CTAs can hold 2 p floats and the batch is at most
 *                         64 rows; otherwise, or with 0, three kernels per round).  The two paths
 *                         add the sparse dot products up in different orders: they agree to
 *                         rounding, each of them bit for bit from run to run.  To be set before
 *                         rfast_load_schedule (RFAST_ESTATE afterwards).
 *   RFAST_OPT_CLUSTER_SIZE  CTAs per activation on that path: 0 (default) = the smallest of 1, 2,
 *                         4, 8 that fits; RFAST_EINVAL if the given size does not fit.  The
 *                         partial dot products are added per CTA, so results agree to rounding
 *                         across sizes.  To be set before rfast_load_schedule.
 *   RFAST_OPT_OPEN_END    1: schedules are loaded open-ended, so that rfast_append_schedule can
 *                         add rounds later (a few more version rows stay occupied at the end of
 *                         what is loaded; values and byte counts do not change).  Default 0.
 *                         To be set before rfast_load_schedule; RFAST_EINVAL with
 *                         RFAST_TRACKER_BUCKETS. */
enum { RFAST_OPT_PERSISTENT = 0, RFAST_OPT_GRAPHS = 1, RFAST_OPT_WAIT_LIMIT_MS = 2, RFAST_OPT_PHANTOM_ARRIVALS = 3,
       RFAST_OPT_ONE_PASS = 4, RFAST_OPT_CLUSTER_SIZE = 5, RFAST_OPT_OPEN_END = 6 };
int rfast_set_option(rfast_ctx* ctx, int option, int64_t value);

/* Read-back of x and y that runs under the work that follows (no counterpart in the paper: a
 * service call for callers that run one schedule after another).  rfast_snapshot enqueues, on the
 * handle's stream, a copy of x and y -- as of everything enqueued so far -- into a second pair of
 * device arrays (allocated at the first call, kept for the life of the handle: 2 n p floats), and on
 * a stream of the handle's own the transfer of that copy into x_dst and y_dst, caller-owned HOST
 * arrays float [n][p] (unpadded, as RFAST_STATE_X / RFAST_STATE_Y deliver them; page-locked memory
 * if the transfer is to overlap anything).  It returns at once; rfast_load_schedule, rfast_reset
 * and rfast_run may follow immediately and do not disturb the snapshot.  The destinations hold the
 * snapshot after rfast_snapshot_wait has returned; a second rfast_snapshot before that queues
 * behind the first (on the device, the host does not wait) and its transfer may overwrite the
 * same destinations.  The values are bit for bit those of rfast_read_state at the same point.
 * RFAST_EINVAL on a null destination, RFAST_ENOMEM / RFAST_ECUDA as reported by the runtime. */
int rfast_snapshot(rfast_ctx* ctx, float* x_dst, float* y_dst);
int rfast_snapshot_wait(rfast_ctx* ctx);

/* Waits for the handle's stream; reports a pending asynchronous error. */
int rfast_sync(rfast_ctx* ctx);

/* Checkpoint / resume.  The blob holds the complete device state of the handle -- x, the
 * trackers, the remembered gradients, every live packet version (published v and running sums
 * rho, i.e. also the packets still in flight) and the round counter -- so that
 *     create + load_schedule(same schedule) + checkpoint_load + run(K - r)
 * continues bit for bit where  run(r) + checkpoint_save  stopped.  The blob is opaque and tied
 * to the problem's shape and to the loaded schedule (a hash of its arrays is checked);
 * RFAST_ESTATE if no schedule is loaded, RFAST_EINVAL on a size or identity mismatch.
 * dst / src are caller-owned HOST buffers of rfast_checkpoint_size() bytes. */
int64_t rfast_checkpoint_size(rfast_ctx* ctx);
int     rfast_checkpoint_save(rfast_ctx* ctx, void* dst, size_t bytes);
int     rfast_checkpoint_load(rfast_ctx* ctx, const void* src, size_t bytes);

/* On-device diagnostics of the current state (off the hot path; reads every state row once):
 *   out[0] consensus error  || x - 1 xbar^T ||_F        (xbar = mean of the x_i)
 *   out[1] || xbar ||_2
 *   out[2] conservation residual of Lemma 3:
 *          max_c | sum_i z_i + sum_e (rho_e - rho~_e) - sum_i g_i |   (0 up to rounding; with
 *          RFAST_TRACKER_BUCKETS the mass in transit sum_e (rho_e - rho~_e) is the content of the
 *          buckets begun and not yet consumed)
 *   out[3] max_c | sum_i g_i |   (the scale of out[2])
 *   out[4] || z ||_F
 *   out[5] || grad F(xbar) ||_2, the full gradient of F = sum_i f_i (every row of every shard,
 *          no sampling) at the mean iterate.  For the objectives that sample minibatches
 *          (softmax, MLP, sparse logistic) it is formed with the kernels the activations use,
 *          the shards walked in chunks of B rows from a state whose rows all hold xbar; x is
 *          moved aside and put back bit for bit, the first such call allocates its scratch (a
 *          copy of x, a double per coordinate) and keeps it for the life of the handle.
 *          NaN where the shard size is not a multiple of B
 *   out[6] the merit function of the non-convex analysis (Section V-B),
 *          M_F(x) = || grad F(xbar) ||^2 + || x - 1 xbar^T ||^2 = out[5]^2 + out[0]^2 (NaN where out[5] is)
 *   out[7] F(xbar) = sum_i f_i(xbar), the objective of eq. (1) at the mean iterate over every row
 *          of every shard (the loss curve of the experiments in Section VI); NaN for a softmax
 *          objective with more than 32 classes
 * n_out is 5 (the first five only), 7 or 8; RFAST_EINVAL otherwise.  out is a caller-owned HOST
 * array of doubles. */
int rfast_diagnostics(rfast_ctx* ctx, double* out, int32_t n_out);

/* Host-only companion of rfast_load_schedule (needs no CUDA device): compiles the schedule
 * for the two graphs of `prob` (only n, root, batch, rows, model, G_R, G_C are read) and
 * writes the integer artefacts into caller-owned HOST arrays, any of which may be NULL:
 *   used_tau_v   [sum over events of indeg_R(node)]   stamp mixed in per (event, in-edge)
 *   used_tau_rho [sum over events of indeg_C(node)]   stamp consumed per (event, in-edge)
 *   v_ver        [events][3]       per v packet version:   row (-1: never leaves the node),
 *   rho_ver      [n_send_c][3]     per rho packet version: write round, last round read
 *   counts       [4]               v rows, rho rows, events, algorithmic floats per coordinate
 * Two versions may share a row only if the earlier one is last read strictly before the round
 * the later one is written (or, for rho, the later one is the same sender's in-place update). */
int rfast_compile_host(const rfast_problem* prob, const rfast_schedule* s,
                       int32_t* used_tau_v, int32_t* used_tau_rho,
                       int32_t* v_ver, int32_t* rho_ver, int64_t* counts,
                       char* err, size_t err_len);

/* Host-only, like rfast_compile_host: compiles the schedule and folds everything the kernels are
 * driven by (event descriptors, mixing / news / running-sum row lists and weights, the byte
 * counts per round) into one 64-bit number.  Two compilations of the same problem and schedule
 * give the same number whatever the number of host threads the compiler used
 * (environment variable RFAST_COMPILE_THREADS caps it; long schedules use up to 8). */
int rfast_compile_digest(const rfast_problem* prob, const rfast_schedule* s, uint64_t* digest,
                         char* err, size_t err_len);

/* Host-only companion of rfast_append_schedule (needs no CUDA device): compiles `first`
 * open-ended, then `first` followed by `more` the way rfast_append_schedule does, and checks
 * (1) that no version row, row list or event descriptor of the rounds of `first` differs
 * between the two and (2) that the stamps consumed (tau_v, tau_rho per event and in-edge) and
 * the final counters t_i are those of the whole schedule compiled in one piece.
 * counts (optional, int64[6]): version rows of v and of rho for `first` open-ended, for the
 * appended whole, for the whole compiled in one piece (closed end).  RFAST_OK if both hold,
 * RFAST_ESCHED with a message otherwise. */
int rfast_compile_append_check(const rfast_problem* prob, const rfast_schedule* first,
                               const rfast_schedule* more, int64_t* counts, char* err, size_t err_len);

/* No counterpart in the paper: a service entry point for callers that are not allowed to
 * allocate device memory.  Some hosts of this library cannot call cudaMalloc where they need a
 * gradient: a framework that hands the whole GPU to its own memory pool up front, a latency-
 * critical loop in which cudaMalloc's implicit device-wide synchronisation is unacceptable, or
 * code that runs after memory has been budgeted to the last byte.  For them this call computes
 * the full-shard least-squares gradient
 *     grad = (1/rows) * feat^T (feat x - target) + l2 * x
 * (the LEAST_SQUARES objective above with batch = 0, for one node) without allocating anything:
 * the per-row residuals that the handle-based path keeps in an allocated buffer live in a fixed
 * array inside the library image, RFAST_STATIC_MAX_ROWS floats (256 KiB) that every GPU loading
 * the library holds until the process exits.
 *   d_feat [rows][n_features], d_target [rows], d_x [n_features]: DEVICE pointers, inputs;
 *   d_grad [n_features]: DEVICE pointer, output; all owned by the caller, row-major fp32.
 *   cuda_stream: cudaStream_t as void* (NULL: legacy default stream); the work is enqueued
 *   there and the call returns without waiting.
 * The device that is current at the call is used.  The first call made on a device looks up
 * the array's device address (cudaGetSymbolAddress) and remembers it; make that first call
 * before starting any stream capture.  rows > RFAST_STATIC_MAX_ROWS is rejected with
 * RFAST_EINVAL and a message in err (err may be NULL).  All calls share the one array, which
 * keeps the previous call's contents; the part a call uses is cleared first.  Two calls whose
 * work overlaps on the GPU (different streams, or different host threads without ordering)
 * race on it: order them on one stream or with events.  Calls no cudaMalloc / cudaFree. */
#define RFAST_STATIC_MAX_ROWS 65536
int rfast_ls_gradient_static(const float* d_feat, const float* d_target, const float* d_x,
                             float* d_grad, int32_t rows, int32_t n_features, float l2,
                             void* cuda_stream, char* err, size_t err_len);

void        rfast_destroy(rfast_ctx* ctx);
const char* rfast_last_error(const rfast_ctx* ctx);   /* ctx may be NULL: last create error */
const char* rfast_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RFAST_H */
