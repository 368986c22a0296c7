// Internal structures of librfast: host graphs, the compiled schedule and the device
// descriptors the kernels read.  Nothing here is part of the public ABI.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "rfast.h"

namespace rfast {

// Weight matrix by receiver (as given) plus the derived sender-side lists.
struct HostGraph {
    int n = 0, E = 0;
    std::vector<int>   rowptr, col, recv;   // recv[e]: receiver of edge e
    std::vector<float> w, diag;
    std::vector<int>   optr;                // [n+1] out-edge ranges per sender
    std::vector<int>   oeid;                // [E]   edge ids, per sender by ascending receiver
    std::vector<int>   opos;                // [E]   position of edge e inside its sender's list
    int indeg(int i) const { return rowptr[i + 1] - rowptr[i]; }
    int outdeg(int i) const { return optr[i + 1] - optr[i]; }
};

// One activation event as the kernels see it (64 bytes).
struct EvDesc {
    int32_t node;
    int32_t v_out;               // version row that receives v = x - alpha z; -1: no packet leaves
    int32_t mix_beg, mix_cnt;    // range in mix_slot / mix_w: in-neighbours of G_R holding a non-zero v
    int32_t news_beg, news_cnt;  // range in news_new / news_prev: G_C in-edges with a newer packet
    int32_t out_beg, out_cnt;    // range in out_cur / out_new / out_a: G_C out-edges
    float   w_self, a_self;      // w_ii, a_ii
    int32_t g_par;               // gradient buffer (0/1) holding the remembered gradient
    int32_t sample;              // index of this event's minibatch (n + event id)
    int32_t stamp;               // t_i + 1, the stamp the outgoing packets carry
    int32_t pad[3];
};
static_assert(sizeof(EvDesc) == 64, "EvDesc must stay 64 bytes");

struct Compiled {
    int     K = 0;
    int64_t n_events = 0;
    std::vector<int>     act_ptr, act_node;
    std::vector<int64_t> in_r_off, in_c_off, out_r_off, out_c_off;   // per event (+1)
    // integer artefacts of Algorithm 1 / 2
    std::vector<int> used_tau_v, used_tau_rho, prev_tau_rho;
    std::vector<int> tau_v_end, tau_rho_end, t_end;
    // packet versions: v per event, rho per (event, G_C out-edge)
    std::vector<int> v_slot, v_write, v_last;
    std::vector<int> rho_slot, rho_write, rho_last;
    int n_v_slots = 0, n_rho_slots = 0;
    // mass-bucket tracker: the contributions consumed together share a row; rho_leader[v] is the
    // first of them (it owns the row; rho_write / rho_last of a leader: first write, consumption)
    bool buckets = false;
    std::vector<int64_t> rho_leader;
    // device descriptors
    std::vector<EvDesc> ev;
    std::vector<int>    mix_slot;  std::vector<float> mix_w;
    std::vector<int>    news_new, news_prev, news_edge;
    std::vector<int>    out_cur, out_new, out_edge;  std::vector<float> out_a;
    // fp32 streams per coordinate (method traffic), prefix sums over rounds
    std::vector<int64_t> round_streams;          // [K+1] streams the kernels touch
    std::vector<int64_t> round_streams_method;   // [K+1] streams the method itself must move
    std::vector<std::vector<int>> ev_of;         // node -> event id of its stamp s at [s-1]
};

// Arguments shared by the sample-gradient kernels.
struct GradArgs {
    const EvDesc* ev;
    const float*  x;          // [n][stride]
    float*        gbuf;       // [2][n][stride]
    int64_t stride, gplane;
    const int*    batch_idx;  // [(n + events) * B]
    int B, rows, F, C, H;
    int64_t p;
    float l2;
};

// What the byte accounting needs to know about the model.
struct ModelTraffic {
    bool elementwise = false;   // one fused pass, gradient recomputed instead of stored
    int  data_streams = 0;      // model data streams per coordinate in the fused pass
    int  grad_track_streams = 5; // split path: gradient reads x, writes g; tracking reads z, g_old, g_new
    int  method_streams = 2;     // the method's own count beyond x, z, packets: the remembered gradient read,
                                 // the new one written (element-wise objective: its two data streams,
                                 // the remembered gradient being recomputed)
};

int build_host_graph(const rfast_graph& g, int n, bool row_stochastic, HostGraph& out, std::string& err);
int check_roots(const HostGraph& R, const HostGraph& C, int root, std::string& err);
// holds (optional): ascending rounds b in 0 .. K at which everything a later activation may still
// read is kept in its row through round b (b = K: the schedule is open-ended).  The rows of the
// rounds before a hold do not depend on the rounds after it.
int compile_schedule(const HostGraph& R, const HostGraph& C, const rfast_schedule* s, int batch,
                     int rows, const ModelTraffic& mt, bool buckets, Compiled& out, std::string& err,
                     const std::vector<int>* holds = nullptr);

}  // namespace rfast
