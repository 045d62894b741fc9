// extern "C" entry points of libumlmd (see include/umlmd.h for the contract).
#include <cmath>
#include <cstring>
#include <new>

#include "alloc.h"
#include "kernels.h"
#include "mlp_gemm.h"
#include "model.h"

using namespace umd;

struct umlmd {
    HostModel hm;
    ModelDev md{};
    Dims d{};
    cudaStream_t st = nullptr;
    std::string err;
    NeighborDev nb;
    int node_tile = 524288;
    int mlp_path = 2;   // tensor-core GEMM wherever it applies, CUDA-core GEMM otherwise
    int gemm_spin_limit = 0;      // polls before a tensor-core pipeline wait gives up (0 = default)
    int fault_skip_stage = 0;     // diagnostic, consumed by the first evaluation: see umlmd_options
    bool have_list = false;
    bool on_device = false;
    std::vector<void*> model_allocs;
    // workspace
    float* state = nullptr; float* desc = nullptr; float* pre = nullptr; float* hbuf = nullptr;
    __half* tc_hi = nullptr; __half* tc_lo = nullptr;   // half-precision split of the current GEMM's activations
    int64_t tile_cap = 0;
    float* g = nullptr; int64_t g_cap = 0;
    double* e_atom = nullptr; double* f_sorted = nullptr; int* type_o = nullptr; int64_t n_cap = 0;
    double* virial_part = nullptr; int64_t vpart_cap = 0;
    double* frame_out = nullptr; int64_t frame_out_cap = 0;     // batched evaluation: [n_frames][10] energy, virial
    double* scratch = nullptr; double* d_out = nullptr; int* d_err = nullptr;
    double* h_out = nullptr; int* h_err = nullptr;      // pinned
    // per-pair amplitude tables of the species present (set up by umlmd_build_neighbors)
    int64_t pair_table_budget = 192ll << 20;            // bytes; negative = never build them
    bool pair_tables = false;                           // in use for the current system
    std::vector<int> present;                           // species the tables were built for, ascending
    float* table_uni = nullptr; size_t table_uni_cap = 0;   // [present^2][n_rows][3][C0], capacity in floats
    float* uni_scale = nullptr;                         // [2] largest |c2|, |c3| of those tables
    int* d_species = nullptr;                           // [3T]: occurrence flags, species -> slot, present list
    int* h_species = nullptr;                           // pinned [T]
    // MD
    double* md_pos = nullptr; double* md_vel = nullptr; double* md_force = nullptr; int64_t md_cap = 0;
    double* d_mass = nullptr; double* d_inv_mass = nullptr;
    bool have_md = false, have_force = false;
    bool have_edge_grad = false;     // h->g holds the edge gradients of the positions in nb.xs
    int steps_since_build = 0;
    double* d_nhc = nullptr;      // thermostat chain on the device: eta[M], v_eta[M], scale, kinetic energy
    bool nhc_reset = true;
    // launch accounting and optional per-class timing
    bool prof_on = false;
    struct Span { int cls; cudaEvent_t a, b; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> free_events;
    double prof_ms[16] = {0};
    int64_t prof_launches[16] = {0};
    int64_t launches_total = 0;
    // replay of repeated launch sequences as CUDA graphs (see run_replayed)
    struct Replay {
        cudaGraphExec_t exec = nullptr;
        const void* key[4] = {nullptr, nullptr, nullptr, nullptr}; double key_dt = 0, key_x0 = 0, key_x1 = 0; int64_t key_serial = -1; int key_flags = 0;
        bool seen = false;                           // the key's sequence has run once as plain launches
        int64_t launches[16] = {0}; int64_t total = 0;   // what one replay launches, per class
    };
    Replay rp_compute, rp_step, rp_nvt;
    int launch_graphs = 0;                           // option: 0 = automatic, 1 = always, -1 = never
    bool graphs_broken = false;                      // a capture failed on this handle: plain launches from then on
    cudaStream_t cap_st = nullptr;                   // stream the sequences are captured on
    int64_t n_owned = -1;                            // atoms [n_owned, N) are ghosts (neighbours only); negative = none
    int64_t graph_replays = 0;
    int64_t list_serial = 0;                         // bumped by everything that changes what a sequence launches
};

enum KernelClass { kGather = 0, kEdgeFwd, kInvFwd, kMlpFwd, kMlpBwd, kInvBwd, kEdgeBwd, kForce, kReduce, kIntegrate,
                   kNeighbor, kClassCount };
static const char* const kClassNames[kClassCount] = {
    "gather_positions", "edge_forward", "invariants_forward", "mlp_forward", "mlp_backward", "invariants_backward",
    "edge_backward", "force_assembly", "energy_virial_reduce", "integrate", "neighbor_build"};

namespace {

// counts the kernels a call site launches and, when profiling is on, brackets them with events
struct Scope {
    umlmd_t* h; int cls; cudaEvent_t a = nullptr;
    static cudaEvent_t get(umlmd_t* h) {
        cudaEvent_t e = nullptr;
        if (!h->free_events.empty()) { e = h->free_events.back(); h->free_events.pop_back(); }
        else cudaEventCreate(&e);
        return e;
    }
    Scope(umlmd_t* h_, int cls_, int n) : h(h_), cls(cls_) {
        h->launches_total += n; h->prof_launches[cls] += n;
        if (h->prof_on) { a = get(h); cudaEventRecord(a, h->st); }
    }
    ~Scope() {
        if (a) { cudaEvent_t b = get(h); cudaEventRecord(b, h->st); h->spans.push_back({cls, a, b}); }
    }
};

int fail(umlmd_t* h, int code, const std::string& msg) {
    if (h) h->err = msg;
    return code;
}

#define API_CUDA(h, call)                                                                     \
    do {                                                                                      \
        cudaError_t e__ = (call);                                                             \
        if (e__ != cudaSuccess)                                                               \
            return fail(h, UMLMD_E_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__)); \
    } while (0)

template <typename T>
cudaError_t upload(umlmd_t* h, const std::vector<T>& v, T** out) {
    *out = nullptr;
    void* p = nullptr;
    cudaError_t e = dev_malloc(&p, v.size() * sizeof(T) + 16);
    if (e != cudaSuccess) return e;
    h->model_allocs.push_back(p);
    if (!v.empty()) e = cudaMemcpyAsync(p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice, h->st);
    *out = static_cast<T*>(p);
    return e;
}

void fill_info(const Dims& d, umlmd_info* o) {
    o->C0 = d.C0; o->L = d.L; o->R = d.R; o->N_rbf = d.N_rbf; o->n_hidden = d.n_hidden; o->F = d.F; o->T = d.T;
    o->C1 = d.C[1]; o->C2 = d.C[2]; o->K1 = d.K[1]; o->K2 = d.K[2]; o->S = d.S; o->D_out = d.D_out;
    o->H = d.H; o->H_pair = d.Hp; o->table_rows = d.n_rows;
}

// the fp32 feature rows and the state of a small single-tile system stay readable after an
// evaluation (umlmd_get_intermediates); larger systems skip the copy nothing else reads
constexpr int64_t kIntermediatesMaxAtoms = 65536;
bool keeps_intermediates(const umlmd_t* h) { return h->nb.N < kIntermediatesMaxAtoms && h->nb.N <= h->node_tile; }

int ensure_workspace(umlmd_t* h) {
    const Dims& d = h->d;
    const int64_t N = h->nb.N, E = h->nb.E;
    const int64_t B = N < h->node_tile ? N : h->node_tile;
    if (B > h->tile_cap || !h->state) {
        int64_t c;
        c = 0; API_CUDA(h, dev_ensure(&h->state, &c, B * d.SP));
        c = 0; API_CUDA(h, dev_ensure(&h->desc, &c, B * d.DP));
        c = 0; API_CUDA(h, dev_ensure(&h->pre, &c, B * d.F * d.n_hidden));
        c = 0; API_CUDA(h, dev_ensure(&h->hbuf, &c, B * d.F * 2));
        const int64_t wmax = d.DP > d.F ? d.DP : d.F;
        c = 0; API_CUDA(h, dev_ensure(&h->tc_hi, &c, 2 * B * wmax));
        c = 0; API_CUDA(h, dev_ensure(&h->tc_lo, &c, 2 * B * wmax));
        h->tile_cap = B;
    }
    if (E > h->g_cap || !h->g) { API_CUDA(h, dev_ensure(&h->g, &h->g_cap, E * 3, 1.1)); h->g_cap /= 3; }
    if (N > h->n_cap || !h->e_atom) {
        int64_t c;
        c = 0; API_CUDA(h, dev_ensure(&h->e_atom, &c, N));
        c = 0; API_CUDA(h, dev_ensure(&h->f_sorted, &c, N * 3));
        c = 0; API_CUDA(h, dev_ensure(&h->type_o, &c, N));
        h->n_cap = N;
    }
    const int64_t n_tiles = B > 0 ? (N + B - 1) / B : 0;
    const int64_t vneed = (N / 4 + n_tiles + 2) * 9;
    if (vneed > h->vpart_cap || !h->virial_part) API_CUDA(h, dev_ensure(&h->virial_part, &h->vpart_cap, vneed));
    return UMLMD_OK;
}

int decode_device_errors(umlmd_t* h, int word) {
    if (word & kErrSpecies) return fail(h, UMLMD_E_INVALID_ARG, "species index outside [0, T)");
    if (word & kErrNonFinite) return fail(h, UMLMD_E_NONFINITE, "non-finite value in positions, energy or forces");
    if (word & kErrPipelineTimeout) return fail(h, UMLMD_E_CUDA, "tensor-core GEMM pipeline wait expired");
    if (word & kErrShiftRange) return fail(h, UMLMD_E_UNSUPPORTED_CELL, "periodic image index outside [-127, 127]");
    if (word & kErrStale)
        return fail(h, UMLMD_E_STALE_NEIGHBORS, "an atom moved more than skin/2 since the neighbor list was built");
    return UMLMD_OK;
}

// enqueue one full evaluation; results stay on the device (d_out[0] energy, d_out[1..9] virial)
int enqueue_compute(umlmd_t* h, const double* d_pos, bool want_grad, double* d_force, double* d_atom_energy) {
    const Dims& d = h->d;
    NeighborDev& nb = h->nb;
    const int N = (int)nb.N;
    const int NR = (int)nb.n_owned;      // rows that are evaluated: the owned atoms, first in the internal order
    // (a batched list was built from these very positions: nothing to gather)
    if (!nb.batch) { Scope sc(h, kGather, 1); API_CUDA(h, launch_gather_positions(nb, d_pos, h->d_err, h->st)); }
    const int B = N < h->node_tile ? N : h->node_tile;
    int vpart_used = 0;
    for (int a0 = 0; a0 < NR; a0 += B) {
        const int n = NR - a0 < B ? NR - a0 : B;
        EdgeArgs ea;
        ea.d = d; ea.table = h->md.table; ea.pairmod = h->md.pairmod; ea.xs = nb.xs; ea.rec = nb.rec; ea.type_s = nb.type_s;
        ea.table_uni = h->pair_tables ? h->table_uni : nullptr;
        ea.uni_scale = h->uni_scale;
        ea.species_slot = h->d_species + d.T; ea.n_present = (int)h->present.size();
        ea.frames = nb.batch ? nb.frames : nullptr; ea.frame_of = nb.frame_of;
        ea.row_ptr = nb.row_ptr; ea.src = nb.src; ea.shift = nb.shift;
        ea.Lx = nb.L[0]; ea.Ly = nb.L[1]; ea.Lz = nb.L[2];
        for (int k = 0; k < 9; ++k) ea.H[k] = nb.H[k];
        ea.tri = nb.tri;
        ea.a0 = a0; ea.a1 = a0 + n; ea.state = h->state; ea.g = h->g;
        ea.virial_part = h->virial_part + (size_t)vpart_used * 9;
        { Scope sc(h, kEdgeFwd, 1); API_CUDA(h, launch_edge_forward(ea, h->st)); }
        InvArgs ia;
        ia.d = d; ia.m = h->md; ia.type_s = nb.type_s; ia.a0 = a0; ia.n = n; ia.state = h->state; ia.desc = h->desc;
        // tensor-core MLP: the invariants kernel writes the first GEMM's operand split itself; the
        // fp32 feature rows are then only kept where something still reads them (the identity
        // residual of a first layer as wide as the feature vector, or the intermediates query of a
        // system smaller than one node tile)
        const bool presplit = mlp_uses_tc(d.F, h->mlp_path);
        ia.desc_hi = presplit ? h->tc_hi : nullptr; ia.desc_lo = presplit ? h->tc_lo : nullptr;
        ia.write_desc = !presplit || d.D_out == d.F || keeps_intermediates(h);
        const bool fold_x0 = presplit && d.D_out != d.F;      // first GEMM skips the per-species constant columns
        ia.skip_x0_split = fold_x0;
        { Scope sc(h, kInvFwd, 1); API_CUDA(h, launch_invariants_forward(ia, h->st)); }
        MlpArgs ma;
        ma.d = d; ma.m = h->md; ma.type_s = nb.type_s; ma.a0 = a0; ma.n = n; ma.desc = h->desc; ma.pre = h->pre;
        ma.hbuf = h->hbuf; ma.e_atom = h->e_atom; ma.path = h->mlp_path; ma.want_grad = want_grad;
        ma.tc_hi = h->tc_hi; ma.tc_lo = h->tc_lo; ma.err = h->d_err; ma.desc_presplit = presplit; ma.fold_x0 = fold_x0;
        ma.tc_slot = (size_t)h->tile_cap * (size_t)(d.DP > d.F ? d.DP : d.F);
        ma.spin_limit = h->gemm_spin_limit; ma.test_skip_kblock = h->fault_skip_stage;
        h->fault_skip_stage = 0;                      // one shot
        { Scope sc(h, kMlpFwd, d.n_hidden + 1); API_CUDA(h, launch_mlp_forward(ma, h->st)); }
        if (want_grad) {
            { Scope sc(h, kMlpBwd, d.n_hidden); API_CUDA(h, launch_mlp_backward(ma, h->st)); }
            { Scope sc(h, kInvBwd, 1); API_CUDA(h, launch_invariants_backward(ia, h->st)); }
            int blocks = 0;
            { Scope sc(h, kEdgeBwd, 1); API_CUDA(h, launch_edge_backward(ea, &blocks, h->st)); }
            vpart_used += blocks;
        }
    }
    h->have_edge_grad = want_grad;
    if (want_grad) {
        Scope sc(h, kForce, 1);
        API_CUDA(h, launch_force_assembly(nb, h->g, d_force ? nullptr : h->f_sorted, d_force, h->d_err, h->st));
    }
    Scope sc(h, kReduce, (N <= 4096 ? 1 : 2) + (d_atom_energy ? 1 : 0));      // one reduction launch for a single slice of energies
    API_CUDA(h, launch_reduce_energy_virial(h->e_atom, N, h->virial_part, vpart_used, h->scratch, h->d_out,
                                            h->d_err, h->st));
    if (d_atom_energy) API_CUDA(h, launch_scatter_atom_energy(nb, h->e_atom, d_atom_energy, h->st));
    return UMLMD_OK;
}

// copy results and the error word to the host and clear the error word (enqueue_fetch), then
// synchronise and decode (finish_fetch)
int enqueue_fetch(umlmd_t* h, int n_out) {
    API_CUDA(h, cudaMemcpyAsync(h->h_out, h->d_out, sizeof(double) * n_out, cudaMemcpyDeviceToHost, h->st));
    API_CUDA(h, cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, h->st));
    API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
    return UMLMD_OK;
}
int finish_fetch(umlmd_t* h) {
    API_CUDA(h, cudaStreamSynchronize(h->st));
    return decode_device_errors(h, *h->h_err);
}
int fetch_results(umlmd_t* h, int n_out) {
    int rc = enqueue_fetch(h, n_out);
    return rc != UMLMD_OK ? rc : finish_fetch(h);
}

// Replay of a repeated launch sequence.  A system of a few thousand atoms spends more time between
// its two dozen kernels than inside them, so a sequence that recurs with the same arguments (an
// evaluation of the same buffers, a middle step of an MD run between two list builds) is recorded
// once as a CUDA graph and replayed with one launch.  `body` enqueues the sequence on h->st; `key`
// names everything its launches depend on besides the handle's own state, which list_serial covers.
// The first occurrence of a key runs as plain launches (it also performs every lazy one-time
// initialisation of the launch helpers), the second is captured on a stream of the handle's own
// (the caller's may be the legacy default stream, which cannot capture) and every later one
// replayed.  A capture that fails for any reason leaves the handle on plain launches for good.
bool replay_allowed(const umlmd_t* h) {
    if (h->graphs_broken || h->prof_on || h->fault_skip_stage || h->launch_graphs < 0) return false;
    if (h->launch_graphs > 0) return true;
    return h->nb.N <= 65536 && h->nb.N <= h->node_tile;       // automatic: systems where launch latency shows
}
void replay_drop(umlmd_t::Replay& r) {
    if (r.exec) cudaGraphExecDestroy(r.exec);
    r.exec = nullptr;
}
template <class Body>
int run_replayed(umlmd_t* h, umlmd_t::Replay& r, const void* k0, const void* k1, const void* k2, const void* k3,
                 double dt, int flags, Body body, double x0 = 0.0, double x1 = 0.0) {
    if (!replay_allowed(h)) return body();
    const bool same = r.key[0] == k0 && r.key[1] == k1 && r.key[2] == k2 && r.key[3] == k3 && r.key_dt == dt && r.key_x0 == x0 && r.key_x1 == x1 &&
                      r.key_flags == flags && r.key_serial == h->list_serial;
    if (!same) {
        replay_drop(r);
        r.key[0] = k0; r.key[1] = k1; r.key[2] = k2; r.key[3] = k3; r.key_dt = dt; r.key_x0 = x0; r.key_x1 = x1; r.key_flags = flags;
        r.key_serial = h->list_serial; r.seen = true;
        return body();
    }
    if (!r.exec) {
        if (!h->cap_st && cudaStreamCreateWithFlags(&h->cap_st, cudaStreamNonBlocking) != cudaSuccess) {
            cudaGetLastError(); h->graphs_broken = true;
            return body();
        }
        int64_t before[16], total = h->launches_total;
        for (int c = 0; c < 16; ++c) before[c] = h->prof_launches[c];
        cudaStream_t real = h->st;
        h->st = h->cap_st;
        int rc = UMLMD_OK;
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamBeginCapture(h->cap_st, cudaStreamCaptureModeRelaxed);
        if (e == cudaSuccess) {
            rc = body();
            e = cudaStreamEndCapture(h->cap_st, &graph);
            if (rc == UMLMD_OK && e == cudaSuccess) e = cudaGraphInstantiate(&r.exec, graph, 0);
            if (graph) cudaGraphDestroy(graph);
        }
        h->st = real;
        for (int c = 0; c < 16; ++c) { r.launches[c] = h->prof_launches[c] - before[c]; h->prof_launches[c] = before[c]; }
        r.total = h->launches_total - total; h->launches_total = total;      // nothing has run yet
        if (rc != UMLMD_OK || e != cudaSuccess || !r.exec) {
            cudaGetLastError();
            replay_drop(r);
            h->graphs_broken = true;
            h->err.clear();
            return body();
        }
    }
    for (int c = 0; c < 16; ++c) h->prof_launches[c] += r.launches[c];
    h->launches_total += r.total;
    ++h->graph_replays;
    API_CUDA(h, cudaGraphLaunch(r.exec, h->st));
    return UMLMD_OK;
}

// first use on a device: upload the model constants and allocate the small result buffers
int ensure_device_model(umlmd_t* h) {
    if (h->on_device) return UMLMD_OK;
    const HostModel& m = h->hm;
    ModelDev& md = h->md;
    cudaError_t e = cudaSuccess;
    auto up = [&](const std::vector<float>& v, float** p) { if (e == cudaSuccess) e = upload(h, v, p); };
    auto uph = [&](const std::vector<__half>& v, __half** p) { if (e == cudaSuccess) e = upload(h, v, p); };
    up(m.table, &md.table); up(m.pairmod, &md.pairmod); up(m.X0, &md.X0); up(m.W1p, &md.W1p); up(m.W2p, &md.W2p);
    up(m.A1, &md.A1); up(m.A2, &md.A2); up(m.mu, &md.mu); up(m.inv_sigma, &md.inv_sigma);
    up(m.type_bias, &md.type_bias);
    for (int t = 0; t < h->d.n_hidden; ++t) { up(m.theta[t], &md.theta[t]); up(m.thetaT[t], &md.thetaT[t]); up(m.bias[t], &md.bias[t]);
        uph(m.theta_hi[t], &md.theta_hi[t]); uph(m.theta_lo[t], &md.theta_lo[t]);
        uph(m.thetaT_hi[t], &md.thetaT_hi[t]); uph(m.thetaT_lo[t], &md.thetaT_lo[t]);
        md.w_scale_inv[t] = 1.0f / m.w_scale[t]; }
    md.grad_scale = m.grad_scale;
    up(m.w_head, &md.w_head); up(m.e_ref, &md.e_ref);
    md.b_head = m.b_head;
    if (e == cudaSuccess && h->d.L >= 3) {
        std::vector<GauntSparse> g1(1, m.g123), g2(1, m.g233);
        e = upload(h, g1, &md.g123);
        if (e == cudaSuccess) e = upload(h, g2, &md.g233);
    }
    if (e == cudaSuccess && h->d.L >= 4) e = upload(h, m.g4, &md.g4);
    void* p = nullptr;
    if (e == cudaSuccess) { e = dev_malloc(&p, sizeof(double) * (reduce_scratch_doubles(0) + 16)); h->scratch = (double*)p; }
    if (e == cudaSuccess) { e = dev_malloc(&p, sizeof(double) * 16); h->d_out = (double*)p; }
    if (e == cudaSuccess) { e = dev_malloc(&p, sizeof(int) * 4); h->d_err = (int*)p; }
    if (e == cudaSuccess) e = cudaMemsetAsync(h->d_err, 0, sizeof(int) * 4, h->st);
    if (e == cudaSuccess) e = cudaMallocHost((void**)&h->h_out, sizeof(double) * 16);
    if (e == cudaSuccess) e = cudaMallocHost((void**)&h->h_err, sizeof(int) * 4);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->st);
    if (e != cudaSuccess) return fail(h, UMLMD_E_CUDA, std::string("model upload: ") + cudaGetErrorString(e));
    h->on_device = true;
    return UMLMD_OK;
}

int build_list(umlmd_t* h, int64_t N, const double* d_pos, const int32_t* d_type, const double cell[9],
               const int pbc[3], double skin) {
    int rc = ensure_device_model(h);
    if (rc != UMLMD_OK) return rc;
    { Scope sc(h, kNeighbor, 7); rc = neighbor_build(&h->nb, N, h->n_owned, d_pos, d_type, cell, pbc, skin, h->hm.rc, h->d_err, h->st, &h->err); }
    if (rc != UMLMD_OK) { h->have_list = false; return rc; }
    h->have_list = true;
    h->have_edge_grad = false;       // edges were renumbered
    h->steps_since_build = 0;
    ++h->list_serial;                // recorded launch sequences name the old list
    rc = ensure_workspace(h);
    if (rc != UMLMD_OK) return rc;
    if (h->nb.n_owned < h->nb.N) {
        // ghost atoms come last in the internal order and no stage visits their rows: their atomic
        // energies and the gradients of their edges are zero from here until the next build
        API_CUDA(h, cudaMemsetAsync(h->e_atom + h->nb.n_owned, 0, sizeof(double) * (size_t)(h->nb.N - h->nb.n_owned), h->st));
        if (h->nb.E > h->nb.E_owned)
            API_CUDA(h, cudaMemsetAsync(h->g + 3 * (size_t)h->nb.E_owned, 0, sizeof(float) * 3 * (size_t)(h->nb.E - h->nb.E_owned), h->st));
    }
    return UMLMD_OK;
}

// With few species present, psi_c(rho) of every ordered pair among them is tabulated by itself,
// so that the edge kernels read one table row per edge and neither pair rows nor shared modes.
// The tables depend on the model and the set of species only, so they are kept across builds.
int setup_pair_tables(umlmd_t* h) {
    const Dims& d = h->d;
    std::vector<int> present;
    for (int t = 0; t < d.T; ++t) if (h->h_species[t]) present.push_back(t);
    const size_t np = present.size();
    const size_t floats = np * np * (size_t)d.n_rows * 3 * d.C0;
    h->pair_tables = np > 0 && h->pair_table_budget >= 0 && floats * sizeof(float) <= (size_t)h->pair_table_budget;
    if (!h->pair_tables || present == h->present) return UMLMD_OK;
    if (floats > h->table_uni_cap) {
        dev_free(h->table_uni); h->table_uni = nullptr; h->table_uni_cap = 0;
        void* p = nullptr;
        API_CUDA(h, dev_malloc(&p, sizeof(float) * floats));
        h->table_uni = (float*)p; h->table_uni_cap = floats;
    }
    std::vector<int> up(2 * (size_t)d.T, 0);          // species -> slot, then the present list
    for (size_t k = 0; k < np; ++k) { up[present[k]] = (int)k; up[d.T + k] = present[k]; }
    API_CUDA(h, cudaMemcpyAsync(h->d_species + d.T, up.data(), sizeof(int) * up.size(), cudaMemcpyHostToDevice, h->st));
    if (!h->uni_scale) { void* p = nullptr; API_CUDA(h, dev_malloc(&p, 4 * sizeof(float))); h->uni_scale = (float*)p; }
    API_CUDA(h, launch_fuse_pair_tables(d, h->md.table, h->md.pairmod, h->d_species + 2 * d.T, (int)np, h->uni_scale, h->table_uni, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));       // `up` is pageable host memory
    h->launches_total += 2;
    h->present = present;
    return UMLMD_OK;
}

}  // namespace

extern "C" {

int umlmd_profile_widths(int32_t C0, int32_t L, int32_t R, umlmd_info* out) {
    if (!out) return UMLMD_E_INVALID_ARG;
    Dims d;
    if (!derive_dims(C0, L, R, &d)) return UMLMD_E_UNSUPPORTED_PROFILE;
    std::memset(out, 0, sizeof(*out));
    fill_info(d, out);
    return UMLMD_OK;
}

int umlmd_create(const void* blob, size_t blob_bytes, const umlmd_options* opt, void* stream, umlmd_t** out) {
    if (!blob || !out) return UMLMD_E_INVALID_ARG;
    *out = nullptr;
    umlmd_t* h = new (std::nothrow) umlmd();
    if (!h) return UMLMD_E_INVALID_ARG;
    h->st = static_cast<cudaStream_t>(stream);
    double dx_override = 0;
    if (opt) {
        if (opt->struct_bytes != sizeof(umlmd_options)) { delete h; return UMLMD_E_INVALID_ARG; }
        if (opt->table_dx < 0 || opt->node_tile < 0 || opt->mlp_path < 0 || opt->mlp_path > 4) { delete h; return UMLMD_E_INVALID_ARG; }
        dx_override = opt->table_dx;
        if (opt->node_tile > 0) h->node_tile = opt->node_tile;
        if (opt->mlp_path > 0) h->mlp_path = opt->mlp_path;
        if (opt->pair_table_mb != 0) h->pair_table_budget = opt->pair_table_mb < 0 ? -1 : (int64_t)opt->pair_table_mb << 20;
        if (opt->gemm_spin_limit < 0 || opt->fault_skip_gemm_stage < 0) { delete h; return UMLMD_E_INVALID_ARG; }
        h->gemm_spin_limit = opt->gemm_spin_limit;
        h->fault_skip_stage = opt->fault_skip_gemm_stage;
        if (opt->launch_graphs < -1 || opt->launch_graphs > 1) { delete h; return UMLMD_E_INVALID_ARG; }
        h->launch_graphs = opt->launch_graphs;
    }
    int rc = build_host_model(blob, blob_bytes, dx_override, &h->hm, &h->err);
    if (rc != UMLMD_OK) { delete h; return rc; }
    h->d = h->hm.d;
    *out = h;
    return UMLMD_OK;
}

int umlmd_destroy(umlmd_t* h) {
    if (!h) return UMLMD_OK;
    if (h->on_device) cudaStreamSynchronize(h->st);
    for (void* p : h->model_allocs) dev_free(p);
    neighbor_free(&h->nb);
    void* ptrs[] = {h->frame_out, h->state, h->desc, h->pre, h->hbuf, h->tc_hi, h->tc_lo, h->g, h->e_atom, h->f_sorted, h->type_o, h->virial_part,
                    h->scratch, h->d_out, h->d_err, h->md_force, h->d_mass, h->d_inv_mass, h->d_nhc, h->table_uni, h->d_species, h->uni_scale};
    for (void* p : ptrs) dev_free(p);
    for (auto& sp : h->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (cudaEvent_t e : h->free_events) cudaEventDestroy(e);
    if (h->rp_compute.exec) cudaGraphExecDestroy(h->rp_compute.exec);
    if (h->rp_step.exec) cudaGraphExecDestroy(h->rp_step.exec);
    if (h->rp_nvt.exec) cudaGraphExecDestroy(h->rp_nvt.exec);
    if (h->cap_st) cudaStreamDestroy(h->cap_st);
    if (h->h_out) cudaFreeHost(h->h_out);
    if (h->h_err) cudaFreeHost(h->h_err);
    if (h->h_species) cudaFreeHost(h->h_species);
    delete h;
    return UMLMD_OK;
}

int umlmd_query(const umlmd_t* h, umlmd_info* out) {
    if (!h || !out) return UMLMD_E_INVALID_ARG;
    std::memset(out, 0, sizeof(*out));
    fill_info(h->d, out);
    out->rc = h->hm.rc; out->table_dx = h->hm.dx;
    out->n_atoms = h->have_list ? h->nb.N : 0;
    out->n_edges = h->have_list ? h->nb.E : 0;
    out->device_bytes = dev_bytes_held();
    out->kernel_launches = h->launches_total;
    out->graph_replays = h->graph_replays;
    return UMLMD_OK;
}

const char* umlmd_last_error(const umlmd_t* h) { return h ? h->err.c_str() : "null handle"; }

int umlmd_build_neighbors(umlmd_t* h, int64_t N, const double* d_pos, const int32_t* d_type, const double cell[9],
                          const int pbc[3], double skin) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (N < 0 || !cell || !pbc || !(skin >= 0) || !std::isfinite(skin) || (N > 0 && (!d_pos || !d_type)))
        return fail(h, UMLMD_E_INVALID_ARG, "bad argument to umlmd_build_neighbors");
    bool diagonal = true;
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            const double v = cell[3 * i + j];
            if (!std::isfinite(v)) return fail(h, UMLMD_E_UNSUPPORTED_CELL, "non-finite cell");
            if (i != j && v != 0.0) diagonal = false;
        }
    if (diagonal)
        for (int i = 0; i < 3; ++i)
            if (!(cell[4 * i] > 0.0)) return fail(h, UMLMD_E_UNSUPPORTED_CELL, "cell edges must be positive");
    h->have_md = false;
    int rc = build_list(h, N, d_pos, d_type, cell, pbc, skin);
    if (rc != UMLMD_OK) return rc;
    if (N > 0) API_CUDA(h, cudaMemcpyAsync(h->type_o, d_type, sizeof(int) * N, cudaMemcpyDeviceToDevice, h->st));
    // which species occur: few enough of them get per-pair amplitude tables (see below)
    const int T = h->d.T;
    if (!h->d_species) {
        void* p = nullptr;
        API_CUDA(h, dev_malloc(&p, sizeof(int) * 3 * (size_t)T));
        h->d_species = (int*)p;
        API_CUDA(h, cudaMallocHost((void**)&h->h_species, sizeof(int) * (size_t)T));
    }
    API_CUDA(h, launch_species_present(N, d_type, T, h->d_species, h->d_err, h->st));
    h->launches_total += N > 0;
    API_CUDA(h, cudaMemcpyAsync(h->h_species, h->d_species, sizeof(int) * (size_t)T, cudaMemcpyDeviceToHost, h->st));
    // surface device-side findings of the build (non-finite positions, image range)
    API_CUDA(h, cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, h->st));
    API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    rc = decode_device_errors(h, *h->h_err);
    if (rc != UMLMD_OK) { h->have_list = false; return rc; }
    return setup_pair_tables(h);
}

int umlmd_get_neighbors(umlmd_t* h, int32_t* d_row_ptr, int32_t* d_src, int8_t* d_shift, int64_t cap,
                        int64_t* n_edges) {
    if (!h || !n_edges) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "no neighbor list built");
    *n_edges = h->nb.E;
    if (cap == 0) return UMLMD_OK;
    if (cap < h->nb.E) return fail(h, UMLMD_E_CAPACITY, "edge buffers smaller than the list");
    if (h->nb.E > 0x7fffffffll) return fail(h, UMLMD_E_CAPACITY, "the export has 32-bit row pointers; this list has more than 2^31 - 1 edges");
    if (!d_row_ptr || (h->nb.E > 0 && (!d_src || !d_shift))) return fail(h, UMLMD_E_INVALID_ARG, "null output buffer");
    int rc = neighbor_export(&h->nb, d_row_ptr, d_src, d_shift, h->st, &h->err);
    if (rc != UMLMD_OK) return rc;
    API_CUDA(h, cudaStreamSynchronize(h->st));
    return UMLMD_OK;
}

int umlmd_get_neighbor_rows(umlmd_t* h, int64_t first_row, int64_t n_rows, int64_t* d_row_ptr, int32_t* d_src,
                            int8_t* d_shift, int64_t cap, int64_t* n_edges) {
    if (!h || !n_edges) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "no neighbor list built");
    if (first_row < 0 || n_rows < 0 || first_row + n_rows > h->nb.N) return fail(h, UMLMD_E_INVALID_ARG, "row range outside [0, N)");
    if (!d_row_ptr) return fail(h, UMLMD_E_INVALID_ARG, "null row offsets");
    if (cap < 0 || (cap > 0 && (!d_src || !d_shift))) return fail(h, UMLMD_E_INVALID_ARG, "null edge buffers");
    int rc = neighbor_export_rows(&h->nb, first_row, n_rows, d_row_ptr, d_src, d_shift, cap, h->st, &h->err);
    if (rc != UMLMD_OK) return rc;
    int64_t total = 0;
    API_CUDA(h, cudaMemcpyAsync(&total, d_row_ptr + n_rows, sizeof(total), cudaMemcpyDeviceToHost, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    *n_edges = total;
    if (cap > 0 && cap < total) return fail(h, UMLMD_E_CAPACITY, "edge buffers smaller than the rows asked for");
    return UMLMD_OK;
}

int umlmd_workspace_bytes(const umlmd_t* h, int64_t N, int64_t n_edges, int64_t* bytes) {
    if (!h || !bytes || N < 0 || n_edges < 0) return UMLMD_E_INVALID_ARG;
    const Dims& d = h->d;
    const HostModel& m = h->hm;
    auto buf = [](int64_t n, int64_t elem) { return (n + 16) * elem; };          // dev_ensure pads by 16 elements
    auto grown = [](int64_t n, int64_t elem) { return ((int64_t)(n * 1.1) + 16) * elem; };
    int64_t t = 0;
    // model constants (uploaded by the first build)
    auto vec = [&](size_t n, size_t elem) { t += (int64_t)(n * elem + 16); };
    vec(m.table.size(), 4); vec(m.pairmod.size(), 4); vec(m.X0.size(), 4); vec(m.W1p.size(), 4); vec(m.W2p.size(), 4);
    vec(m.A1.size(), 4); vec(m.A2.size(), 4); vec(m.mu.size(), 4); vec(m.inv_sigma.size(), 4); vec(m.type_bias.size(), 4);
    for (int k = 0; k < d.n_hidden; ++k) {
        vec(m.theta[k].size(), 4); vec(m.thetaT[k].size(), 4); vec(m.bias[k].size(), 4);
        vec(m.theta_hi[k].size(), 2); vec(m.theta_lo[k].size(), 2); vec(m.thetaT_hi[k].size(), 2); vec(m.thetaT_lo[k].size(), 2);
    }
    vec(m.w_head.size(), 4); vec(m.e_ref.size(), 4);
    if (d.L >= 3) t += 2 * (int64_t)(sizeof(GauntSparse) + 16);
    if (d.L >= 4) t += (int64_t)(5 * sizeof(GauntSparseBig) + 16);
    t += 8 * (reduce_scratch_doubles(0) + 16) + 8 * 16 + 4 * 4 + 4 * 3 * d.T + 16;
    // neighbor list: per-atom arrays, cell table (at most 8 N + 64 cells), edges, sort / scan scratch
    const int64_t A = N + 1;
    t += buf(3 * A, 8) * 3 + buf(6 * A, 4) + buf(A, 4) * 2 + buf(A + 1, 8) + buf(A, 4) * 4 + buf(A + 1, 4);
    t += buf(8 * N + 64 + 2, 4);
    t += grown(n_edges, 4) * 2 + grown(n_edges, 8);
    t += 16 * A + (2 << 20);
    // evaluation workspace of one node tile, per-edge gradients, per-atom results, MD forces
    const int64_t Bt = N < h->node_tile ? N : h->node_tile;
    const int64_t wmax = d.DP > d.F ? d.DP : d.F;
    t += buf(Bt * d.SP, 4) + buf(Bt * d.DP, 4) + buf(Bt * d.F * d.n_hidden, 4) + buf(Bt * d.F * 2, 4) + 2 * buf(2 * Bt * wmax, 2);
    t += grown(3 * n_edges, 4);
    t += buf(N, 8) + buf(3 * N, 8) + buf(N, 4);
    const int64_t tiles = Bt > 0 ? (N + Bt - 1) / Bt : 0;
    t += buf((N / 4 + tiles + 2) * 9, 8);
    t += buf(3 * N, 8) + 2 * buf(d.T, 8) + buf(2 * kNhcChain + 2, 8);
    *bytes = t;
    return UMLMD_OK;
}

int umlmd_get_nvt_state(umlmd_t* h, double state[UMLMD_NVT_STATE_DOUBLES]) {
    if (!h || !state) return UMLMD_E_INVALID_ARG;
    static_assert(UMLMD_NVT_STATE_DOUBLES == 2 * kNhcChain, "thermostat state size");
    for (int k = 0; k < UMLMD_NVT_STATE_DOUBLES; ++k) state[k] = 0.0;
    if (!h->d_nhc || h->nhc_reset) return UMLMD_OK;            // chain at rest
    API_CUDA(h, cudaMemcpyAsync(state, h->d_nhc, sizeof(double) * UMLMD_NVT_STATE_DOUBLES, cudaMemcpyDeviceToHost, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    return UMLMD_OK;
}

int umlmd_set_nvt_state(umlmd_t* h, const double state[UMLMD_NVT_STATE_DOUBLES]) {
    if (!h || !state) return UMLMD_E_INVALID_ARG;
    if (!h->have_md) return fail(h, UMLMD_E_NO_MD_STATE, "umlmd_set_md_state must be called first");
    for (int k = 0; k < UMLMD_NVT_STATE_DOUBLES; ++k)
        if (!std::isfinite(state[k])) return fail(h, UMLMD_E_INVALID_ARG, "non-finite thermostat state");
    if (!h->d_nhc) { int64_t c = 0; API_CUDA(h, dev_ensure(&h->d_nhc, &c, 2 * kNhcChain + 2)); }
    double full[2 * kNhcChain + 2] = {0};
    for (int k = 0; k < UMLMD_NVT_STATE_DOUBLES; ++k) full[k] = state[k];
    full[2 * kNhcChain] = 1.0;
    API_CUDA(h, cudaMemcpyAsync(h->d_nhc, full, sizeof(full), cudaMemcpyHostToDevice, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    h->nhc_reset = false;
    return UMLMD_OK;
}

int umlmd_compute(umlmd_t* h, const double* d_pos, double* energy, double* d_force, double virial[9],
                  double* d_atom_energy) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "umlmd_build_neighbors must be called first");
    if (h->nb.N > 0 && !d_pos) return fail(h, UMLMD_E_INVALID_ARG, "null positions");
    const bool want_grad = d_force != nullptr || virial != nullptr;
    if (h->nb.N == 0) {
        if (energy) *energy = 0;
        if (virial) for (int k = 0; k < 9; ++k) virial[k] = 0;
        return UMLMD_OK;
    }
    int rc = run_replayed(h, h->rp_compute, d_pos, d_force, d_atom_energy, nullptr, 0.0, want_grad ? 1 : 0, [&]() {
        int r = enqueue_compute(h, d_pos, want_grad, d_force, d_atom_energy);
        return r != UMLMD_OK ? r : enqueue_fetch(h, 10);
    });
    if (rc != UMLMD_OK) return rc;
    rc = finish_fetch(h);
    if (rc != UMLMD_OK) return rc;
    if (energy) *energy = h->h_out[0];
    if (virial) for (int k = 0; k < 9; ++k) virial[k] = h->h_out[1 + k];
    return UMLMD_OK;
}

int umlmd_compute_batch(umlmd_t* h, int32_t n_frames, const int64_t* frame_offsets, const double* d_pos,
                        const int32_t* d_type, const double* cells, const int pbc[3], double* energies, double* d_force,
                        double* virials, double* d_atom_energy) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (n_frames < 0 || (n_frames > 0 && (!frame_offsets || !cells)) || !pbc)
        return fail(h, UMLMD_E_INVALID_ARG, "bad argument to umlmd_compute_batch");
    if (n_frames == 0) return UMLMD_OK;
    if (frame_offsets[0] != 0) return fail(h, UMLMD_E_INVALID_ARG, "frame_offsets must start at 0");
    for (int f = 0; f < n_frames; ++f) {
        const int64_t n = frame_offsets[f + 1] - frame_offsets[f];
        if (n < 0) return fail(h, UMLMD_E_INVALID_ARG, "frame_offsets must not decrease");
        if (n > UMLMD_BATCH_MAX_FRAME_ATOMS)
            return fail(h, UMLMD_E_CAPACITY, "a frame of a batch holds more atoms than the exhaustive per-frame search is meant for; use umlmd_build_neighbors");
    }
    const int64_t N = frame_offsets[n_frames];
    if (N > 0x7fff0000LL) return fail(h, UMLMD_E_INVALID_ARG, "too many atoms for 32-bit indices");
    if (N > 0 && (!d_pos || !d_type)) return fail(h, UMLMD_E_INVALID_ARG, "null positions or species");
    int rc = ensure_device_model(h);
    if (rc != UMLMD_OK) return rc;
    h->have_list = false; h->have_md = false; h->have_edge_grad = false;     // the handle's list is replaced
    ++h->list_serial;
    { Scope sc(h, kNeighbor, 5); rc = neighbor_build_batch(&h->nb, n_frames, frame_offsets, cells, pbc, d_pos, d_type, h->d.T, h->hm.rc, h->d_err, h->st, &h->err); }
    if (rc != UMLMD_OK) return rc;
    const bool want_grad = d_force != nullptr || virials != nullptr;
    if (N > 0) {
        if ((rc = ensure_workspace(h)) != UMLMD_OK) return rc;
        const int T = h->d.T;
        if (!h->d_species) {
            void* p = nullptr;
            API_CUDA(h, dev_malloc(&p, sizeof(int) * 3 * (size_t)T));
            h->d_species = (int*)p;
            API_CUDA(h, cudaMallocHost((void**)&h->h_species, sizeof(int) * (size_t)T));
        }
        API_CUDA(h, launch_species_present(N, h->nb.type_s, T, h->d_species, h->d_err, h->st));
        h->launches_total += 1;
        API_CUDA(h, cudaMemcpyAsync(h->h_species, h->d_species, sizeof(int) * (size_t)T, cudaMemcpyDeviceToHost, h->st));
        API_CUDA(h, cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, h->st));
        API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
        API_CUDA(h, cudaStreamSynchronize(h->st));
        if ((rc = decode_device_errors(h, *h->h_err)) != UMLMD_OK) return rc;
        if ((rc = setup_pair_tables(h)) != UMLMD_OK) return rc;
        if ((rc = enqueue_compute(h, d_pos, want_grad, d_force, d_atom_energy)) != UMLMD_OK) return rc;
    }
    API_CUDA(h, dev_ensure(&h->frame_out, &h->frame_out_cap, (int64_t)n_frames * 10));
    if (N > 0) {
        Scope sc(h, kReduce, 1);
        API_CUDA(h, launch_frame_reduce(h->nb, h->e_atom, h->g, virials != nullptr, h->frame_out, h->st));
    } else {
        API_CUDA(h, cudaMemsetAsync(h->frame_out, 0, sizeof(double) * 10 * (size_t)n_frames, h->st));
    }
    std::vector<double> host((size_t)n_frames * 10);
    API_CUDA(h, cudaMemcpyAsync(host.data(), h->frame_out, sizeof(double) * host.size(), cudaMemcpyDeviceToHost, h->st));
    if (N > 0) { if ((rc = fetch_results(h, 10)) != UMLMD_OK) return rc; }
    else API_CUDA(h, cudaStreamSynchronize(h->st));
    for (int f = 0; f < n_frames; ++f) {
        if (energies) energies[f] = host[10 * (size_t)f];
        if (virials) for (int k = 0; k < 9; ++k) virials[9 * (size_t)f + k] = host[10 * (size_t)f + 1 + k];
    }
    return UMLMD_OK;
}

int umlmd_set_md_state(umlmd_t* h, double* d_pos, double* d_vel, const double* mass_per_type) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "umlmd_build_neighbors must be called first");
    if (!d_pos || !d_vel || !mass_per_type) return fail(h, UMLMD_E_INVALID_ARG, "null MD state");
    const int T = h->d.T;
    std::vector<double> m(T), im(T);
    for (int t = 0; t < T; ++t) {
        if (!(mass_per_type[t] > 0) || !std::isfinite(mass_per_type[t])) return fail(h, UMLMD_E_INVALID_ARG, "masses must be positive");
        m[t] = mass_per_type[t]; im[t] = 1.0 / mass_per_type[t];
    }
    int64_t c;
    if (!h->d_mass) { c = 0; API_CUDA(h, dev_ensure(&h->d_mass, &c, T)); c = 0; API_CUDA(h, dev_ensure(&h->d_inv_mass, &c, T)); }
    API_CUDA(h, cudaMemcpyAsync(h->d_mass, m.data(), sizeof(double) * T, cudaMemcpyHostToDevice, h->st));
    API_CUDA(h, cudaMemcpyAsync(h->d_inv_mass, im.data(), sizeof(double) * T, cudaMemcpyHostToDevice, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    if (h->nb.N > h->md_cap || !h->md_force) API_CUDA(h, dev_ensure(&h->md_force, &h->md_cap, h->nb.N * 3));
    h->md_pos = d_pos; h->md_vel = d_vel;
    h->have_md = true; h->have_force = false; h->nhc_reset = true;
    ++h->list_serial;                // masses and buffers of the recorded step sequence may have changed
    return UMLMD_OK;
}

// after a drift: rebuild the list if the schedule (rebuild_every > 0) or the displacement
// criterion (rebuild_every < 0) asks for it
static int maybe_rebuild(umlmd_t* h, int rebuild_every) {
    const int64_t N = h->nb.N;
    bool rebuild = rebuild_every > 0 && h->steps_since_build >= rebuild_every;
    if (rebuild_every < 0) {
        // displacement-triggered: the gather pass flags any atom that has moved more than half
        // the skin since the build; read the flag (one host synchronisation per step)
        API_CUDA(h, launch_gather_positions(h->nb, h->md_pos, h->d_err, h->st));
        API_CUDA(h, cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, h->st));
        API_CUDA(h, cudaStreamSynchronize(h->st));
        const int word = *h->h_err;
        if (word & ~kErrStale) {
            API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
            return decode_device_errors(h, word & ~kErrStale);
        }
        if (word & kErrStale) {
            API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
            rebuild = true;
        }
    }
    if (rebuild) {
        const double skin = h->nb.skin;
        double cell[9];
        for (int k = 0; k < 9; ++k) cell[k] = h->nb.H[k];
        const int pbc[3] = {h->nb.pbc[0], h->nb.pbc[1], h->nb.pbc[2]};
        // The build synchronises the stream anyway (it reads the edge count), so this is the place
        // to look at what the steps since the previous build reported: a list that went stale, or a
        // non-finite value, ends the run here instead of after the last step.
        API_CUDA(h, cudaMemcpyAsync(h->h_err, h->d_err, sizeof(int), cudaMemcpyDeviceToHost, h->st));
        int rc = build_list(h, N, h->md_pos, h->type_o, cell, pbc, skin);
        if (rc != UMLMD_OK) return rc;
        const int word = *h->h_err;                  // the build has synchronised the stream since the copy
        if (word) {
            API_CUDA(h, cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st));
            return decode_device_errors(h, word);
        }
    }
    return UMLMD_OK;
}

// error exit of a stepping loop: the error word must not leak into the next call, and the forces
// kept for the next step's opening kick no longer match the positions
static int stop_run(umlmd_t* h, int rc) {
    h->have_force = false;
    if (h->d_err) cudaMemsetAsync(h->d_err, 0, sizeof(int), h->st);
    return rc;
}

int umlmd_step(umlmd_t* h, int nsteps, double dt_ps, int rebuild_every, double* e_pot, double* e_kin) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "umlmd_build_neighbors must be called first");
    if (!h->have_md) return fail(h, UMLMD_E_NO_MD_STATE, "umlmd_set_md_state must be called first");
    if (nsteps < 0 || !(dt_ps > 0) || !std::isfinite(dt_ps)) return fail(h, UMLMD_E_INVALID_ARG, "bad step count or time step");
    if (h->nb.n_owned < h->nb.N)
        return fail(h, UMLMD_E_INVALID_ARG, "this driver integrates every atom of the handle; with ghost atoms use umlmd_compute and umlmd_vv_update");
    const int64_t N = h->nb.N;
    int rc;
    if (!h->have_force) {
        if ((rc = enqueue_compute(h, h->md_pos, true, h->md_force, nullptr)) != UMLMD_OK) return rc;
        h->have_force = true;
    }
    for (int s = 0; s < nsteps; ++s) {
        // opening half kick and drift; from the second step on they were fused with the previous
        // step's closing half kick
        if (s == 0) { Scope sc(h, kIntegrate, 1); API_CUDA(h, launch_vv_kick_drift(N, h->md_pos, h->md_vel, h->md_force, h->type_o, h->d_inv_mass, dt_ps, 1, true, nullptr, h->st)); }
        ++h->steps_since_build;
        if ((rc = maybe_rebuild(h, rebuild_every)) != UMLMD_OK) return stop_run(h, rc);
        const bool last = s + 1 == nsteps;
        auto body = [&]() {
            int r = enqueue_compute(h, h->md_pos, true, h->md_force, nullptr);
            if (r != UMLMD_OK) return r;
            Scope sc(h, kIntegrate, 1);
            API_CUDA(h, launch_vv_kick_drift(N, h->md_pos, h->md_vel, h->md_force, h->type_o, h->d_inv_mass, dt_ps, last ? 1 : 2, !last, nullptr, h->st));
            return (int)UMLMD_OK;
        };
        // a middle step between two list builds launches the same sequence as the one before it
        rc = last ? body() : run_replayed(h, h->rp_step, h->md_pos, h->md_vel, h->md_force, nullptr, dt_ps, 0, body);
        if (rc != UMLMD_OK) return stop_run(h, rc);
    }
    { Scope sc(h, kIntegrate, 2); API_CUDA(h, launch_kinetic_energy(N, h->md_vel, h->type_o, h->d_mass, h->scratch, h->d_out + 10, h->st)); }
    rc = fetch_results(h, 11);
    if (rc != UMLMD_OK) return stop_run(h, rc);
    if (e_pot) *e_pot = h->h_out[0];
    if (e_kin) *e_kin = h->h_out[10];
    return UMLMD_OK;
}

int umlmd_step_nvt(umlmd_t* h, int nsteps, double dt_ps, int rebuild_every, double temperature_K, double t_damp_ps,
                   double* e_pot, double* e_kin, double* e_conserved) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "umlmd_build_neighbors must be called first");
    if (!h->have_md) return fail(h, UMLMD_E_NO_MD_STATE, "umlmd_set_md_state must be called first");
    if (nsteps < 0 || !(dt_ps > 0) || !std::isfinite(dt_ps) || !(temperature_K > 0) || !std::isfinite(temperature_K) ||
        !(t_damp_ps > 0) || !std::isfinite(t_damp_ps))
        return fail(h, UMLMD_E_INVALID_ARG, "bad step count, time step, temperature or damping time");
    const int64_t N = h->nb.N;
    if (h->nb.n_owned < N)
        return fail(h, UMLMD_E_INVALID_ARG, "this driver integrates every atom of the handle; with ghost atoms use umlmd_compute and umlmd_vv_update");
    if (N < 2) return fail(h, UMLMD_E_INVALID_ARG, "the thermostat needs at least two atoms");
    constexpr int M = kNhcChain;
    int rc;
    if (!h->d_nhc) { int64_t c = 0; API_CUDA(h, dev_ensure(&h->d_nhc, &c, 2 * M + 2)); h->nhc_reset = true; }
    if (h->nhc_reset) { API_CUDA(h, cudaMemsetAsync(h->d_nhc, 0, sizeof(double) * (2 * M + 2), h->st)); h->nhc_reset = false; }
    NhcParams p;
    p.dof = 3.0 * (double)N - 3.0;
    p.kT = kBoltzmann * temperature_K;
    p.Q[0] = p.dof * p.kT * t_damp_ps * t_damp_ps;
    for (int k = 1; k < M; ++k) p.Q[k] = p.kT * t_damp_ps * t_damp_ps;
    p.dt_half = 0.5 * dt_ps;
    if (!h->have_force) {
        if ((rc = enqueue_compute(h, h->md_pos, true, h->md_force, nullptr)) != UMLMD_OK) return rc;
        h->have_force = true;
    }
    double* d_ke = h->d_out + 10;
    double* d_scale = h->d_nhc + 2 * M;
    if (nsteps > 0) {      // opening half step of the chain for the first step
        Scope sc(h, kIntegrate, 3);
        API_CUDA(h, launch_kinetic_energy(N, h->md_vel, h->type_o, h->d_mass, h->scratch, d_ke, h->st));
        API_CUDA(h, launch_nhc(h->d_nhc, d_ke, 1, p, h->st));
    }
    for (int s = 0; s < nsteps; ++s) {
        { Scope sc(h, kIntegrate, 1); API_CUDA(h, launch_vv_kick_drift(N, h->md_pos, h->md_vel, h->md_force, h->type_o, h->d_inv_mass, dt_ps, 1, true, d_scale, h->st)); }
        ++h->steps_since_build;
        if ((rc = maybe_rebuild(h, rebuild_every)) != UMLMD_OK) return stop_run(h, rc);
        const bool last = s + 1 == nsteps;
        auto body = [&]() {
            int r = enqueue_compute(h, h->md_pos, true, h->md_force, nullptr);
            if (r != UMLMD_OK) return r;
            Scope sc(h, kIntegrate, 4);
            API_CUDA(h, launch_vv_kick_drift(N, h->md_pos, h->md_vel, h->md_force, h->type_o, h->d_inv_mass, dt_ps, 1, false, nullptr, h->st));
            API_CUDA(h, launch_kinetic_energy(N, h->md_vel, h->type_o, h->d_mass, h->scratch, d_ke, h->st));
            // closing half step of the chain, and the next step's opening one in the same launch
            API_CUDA(h, launch_nhc(h->d_nhc, d_ke, last ? 1 : 2, p, h->st));
            return (int)UMLMD_OK;
        };
        // a middle step between two list builds launches the same sequence as the one before it (the
        // opening kick and drift above differ between the first step of a call and the others: plain)
        rc = last ? body() : run_replayed(h, h->rp_nvt, h->md_pos, h->md_vel, h->md_force, h->d_nhc, dt_ps, 0, body,
                                          temperature_K, t_damp_ps);
        if (rc != UMLMD_OK) return stop_run(h, rc);
    }
    if (nsteps > 0) {      // the last scale factor has not been applied to the velocities yet
        Scope sc(h, kIntegrate, 1);
        API_CUDA(h, launch_vv_kick_drift(N, h->md_pos, h->md_vel, h->md_force, h->type_o, h->d_inv_mass, dt_ps, 0, false, d_scale, h->st));
    } else {
        Scope sc(h, kIntegrate, 2);
        API_CUDA(h, launch_kinetic_energy(N, h->md_vel, h->type_o, h->d_mass, h->scratch, d_ke, h->st));
        API_CUDA(h, cudaMemcpyAsync(h->d_nhc + 2 * M + 1, d_ke, sizeof(double), cudaMemcpyDeviceToDevice, h->st));
    }
    double chain[2 * M + 2];
    API_CUDA(h, cudaMemcpyAsync(chain, h->d_nhc, sizeof(chain), cudaMemcpyDeviceToHost, h->st));
    rc = fetch_results(h, 10);
    if (rc != UMLMD_OK) return stop_run(h, rc);
    const double ke = chain[2 * M + 1];
    if (e_pot) *e_pot = h->h_out[0];
    if (e_kin) *e_kin = ke;
    if (e_conserved) {
        double e = h->h_out[0] + ke + p.dof * p.kT * chain[0];
        for (int k = 0; k < M; ++k) e += 0.5 * p.Q[k] * chain[M + k] * chain[M + k];
        for (int k = 1; k < M; ++k) e += p.kT * chain[k];
        *e_conserved = e;
    }
    return UMLMD_OK;
}

int umlmd_atom_virial(umlmd_t* h, double* d_atom_virial) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "umlmd_build_neighbors must be called first");
    if (!h->have_edge_grad) return fail(h, UMLMD_E_INVALID_ARG, "no evaluation with forces or virial since the last build");
    if (h->nb.N > 0 && !d_atom_virial) return fail(h, UMLMD_E_INVALID_ARG, "null output buffer");
    { Scope sc(h, kForce, 1); API_CUDA(h, launch_atom_virial(h->nb, h->g, d_atom_virial, h->st)); }
    API_CUDA(h, cudaStreamSynchronize(h->st));
    return UMLMD_OK;
}

int umlmd_set_owned_atoms(umlmd_t* h, int64_t n_owned) {
    if (!h) return UMLMD_E_INVALID_ARG;
    h->n_owned = n_owned < 0 ? -1 : n_owned;
    // the internal order of the atoms depends on it: the next evaluation needs a new list
    h->have_list = false; h->have_md = false; h->have_force = false; h->have_edge_grad = false;
    ++h->list_serial;
    return UMLMD_OK;
}

int umlmd_vv_update(int64_t N, double* d_pos, double* d_vel, const double* d_force, const int32_t* d_type,
                    const double* d_inv_mass_per_type, double dt_ps, int32_t half_kicks, int32_t drift, void* stream) {
    if (N < 0 || half_kicks < 0 || half_kicks > 2 || !(dt_ps > 0) || !std::isfinite(dt_ps)) return UMLMD_E_INVALID_ARG;
    if (N > 0 && (!d_vel || !d_type || !d_inv_mass_per_type || (half_kicks > 0 && !d_force) || (drift && !d_pos)))
        return UMLMD_E_INVALID_ARG;
    if (N == 0 || (half_kicks == 0 && !drift)) return UMLMD_OK;
    cudaError_t e = launch_vv_kick_drift(N, d_pos, d_vel, d_force, d_type, d_inv_mass_per_type, dt_ps, half_kicks, drift != 0,
                                         nullptr, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? UMLMD_OK : UMLMD_E_CUDA;
}

int umlmd_get_intermediates(umlmd_t* h, float* d_state, float* d_desc) {
    if (!h) return UMLMD_E_INVALID_ARG;
    if (!h->have_list) return fail(h, UMLMD_E_NO_NEIGHBORS, "no neighbor list built");
    if (!keeps_intermediates(h)) return fail(h, UMLMD_E_CAPACITY, "intermediates are only kept for systems of one tile and fewer than 65536 atoms");
    if (d_state) API_CUDA(h, launch_unsort_state(h->nb, h->state, h->d.SP, h->d.S + 2, d_state, h->st));
    if (d_desc) API_CUDA(h, launch_unsort_state(h->nb, h->desc, h->d.DP, h->d.D_out, d_desc, h->st));
    API_CUDA(h, cudaStreamSynchronize(h->st));
    return UMLMD_OK;
}

int umlmd_eval_radial_table(const umlmd_t* h, int64_t n, const double* rho, double* out_g, double* out_dg) {
    if (!h || n < 0 || (n > 0 && (!rho || !out_g))) return UMLMD_E_INVALID_ARG;
    const Dims& d = h->d;
    const int NC = d.C0 + d.R;
    for (int64_t i = 0; i < n; ++i) {
        int row = (int)std::floor(rho[i] / h->hm.dx);
        if (row < 0) row = 0;
        if (row > d.n_rows - 1) row = d.n_rows - 1;
        const double t = rho[i] - row * h->hm.dx;
        const float* p = &h->hm.table[(size_t)row * 3 * d.CP];
        for (int c = 0; c < NC; ++c) {
            unsigned w;
            std::memcpy(&w, &p[2 * d.CP + c], sizeof(w));
            float h2, h3;
            tab_unpack(w, d.tab_k2, d.tab_k3, &h2, &h3);
            const double c0 = p[c], c1 = p[d.CP + c], c2 = h2, c3 = h3;
            out_g[i * NC + c] = ((c3 * t + c2) * t + c1) * t + c0;
            if (out_dg) out_dg[i * NC + c] = (3 * c3 * t + 2 * c2) * t + c1;
        }
    }
    return UMLMD_OK;
}

int umlmd_set_profiling(umlmd_t* h, int enabled) {
    if (!h) return UMLMD_E_INVALID_ARG;
    h->prof_on = enabled != 0;
    return UMLMD_OK;
}

int umlmd_get_profile(umlmd_t* h, int32_t max_classes, double* ms, int64_t* launches, int32_t* n_classes) {
    if (!h || !n_classes || max_classes < 0) return UMLMD_E_INVALID_ARG;
    if (h->on_device) API_CUDA(h, cudaStreamSynchronize(h->st));
    for (auto& sp : h->spans) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, sp.a, sp.b) == cudaSuccess) h->prof_ms[sp.cls] += t;
        h->free_events.push_back(sp.a);
        h->free_events.push_back(sp.b);
    }
    h->spans.clear();
    *n_classes = kClassCount;
    for (int k = 0; k < kClassCount && k < max_classes; ++k) {
        if (ms) ms[k] = h->prof_ms[k];
        if (launches) launches[k] = h->prof_launches[k];
    }
    for (int k = 0; k < kClassCount; ++k) { h->prof_ms[k] = 0; h->prof_launches[k] = 0; }
    return UMLMD_OK;
}

const char* umlmd_profile_class_name(int32_t cls) {
    return (cls >= 0 && cls < kClassCount) ? kClassNames[cls] : "";
}

int umlmd_eval_pair_cache(const umlmd_t* h, int32_t type_i, int32_t type_j, double* out) {
    if (!h || !out) return UMLMD_E_INVALID_ARG;
    const Dims& d = h->d;
    if (type_i < 0 || type_j < 0 || type_i >= d.T || type_j >= d.T) return UMLMD_E_INVALID_ARG;
    const size_t n = (size_t)(2 + d.R) * d.C0;
    const float* p = &h->hm.pairmod[(size_t)(type_i * d.T + type_j) * n];
    for (size_t k = 0; k < n; ++k) out[k] = p[k];
    return UMLMD_OK;
}

}  // extern "C"
