// C ABI of the library: argument validation, workspace carving, launch sequencing.
#include <algorithm>
#include <atomic>
#include <mutex>

#include "internal.cuh"

namespace aaac {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {
std::atomic<unsigned long long> g_launches{0};
}
void note_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

namespace {

constexpr size_t kAlign = 256;
size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Candidate list of the quantile start: by default a sixteenth of the layer's weights (what the
// <= 64 histogram bins of the requested order statistics hold is usually 1-3 %), never less than
// the fit's selection words [N][ceil(K/256)] that later reuse the space.
size_t g_debug_qcap = 0;         // aaac_debug_quantile_cap: a forced list capacity (0 = none)

size_t default_qcap(int64_t N, int64_t K) {
    if (N <= 0 || K <= 0) return 1;
    const size_t nk = (size_t)N * (size_t)K;
    size_t cap = nk / 16;
    if (cap < ((size_t)1 << 18)) cap = nk < ((size_t)1 << 18) ? nk : ((size_t)1 << 18);
    const size_t sig = (size_t)N * (size_t)((K + 255) / 256);
    return cap < sig ? sig : cap;
}

// Lays the scratch regions out after `base` (which may be null to measure only).  qcap = entries
// of the candidate list; with a real workspace the list takes whatever the caller's buffer holds
// beyond the fixed regions (at most one entry per weight).
Workspace carve(void* base, int mode, int64_t N, int64_t K, size_t ws_bytes = 0, bool full = false) {
    Workspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void* p = base ? static_cast<char*>(base) + off : nullptr;
        off += up(bytes);
        return p;
    };
    const int g = mode == AAAC_INT4 ? 128 : 16;
    const int64_t K8 = (K + 7) / 8 * 8;
    w.ctrl = static_cast<Ctrl*>(take(sizeof(Ctrl)));
    w.part = static_cast<double*>(take(sizeof(double) * kMaxBlocks * kPartStride));
    w.rinv = static_cast<float*>(take(sizeof(float) * (size_t)(mode == AAAC_INT4 && N > 0 && K > 0 ? N * (K / g + 1) : 1)));
    w.I = static_cast<float*>(take(sizeof(float) * (size_t)(K8 > 0 ? K8 : 8)));
    w.act_part = static_cast<double*>(take(sizeof(double) * (size_t)act_splits_max(K) * (size_t)(K8 > 0 ? K8 : 8)));
    w.qhist = static_cast<uint32_t*>(take(sizeof(uint32_t) * kQBins));
    w.qslot_of_bin = static_cast<uint8_t*>(take(kQBins));
    const size_t nk = (size_t)(N > 0 && K > 0 ? N * K : 1);
    size_t cap = full ? nk : default_qcap(N, K);
    if (base && ws_bytes > off + cap * sizeof(uint32_t)) {
        cap = (ws_bytes - off) / sizeof(uint32_t);
        if (cap > nk) cap = nk;
    }
    if (g_debug_qcap && g_debug_qcap < cap) cap = g_debug_qcap;
    const size_t sig = (size_t)(N > 0 ? N : 1) * (size_t)((K + 255) / 256);
    if (cap < sig) cap = sig;                       // the fit's selection words reuse the list
    w.qcap = cap;
    w.qlist = static_cast<uint32_t*>(take(sizeof(uint32_t) * cap));
    w.bytes = off;
    return w;
}

// selection group sizes the kernels are built for: S = g, and S = 16 inside INT4's g = 128
bool sel_ok(int mode, int group, int sel_group) {
    return sel_group == group || (mode == AAAC_INT4 && group == 128 && sel_group == 16);
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_layer(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group) {
    if (!W) return AAAC_ERR_NULL;
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return AAAC_ERR_MODE;
    if (group != (mode == AAAC_INT4 ? 128 : 16)) return AAAC_ERR_MODE;
    if (N < 1 || K < 1 || K % group || K % 8 || ldw < K || ldw % 8) return AAAC_ERR_SHAPE;
    if (!aligned(W, 16)) return AAAC_ERR_ALIGN;
    return AAAC_OK;
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
    if (!ws) return AAAC_ERR_NULL;
    if (!aligned(ws, kAlign)) return AAAC_ERR_ALIGN;
    if (ws_bytes < need) return AAAC_ERR_WORKSPACE;
    return AAAC_OK;
}

// ---- optional per-launch timing of the fit-round kernel ----
struct Timing {
    std::mutex mu;
    bool on = false;
    int cap = 0, n = 0;
    cudaEvent_t* ev = nullptr;      // 2 per launch
} g_timing;

// Side streams of one device.  The layers of a batch are independent until their common fit
// launch, so their scales and start passes are queued on streams of their own, forked from the
// caller's stream and joined back to it: the small latency-bound kernels of one layer (plan,
// selection, the tails of the streaming passes) then run under the bandwidth-bound passes of another.
constexpr int kSideStreams = 7;
constexpr int kMaxDevices = 64;
struct SideStreams {
    bool tried = false, ok = false;
    cudaStream_t s[kSideStreams];
    cudaEvent_t fork, join[kSideStreams];
};
std::mutex g_side_mu;                  // held while a call queues work on the side streams
SideStreams g_side[kMaxDevices];

// the current device's side streams (created on first use), or nullptr: then everything stays on the caller's stream
SideStreams* side_streams() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    SideStreams& p = g_side[dev];
    if (!p.tried) {
        p.tried = true;
        bool ok = cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < kSideStreams && ok; ++i)
            ok = cudaStreamCreateWithFlags(&p.s[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.join[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) cudaGetLastError();
        p.ok = ok;
    }
    return p.ok ? &p : nullptr;
}

// Lanes for n independent pieces of work: lane 0 is the caller's stream, the others are side
// streams that wait for what the caller's stream holds so far; join() makes the caller's stream
// wait for all of them again.  One lane (no side streams, or n = 1) is the caller's stream alone.
class Lanes {
public:
    Lanes(cudaStream_t st, int n) : lk_(g_side_mu, std::defer_lock), st_(st) {
        if (n > 1) {
            lk_.lock();
            side_ = side_streams();
        }
        lanes_ = side_ ? std::min(n, kSideStreams + 1) : 1;
        if (lanes_ > 1) {
            ok_ = cudaEventRecord(side_->fork, st_) == cudaSuccess;
            for (int i = 0; i + 1 < lanes_ && ok_; ++i) ok_ = cudaStreamWaitEvent(side_->s[i], side_->fork, 0) == cudaSuccess;
        }
    }
    bool ok() const { return ok_; }
    cudaStream_t of(int l) const {
        const int lane = l % lanes_;
        return lane == 0 ? st_ : side_->s[lane - 1];
    }
    // always called, also after an error, so that no side stream is left outside the caller's stream's order
    bool join() {
        for (int i = 0; i + 1 < lanes_; ++i)
            if (cudaEventRecord(side_->join[i], side_->s[i]) != cudaSuccess ||
                cudaStreamWaitEvent(st_, side_->join[i], 0) != cudaSuccess)
                ok_ = false;
        lanes_ = 1;
        return ok_;
    }
private:
    std::unique_lock<std::mutex> lk_;
    SideStreams* side_ = nullptr;
    cudaStream_t st_;
    int lanes_ = 1;
    bool ok_ = true;
};

}  // namespace
}  // namespace aaac

using namespace aaac;

extern "C" {

const char* aaac_status_string(int status) {
    switch (status) {
        case AAAC_OK: return "ok";
        case AAAC_ERR_NULL: return "a required pointer is NULL";
        case AAAC_ERR_MODE: return "unknown mode or init, or group size does not match the mode";
        case AAAC_ERR_SHAPE: return "bad shape (N, K, T, leading dimension or iteration count)";
        case AAAC_ERR_ALIGN: return "pointer not sufficiently aligned";
        case AAAC_ERR_WORKSPACE: return "workspace too small";
        case AAAC_ERR_CUDA: return "CUDA runtime call or kernel launch failed";
        case AAAC_ERR_NONFINITE: return "input holds Inf or NaN";
        case AAAC_ERR_UNIMPLEMENTED: return "not implemented";
        case AAAC_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this no-allocation entry point";
        case AAAC_ERR_TIMEOUT: return "a bounded wait between the blocks of a kernel ran out; results are not valid";
        default: return "unknown status";
    }
}

size_t aaac_workspace_bytes(int mode, int64_t N, int64_t K, int64_t T) {
    (void)T;
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return 0;
    return carve(nullptr, mode, N, K).bytes;
}

size_t aaac_workspace_bytes_full(int mode, int64_t N, int64_t K, int64_t T) {
    (void)T;
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return 0;
    return carve(nullptr, mode, N, K, 0, true).bytes;
}

int aaac_act_stats(const void* X, int64_t T, int64_t K, int64_t ldx, float* I, int accumulate,
                   uint32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
    if (!X || !I) return AAAC_ERR_NULL;
    if (T < 1 || K < 1 || K % 8 || ldx < K || ldx % 8) return AAAC_ERR_SHAPE;
    if (!aligned(X, 16) || !aligned(I, 4)) return AAAC_ERR_ALIGN;
    // only the small regions are used; size the check for a 1-row layer of this width
    int rc = check_ws(ws, ws_bytes, carve(nullptr, AAAC_NVFP4, 1, K).bytes);
    if (rc) return rc;
    Workspace w = carve(ws, AAAC_NVFP4, 1, K, ws_bytes);
    return launch_act_stats(static_cast<const uint16_t*>(X), T, K, ldx, I, accumulate, dev_status, w,
                            static_cast<cudaStream_t>(stream)) == cudaSuccess ? AAAC_OK : AAAC_ERR_CUDA;
}

int aaac_fit_layer(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group,
                   const float* I, const void* X, int64_t T, int64_t ldx,
                   int n_outer, int n_inner, int init,
                   float* T01, void* scales, float* tensor_scale, double* err_trace,
                   uint32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
    return aaac_fit_layer_sel(W, N, K, ldw, mode, group, group, I, X, T, ldx, n_outer, n_inner, init, T01, scales,
                              tensor_scale, err_trace, dev_status, ws, ws_bytes, stream);
}

namespace {
// argument checks of one layer of a fit call
int check_fit_layer(const aaac_layer& L, int mode, int group, int sel_group, int n_outer, int n_inner, int init) {
    int rc = check_layer(L.W, L.N, L.K, L.ldw, mode, group);
    if (rc) return rc;
    if (!sel_ok(mode, group, sel_group)) return AAAC_ERR_MODE;
    if (!L.T01 || !L.scales || !L.tensor_scale) return AAAC_ERR_NULL;
    if (!L.I && !L.X) return AAAC_ERR_NULL;
    // the fit kernels index a layer's elements with 32 bits
    if ((unsigned long long)L.N * (unsigned long long)L.ldw >= (1ull << 32)) return AAAC_ERR_TOO_LARGE;
    if (init != AAAC_INIT_QUANTILE && init != AAAC_INIT_GRID && init != AAAC_INIT_USER) return AAAC_ERR_MODE;
    if (n_outer < 0) return AAAC_ERR_SHAPE;
    if (n_inner < 1 || (int64_t)n_outer * n_inner > (1 << 20)) return AAAC_ERR_SHAPE;
    if (!L.I && (L.T < 1 || L.ldx < L.K || L.ldx % 8)) return AAAC_ERR_SHAPE;
    if (!L.I && !aligned(L.X, 16)) return AAAC_ERR_ALIGN;
    if (L.I && !aligned(L.I, 16)) return AAAC_ERR_ALIGN;
    if (!aligned(L.scales, mode == AAAC_INT4 ? 2 : 1) || !aligned(L.T01, 4)) return AAAC_ERR_ALIGN;
    return check_ws(L.ws, L.ws_bytes, carve(nullptr, mode, L.N, L.K).bytes);
}

// Layers of a batch that are given the same activations (pointer, T, K, ldx) share their importances:
// they are computed once, into the workspace of the first such layer.  Returns that layer's index
// (l itself for a layer with importances of its own or activations nobody before it has).
int importance_owner(const aaac_layer* layers, int l) {
    const aaac_layer& L = layers[l];
    if (L.I) return l;
    for (int k = 0; k < l; ++k) {
        const aaac_layer& M = layers[k];
        if (!M.I && M.X == L.X && M.T == L.T && M.K == L.K && M.ldx == L.ldx) return k;
    }
    return l;
}

// Alg. 1 lines 1-5 of one layer: importance (if from X and not shared with an earlier layer, whose
// `shared_I` is then passed), scales, start tables; returns the importance used
int prepare_fit_layer(const aaac_layer& L, int mode, int init, uint32_t* dev_status, const Workspace& w, cudaStream_t st,
                      const float* shared_I, const float** I_used) {
    const uint16_t* Wp = static_cast<const uint16_t*>(L.W);
    if (cudaMemsetAsync(w.ctrl, 0, sizeof(Ctrl), st) != cudaSuccess) return AAAC_ERR_CUDA;
    const float* I = L.I ? L.I : shared_I;
    if (!I) {
        if (launch_act_stats(static_cast<const uint16_t*>(L.X), L.T, L.K, L.ldx, w.I, 0, dev_status, w, st) != cudaSuccess)
            return AAAC_ERR_CUDA;
        I = w.I;
    }
    const bool fused = init == AAAC_INIT_QUANTILE;      // the scales pass counts the quantile start's histogram on its way
    if (launch_scales(Wp, L.N, L.K, L.ldw, mode, L.scales, L.tensor_scale, dev_status, w, st, fused) != cudaSuccess) return AAAC_ERR_CUDA;
    if (launch_init(Wp, L.N, L.K, L.ldw, mode, init, L.scales, L.T01, dev_status, w, st, fused) != cudaSuccess) return AAAC_ERR_CUDA;
    *I_used = I;
    return AAAC_OK;
}
}  // namespace

int aaac_fit_layers(const aaac_layer* layers, int n_layers, int mode, int group, int sel_group,
                    int n_outer, int n_inner, int init, uint32_t* dev_status, void* stream) {
    if (!layers) return AAAC_ERR_NULL;
    if (n_layers < 1 || n_layers > 4096) return AAAC_ERR_SHAPE;
    for (int l = 0; l < n_layers; ++l) {
        const int rc = check_fit_layer(layers[l], mode, group, sel_group, n_outer, n_inner, init);
        if (rc) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    FitLayerArgs* args = new FitLayerArgs[(size_t)n_layers];
    int rc = AAAC_OK;
    {
        Lanes lanes(st, n_layers);
        if (!lanes.ok()) rc = AAAC_ERR_CUDA;
        for (int l = 0; l < n_layers && rc == AAAC_OK; ++l) {
            const aaac_layer& L = layers[l];
            const Workspace w = carve(L.ws, mode, L.N, L.K, L.ws_bytes);
            const float* I = nullptr;
            // (the passes queued here do not read the importances; the fit launch, after the join, does)
            const int owner = importance_owner(layers, l);
            const float* shared_I = owner == l ? nullptr
                                               : carve(layers[owner].ws, mode, layers[owner].N, layers[owner].K, layers[owner].ws_bytes).I;
            rc = prepare_fit_layer(L, mode, init, dev_status, w, lanes.of(l), shared_I, &I);
            args[l] = FitLayerArgs{static_cast<const uint16_t*>(L.W), L.N, L.K, L.ldw, L.scales, I, L.err_trace, L.T01, w};
        }
        if (!lanes.join() && rc == AAAC_OK) rc = AAAC_ERR_CUDA;
    }
    if (rc == AAAC_OK) {
        // all rounds run in one launch per batch; the optional timing brackets the launches of this call
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (n_outer > 0) {
            std::lock_guard<std::mutex> lk(g_timing.mu);
            if (g_timing.on && g_timing.n < g_timing.cap) {
                e0 = g_timing.ev[2 * g_timing.n];
                e1 = g_timing.ev[2 * g_timing.n + 1];
                ++g_timing.n;
            }
        }
        if (e0) cudaEventRecord(e0, st);
        if (launch_fit_rounds_batch(args, n_layers, mode, sel_group, n_outer, n_inner, dev_status, st) != cudaSuccess) rc = AAAC_ERR_CUDA;
        if (e1) cudaEventRecord(e1, st);
    }
    // with rounds to run the last fit launch writes the tables out itself; with none, a small kernel does
    for (int l = 0; l < n_layers && rc == AAAC_OK && n_outer == 0; ++l)
        if (launch_export_tables(layers[l].T01, args[l].ws, st) != cudaSuccess) rc = AAAC_ERR_CUDA;
    delete[] args;
    return rc;
}

int aaac_fit_layer_sel(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group, int sel_group,
                       const float* I, const void* X, int64_t T, int64_t ldx,
                       int n_outer, int n_inner, int init,
                       float* T01, void* scales, float* tensor_scale, double* err_trace,
                       uint32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
    const aaac_layer L{W, N, K, ldw, I, X, T, ldx, T01, scales, tensor_scale, err_trace, ws, ws_bytes};
    return aaac_fit_layers(&L, 1, mode, group, sel_group, n_outer, n_inner, init, dev_status, stream);
}

namespace {
// the pack pass of one layer on `st`; arguments already checked
int enqueue_pack(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int sel_group,
                 const float* I, const float* T01_f32, uint16_t* T01_bf16,
                 void* scales, const float* tensor_scale, uint8_t* codes, uint8_t* sigma_bits,
                 double* err_out, uint64_t* stats, void* ws, size_t ws_bytes, cudaStream_t stream) {
    Workspace w = carve(ws, mode, N, K, ws_bytes);
    cudaStream_t st = stream;
    // the pack pass uses only the block counter and its own result fields of the control block
    if (cudaMemsetAsync(&w.ctrl->done, 0, sizeof(uint32_t), st) != cudaSuccess) return AAAC_ERR_CUDA;
    if (cudaMemsetAsync(w.ctrl->pack_err, 0, sizeof(double) * 2 + sizeof(unsigned long long) * 4, st) != cudaSuccess)
        return AAAC_ERR_CUDA;
    return launch_pack(static_cast<const uint16_t*>(W), N, K, ldw, mode, sel_group, I, T01_f32, T01_bf16, scales,
                       tensor_scale, codes, sigma_bits, err_out, reinterpret_cast<unsigned long long*>(stats), w, st) == cudaSuccess
               ? AAAC_OK : AAAC_ERR_CUDA;
}
}  // namespace

int aaac_pack(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group,
              const float* I, const float* T01_f32, uint16_t* T01_bf16,
              void* scales, const float* tensor_scale, uint8_t* codes,
              double* err_out, uint64_t* stats, void* ws, size_t ws_bytes, void* stream) {
    return aaac_pack_sel(W, N, K, ldw, mode, group, group, I, T01_f32, T01_bf16, scales, tensor_scale, codes, nullptr,
                         err_out, stats, ws, ws_bytes, stream);
}

int aaac_pack_sel(const void* W, int64_t N, int64_t K, int64_t ldw, int mode, int group, int sel_group,
                  const float* I, const float* T01_f32, uint16_t* T01_bf16,
                  void* scales, const float* tensor_scale, uint8_t* codes, uint8_t* sigma_bits,
                  double* err_out, uint64_t* stats, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_layer(W, N, K, ldw, mode, group);
    if (rc) return rc;
    if (!sel_ok(mode, group, sel_group)) return AAAC_ERR_MODE;
    if (sel_group != group && !sigma_bits) return AAAC_ERR_NULL;
    if (sel_group == group) sigma_bits = nullptr;
    if (!I || !T01_f32 || !T01_bf16 || !scales || !codes) return AAAC_ERR_NULL;
    if (mode == AAAC_NVFP4 && !tensor_scale) return AAAC_ERR_NULL;
    if (!aligned(I, 16) || !aligned(codes, 16) || !aligned(T01_bf16, 2)) return AAAC_ERR_ALIGN;
    // the pack kernel, like the fit kernels, indexes a layer's elements with 32 bits
    if ((unsigned long long)N * (unsigned long long)ldw >= (1ull << 32)) return AAAC_ERR_TOO_LARGE;
    rc = check_ws(ws, ws_bytes, carve(nullptr, mode, N, K).bytes);
    if (rc) return rc;
    return enqueue_pack(W, N, K, ldw, mode, sel_group, I, T01_f32, T01_bf16, scales, tensor_scale, codes, sigma_bits,
                        err_out, stats, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

int aaac_quantize_layers(const aaac_layer* layers, const aaac_layer_out* outs, int n_layers, int mode, int group,
                         int sel_group, int n_outer, int n_inner, int init, uint32_t* dev_status, void* stream) {
    if (!layers || !outs) return AAAC_ERR_NULL;
    if (n_layers < 1 || n_layers > 4096) return AAAC_ERR_SHAPE;
    for (int l = 0; l < n_layers; ++l) {
        const aaac_layer& L = layers[l];
        const aaac_layer_out& O = outs[l];
        const int rc = check_fit_layer(L, mode, group, sel_group, n_outer, n_inner, init);
        if (rc) return rc;
        if (!O.T01_bf16 || !O.codes) return AAAC_ERR_NULL;
        if (sel_group != group && !O.sigma_bits) return AAAC_ERR_NULL;
        if (!aligned(O.codes, 16) || !aligned(O.T01_bf16, 2)) return AAAC_ERR_ALIGN;
        if (O.What && (O.ldo < L.K || O.ldo % 8)) return AAAC_ERR_SHAPE;
        if (O.What && !aligned(O.What, 16)) return AAAC_ERR_ALIGN;
    }
    int rc = aaac_fit_layers(layers, n_layers, mode, group, sel_group, n_outer, n_inner, init, dev_status, stream);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Lanes lanes(st, n_layers);
    if (!lanes.ok()) rc = AAAC_ERR_CUDA;
    for (int l = 0; l < n_layers && rc == AAAC_OK; ++l) {
        const aaac_layer& L = layers[l];
        const aaac_layer_out& O = outs[l];
        // the importance the fit used: the caller's, or the one the fit computed from X into a workspace
        const aaac_layer& Lo = layers[importance_owner(layers, l)];
        const float* I = L.I ? L.I : carve(Lo.ws, mode, Lo.N, Lo.K, Lo.ws_bytes).I;
        uint8_t* sg = sel_group == group ? nullptr : O.sigma_bits;
        rc = enqueue_pack(L.W, L.N, L.K, L.ldw, mode, sel_group, I, L.T01, O.T01_bf16, L.scales, L.tensor_scale, O.codes, sg,
                          O.err_out, O.stats, L.ws, L.ws_bytes, lanes.of(l));
        if (rc == AAAC_OK && O.What &&
            launch_dequant(O.codes, L.scales, sg, L.tensor_scale, O.T01_bf16, L.N, L.K, mode, static_cast<uint16_t*>(O.What),
                           O.ldo, lanes.of(l)) != cudaSuccess)
            rc = AAAC_ERR_CUDA;
    }
    if (!lanes.join() && rc == AAAC_OK) rc = AAAC_ERR_CUDA;
    return rc;
}

int aaac_dequant(const uint8_t* codes, const void* scales, const float* tensor_scale,
                 const uint16_t* T01_bf16, int64_t N, int64_t K, int mode, int group,
                 void* What, int64_t ldo, void* stream) {
    return aaac_dequant_sel(codes, scales, nullptr, tensor_scale, T01_bf16, N, K, mode, group, group, What, ldo, stream);
}

int aaac_dequant_sel(const uint8_t* codes, const void* scales, const uint8_t* sigma_bits, const float* tensor_scale,
                     const uint16_t* T01_bf16, int64_t N, int64_t K, int mode, int group, int sel_group,
                     void* What, int64_t ldo, void* stream) {
    if (!codes || !scales || !T01_bf16 || !What) return AAAC_ERR_NULL;
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return AAAC_ERR_MODE;
    if (group != (mode == AAAC_INT4 ? 128 : 16)) return AAAC_ERR_MODE;
    if (!sel_ok(mode, group, sel_group)) return AAAC_ERR_MODE;
    if (sel_group != group && !sigma_bits) return AAAC_ERR_NULL;
    if (sel_group == group) sigma_bits = nullptr;
    if (mode == AAAC_NVFP4 && !tensor_scale) return AAAC_ERR_NULL;
    if (N < 1 || K < 1 || K % group || K % 8 || ldo < K || ldo % 8) return AAAC_ERR_SHAPE;
    if (!aligned(codes, 4) || !aligned(What, 16)) return AAAC_ERR_ALIGN;
    return launch_dequant(codes, scales, sigma_bits, tensor_scale, T01_bf16, N, K, mode, static_cast<uint16_t*>(What), ldo,
                          static_cast<cudaStream_t>(stream)) == cudaSuccess ? AAAC_OK : AAAC_ERR_CUDA;
}

int aaac_prescale_columns(const void* W, int64_t N, int64_t K, int64_t ldw, const float* a,
                          void* W_out, int64_t ldo, const float* I, float* I_out,
                          uint32_t* dev_status, void* stream) {
    if (!W || !a || !W_out) return AAAC_ERR_NULL;
    if ((I == nullptr) != (I_out == nullptr)) return AAAC_ERR_NULL;
    if (N < 1 || K < 1 || K % 8 || ldw < K || ldw % 8 || ldo < K || ldo % 8) return AAAC_ERR_SHAPE;
    if (!aligned(W, 16) || !aligned(W_out, 16) || !aligned(a, 16)) return AAAC_ERR_ALIGN;
    return launch_prescale(static_cast<const uint16_t*>(W), N, K, ldw, a, static_cast<uint16_t*>(W_out), ldo, I, I_out,
                           dev_status, static_cast<cudaStream_t>(stream)) == cudaSuccess ? AAAC_OK : AAAC_ERR_CUDA;
}

// ---- host-buffer path ----

namespace {
struct HostLayout {
    size_t W, X, I, T01, Tb, scales, ts, codes, err, status, ws, total;
};
HostLayout host_layout(int mode, int64_t N, int64_t K, int64_t T) {
    HostLayout h{};
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += up(b); return o; };
    const int g = mode == AAAC_INT4 ? 128 : 16;
    h.W = take((size_t)N * K * 2);
    h.X = take((size_t)T * K * 2);
    h.I = take((size_t)K * 4);
    h.T01 = take(2 * kM * 4);
    h.Tb = take(2 * kM * 2);
    h.scales = take((size_t)N * (K / g) * (mode == AAAC_INT4 ? 2 : 1));
    h.ts = take(4);
    h.codes = take((size_t)N * K / 2);
    h.err = take(16);
    h.status = take(4);
    h.ws = take(carve(nullptr, mode, N, K).bytes);
    h.total = off;
    return h;
}
}  // namespace

size_t aaac_host_workspace_bytes(int mode, int64_t N, int64_t K, int64_t T) {
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return 0;
    return host_layout(mode, N, K, T).total;
}

int aaac_quantize_layer_host(const void* W_host, int64_t N, int64_t K, int mode, int group,
                             const void* X_host, int64_t T, int n_outer, int init,
                             float* T01_host, uint16_t* T01_bf16_host, void* scales_host,
                             float* tensor_scale_host, uint8_t* codes_host, double* err_out_host,
                             void* ws, size_t ws_bytes, void* stream) {
    uint32_t hstatus = 0;
    const int rc = aaac_quantize_layer_host_async(W_host, N, K, mode, group, X_host, T, n_outer, init, T01_host,
                                                  T01_bf16_host, scales_host, tensor_scale_host, codes_host,
                                                  err_out_host, &hstatus, ws, ws_bytes, stream);
    if (rc) return rc;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return AAAC_ERR_CUDA;
    if (hstatus & AAAC_DEV_TIMEOUT) return AAAC_ERR_TIMEOUT;
    if (hstatus & AAAC_DEV_SCRATCH) return AAAC_ERR_WORKSPACE;
    return (hstatus & AAAC_DEV_NONFINITE) ? AAAC_ERR_NONFINITE : AAAC_OK;
}

int aaac_quantize_layer_host_async(const void* W_host, int64_t N, int64_t K, int mode, int group,
                                   const void* X_host, int64_t T, int n_outer, int init,
                                   float* T01_host, uint16_t* T01_bf16_host, void* scales_host,
                                   float* tensor_scale_host, uint8_t* codes_host, double* err_out_host,
                                   uint32_t* status_host, void* ws, size_t ws_bytes, void* stream) {
    if (!status_host) return AAAC_ERR_NULL;
    if (!W_host || !X_host || !T01_host || !T01_bf16_host || !scales_host || !tensor_scale_host || !codes_host)
        return AAAC_ERR_NULL;
    if (mode != AAAC_INT4 && mode != AAAC_NVFP4) return AAAC_ERR_MODE;
    if (group != (mode == AAAC_INT4 ? 128 : 16)) return AAAC_ERR_MODE;
    if (N < 1 || K < 1 || T < 1 || K % group || K % 8 || n_outer < 0) return AAAC_ERR_SHAPE;
    if (init != AAAC_INIT_QUANTILE && init != AAAC_INIT_GRID) return AAAC_ERR_MODE;
    const HostLayout h = host_layout(mode, N, K, T);
    int rc = check_ws(ws, ws_bytes, h.total);
    if (rc) return rc;
    char* d = static_cast<char*>(ws);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int g = group;
    const size_t scale_bytes = (size_t)N * (K / g) * (mode == AAAC_INT4 ? 2 : 1);
    uint32_t* dstatus = reinterpret_cast<uint32_t*>(d + h.status);
    if (cudaMemsetAsync(dstatus, 0, 4, st) != cudaSuccess) return AAAC_ERR_CUDA;
    if (cudaMemcpyAsync(d + h.X, X_host, (size_t)T * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return AAAC_ERR_CUDA;
    if (cudaMemcpyAsync(d + h.W, W_host, (size_t)N * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return AAAC_ERR_CUDA;
    void* lws = d + h.ws;
    const size_t lws_bytes = ws_bytes - h.ws;
    float* I = reinterpret_cast<float*>(d + h.I);
    float* T01 = reinterpret_cast<float*>(d + h.T01);
    rc = aaac_act_stats(d + h.X, T, K, K, I, 0, dstatus, lws, lws_bytes, stream);
    if (rc) return rc;
    rc = aaac_fit_layer(d + h.W, N, K, K, mode, group, I, nullptr, 0, 0, n_outer, 1, init, T01, d + h.scales,
                        reinterpret_cast<float*>(d + h.ts), nullptr, dstatus, lws, lws_bytes, stream);
    if (rc) return rc;
    rc = aaac_pack(d + h.W, N, K, K, mode, group, I, T01, reinterpret_cast<uint16_t*>(d + h.Tb), d + h.scales,
                   reinterpret_cast<float*>(d + h.ts), reinterpret_cast<uint8_t*>(d + h.codes),
                   reinterpret_cast<double*>(d + h.err), nullptr, lws, lws_bytes, stream);
    if (rc) return rc;
    cudaError_t e = cudaSuccess;
    auto back = [&](void* dst, size_t off, size_t bytes) {
        if (e == cudaSuccess && dst) e = cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, st);
    };
    back(codes_host, h.codes, (size_t)N * K / 2);
    back(scales_host, h.scales, scale_bytes);
    back(T01_host, h.T01, 2 * kM * 4);
    back(T01_bf16_host, h.Tb, 2 * kM * 2);
    back(tensor_scale_host, h.ts, 4);
    back(err_out_host, h.err, 16);
    back(status_host, h.status, 4);
    return e == cudaSuccess ? AAAC_OK : AAAC_ERR_CUDA;
}

int aaac_debug_quantile_cap(size_t entries) {
    g_debug_qcap = entries;
    return AAAC_OK;
}

int aaac_debug_fit_wait(int extra_arrivals, unsigned spin_limit) {
    set_fit_wait(extra_arrivals, spin_limit);
    return AAAC_OK;
}

unsigned long long aaac_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

// ---- timing of the fit-round kernel ----

int aaac_timing_begin(int max_launches) {
    std::lock_guard<std::mutex> lk(g_timing.mu);
    if (g_timing.ev) {
        for (int i = 0; i < 2 * g_timing.cap; ++i) cudaEventDestroy(g_timing.ev[i]);
        delete[] g_timing.ev;
        g_timing.ev = nullptr;
    }
    g_timing.on = false;
    g_timing.n = 0;
    g_timing.cap = 0;
    if (max_launches <= 0) return AAAC_OK;
    g_timing.ev = new cudaEvent_t[2 * (size_t)max_launches];
    for (int i = 0; i < 2 * max_launches; ++i)
        if (cudaEventCreate(&g_timing.ev[i]) != cudaSuccess) return AAAC_ERR_CUDA;
    g_timing.cap = max_launches;
    g_timing.on = true;
    return AAAC_OK;
}

int aaac_timing_end(float* ms_host, int capacity) {
    std::lock_guard<std::mutex> lk(g_timing.mu);
    g_timing.on = false;
    int n = g_timing.n < capacity ? g_timing.n : capacity;
    for (int i = 0; i < n; ++i) {
        if (cudaEventSynchronize(g_timing.ev[2 * i + 1]) != cudaSuccess) return -1;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_timing.ev[2 * i], g_timing.ev[2 * i + 1]) != cudaSuccess) return -1;
        if (ms_host) ms_host[i] = ms;
    }
    for (int i = 0; i < 2 * g_timing.cap; ++i) cudaEventDestroy(g_timing.ev[i]);
    delete[] g_timing.ev;
    g_timing.ev = nullptr;
    g_timing.cap = 0;
    g_timing.n = 0;
    return n;
}

}  // extern "C"
