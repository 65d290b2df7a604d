// Host side of libsdnn.so: the C ABI declared in include/sdnn.h.
// Validation, re-layout of the stored entries into the kernels' sliced format, device memory, the
// per-layer launch sequences (optionally as a CUDA graph) and the staging of host buffers.  Every
// arithmetic step runs in the kernels of kernels.cuh.
#include "../../include/sdnn.h"
#include "kernels.cuh"
#include "reorder.h"

#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <tuple>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

using namespace sdnn_kernels;

namespace {

thread_local std::string g_create_error;

// Host description of a layer's stored entries, kept for get/set_weights: either every row has the same
// number of entries (no array needed) or the caller's row_ptr is remembered.
struct RowShape {
    int uniform_k = -1;
    std::vector<int> row_ptr;
    int len(int i) const { return uniform_k >= 0 ? uniform_k : row_ptr[i + 1] - row_ptr[i]; }
    int64_t start(int i) const { return uniform_k >= 0 ? (int64_t)i * uniform_k : row_ptr[i]; }
};

// Buffers of one inference tile in flight.  Tiles are independent of one another (so are the inputs), and a
// handle may work on two at a time, each on its own stream, so that the ramp and tail of one tile's launches are
// filled by the other's.
struct InferLane {
    cudaStream_t stream = nullptr;         // lane 0: the handle's stream
    float* tile[2] = {nullptr, nullptr};   // ping-pong activation tiles
    int* seg_cnt = nullptr;
    int* tile_cnt = nullptr;
    long long* offs = nullptr;
    ColState cs{};                         // live-column bookkeeping (SDNN_FLAG_SKIP_DEAD)
    int* live_hist = nullptr;              // [L] live inputs after each layer of this lane's most recent tile
    float* stage_out = nullptr;            // host entry point: staged x^L and counts of this lane's tile
    int* stage_cnt = nullptr;
    cudaEvent_t ev_scan = nullptr;         // this lane's last scan of the running id total is done
    cudaEvent_t ev_done = nullptr;         // everything this lane was given in the current call is done
    bool ready = false;
};

struct LayerMem {
    int64_t r_elems = 0, c_elems = 0;      // padded lengths of the two sliced copies
    int c_max_chunks = 0;                  // chunks of the widest slice of the transposed copy
    bool r_chunks_mult4 = false;           // every slice of the row-major copy has a multiple of 4 chunks
    int* r_idx = nullptr; float* r_val = nullptr; float* r_grad = nullptr;
    int* c_idx = nullptr; float* c_val = nullptr;
    std::vector<int> r_slice_off;          // host copy of the row-major slice offsets
    RowShape shape;
    // set-up reordering (SDNN_FLAG_REORDER): how the stored rows and entries map back to the caller's CSR arrays
    std::vector<int> row_src;              // [N] stored row -> caller's row (empty: identity)
    std::vector<int> entry_src;            // [nnz] entry in stored order (stored rows, their entries in stored order) -> caller's position
    int* r_out = nullptr;                  // grouped layer in the default layout: tile row each stored row writes (device, [N])
    int* r_row_of = nullptr;               // ... and its inverse: stored row that holds neuron (tile row) i (device, [N])
    // windowed layer: rows grouped by shared columns, the group's window staged in shared memory (forward_window_kernel)
    bool windowed = false;
    int groups = 0, max_wlen = 0;
    std::vector<int> w_row_at;             // [N] host: offset of each stored row's entries in w_col / w_val
    int64_t w_elems = 0;                   // padded entries
    unsigned short* w_col = nullptr; float* w_val = nullptr; int* w_out = nullptr;
    int* w_g_row0 = nullptr; int* w_g_c0 = nullptr; int* w_g_wlen = nullptr; int* w_g_ebase = nullptr; int* w_g_k = nullptr;
};

// caller's arrays of one layer, kept on the host until sdnn_finalize when the neurons are to be reordered
struct HostLayer {
    std::vector<int> rp, col;
    std::vector<float> val, bias;
};

}  // namespace

struct sdnn {
    int L = 0, N = 0, NS = 0;           // layers, neurons, slices of SLICE rows
    sdnn_config cfg{};
    cudaStream_t stream = nullptr;
    bool own_stream = false;
    int device = 0, sms = 0;
    bool finalized = false, stepped = false;
    bool mirror = false;                // training with the transposed copy (no atomics)
    bool idx16 = false;                 // the sliced copies hold 16-bit indices (at most 65536 neurons, SDNN_FLAG_IDX32 not set)
    bool pdl = false;                   // programmatic dependent launch between the layer kernels
    int fwd_pdl = 2;                    // PDL_EARLY; when a forward launch lets the next one go (PDL_EARLY, or PDL_AT_END while two tiles are in flight)
    std::vector<int64_t> nnz;
    std::vector<char> loaded;
    std::vector<LayerMem> lay;
    int ld_max = 0;                     // padded width of the widest tile this handle processes

    int* d_r_slice_off = nullptr;       // [L][NS+1]
    int* d_r_len = nullptr;             // [L][N]
    int* d_c_slice_off = nullptr;       // [L][NS+1]   (mirror)
    int* d_c_len = nullptr;             // [L][N]
    int* d_c_order = nullptr;           // [L][N]
    float* d_bias = nullptr;            // [L][N]

    // training
    float* d_acts = nullptr;            // [(L+1)][N][ld]: x^0 .. x^L of the current step
    float* d_s[2] = {nullptr, nullptr}; // atomics: alternating S = W^T delta tiles (all-zero between steps); mirror: delta tiles
    float* d_dl = nullptr;              // delta^L tile (atomics realisation)
    float* d_delta_all = nullptr;       // split backward: [L][N][ld], every delta^k of the step
    bool split = false;                 // transposed realisation with the row units as launches of their own on side streams
    static constexpr int MAX_SIDE = 2;
    cudaStream_t side_streams[MAX_SIDE] = {nullptr, nullptr};   // the row-unit launches alternate between these
    cudaEvent_t ev_side_join[MAX_SIDE] = {nullptr, nullptr};
    int n_side = 0;
    cudaStream_t launch_stream = nullptr;     // where launch_k currently enqueues (NULL = stream)
    std::vector<cudaEvent_t> ev_delta;  // [L] delta^k (0-based layer) complete
    cudaEvent_t ev_fork = nullptr;
    float* d_yt = nullptr;              // target tile
    StepParams* d_sp = nullptr;
    double* d_loss = nullptr;
    float* d_dbg_delta = nullptr;       // [L][N][ld]   (KEEP_DEBUG)
    unsigned long long* d_mismatch = nullptr;
    int last_b = 0, last_ld = 0;        // batch and padded width of the last step's activations
    int last_delta_b = 0, last_delta_ld = 0;   // ... of its deltas (1 and 4 after a step in the averaged form)
    // averaged form of the minibatch step (allocated at its first use)
    float* d_mean = nullptr;            // [(L+1)][N][4]: batch means of x^0 .. x^L
    StepParams* d_sp_batch = nullptr;   // the real batch, while d_sp describes the single backpropagated vector
    const float* bwd_acts = nullptr;    // activations the backward launches read (NULL: d_acts)
    cudaGraphExec_t graph = nullptr, graph_avg = nullptr;
    int graph_ld = 0, graph_avg_ld = 0;
    int64_t graph_launches = 0, graph_avg_launches = 0;   // kernel nodes of the captured steps
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};   // before forward chain, between, after backward chain

    // inference
    InferLane lane[2];
    InferLane* cur = nullptr;           // lane the launch helpers currently work for
    cudaEvent_t last_scan_ev = nullptr, ev_lane_start = nullptr;
    int live_lane = 0;
    long long* d_running = nullptr;
    int l2_bytes = 0;
    std::vector<char> local_pattern;    // per layer: blocks of 1024 rows touch few distinct columns (see infer_tile_width)
    bool reorder = false;               // SDNN_FLAG_REORDER: layers are analysed and laid out at sdnn_finalize
    int grouped_layers = 0;             // layers for which the analysis found groups of rows sharing a window of columns
    std::vector<HostLayer> pending;     // their arrays until then
    int* d_in_label = nullptr;          // [N] tile row of input neuron i (NULL: identity)
    std::vector<std::vector<int>> labels;   // [L + 1] host: tile row of neuron i at boundary k (x^k, delta^k); empty = identity
    int windowed_layers = 0;
    bool compaction = false;            // SDNN_FLAG_SKIP_DEAD asked for; effective while no bias is positive
    std::vector<char> bias_nonpositive; // per layer
    bool live_valid = false;

    // staging for the *_host entry points (allocated on first use)
    float* d_stage_a = nullptr;
    float* d_stage_b = nullptr;
    float* d_stage_a2 = nullptr;        // second input stage of sdnn_infer_batch_host: tile t+1 is copied while tile t computes
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr}, ev_consumed[2] = {nullptr, nullptr};
    int* d_stage_cnt = nullptr;
    int* d_stage_idx = nullptr;
    int64_t stage_idx_cap = 0;

    std::map<std::tuple<const void*, int, int>, std::pair<int, int>> plans;   // (kernel, units, chunks) -> (grid.x, block)
    std::map<std::pair<const void*, int>, int> occupancy;                     // (kernel, block) -> resident CTAs per SM

    int64_t launches = 0;
    int64_t dev_bytes = 0;
    std::vector<void*> allocs;
    std::string err;
};

namespace {

int fail(sdnn* h, int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (h) h->err = buf;
    g_create_error = buf;
    return code;
}

int cuda_fail(sdnn* h, cudaError_t e, const char* what) {
    int code = (e == cudaErrorMemoryAllocation) ? SDNN_ERR_OOM : SDNN_ERR_CUDA;
    return fail(h, code, "%s: %s", what, cudaGetErrorString(e));
}

#define CU(h, call)                                                  \
    do {                                                             \
        cudaError_t e_ = (call);                                     \
        if (e_ != cudaSuccess) return cuda_fail((h), e_, #call);     \
    } while (0)

template <typename T>
int dev_alloc(sdnn* h, T** out, size_t count, bool zero) {
    size_t bytes = count * sizeof(T);
    if (bytes == 0) bytes = sizeof(T);
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(h, e, "cudaMalloc"); }
    h->allocs.push_back(p);
    h->dev_bytes += (int64_t)bytes;
    if (zero) CU(h, cudaMemsetAsync(p, 0, bytes, h->stream));
    *out = static_cast<T*>(p);
    return SDNN_OK;
}

// Programmatic dependent launch, the kernels' `pdl` argument: 0 = off; 1 = a CTA lets the next launch go when it is
// done; 2 = as soon as its own wait for the previous launch has returned, so that CTAs of the next launch move into SM
// slots as they fall free and run their prologue (shapes, first indices) under this launch's tail.  2 is used where
// the launch has the device to itself (the forward chains: config 5 13.5 -> 13.1 us per layer, config 3 9.3 -> 8.9 us,
// a 1024-neuron layer 2.7 -> 1.9 us) and for backward launches of at most one CTA per SM; a larger backward launch
// shares the SMs with the row-unit launches of the side streams, and early CTAs of the next layer, which only wait,
// then stand in their way (N = 16384, B = 1: 6 % slower).
constexpr int PDL_AT_END = 1, PDL_EARLY = 2;

// padded batch width: 4, 8, .., 256, then multiples of 256
int padded_width(int b) {
    if (b <= 4) return 4;
    if (b <= 256) { int w = 4; while (w < b) w <<= 1; return w; }
    return (b + 255) / 256 * 256;
}

// lanes per row group (g), batch entries per lane (v), (g*v)-wide chunks per tile row
struct Geometry { int g; int v; int chunks; };
Geometry geometry(int cols) {
    if (cols <= 4) return {1, 4, 1};
    if (cols <= 256) return {cols / 8, 8, 1};
    return {32, 8, cols / 256};
}

int validate_cfg(const sdnn_config* cfg) {
    if (!cfg) return fail(nullptr, SDNN_ERR_INVALID_ARG, "cfg is NULL");
    if (cfg->activation != SDNN_ACT_CLAMPED_RELU && cfg->activation != SDNN_ACT_SIGMOID)
        return fail(nullptr, SDNN_ERR_UNIMPLEMENTED, "activation must be 0 (clamped ReLU) or 1 (sigmoid)");
    if (cfg->activation == SDNN_ACT_CLAMPED_RELU && (!(cfg->clamp > 0.0f) || !std::isfinite(cfg->clamp)))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "clamp must be finite and > 0");
    if (cfg->max_batch < 1) return fail(nullptr, SDNN_ERR_INVALID_ARG, "max_batch must be >= 1");
    if (cfg->max_batch > (1 << 30))      // rounding up to the tile width must stay inside 32 bits
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "max_batch must be at most 2^30");
    if (cfg->train && cfg->max_batch > 128) return fail(nullptr, SDNN_ERR_INVALID_ARG, "training handles support max_batch <= 128");
    if ((cfg->flags & SDNN_FLAG_BWD_ATOMICS) && (cfg->flags & SDNN_FLAG_BWD_CSC))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "choose one backward strategy");
    if ((cfg->flags & SDNN_FLAG_SMEM_WINDOWS) && cfg->train)
        return fail(nullptr, SDNN_ERR_UNIMPLEMENTED, "SDNN_FLAG_SMEM_WINDOWS is implemented for inference handles (train = 0)");
    if ((cfg->flags & SDNN_FLAG_SMEM_WINDOWS) && !(cfg->flags & SDNN_FLAG_REORDER))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "SDNN_FLAG_SMEM_WINDOWS needs SDNN_FLAG_REORDER");
    if ((cfg->flags & SDNN_FLAG_SMEM_WINDOWS) && (cfg->flags & SDNN_FLAG_SKIP_DEAD))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "SDNN_FLAG_SMEM_WINDOWS and SDNN_FLAG_SKIP_DEAD cannot be combined "
                                                  "(the window kernels do not keep track of live inputs)");
    return SDNN_OK;
}

// Host-side check of one layer: returns SDNN_OK or fills the message.
int validate_layer(sdnn* h, int layer, int n, int64_t expect_nnz, const int32_t* rp, const int32_t* col,
                   const float* val, const float* bias) {
    if (!rp || !bias) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d: NULL row_ptr or bias", layer);
    if (rp[0] != 0) return fail(h, SDNN_ERR_BAD_CSR, "layer %d: row_ptr[0] = %d, expected 0", layer, rp[0]);
    for (int i = 0; i < n; ++i)
        if (rp[i + 1] < rp[i]) return fail(h, SDNN_ERR_BAD_CSR, "layer %d: row_ptr decreases at row %d", layer, i);
    if ((int64_t)rp[n] != expect_nnz)
        return fail(h, SDNN_ERR_BAD_CSR, "layer %d: row_ptr[N] = %d but %lld stored entries were announced", layer, rp[n],
                    (long long)expect_nnz);
    if (expect_nnz > 0 && (!col || !val)) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d: NULL col_idx or values", layer);
    int bad_row = -1, bad_kind = 0;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < n; ++i) {
        int kind = 0;
        if (!std::isfinite(bias[i])) kind = 4;
        for (int p = rp[i]; p < rp[i + 1] && !kind; ++p) {
            if (col[p] < 0 || col[p] >= n) kind = 1;
            else if (p > rp[i] && col[p] <= col[p - 1]) kind = (col[p] == col[p - 1]) ? 2 : 3;
            else if (!std::isfinite(val[p])) kind = 5;
        }
        if (kind) {
#pragma omp critical
            if (bad_row < 0 || i < bad_row) { bad_row = i; bad_kind = kind; }
        }
    }
    if (bad_row >= 0) {
        static const char* what[] = {"", "column index out of range", "duplicate column", "columns not ascending",
                                     "non-finite bias", "non-finite value"};
        return fail(h, SDNN_ERR_BAD_CSR, "layer %d, row %d: %s", layer, bad_row, what[bad_kind]);
    }
    return SDNN_OK;
}

// ---------------------------------------------------------------------------------------------
// Sliced layout (see kernels.cuh): slices of SLICE units, chunks of 4 entries interleaved over the units of a slice.
inline int64_t sliced_pos(const int* slice_off, int unit, int q) {
    return (int64_t)slice_off[unit / SLICE] + (int64_t)(q >> 2) * CHUNK_ROW + (unit % SLICE) * 4 + (q & 3);
}

// slice offsets from unit lengths; returns the padded element count or -1 if it does not fit int32
template <typename LenFn>
int64_t build_slice_offsets(int n, LenFn len, std::vector<int>& off) {
    const int ns = (n + SLICE - 1) / SLICE;
    off.assign(ns + 1, 0);
    int64_t run = 0;
    for (int s = 0; s < ns; ++s) {
        int w = 0;
        for (int i = s * SLICE; i < std::min(n, (s + 1) * SLICE); ++i) w = std::max(w, len(i));
        w = (w + 7) / 8 * 8;      // whole pipeline steps of two chunks
        run += (int64_t)SLICE * w;
        if (run > INT32_MAX) return -1;
        off[s + 1] = (int)run;
    }
    return run;
}

void count_launch(sdnn* h, int k = 1) { h->launches += k; }

// NVTX range on the calling host thread (a timeline tool shows which launches a call or a layer pass enqueued; for a
// captured step the ranges cover the capture, the replays appear under the range of the call that launches the graph)
struct NvtxRange {
    explicit NvtxRange(const char* what, int k = -1) {
        if (k < 0) { nvtxRangePushA(what); return; }
        char buf[48];
        snprintf(buf, sizeof buf, "%s %d", what, k);
        nvtxRangePushA(buf);
    }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

// ---------------------------------------------------------------------------------------------
// Launch shapes.  The layer kernels are persistent: warps take units in a grid-stride loop.  The number of
// warps per SM is chosen so that the last round of the loop is as full as possible (a nearly empty last
// round leaves too few requests in flight to keep the memory system busy).
int resident_ctas(sdnn* h, const void* kernel, int block) {
    auto key = std::make_pair(kernel, block);
    auto it = h->occupancy.find(key);
    if (it != h->occupancy.end()) return it->second;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, block, 0) != cudaSuccess || occ < 1) { cudaGetLastError(); occ = 1; }
    h->occupancy[key] = occ;
    return occ;
}

std::pair<int, int> plan_grid(sdnn* h, const void* kernel, int units, int chunks, int oneshot_wpb = 0) {
    auto key = std::make_tuple(kernel, units, chunks);
    auto it = h->plans.find(key);
    if (it != h->plans.end()) return it->second;
    double best = -1.0;
    std::pair<int, int> pick{1, 256};
    for (int wpb = 8; wpb >= 4; --wpb) {
        const int block = wpb * 32;
        const int occ = resident_ctas(h, kernel, block);
        for (int c = occ; c >= 1; --c) {
            const int per_sm_warps = c * wpb;
            if (per_sm_warps < 16 && c != occ) continue;
            int gx = std::max(1, h->sms * c / chunks);
            const int64_t warps = (int64_t)gx * wpb;
            if (warps >= units) {      // one round: a plain grid of ceil(units / wpb) CTAs does it
                gx = (units + wpb - 1) / wpb;
                const double eff = 1.0 + 1e-3 / wpb;      // ties: smaller CTAs, which spread over more SMs (config 1 inference: 0.51 -> 0.49 ms)
                if (eff > best) { best = eff; pick = {gx, block}; }
                continue;
            }
            const int64_t rounds = (units + warps - 1) / warps;
            double eff = (double)units / (double)(rounds * warps) + 1e-3 * per_sm_warps / 64.0;   // ties: more warps
            if (eff > best) { best = eff; pick = {gx, block}; }
        }
    }
    if (oneshot_wpb > 0) {
        // one-shot grid.  Where the units outnumber the resident warps by half or more, a warp takes two units (the second
        // one's entries are on their way while it works on the first): the grid then fits the device in one round.
        // Measured per backward layer, one / two units per warp: 65536 neurons B = 16 23.4 / 23.0 us, 131072: 51.1 / 48.2,
        // 16384 neurons B = 64 17.6 / 16.8; with fewer units than that two per warp lose (32768 neurons B = 16: 12.9 / 16.3).
        const int64_t slots = (int64_t)h->sms * std::max(1, resident_ctas(h, kernel, oneshot_wpb * 32)) * oneshot_wpb;
        const int upw = (2 * (int64_t)units >= 3 * slots) ? 2 : 1;
        pick = {(units + oneshot_wpb * upw - 1) / (oneshot_wpb * upw), oneshot_wpb * 32};
    }
    h->plans[key] = pick;
    return pick;
}

Sliced rows_of(sdnn* h, int layer) {
    Sliced m;
    m.slice_off = h->d_r_slice_off + (size_t)layer * (h->NS + 1);
    m.len = h->d_r_len + (size_t)layer * h->N;
    m.idx = h->lay[layer].r_idx;
    m.val = h->lay[layer].r_val;
    m.order = nullptr;
    m.idx16 = h->idx16 ? 1 : 0;
    m.out = h->lay[layer].r_out;
    return m;
}

Sliced cols_of(sdnn* h, int layer) {
    Sliced m;
    m.slice_off = h->d_c_slice_off + (size_t)layer * (h->NS + 1);
    m.len = h->d_c_len + (size_t)layer * h->N;
    m.idx = h->lay[layer].c_idx;
    m.val = h->lay[layer].c_val;
    m.order = h->d_c_order + (size_t)layer * h->N;
    m.idx16 = h->idx16 ? 1 : 0;
    m.out = nullptr;
    return m;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_k(sdnn* h, void (*kernel)(KArgs...), dim3 grid, dim3 block, bool pdl, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = 0; lc.stream = h->launch_stream ? h->launch_stream : h->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernel, KArgs(args)...);
}

template <bool I16, int G, int V, int CPS = 2>
void launch_forward_gv(sdnn* h, int layer, const float* xin, float* xout, int ld, int chunks, bool track) {
    constexpr int RPW = 32 / G;
    const int units = (h->N + RPW - 1) / RPW;
    const float* bias = h->d_bias + (size_t)layer * h->N;
    auto plan = plan_grid(h, (const void*)forward_kernel<G, V, CPS, I16>, units, chunks);
    // A persistent grid gives every CTA a run of consecutive units, so that its entries are one contiguous stretch of the
    // layer's arrays: 3 % faster than a grid-stride walk at configs 3 and 5, 15 % on a local pattern with 256-input tiles.
    // Tiles of one chunk (up to 256 inputs) only: with several chunks per tile the grid-stride walk measured 1 % faster
    // (config 2: 5.00e12 against 4.95e12 edges/s).
    // Not where the input tile outgrows L2: there a grid-stride walk keeps all SMs inside the same few row blocks at any
    // time, and on a local pattern (config 4, 1024-input tiles: 268 MB) that is what keeps their window of the tile in
    // L2 (the blocked walk measured 2.4e12 against 4.6e12 edges/s there).
    int span = 0;
    const double tile_bytes = (double)h->N * ld * sizeof(float);
    if (chunks == 1 && plan.first * (plan.second / 32) < units && (h->l2_bytes <= 0 || tile_bytes <= 0.55 * (double)h->l2_bytes))
        span = (units + plan.first - 1) / plan.first;
    // 64-byte rows of a layer whose rows all have the same length (no padding entries, which all point at tile row 0: L1
    // absorbs those, one L2 slice would not): the instantiation whose gathers go past L1
    const bool cg = G == 2 && V == 8 && CPS == 2 && h->lay[layer].shape.uniform_k > 0 && h->N % SLICE == 0;
#define SDNN_FWD(CG_, SPAN_)                                                                                                   \
    launch_k(h, forward_kernel<G, V, CPS, I16, CG_, SPAN_>, dim3(plan.first, chunks), dim3(plan.second), h->pdl, rows_of(h, layer), \
             bias, xin, xout, h->N, ld, h->cfg.clamp, h->cfg.activation, h->pdl ? h->fwd_pdl : 0,                              \
             track ? (const int*)h->cur->cs.ncols : (const int*)nullptr, track ? h->cur->cs.flags : (int*)nullptr, span)
    // the grid-stride instantiation is the one the wide inference tiles take: it carries nothing of the other walk
    if (cg) { if (span > 0) SDNN_FWD((G == 2 && V == 8 && CPS == 2), true); else SDNN_FWD((G == 2 && V == 8 && CPS == 2), false); }
    else if (span > 0) SDNN_FWD(false, true);
    else SDNN_FWD(false, false);
#undef SDNN_FWD
}

// track: compaction mode (process only the live columns, mark the columns that stay live)
// Tiles of padded width 4 take the kernels that give a lane a row's chunk instead of a row (see kernels.cuh), unless
// the handle asked for one of the other backward realisations: those keep the common kernels at every width.
bool entry_parallel(const sdnn* h, int ld) {
    return ld == 4 && !(h->cfg.flags & (SDNN_FLAG_BWD_ATOMICS | SDNN_FLAG_BWD_ONE_LAUNCH));
}

template <bool I16>
void launch_forward_i(sdnn* h, int layer, const float* xin, float* xout, int ld, int cols, bool track) {
    const Geometry q = geometry(cols);
    if (q.v == 4 && !track && entry_parallel(h, ld)) {
        const int wf = h->NS <= h->sms ? 1 : 4;      // few slices: one per CTA, so that they spread over as many SMs
        launch_k(h, forward_ep_kernel<I16>, dim3((h->NS + wf - 1) / wf), dim3(32 * wf), h->pdl, rows_of(h, layer),
                 (const float*)(h->d_bias + (size_t)layer * h->N), xin, xout, h->N, h->cfg.clamp, h->cfg.activation, h->pdl ? h->fwd_pdl : 0);
    } else if (q.v == 4) launch_forward_gv<I16, 1, 4>(h, layer, xin, xout, ld, q.chunks, track);
    else switch (q.g) {
        case 1: launch_forward_gv<I16, 1, 8>(h, layer, xin, xout, ld, q.chunks, track); break;
        case 2: launch_forward_gv<I16, 2, 8>(h, layer, xin, xout, ld, q.chunks, track); break;
        case 4: launch_forward_gv<I16, 4, 8>(h, layer, xin, xout, ld, q.chunks, track); break;
        case 8: launch_forward_gv<I16, 8, 8>(h, layer, xin, xout, ld, q.chunks, track); break;
        case 16: launch_forward_gv<I16, 16, 8>(h, layer, xin, xout, ld, q.chunks, track); break;
        default:
            // a launch of at most one warp-row per resident slot is bound by its chain of round trips: four chunks (16
            // entries) of a row in flight per step instead of two, where every slice has whole steps of that size
            if (!track && h->lay[layer].r_chunks_mult4 && (int64_t)h->N * q.chunks <= (int64_t)h->sms * 8)
                launch_forward_gv<I16, 32, 8, 4>(h, layer, xin, xout, ld, q.chunks, track);
            else launch_forward_gv<I16, 32, 8>(h, layer, xin, xout, ld, q.chunks, track);
            break;
    }
    count_launch(h);
}

// the kernels are instantiated for both index widths of the sliced copies
void launch_forward(sdnn* h, int layer, const float* xin, float* xout, int ld, int cols, bool track = false) {
    if (h->idx16) launch_forward_i<true>(h, layer, xin, xout, ld, cols, track);
    else launch_forward_i<false>(h, layer, xin, xout, ld, cols, track);
}

// Windowed layers (rows grouped by shared columns at set-up): the group's window of the input tile is staged in shared
// memory.  One CTA per SM (the window takes most of its shared memory), items = groups x chunks of up to 32 inputs.
constexpr int WINDOW_COL_CAP = 1536;      // tile rows a window may span: 1536 x 32 inputs x 4 bytes = 192 KB of shared memory
constexpr int WINDOW_ROW_CAP = 2048;      // rows per group

template <int TC>
cudaError_t launch_forward_window_tc(sdnn* h, const LayerMem& lm, const Windowed& m, const float* xin, float* xout, int ld, int cols) {
    static bool configured[64] = {};
    if (h->device < 64 && !configured[h->device]) {
        cudaError_t e = cudaFuncSetAttribute(forward_window_kernel<TC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             WINDOW_RING_BYTES + WINDOW_COL_CAP * TC * 4);
        if (e != cudaSuccess) return e;
        configured[h->device] = true;
    }
    const int chunks = cols / TC;
    // too few (group, chunk) pairs for the device: split the rows of a group over several items (each stages the window);
    // an item keeps at least 64 rows per warp-row of work so that the staging stays a small part of it
    int splits = 1;
    const int avg_rows = std::max(1, h->N / std::max(1, lm.groups));
    while (lm.groups * chunks * splits < 2 * h->sms && avg_rows / (splits * 2) >= 64 && splits < 32) splits *= 2;
    const int items = lm.groups * chunks * splits;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(std::max(1, std::min(items, h->sms))); lc.blockDim = dim3(WINDOW_THREADS);
    lc.dynamicSmemBytes = WINDOW_RING_BYTES + (size_t)std::max(lm.max_wlen, 1) * TC * sizeof(float);
    lc.stream = h->launch_stream ? h->launch_stream : h->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = h->pdl ? 1 : 0;
    return cudaLaunchKernelEx(&lc, forward_window_kernel<TC>, m, xin, xout, ld, chunks, splits, h->cfg.clamp, (int)h->cfg.activation,
                              h->pdl ? PDL_AT_END : 0);
}

// chunks of 32 inputs: the kernel with four rows side by side in a warp, where its larger entry ring leaves room for the window
cudaError_t launch_forward_window32(sdnn* h, const LayerMem& lm, const Windowed& m, const float* xin, float* xout, int ld, int cols) {
    static bool configured[64] = {};
    if (h->device < 64 && !configured[h->device]) {
        cudaError_t e = cudaFuncSetAttribute(forward_window32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        configured[h->device] = true;
    }
    const int chunks = cols / 32;
    int splits = 1;
    const int avg_rows = std::max(1, h->N / std::max(1, lm.groups));
    while (lm.groups * chunks * splits < 2 * h->sms && avg_rows / (splits * 2) >= 128 && splits < 32) splits *= 2;
    const int items = lm.groups * chunks * splits;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(std::max(1, std::min(items, h->sms))); lc.blockDim = dim3(W32_THREADS);
    lc.dynamicSmemBytes = W32_RING_BYTES + (size_t)std::max(lm.max_wlen, 1) * 32 * sizeof(float);
    lc.stream = h->launch_stream ? h->launch_stream : h->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = h->pdl ? 1 : 0;
    return cudaLaunchKernelEx(&lc, forward_window32_kernel, m, xin, xout, ld, chunks, splits, h->cfg.clamp, (int)h->cfg.activation,
                              h->pdl ? PDL_AT_END : 0);
}

void launch_forward_window(sdnn* h, int layer, const float* xin, float* xout, int ld, int cols) {
    const LayerMem& lm = h->lay[layer];
    Windowed m;
    m.col = lm.w_col; m.val = lm.w_val; m.out = lm.w_out;
    m.bias = h->d_bias + (size_t)layer * h->N;
    m.g_row0 = lm.w_g_row0; m.g_c0 = lm.w_g_c0; m.g_wlen = lm.w_g_wlen; m.g_ebase = lm.w_g_ebase; m.g_k = lm.w_g_k; m.groups = lm.groups;
    if (cols >= 32 && W32_RING_BYTES + (size_t)lm.max_wlen * 128 <= 227u * 1024u) launch_forward_window32(h, lm, m, xin, xout, ld, cols);
    else if (cols >= 32) launch_forward_window_tc<32>(h, lm, m, xin, xout, ld, cols);
    else if (cols == 16) launch_forward_window_tc<16>(h, lm, m, xin, xout, ld, cols);
    else if (cols == 8) launch_forward_window_tc<8>(h, lm, m, xin, xout, ld, cols);
    else launch_forward_window_tc<4>(h, lm, m, xin, xout, ld, cols);
    count_launch(h);
}

// delta tile of layer `layer` (0-based; the paper's delta^{layer+1}) in the transposed realisation
float* delta_tile(sdnn* h, int layer, size_t tile) {
    if (h->d_dbg_delta) return h->d_dbg_delta + (size_t)layer * tile;
    if (h->d_delta_all) return h->d_delta_all + (size_t)layer * tile;
    return h->d_s[layer & 1];
}

// part: 0 = the whole layer in one launch; 1 = column units only; 2 = row units only (transposed realisation)
template <bool I16, int G, int V, int CPS>
void launch_backward_gvc(sdnn* h, int layer, int ld, int part) {
    constexpr int RPW = 32 / G;
    const size_t tile = (size_t)h->N * ld;
    const bool last = layer == h->L - 1, prop = layer > 0;
    const int units = (h->N + RPW - 1) / RPW;
    BackwardArgs a{};
    a.rows = rows_of(h, layer);
    a.bias = h->d_bias + (size_t)layer * h->N;
    const float* acts = h->bwd_acts ? h->bwd_acts : h->d_acts;
    a.xk = acts + (size_t)(layer + 1) * tile;
    a.xprev = acts + (size_t)layer * tile;
    a.dbg_grad = h->lay[layer].r_grad;
    a.sp = h->d_sp;
    a.n = h->N;
    a.clamp = h->cfg.clamp;
    a.act = h->cfg.activation;
    a.update_bias = h->cfg.update_bias ? 1 : 0;
    a.skip_dead = (h->cfg.flags & SDNN_FLAG_SKIP_DEAD) ? 1 : 0;
    a.pdl = h->pdl ? PDL_AT_END : 0;
    a.warm = (layer >= 1) ? acts + (size_t)(layer - 1) * tile : nullptr;
    a.warm_bytes = (unsigned)(tile * sizeof(float));
    // The two launches of a layer in the split realisation run beside each other (and beside those of the next layer):
    // one warp per CTA and one unit per warp lets the hardware interleave them unit by unit, which measured 6 % (config 5)
    // and 9 % (config 3) faster than two persistent grids sharing the SMs.  Alone on the device (forward, one launch per
    // layer) the persistent grid is the faster one.
    const int os_ = (h->split && part != 0) ? 1 : 0;
#define SDNN_BWD(FROM_S, SCAT, MIR)                                                            \
    do {                                                                                       \
        if (a.dbg_grad) {                                                                      \
            auto plan = plan_grid(h, (const void*)backward_kernel<G, V, CPS, I16, FROM_S, SCAT, MIR, true>, units, 1, os_);   \
            if (a.pdl && (plan.first <= h->sms || MIR)) a.pdl = PDL_EARLY;                     \
            launch_k(h, backward_kernel<G, V, CPS, I16, FROM_S, SCAT, MIR, true>, dim3(plan.first), dim3(plan.second), a.pdl != 0, a); \
        } else {                                                                               \
            auto plan = plan_grid(h, (const void*)backward_kernel<G, V, CPS, I16, FROM_S, SCAT, MIR, false>, units, 1, os_);  \
            if (a.pdl && (plan.first <= h->sms || MIR)) a.pdl = PDL_EARLY;                     \
            launch_k(h, backward_kernel<G, V, CPS, I16, FROM_S, SCAT, MIR, false>, dim3(plan.first), dim3(plan.second), a.pdl != 0, a); \
        }                                                                                      \
    } while (0)
    if (h->mirror) {
        a.dk = delta_tile(h, layer, tile);
        if (prop && part != 2) {
            a.cols = cols_of(h, layer);
            a.dprev = delta_tile(h, layer - 1, tile);
            a.cols_only = part == 1 ? 1 : 0;
            SDNN_BWD(false, false, true);
        } else if (part != 1) {
            if (part == 2) { a.pdl = 0; a.warm = nullptr; }
            SDNN_BWD(false, false, false);
        }
    } else {
        float* dl = h->d_dbg_delta ? h->d_dbg_delta + (size_t)layer * tile : h->d_dl;
        a.dk = last ? dl : h->d_s[(layer + 1) & 1];
        a.dprev = h->d_s[layer & 1];
        a.dbg_delta = (!last && h->d_dbg_delta) ? h->d_dbg_delta + (size_t)layer * tile : nullptr;
        if (last && prop) SDNN_BWD(false, true, false);
        else if (last) SDNN_BWD(false, false, false);
        else if (prop) SDNN_BWD(true, true, false);
        else SDNN_BWD(true, false, false);
    }
#undef SDNN_BWD
}

template <bool I16, int G, int V>
void launch_backward_gv(sdnn* h, int layer, int ld, int part) {
    launch_backward_gvc<I16, G, V, 2>(h, layer, ld, part);
}

// the two launches of a layer in the split transposed realisation, for tiles of padded width 4
template <bool I16>
void launch_backward_ep(sdnn* h, int layer, int part) {
    const size_t tile = (size_t)h->N * 4;
    const float* acts = h->bwd_acts ? h->bwd_acts : h->d_acts;
    const float* xprev = acts + (size_t)layer * tile;
    const float* dk = delta_tile(h, layer, tile);
    const int wb = h->NS <= h->sms ? 1 : 4;          // few slices: one per CTA (a 1024-neuron net: 0.56 -> 0.51 ms per step)
    const dim3 grid((h->NS + wb - 1) / wb), block(32 * wb);
    if (part == 1) {
        const int pdl = h->pdl ? PDL_EARLY : 0;      // indices, lengths and order are read in front of the wait
        // a launch of at most one CTA per SM is bound by its chain of round trips: take a long column in one go
        if ((int)grid.x <= h->sms && h->lay[layer].c_max_chunks > 2 * EP_IT)
            launch_k(h, backward_col_ep_kernel<2 * EP_IT, I16>, grid, block, h->pdl, cols_of(h, layer), xprev, dk, delta_tile(h, layer - 1, tile),
                     h->N, h->cfg.clamp, h->cfg.activation, (const StepParams*)h->d_sp, pdl);
        else
            launch_k(h, backward_col_ep_kernel<EP_IT, I16>, grid, block, h->pdl, cols_of(h, layer), xprev, dk, delta_tile(h, layer - 1, tile),
                     h->N, h->cfg.clamp, h->cfg.activation, (const StepParams*)h->d_sp, pdl);
    } else {
        float* bias = h->d_bias + (size_t)layer * h->N;
        float* grad = h->lay[layer].r_grad;
        if (grad) launch_k(h, backward_row_ep_kernel<true, I16>, grid, block, false, rows_of(h, layer), bias, xprev, dk, grad, h->N,
                           (const StepParams*)h->d_sp, h->cfg.update_bias ? 1 : 0, 0);
        else launch_k(h, backward_row_ep_kernel<false, I16>, grid, block, false, rows_of(h, layer), bias, xprev, dk, grad, h->N,
                      (const StepParams*)h->d_sp, h->cfg.update_bias ? 1 : 0, 0);
    }
}

template <bool I16>
void launch_backward_i(sdnn* h, int layer, int ld, int part) {
    const Geometry q = geometry(ld);
    if (q.v == 4 && h->split && part != 0 && entry_parallel(h, ld)) launch_backward_ep<I16>(h, layer, part);
    else if (q.v == 4) launch_backward_gv<I16, 1, 4>(h, layer, ld, part);
    else switch (q.g) {
        case 1: launch_backward_gv<I16, 1, 8>(h, layer, ld, part); break;
        case 2: launch_backward_gv<I16, 2, 8>(h, layer, ld, part); break;
        case 4: launch_backward_gv<I16, 4, 8>(h, layer, ld, part); break;
        case 8: launch_backward_gv<I16, 8, 8>(h, layer, ld, part); break;
        default: launch_backward_gv<I16, 16, 8>(h, layer, ld, part); break;
    }
    count_launch(h);
}

void launch_backward(sdnn* h, int layer, int ld, int part = 0) {
    if (h->idx16) launch_backward_i<true>(h, layer, ld, part);
    else launch_backward_i<false>(h, layer, ld, part);
}

void launch_output_gradient(sdnn* h, int ld) {
    const size_t tile = (size_t)h->N * ld;
    float* dl = h->mirror ? delta_tile(h, h->L - 1, tile)
                          : (h->d_dbg_delta ? h->d_dbg_delta + (size_t)(h->L - 1) * tile : h->d_dl);
    const long long vecs = (long long)h->N * (ld / 4);
    const int grid = (int)std::min<long long>((vecs + 255) / 256, (long long)h->sms * 8);
    output_gradient_kernel<<<grid, 256, 0, h->stream>>>(h->d_acts + (size_t)h->L * tile, h->d_yt, dl, h->N, ld, h->cfg.clamp,
                                                        h->cfg.activation, h->d_sp, h->d_loss);
    count_launch(h);
}

void launch_transpose_in(sdnn* h, const float* src, float* dst, int cnt, int cols, int ld, const int* row_map = nullptr) {
    dim3 grid((h->N + 31) / 32, (cols + 31) / 32), block(32, 8);
    transpose_in_kernel<<<grid, block, 0, h->launch_stream ? h->launch_stream : h->stream>>>(src, dst, h->N, cnt, cols, ld, row_map);
    count_launch(h);
}

// backward chain of one train step over tiles of padded width ld
void enqueue_backward_chain(sdnn* h, int ld) {
    if (h->split) {
        // column units chain on the main stream; the row units of layer k only need delta^k and x^{k-1}, so they run on
        // the side streams beside the column units of the layers below
        cudaEventRecord(h->ev_fork, h->stream);
        for (int q = 0; q < h->n_side; ++q) cudaStreamWaitEvent(h->side_streams[q], h->ev_fork, 0);
        cudaEventRecord(h->ev_delta[h->L - 1], h->stream);
        for (int k = h->L - 1; k >= 0; --k) {
            NvtxRange pass("backward layer", k + 1);
            cudaStream_t side = h->side_streams[k % h->n_side];
            cudaStreamWaitEvent(side, h->ev_delta[k], 0);
            h->launch_stream = side;
            launch_backward(h, k, ld, 2);
            h->launch_stream = nullptr;
            if (k > 0) {
                launch_backward(h, k, ld, 1);
                cudaEventRecord(h->ev_delta[k - 1], h->stream);
            }
        }
        for (int q = 0; q < h->n_side; ++q) {
            cudaEventRecord(h->ev_side_join[q], h->side_streams[q]);
            cudaStreamWaitEvent(h->stream, h->ev_side_join[q], 0);
        }
    } else {
        for (int k = h->L - 1; k >= 0; --k) {
            NvtxRange pass("backward layer", k + 1);
            launch_backward(h, k, ld);
        }
    }
}

// forward + backward chain of one train step on the internal buffers; `flags` selects how the three
// timing events are recorded (as external event-record nodes while capturing a graph).
// averaged: the forward chain runs on the whole batch, then the batch means of x^0..x^L and the averaged delta^L are
// formed and the backward chain runs on those single vectors (tiles of padded width 4).
void enqueue_step_body(sdnn* h, int ld, unsigned flags, bool averaged) {
    const size_t tile = (size_t)h->N * ld;
    cudaEventRecordWithFlags(h->ev[0], h->stream, flags);
    {
        NvtxRange chain("sdnn forward chain");
        for (int k = 0; k < h->L; ++k) {
            NvtxRange pass("forward layer", k + 1);
            launch_forward(h, k, h->d_acts + (size_t)k * tile, h->d_acts + (size_t)(k + 1) * tile, ld, ld);
        }
    }
    cudaEventRecordWithFlags(h->ev[1], h->stream, flags);
    NvtxRange chain("sdnn backward chain");
    if (!averaged) {
        launch_output_gradient(h, ld);
        enqueue_backward_chain(h, ld);
    } else {
        const long long rows = (long long)(h->L + 1) * h->N;
        const int grid_m = (int)std::min<long long>((rows + 255) / 256, (long long)h->sms * 16);
        batch_mean_kernel<<<grid_m, 256, 0, h->stream>>>(h->d_acts, h->d_mean, rows, ld, h->d_sp_batch);
        const size_t tile1 = (size_t)h->N * 4;
        float* dl = h->mirror ? delta_tile(h, h->L - 1, tile1)
                              : (h->d_dbg_delta ? h->d_dbg_delta + (size_t)(h->L - 1) * tile1 : h->d_dl);
        const int grid_g = std::min((h->N + 255) / 256, h->sms * 8);
        output_gradient_averaged_kernel<<<grid_g, 256, 0, h->stream>>>(h->d_acts + (size_t)h->L * tile, h->d_yt, dl, h->N, ld,
                                                                     h->cfg.clamp, h->cfg.activation, h->d_sp_batch, h->d_loss);
        count_launch(h, 2);
        h->bwd_acts = h->d_mean;
        enqueue_backward_chain(h, 4);
        h->bwd_acts = nullptr;
    }
    cudaEventRecordWithFlags(h->ev[2], h->stream, flags);
}

int train_step_device(sdnn* h, const float* x0, const float* target, int B, float eta, float* loss_out, bool averaged = false) {
    NvtxRange call(averaged ? "sdnn_train_step_averaged" : "sdnn_train_step");
    const int ld = padded_width(B);
    h->fwd_pdl = PDL_EARLY;
    if (averaged) {
        if (!h->d_mean) {
            int rc;
            if ((rc = dev_alloc(h, &h->d_mean, (size_t)(h->L + 1) * h->N * 4, true))) return rc;
            if ((rc = dev_alloc(h, &h->d_sp_batch, 1, true))) return rc;
        }
        set_step_params_kernel<<<1, 1, 0, h->stream>>>(h->d_sp_batch, eta, B, h->d_loss);
        set_step_params_kernel<<<1, 1, 0, h->stream>>>(h->d_sp, eta, 1, h->d_loss);
        count_launch(h, 2);
    } else {
        set_step_params_kernel<<<1, 1, 0, h->stream>>>(h->d_sp, eta, B, h->d_loss);
        count_launch(h);
    }
    launch_transpose_in(h, x0, h->d_acts, B, ld, ld, h->d_in_label);
    launch_transpose_in(h, target, h->d_yt, B, ld, ld);
    if (h->cfg.flags & SDNN_FLAG_NO_GRAPH) {
        enqueue_step_body(h, ld, cudaEventRecordDefault, averaged);
    } else {
        cudaGraphExec_t& graph = averaged ? h->graph_avg : h->graph;
        int& graph_ld = averaged ? h->graph_avg_ld : h->graph_ld;
        int64_t& graph_launches = averaged ? h->graph_avg_launches : h->graph_launches;
        if (!graph || graph_ld != ld) {
            if (graph) { cudaGraphExecDestroy(graph); graph = nullptr; }
            cudaGraph_t g = nullptr;
            const int64_t before = h->launches;
            CU(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
            enqueue_step_body(h, ld, cudaEventRecordExternal, averaged);
            cudaError_t e = cudaStreamEndCapture(h->stream, &g);
            graph_launches = h->launches - before;
            h->launches = before;
            if (e != cudaSuccess) return cuda_fail(h, e, "cudaStreamEndCapture");
            e = cudaGraphInstantiate(&graph, g, 0);
            cudaGraphDestroy(g);
            if (e != cudaSuccess) { graph = nullptr; return cuda_fail(h, e, "cudaGraphInstantiate"); }
            graph_ld = ld;
        }
        CU(h, cudaGraphLaunch(graph, h->stream));
        count_launch(h, (int)graph_launches);
    }
    CU(h, cudaGetLastError());
    h->stepped = true; h->last_b = B; h->last_ld = ld;
    h->last_delta_b = averaged ? 1 : B; h->last_delta_ld = averaged ? 4 : ld;
    if (loss_out) {
        double j = 0.0;
        CU(h, cudaMemcpyAsync(&j, h->d_loss, sizeof(double), cudaMemcpyDeviceToHost, h->stream));
        CU(h, cudaStreamSynchronize(h->stream));
        *loss_out = (float)j;
    }
    return SDNN_OK;
}

int check_train_args(sdnn* h, const float* x0, const float* target, int B, float eta) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (!h->finalized) return fail(h, SDNN_ERR_STATE, "handle is not finalized");
    if (!h->cfg.train) return fail(h, SDNN_ERR_STATE, "handle was created with train = 0");
    if (!x0 || !target) return fail(h, SDNN_ERR_INVALID_ARG, "x0 or target is NULL");
    if (B < 1 || B > h->cfg.max_batch) return fail(h, SDNN_ERR_INVALID_ARG, "B = %d outside [1, max_batch = %d]", B, h->cfg.max_batch);
    if (!std::isfinite(eta)) return fail(h, SDNN_ERR_INVALID_ARG, "eta is not finite");
    return SDNN_OK;
}

int alloc_lane(sdnn* h, InferLane& ln, bool own_stream) {
    if (ln.ready) return SDNN_OK;
    const size_t N = (size_t)h->N, tile = N * (size_t)h->ld_max, nseg = (N + NZ_SEG - 1) / NZ_SEG;
    int rc;
    if (own_stream) CU(h, cudaStreamCreateWithFlags(&ln.stream, cudaStreamNonBlocking));
    else ln.stream = h->stream;
    CU(h, cudaEventCreateWithFlags(&ln.ev_scan, cudaEventDisableTiming));
    CU(h, cudaEventCreateWithFlags(&ln.ev_done, cudaEventDisableTiming));
    if ((rc = dev_alloc(h, &ln.tile[0], tile, false))) return rc;
    if ((rc = dev_alloc(h, &ln.tile[1], tile, false))) return rc;
    if ((rc = dev_alloc(h, &ln.seg_cnt, nseg * (size_t)h->ld_max, false))) return rc;
    if ((rc = dev_alloc(h, &ln.tile_cnt, (size_t)h->ld_max, false))) return rc;
    if ((rc = dev_alloc(h, &ln.offs, (size_t)h->ld_max, false))) return rc;
    if (h->compaction) {
        int* blk = nullptr;
        if ((rc = dev_alloc(h, &blk, 3 * (size_t)h->ld_max + 4, true))) return rc;
        ln.cs.colmap = blk; ln.cs.perm = blk + h->ld_max; ln.cs.flags = blk + 2 * (size_t)h->ld_max;
        ln.cs.ncols = blk + 3 * (size_t)h->ld_max; ln.cs.old_ncols = ln.cs.ncols + 1; ln.cs.do_compact = ln.cs.ncols + 2;
        if ((rc = dev_alloc(h, &ln.live_hist, (size_t)h->L, true))) return rc;
    }
    ln.ready = true;
    return SDNN_OK;
}

// One tile of inference on device buffers, on lane `ln`: x0 [cnt][N] -> outputs for these cnt inputs.
int infer_tile(sdnn* h, InferLane& ln, const float* x0, int cnt, float* y_out, int* cnt_out, int* idx_out, long long capacity,
               bool want_sets) {
    NvtxRange call("sdnn inference tile");
    const int ld = h->ld_max;
    const int cols = padded_width(cnt);
    cudaStream_t st = ln.stream;
    h->cur = &ln;
    h->launch_stream = st;
    launch_transpose_in(h, x0, ln.tile[0], cnt, cols, ld, h->d_in_label);
    int cur = 0;
    bool track = h->compaction && h->cfg.activation == SDNN_ACT_CLAMPED_RELU;      // sigmoid(b) is never 0: nothing ever dies
    for (int l = 0; l < h->L && track; ++l) track = h->bias_nonpositive[l] != 0;     // the zero vector must be a fixed point
    if (track) {
        const Geometry q = geometry(cols);
        const int chunk = q.g * q.v;
        const int rows_grid = std::min((h->N + 7) / 8, h->sms * 8);
        cols_init_kernel<<<(ld + 255) / 256, 256, 0, st>>>(ln.cs, cnt, ld);
        count_launch(h);
        for (int k = 0; k < h->L; ++k) {
            launch_forward(h, k, ln.tile[cur], ln.tile[cur ^ 1], ld, cols, true);
            cur ^= 1;
            live_kernel<<<1, 1024, 0, st>>>(ln.cs, ln.live_hist + k, chunk);
            compact_kernel<<<rows_grid, 256, 0, st>>>(ln.cs, ln.tile[cur], h->N, ld, chunk);
            count_launch(h, 2);
        }
        expand_kernel<<<rows_grid, 256, 0, st>>>(ln.cs, ln.tile[cur], ln.tile[cur ^ 1], h->N, cols, ld);
        count_launch(h);
        cur ^= 1;
        h->live_valid = true;
        h->live_lane = (int)(&ln - h->lane);
    } else {
        for (int k = 0; k < h->L; ++k) {
            NvtxRange pass("forward layer", k + 1);
            if (h->lay[k].windowed) launch_forward_window(h, k, ln.tile[cur], ln.tile[cur ^ 1], ld, cols);
            else launch_forward(h, k, ln.tile[cur], ln.tile[cur ^ 1], ld, cols);
            cur ^= 1;
        }
    }
    h->launch_stream = nullptr;
    h->cur = &h->lane[0];
    const float* xl = ln.tile[cur];
    if (y_out) {
        dim3 grid((h->N + 31) / 32, (cnt + 31) / 32), block(32, 8);
        transpose_out_kernel<<<grid, block, 0, st>>>(xl, y_out, h->N, cnt, ld);
        count_launch(h);
    }
    if (want_sets) {
        const int nseg = (h->N + NZ_SEG - 1) / NZ_SEG;
        dim3 grid(nseg, (cnt + 127) / 128);
        nz_count_kernel<<<grid, 128, 0, st>>>(xl, ln.seg_cnt, h->N, cnt, ld);
        nz_scan_segments_kernel<<<(cnt + 127) / 128, 128, 0, st>>>(ln.seg_cnt, ln.tile_cnt, nseg, cnt, ld);
        // the running total of ids is carried from tile to tile: the scans of successive tiles run in order
        if (h->last_scan_ev && h->last_scan_ev != ln.ev_scan) CU(h, cudaStreamWaitEvent(st, h->last_scan_ev, 0));
        nz_scan_inputs_kernel<<<1, 1024, 0, st>>>(ln.tile_cnt, ln.offs, h->d_running, cnt_out, cnt);
        CU(h, cudaEventRecord(ln.ev_scan, st));
        h->last_scan_ev = ln.ev_scan;
        count_launch(h, 3);
        if (idx_out) {
            nz_fill_kernel<<<grid, 128, 0, st>>>(xl, ln.seg_cnt, ln.offs, idx_out, capacity, h->N, cnt, ld);
            count_launch(h);
        }
    }
    CU(h, cudaGetLastError());
    return SDNN_OK;
}

// Inputs per inference tile.  The gathers of a layer read the whole activation tile at random, so the two
// ping-pong tiles should sit in L2: unless every layer's pattern is local (each block of rows reads few tile rows,
// which the cache then holds whatever the tile's size), the tile is narrowed to the widest power of two >= 128
// for which both tiles take at most 55 % of the L2.
int infer_tile_width(const sdnn* h) {
    int T = h->cfg.max_batch;
    bool local = true;
    for (char c : h->local_pattern) local = local && c;
    if (local || h->l2_bytes <= 0) return T;
    const double budget = 0.55 * (double)h->l2_bytes;
    while (T > 128 && 2.0 * h->N * padded_width(T) * sizeof(float) > budget) {
        int p = 128;
        while (p * 2 < T) p *= 2;      // largest power of two below T (at least 128)
        T = p;
    }
    return T;
}

// Tiles in flight, each on a stream of its own.  Two: a third adds a percent or two at most and costs two more
// activation tiles.  The gathers of a layer touch its input tile only, so the second lane doubles what should stay
// in L2 from one tile to two, which the tile width already allows for.
int infer_lanes(const sdnn* h, int /*T*/) {
    return (h->cfg.flags & SDNN_FLAG_ONE_TILE) ? 1 : 2;
}

// start / end of a batch that may use the second lane: lane 1 sees what the handle's stream has done so far, and the
// handle's stream ends up behind everything lane 1 did
int lanes_begin(sdnn* h, int lanes) {
    h->last_scan_ev = nullptr;
    // with two tiles in flight, CTAs of a tile's next layer that only wait would hold SM slots the other tile can use
    // (config 4 and uniform N = 65536: 1.4 % slower when released early)
    h->fwd_pdl = lanes > 1 ? PDL_AT_END : PDL_EARLY;
    if (lanes < 2) return SDNN_OK;
    if (!h->ev_lane_start) CU(h, cudaEventCreateWithFlags(&h->ev_lane_start, cudaEventDisableTiming));
    for (int i = 1; i < lanes; ++i) {      // before the event: new buffers are zeroed on the handle's stream
        int rc = alloc_lane(h, h->lane[i], true);
        if (rc) return rc;
    }
    CU(h, cudaEventRecord(h->ev_lane_start, h->stream));
    for (int i = 1; i < lanes; ++i) CU(h, cudaStreamWaitEvent(h->lane[i].stream, h->ev_lane_start, 0));
    return SDNN_OK;
}
int lanes_end(sdnn* h, int lanes) {
    for (int i = 1; i < lanes; ++i) {
        if (!h->lane[i].ready) continue;
        CU(h, cudaEventRecord(h->lane[i].ev_done, h->lane[i].stream));
        CU(h, cudaStreamWaitEvent(h->stream, h->lane[i].ev_done, 0));
    }
    return SDNN_OK;
}

int check_infer_args(sdnn* h, const float* x0, int64_t n_inputs, int32_t* idx, int64_t cap) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (!h->finalized) return fail(h, SDNN_ERR_STATE, "handle is not finalized");
    if (n_inputs < 0) return fail(h, SDNN_ERR_INVALID_ARG, "n_inputs < 0");
    if (n_inputs > 0 && !x0) return fail(h, SDNN_ERR_INVALID_ARG, "x0 is NULL");
    if (idx && cap < 0) return fail(h, SDNN_ERR_INVALID_ARG, "nz_index_capacity < 0");
    return SDNN_OK;
}

int ensure_stage(sdnn* h) {
    if (h->d_stage_a) return SDNN_OK;
    const size_t cnt = (size_t)h->cfg.max_batch * h->N;
    int rc;
    if ((rc = dev_alloc(h, &h->d_stage_a, cnt, false))) return rc;
    if ((rc = dev_alloc(h, &h->d_stage_b, cnt, false))) return rc;
    if ((rc = dev_alloc(h, &h->d_stage_cnt, (size_t)h->cfg.max_batch, false))) return rc;
    return SDNN_OK;
}

// values in the caller's CSR order -> row-major sliced copy (padding zero)
void csr_to_sliced(const sdnn* h, const LayerMem& lm, const float* src, std::vector<float>& dst) {
    dst.assign((size_t)lm.r_elems, 0.0f);
    const int* off = lm.r_slice_off.data();
#pragma omp parallel for schedule(static)
    for (int i = 0; i < h->N; ++i) {
        const int len = lm.shape.len(i);
        const int64_t s = lm.shape.start(i);
        for (int q = 0; q < len; ++q) dst[(size_t)sliced_pos(off, i, q)] = src[s + q];
    }
}

void sliced_to_csr(const sdnn* h, const LayerMem& lm, const std::vector<float>& src, float* dst) {
    const int* off = lm.r_slice_off.data();
#pragma omp parallel for schedule(static)
    for (int i = 0; i < h->N; ++i) {
        const int len = lm.shape.len(i);
        const int64_t s = lm.shape.start(i);
        for (int q = 0; q < len; ++q) dst[s + q] = src[(size_t)sliced_pos(off, i, q)];
    }
}

int refresh_mirror(sdnn* h, int layer, unsigned long long* mismatch_dev) {
    const int wpb = 8;
    mirror_values_kernel<<<(h->N + wpb - 1) / wpb, wpb * 32, 0, h->stream>>>(rows_of(h, layer), cols_of(h, layer), h->N, mismatch_dev,
                                                                             (const int*)h->lay[layer].r_row_of);
    CU(h, cudaGetLastError());
    return SDNN_OK;
}

// Index arrays of the sliced copies: 16 bits per index where the net has at most 65536 neurons (h->idx16), else 32.
int alloc_indices(sdnn* h, int** out, size_t count) {
    if (!h->idx16) return dev_alloc(h, out, count, false);
    unsigned short* p = nullptr;
    int rc = dev_alloc(h, &p, count, false);
    *out = reinterpret_cast<int*>(p);
    return rc;
}
int upload_indices(sdnn* h, int* dst, const std::vector<int>& src) {      // synchronous with respect to `src` when narrowing
    if (!h->idx16) {
        CU(h, cudaMemcpyAsync(dst, src.data(), src.size() * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        return SDNN_OK;
    }
    std::vector<unsigned short> narrow(src.size());
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < (int64_t)src.size(); ++q) narrow[(size_t)q] = (unsigned short)src[(size_t)q];
    CU(h, cudaMemcpyAsync(dst, narrow.data(), narrow.size() * sizeof(unsigned short), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaStreamSynchronize(h->stream));
    return SDNN_OK;
}

// Lays out one validated layer (caller's or reordered CSR, host arrays) in the kernels' sliced format and uploads it.
// out_label (host, or NULL): tile row that each given row writes, for a layer whose rows are stored group by group.
int upload_layer(sdnn* h, int layer, const int32_t* row_ptr, const int32_t* col_idx, const float* values, const float* bias,
                 const int* out_label = nullptr) {
    int rc;
    CU(h, cudaSetDevice(h->device));
    const int N = h->N, NS = h->NS;
    LayerMem& lm = h->lay[layer];

    // ---- row-major sliced copy
    bool uniform = true;
    const int k0 = row_ptr[1] - row_ptr[0];
    for (int i = 1; i < N && uniform; ++i) uniform = (row_ptr[i + 1] - row_ptr[i]) == k0;
    if (uniform) lm.shape.uniform_k = k0; else lm.shape.row_ptr.assign(row_ptr, row_ptr + N + 1);
    std::vector<int> r_len(N);
    for (int i = 0; i < N; ++i) r_len[i] = row_ptr[i + 1] - row_ptr[i];
    lm.r_elems = build_slice_offsets(N, [&](int i) { return r_len[i]; }, lm.r_slice_off);
    if (lm.r_elems < 0) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d: padded sliced layout exceeds 2^31 entries", layer);
    lm.r_chunks_mult4 = true;
    for (int sl = 0; sl < NS; ++sl) lm.r_chunks_mult4 = lm.r_chunks_mult4 && ((lm.r_slice_off[sl + 1] - lm.r_slice_off[sl]) / CHUNK_ROW) % 4 == 0;
    std::vector<int> r_idx((size_t)lm.r_elems, 0);
    std::vector<float> r_val;
    csr_to_sliced(h, lm, values, r_val);
    {
        const int* off = lm.r_slice_off.data();
#pragma omp parallel for schedule(static)
        for (int i = 0; i < N; ++i)
            for (int q = 0; q < r_len[i]; ++q) r_idx[(size_t)sliced_pos(off, i, q)] = col_idx[row_ptr[i] + q];
    }
    if ((rc = alloc_indices(h, &lm.r_idx, (size_t)lm.r_elems))) return rc;
    if ((rc = dev_alloc(h, &lm.r_val, (size_t)lm.r_elems, false))) return rc;
    if (h->cfg.train && (h->cfg.flags & SDNN_FLAG_KEEP_DEBUG))
        if ((rc = dev_alloc(h, &lm.r_grad, (size_t)lm.r_elems, true))) return rc;
    CU(h, cudaMemcpyAsync(h->d_r_slice_off + (size_t)layer * (NS + 1), lm.r_slice_off.data(), (size_t)(NS + 1) * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(h->d_r_len + (size_t)layer * N, r_len.data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(h->d_bias + (size_t)layer * N, bias, (size_t)N * sizeof(float), cudaMemcpyHostToDevice, h->stream));
    if (lm.r_elems) {
        if ((rc = upload_indices(h, lm.r_idx, r_idx))) return rc;
        CU(h, cudaMemcpyAsync(lm.r_val, r_val.data(), (size_t)lm.r_elems * sizeof(float), cudaMemcpyHostToDevice, h->stream));
    }

    if (out_label) {
        std::vector<int> row_of(N);
        for (int i = 0; i < N; ++i) row_of[out_label[i]] = i;
        if ((rc = dev_alloc(h, &lm.r_out, (size_t)N, false))) return rc;
        if ((rc = dev_alloc(h, &lm.r_row_of, (size_t)N, false))) return rc;
        CU(h, cudaMemcpyAsync(lm.r_out, out_label, (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaMemcpyAsync(lm.r_row_of, row_of.data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaStreamSynchronize(h->stream));
    }

    // ---- transposed sliced copy (not needed for the first layer: delta^0 is never formed)
    std::vector<int> c_idx, c_len, order, c_off;
    if (h->mirror && layer > 0) {
        const int64_t nz = h->nnz[layer];
        std::vector<int> deg(N, 0);
        for (int64_t p = 0; p < nz; ++p) ++deg[col_idx[p]];
        int dmax = 0;
        for (int j = 0; j < N; ++j) dmax = std::max(dmax, deg[j]);
        // columns by descending length (stable in j): slices of nearly equal length, little padding
        std::vector<int> bucket(dmax + 2, 0);
        for (int j = 0; j < N; ++j) ++bucket[dmax - deg[j] + 1];
        for (int d = 0; d <= dmax; ++d) bucket[d + 1] += bucket[d];
        order.resize(N);
        std::vector<int> place(N);
        for (int j = 0; j < N; ++j) { const int cc = bucket[dmax - deg[j]]++; order[cc] = j; place[j] = cc; }
        c_len.resize(N);
        for (int cc = 0; cc < N; ++cc) c_len[cc] = deg[order[cc]];
        lm.c_elems = build_slice_offsets(N, [&](int cc) { return c_len[cc]; }, c_off);
        if (lm.c_elems < 0) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d: padded transposed layout exceeds 2^31 entries", layer);
        for (int sl = 0; sl < NS; ++sl) lm.c_max_chunks = std::max(lm.c_max_chunks, (c_off[sl + 1] - c_off[sl]) / CHUNK_ROW);
        c_idx.assign((size_t)lm.c_elems, 0);
        // each thread owns a range of columns and scans all entries in row order: rows ascend within a column
#pragma omp parallel
        {
            int nt = 1, tid = 0;
#ifdef _OPENMP
            nt = omp_get_num_threads(); tid = omp_get_thread_num();
#endif
            const int j0 = (int)((int64_t)N * tid / nt), j1 = (int)((int64_t)N * (tid + 1) / nt);
            std::vector<int> cursor(j1 - j0, 0);
            for (int i = 0; i < N; ++i)
                for (int p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
                    const int j = col_idx[p];
                    if (j < j0 || j >= j1) continue;
                    const int q = cursor[j - j0]++;
                    c_idx[(size_t)sliced_pos(c_off.data(), place[j], q)] = out_label ? out_label[i] : i;      // the delta tile's row
                }
        }
        if ((rc = alloc_indices(h, &lm.c_idx, (size_t)lm.c_elems))) return rc;
        if ((rc = dev_alloc(h, &lm.c_val, (size_t)lm.c_elems, true))) return rc;
        CU(h, cudaMemcpyAsync(h->d_c_slice_off + (size_t)layer * (NS + 1), c_off.data(), (size_t)(NS + 1) * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaMemcpyAsync(h->d_c_len + (size_t)layer * N, c_len.data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaMemcpyAsync(h->d_c_order + (size_t)layer * N, order.data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        if (lm.c_elems && (rc = upload_indices(h, lm.c_idx, c_idx))) return rc;
        if ((rc = refresh_mirror(h, layer, nullptr))) return rc;
    }
    CU(h, cudaStreamSynchronize(h->stream));   // the host vectors above go out of scope; the caller may reuse its arrays
    {
        bool nonpos = true;
        for (int i = 0; i < N && nonpos; ++i) nonpos = !(bias[i] > 0.0f);
        h->bias_nonpositive[layer] = nonpos ? 1 : 0;
    }
    {   // locality of the pattern: distinct columns touched by each block of 1024 consecutive rows, summed over the blocks
        std::vector<int> stamp(N, -1);
        int64_t distinct = 0;
        for (int i = 0; i < N; ++i) {
            const int blk = i >> 10;
            for (int p = row_ptr[i]; p < row_ptr[i + 1]; ++p)
                if (stamp[col_idx[p]] != blk) { stamp[col_idx[p]] = blk; ++distinct; }
        }
        h->local_pattern[layer] = distinct <= 2 * (int64_t)N ? 1 : 0;
    }
    return SDNN_OK;
}

// Entries per (padded) row of every group of a structured layer and the padded total; -1 if padding every row of a
// group to its longest row would more than quadruple the layer (plus a margin of 64 entries per row).
int64_t windowed_padding(int n, const int32_t* rp, const sdnn_reorder::Grouping& g, std::vector<int>* ks) {
    const int groups = (int)g.group_c0.size();
    int64_t total = 0;
    if (ks) ks->assign(groups, 0);
    for (int q = 0; q < groups; ++q) {
        int k = 0;
        for (int s = g.group_row0[q]; s < g.group_row0[q + 1]; ++s) k = std::max(k, rp[g.row_order[s] + 1] - rp[g.row_order[s]]);
        k = (k + 7) / 8 * 8;
        if (ks) (*ks)[q] = k;
        total += (int64_t)k * (g.group_row0[q + 1] - g.group_row0[q]);
    }
    if (total > 4 * (int64_t)rp[n] + 64 * (int64_t)n || total > INT32_MAX) return -1;
    return total;
}

// One structured layer in the windowed layout: rows group by group, every row padded to its group's longest, columns
// relative to the group's window.
//   in_label : new numbers of the layer's input neurons (from this layer's own grouping)
//   out_label: new numbers of its output neurons (from the next layer's grouping), or NULL for the caller's numbering
int build_windowed_layer(sdnn* h, int layer, const HostLayer& hl, const sdnn_reorder::Grouping& g, const std::vector<int>* out_label) {
    const int N = h->N;
    LayerMem& lm = h->lay[layer];
    const int groups = (int)g.group_c0.size();
    std::vector<int> ks, ebase(groups, 0);
    const int64_t padded = windowed_padding(N, hl.rp.data(), g, &ks);
    if (padded < 0) return fail(h, SDNN_ERR_STATE, "layer %d: windowed layout too large", layer);      // excluded by build_reordered
    for (int q = 1; q < groups; ++q) ebase[q] = ebase[q - 1] + ks[q - 1] * (g.group_row0[q] - g.group_row0[q - 1]);
    std::vector<int> stored_rp(N + 1, 0), out(N);
    std::vector<float> bias_s(N);
    lm.w_row_at.assign(N, 0);
    for (int q = 0; q < groups; ++q)
        for (int s = g.group_row0[q]; s < g.group_row0[q + 1]; ++s) lm.w_row_at[s] = ebase[q] + (s - g.group_row0[q]) * ks[q];
    for (int s = 0; s < N; ++s) {
        const int i = g.row_order[s];
        stored_rp[s + 1] = stored_rp[s] + (hl.rp[i + 1] - hl.rp[i]);
        out[s] = out_label ? (*out_label)[i] : i;
        bias_s[s] = hl.bias[i];
    }
    std::vector<unsigned short> wcol((size_t)padded, 0);
    std::vector<float> wval((size_t)padded, 0.0f);
    lm.entry_src.assign((size_t)stored_rp[N], 0);
    int max_wlen = 0;
    for (int q = 0; q < groups; ++q) max_wlen = std::max(max_wlen, g.group_wlen[q]);
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < groups; ++q) {
        std::vector<std::pair<int, int>> ent;      // (column within the window, caller's entry position)
        for (int s = g.group_row0[q]; s < g.group_row0[q + 1]; ++s) {
            const int i = g.row_order[s];
            ent.clear();
            for (int p = hl.rp[i]; p < hl.rp[i + 1]; ++p) ent.emplace_back(g.col_label[hl.col[p]] - g.group_c0[q], p);
            std::sort(ent.begin(), ent.end());
            for (size_t t = 0; t < ent.size(); ++t) {
                wcol[(size_t)lm.w_row_at[s] + t] = (unsigned short)ent[t].first;
                wval[(size_t)lm.w_row_at[s] + t] = hl.val[ent[t].second];
                lm.entry_src[(size_t)stored_rp[s] + t] = ent[t].second;
            }
        }
    }
    lm.windowed = true;
    lm.groups = groups;
    lm.max_wlen = max_wlen;
    lm.w_elems = padded;
    lm.shape.uniform_k = -1;
    lm.shape.row_ptr = stored_rp;
    lm.row_src = g.row_order;
    int rc;
    CU(h, cudaSetDevice(h->device));
    if ((rc = dev_alloc(h, &lm.w_col, (size_t)padded, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_val, (size_t)padded, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_out, (size_t)N, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_g_row0, (size_t)groups + 1, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_g_c0, (size_t)groups, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_g_wlen, (size_t)groups, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_g_ebase, (size_t)groups, false))) return rc;
    if ((rc = dev_alloc(h, &lm.w_g_k, (size_t)groups, false))) return rc;
    if (padded) {
        CU(h, cudaMemcpyAsync(lm.w_col, wcol.data(), (size_t)padded * sizeof(unsigned short), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaMemcpyAsync(lm.w_val, wval.data(), (size_t)padded * sizeof(float), cudaMemcpyHostToDevice, h->stream));
    }
    CU(h, cudaMemcpyAsync(lm.w_out, out.data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(lm.w_g_row0, g.group_row0.data(), ((size_t)groups + 1) * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(lm.w_g_c0, g.group_c0.data(), (size_t)groups * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(lm.w_g_wlen, g.group_wlen.data(), (size_t)groups * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(lm.w_g_ebase, ebase.data(), (size_t)groups * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(lm.w_g_k, ks.data(), (size_t)groups * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(h->d_bias + (size_t)layer * N, bias_s.data(), (size_t)N * sizeof(float), cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaStreamSynchronize(h->stream));
    bool nonpos = true;
    for (int i = 0; i < N && nonpos; ++i) nonpos = !(hl.bias[i] > 0.0f);
    h->bias_nonpositive[layer] = nonpos ? 1 : 0;
    h->local_pattern[layer] = 1;
    ++h->windowed_layers;
    return SDNN_OK;
}

// One structured layer in the default (sliced) layout: rows stored group by group, columns renumbered so that a group
// reads one contiguous window of tile rows (which the caches then hold while the group is worked on), every stored row
// writing the tile row that the next layer's grouping assigned to its neuron.
int build_grouped_layer(sdnn* h, int layer, const HostLayer& hl, const sdnn_reorder::Grouping& g, const std::vector<int>* out_label) {
    const int N = h->N;
    LayerMem& lm = h->lay[layer];
    std::vector<int> rp(N + 1, 0), col((size_t)hl.rp[N]), out(N);
    std::vector<float> val((size_t)hl.rp[N]), bias(N);
    lm.entry_src.assign((size_t)hl.rp[N], 0);
    for (int s = 0; s < N; ++s) {
        const int i = g.row_order[s];
        rp[s + 1] = rp[s] + (hl.rp[i + 1] - hl.rp[i]);
        out[s] = out_label ? (*out_label)[i] : i;
        bias[s] = hl.bias[i];
    }
#pragma omp parallel
    {
        std::vector<std::pair<int, int>> ent;      // (new column number, caller's entry position)
#pragma omp for schedule(static)
        for (int s = 0; s < N; ++s) {
            const int i = g.row_order[s];
            ent.clear();
            for (int p = hl.rp[i]; p < hl.rp[i + 1]; ++p) ent.emplace_back(g.col_label[hl.col[p]], p);
            std::sort(ent.begin(), ent.end());
            for (size_t t = 0; t < ent.size(); ++t) {
                col[(size_t)rp[s] + t] = ent[t].first;
                val[(size_t)rp[s] + t] = hl.val[ent[t].second];
                lm.entry_src[(size_t)rp[s] + t] = ent[t].second;
            }
        }
    }
    lm.row_src = g.row_order;
    return upload_layer(h, layer, rp.data(), col.data(), val.data(), bias.data(), out.data());
}

// A layer without structure keeps the default layout; only its rows move to where the next layer's grouping put its
// output neurons (stored row = new number of the neuron, as the default kernels expect).
int build_plain_layer(sdnn* h, int layer, const HostLayer& hl, const std::vector<int>* out_label) {
    if (!out_label) return upload_layer(h, layer, hl.rp.data(), hl.col.data(), hl.val.data(), hl.bias.data());
    const int N = h->N;
    LayerMem& lm = h->lay[layer];
    std::vector<int> src(N);
    for (int i = 0; i < N; ++i) src[(*out_label)[i]] = i;
    std::vector<int> rp(N + 1, 0), col((size_t)hl.rp[N]);
    std::vector<float> val((size_t)hl.rp[N]), bias(N);
    lm.entry_src.assign((size_t)hl.rp[N], 0);
    for (int s = 0; s < N; ++s) rp[s + 1] = rp[s] + (hl.rp[src[s] + 1] - hl.rp[src[s]]);
#pragma omp parallel for schedule(static)
    for (int s = 0; s < N; ++s) {
        const int i = src[s];
        bias[s] = hl.bias[i];
        for (int t = 0; t < hl.rp[i + 1] - hl.rp[i]; ++t) {
            col[(size_t)rp[s] + t] = hl.col[(size_t)hl.rp[i] + t];
            val[(size_t)rp[s] + t] = hl.val[(size_t)hl.rp[i] + t];
            lm.entry_src[(size_t)rp[s] + t] = hl.rp[i] + t;
        }
    }
    lm.row_src = src;
    return upload_layer(h, layer, rp.data(), col.data(), val.data(), bias.data());
}

// SDNN_FLAG_REORDER: analyse every layer, renumber, lay out, upload (called by sdnn_finalize).
int build_reordered(sdnn* h) {
    const int L = h->L, N = h->N;
    std::vector<sdnn_reorder::Grouping> G(L);
    const bool smem_windows = (h->cfg.flags & SDNN_FLAG_SMEM_WINDOWS) != 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int l = 0; l < L; ++l)
        if (sdnn_reorder::cluster_rows(N, h->pending[l].rp.data(), h->pending[l].col.data(), WINDOW_COL_CAP, WINDOW_ROW_CAP, G[l]) &&
            smem_windows && windowed_padding(N, h->pending[l].rp.data(), G[l], nullptr) < 0)
            G[l] = sdnn_reorder::Grouping();      // a few long rows would blow the padded layout up: keep the default one
    // numbers of the neurons at boundary l (inputs of layer l): given by layer l's grouping; the outputs of the last
    // layer keep the caller's numbers
    auto labels = [&](int boundary) -> const std::vector<int>* {
        return (boundary < L && G[boundary].structured) ? &G[boundary].col_label : nullptr;
    };
    int rc;
    h->labels.assign(L + 1, std::vector<int>());
    for (int k = 0; k <= L; ++k) if (labels(k)) h->labels[k] = *labels(k);
    if (labels(0)) {
        if ((rc = dev_alloc(h, &h->d_in_label, (size_t)N, false))) return rc;
        CU(h, cudaMemcpyAsync(h->d_in_label, labels(0)->data(), (size_t)N * sizeof(int), cudaMemcpyHostToDevice, h->stream));
        CU(h, cudaStreamSynchronize(h->stream));
    }
    for (int l = 0; l < L; ++l) {
        const bool smem = (h->cfg.flags & SDNN_FLAG_SMEM_WINDOWS) != 0;
        rc = !G[l].structured ? build_plain_layer(h, l, h->pending[l], labels(l + 1))
             : smem           ? build_windowed_layer(h, l, h->pending[l], G[l], labels(l + 1))
                              : build_grouped_layer(h, l, h->pending[l], G[l], labels(l + 1));
        if (rc) return rc;
        if (G[l].structured) ++h->grouped_layers;
        h->pending[l] = HostLayer();
        G[l] = sdnn_reorder::Grouping();
    }
    h->pending.clear();
    return SDNN_OK;
}

// values of a layer: the caller's CSR order <-> the order they are stored in (rows and entries may have moved)
void caller_to_stored(const LayerMem& lm, const float* src, std::vector<float>& dst, int64_t nnz) {
    dst.resize((size_t)nnz);
    if (lm.entry_src.empty()) { std::copy(src, src + nnz, dst.begin()); return; }
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < nnz; ++e) dst[(size_t)e] = src[lm.entry_src[(size_t)e]];
}
void stored_to_caller(const LayerMem& lm, const std::vector<float>& src, float* dst, int64_t nnz) {
    if (lm.entry_src.empty()) { std::copy(src.begin(), src.begin() + nnz, dst); return; }
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < nnz; ++e) dst[lm.entry_src[(size_t)e]] = src[(size_t)e];
}

}  // namespace

extern "C" {

const char* sdnn_version(void) { return "sdnn 0.2 (sm_100a)"; }

const char* sdnn_last_error(const sdnn_t* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

int64_t sdnn_kernel_launches(const sdnn_t* h) { return h ? h->launches : 0; }
int32_t sdnn_infer_tile_width(const sdnn_t* h) { return (h && h->finalized) ? infer_tile_width(h) : 0; }
int32_t sdnn_infer_tiles_in_flight(const sdnn_t* h) { return (h && h->finalized) ? infer_lanes(h, infer_tile_width(h)) : 0; }
int64_t sdnn_device_bytes(const sdnn_t* h) { return h ? h->dev_bytes : 0; }
int32_t sdnn_windowed_layers(const sdnn_t* h) { return (h && h->finalized) ? h->windowed_layers : 0; }
int32_t sdnn_grouped_layers(const sdnn_t* h) { return (h && h->finalized) ? h->grouped_layers : 0; }

int sdnn_cluster_layer(int32_t n, const int32_t* row_ptr, const int32_t* col_idx, int32_t col_cap, int32_t row_cap,
                       int32_t* group_of_row, int32_t* col_label, int32_t* n_groups, int32_t* max_window) {
    if (n < 1 || !row_ptr || !group_of_row || !col_label || !n_groups || !max_window || col_cap < 1 || row_cap < 1 ||
        (row_ptr[n] > 0 && !col_idx))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "sdnn_cluster_layer: NULL argument or size below 1");
    *n_groups = 0; *max_window = 0;
    sdnn_reorder::Grouping g;
    if (!sdnn_reorder::cluster_rows(n, row_ptr, col_idx, col_cap, row_cap, g)) return SDNN_OK;
    const int groups = (int)g.group_c0.size();
    for (int q = 0; q < groups; ++q) {
        for (int s = g.group_row0[q]; s < g.group_row0[q + 1]; ++s) group_of_row[g.row_order[s]] = q;
        *max_window = std::max(*max_window, g.group_wlen[q]);
    }
    std::copy(g.col_label.begin(), g.col_label.end(), col_label);
    *n_groups = groups;
    return SDNN_OK;
}

void sdnn_destroy(sdnn_t* h) {
    if (!h) return;
    cudaSetDevice(h->device);
    if (h->stream || h->own_stream) cudaStreamSynchronize(h->stream);
    if (h->graph) cudaGraphExecDestroy(h->graph);
    if (h->graph_avg) cudaGraphExecDestroy(h->graph_avg);
    for (cudaEvent_t e : h->ev) if (e) cudaEventDestroy(e);
    for (InferLane& ln : h->lane) {
        if (ln.ev_scan) cudaEventDestroy(ln.ev_scan);
        if (ln.ev_done) cudaEventDestroy(ln.ev_done);
        if (ln.stream && ln.stream != h->stream) { cudaStreamSynchronize(ln.stream); cudaStreamDestroy(ln.stream); }
    }
    if (h->ev_lane_start) cudaEventDestroy(h->ev_lane_start);
    for (cudaEvent_t e : h->ev_delta) if (e) cudaEventDestroy(e);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    for (cudaEvent_t e : h->ev_side_join) if (e) cudaEventDestroy(e);
    for (cudaStream_t st : h->side_streams) if (st) { cudaStreamSynchronize(st); cudaStreamDestroy(st); }
    for (cudaEvent_t e : h->ev_copied) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_consumed) if (e) cudaEventDestroy(e);
    if (h->copy_stream) { cudaStreamSynchronize(h->copy_stream); cudaStreamDestroy(h->copy_stream); }
    for (void* p : h->allocs) cudaFree(p);
    if (h->own_stream) cudaStreamDestroy(h->stream);
    delete h;
}

int sdnn_create_deferred(sdnn_t** out, int32_t n_layers, int32_t n_neurons, const int64_t* nnz_per_layer,
                         const sdnn_config* cfg) {
    if (!out) return fail(nullptr, SDNN_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    int rc = validate_cfg(cfg);
    if (rc) return rc;
    if (n_layers < 1 || n_neurons < 1) return fail(nullptr, SDNN_ERR_INVALID_ARG, "n_layers and n_neurons must be >= 1");
    if (!nnz_per_layer) return fail(nullptr, SDNN_ERR_INVALID_ARG, "nnz_per_layer is NULL");
    for (int l = 0; l < n_layers; ++l)
        if (nnz_per_layer[l] < 0 || nnz_per_layer[l] > INT32_MAX)
            return fail(nullptr, SDNN_ERR_INVALID_ARG, "layer %d: stored-entry count outside [0, 2^31)", l);
    // the kernels address a tile row with a 32-bit multiply-add: one tile must stay below 4 GiB
    if ((int64_t)n_neurons * padded_width(cfg->max_batch) * (int64_t)sizeof(float) >= (1LL << 32))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "n_neurons * padded(max_batch) * 4 bytes must stay below 4 GiB: lower max_batch (inference works in tiles of max_batch inputs)");

    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || ndev == 0) { cudaGetLastError(); return fail(nullptr, SDNN_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(e)); }

    sdnn* h = new (std::nothrow) sdnn;
    if (!h) return fail(nullptr, SDNN_ERR_OOM, "host allocation failed");
    h->L = n_layers; h->N = n_neurons; h->NS = (n_neurons + SLICE - 1) / SLICE; h->cfg = *cfg;
    h->stream = static_cast<cudaStream_t>(cfg->cuda_stream);
    auto bail = [&](int code) { g_create_error = h->err; sdnn_destroy(h); return code; };
    if (cfg->device >= 0) {
        if (cfg->device >= ndev) { h->err = "device ordinal out of range"; return bail(SDNN_ERR_INVALID_ARG); }
        if ((e = cudaSetDevice(cfg->device)) != cudaSuccess) return bail(cuda_fail(h, e, "cudaSetDevice"));
        h->device = cfg->device;
    } else if ((e = cudaGetDevice(&h->device)) != cudaSuccess) {
        return bail(cuda_fail(h, e, "cudaGetDevice"));
    }
    if ((e = cudaDeviceGetAttribute(&h->sms, cudaDevAttrMultiProcessorCount, h->device)) != cudaSuccess || h->sms < 1)
        return bail(cuda_fail(h, e, "cudaDeviceGetAttribute(multiprocessor count)"));
    if (cudaDeviceGetAttribute(&h->l2_bytes, cudaDevAttrL2CacheSize, h->device) != cudaSuccess) { cudaGetLastError(); h->l2_bytes = 0; }
    if (!h->stream) {   // the legacy default stream cannot be captured into a graph: use a blocking stream of our own,
                        // which still orders itself against work on the legacy default stream
        if ((e = cudaStreamCreate(&h->stream)) != cudaSuccess) { h->stream = nullptr; return bail(cuda_fail(h, e, "cudaStreamCreate")); }
        h->own_stream = true;
    }
    h->mirror = cfg->train && !(cfg->flags & SDNN_FLAG_BWD_ATOMICS);
    h->idx16 = n_neurons <= 65536 && !(cfg->flags & SDNN_FLAG_IDX32);
    h->reorder = (cfg->flags & SDNN_FLAG_REORDER) != 0;
    if (h->reorder) h->pending.resize(n_layers);
    h->pdl = !(cfg->flags & SDNN_FLAG_NO_PDL);
    h->nnz.assign(nnz_per_layer, nnz_per_layer + n_layers);
    h->loaded.assign(n_layers, 0);
    h->lay.resize(n_layers);
    h->ld_max = padded_width(cfg->max_batch);
    const size_t N = (size_t)n_neurons, L = (size_t)n_layers, tile = N * (size_t)h->ld_max;

    if ((rc = dev_alloc(h, &h->d_r_slice_off, L * (h->NS + 1), false))) return bail(rc);
    if ((rc = dev_alloc(h, &h->d_r_len, L * N, false))) return bail(rc);
    if ((rc = dev_alloc(h, &h->d_bias, L * N, false))) return bail(rc);
    if (h->mirror) {
        if ((rc = dev_alloc(h, &h->d_c_slice_off, L * (h->NS + 1), false))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_c_len, L * N, false))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_c_order, L * N, false))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_mismatch, 1, true))) return bail(rc);
    }
    if (cfg->train) {
        for (cudaEvent_t& ev : h->ev)
            if ((e = cudaEventCreate(&ev)) != cudaSuccess) { ev = nullptr; return bail(cuda_fail(h, e, "cudaEventCreate")); }
        if ((rc = dev_alloc(h, &h->d_acts, (L + 1) * tile, false))) return bail(rc);
        h->split = h->mirror && !(cfg->flags & SDNN_FLAG_BWD_ONE_LAUNCH);
        if (h->split) {
            if (!(cfg->flags & SDNN_FLAG_KEEP_DEBUG) && (rc = dev_alloc(h, &h->d_delta_all, L * tile, true))) return bail(rc);
            h->n_side = 2;      // row-unit launches of neighbouring layers do not depend on each other: two streams let them overlap
            for (int q = 0; q < h->n_side; ++q) {
                if ((e = cudaStreamCreateWithFlags(&h->side_streams[q], cudaStreamNonBlocking)) != cudaSuccess) return bail(cuda_fail(h, e, "cudaStreamCreate"));
                if ((e = cudaEventCreateWithFlags(&h->ev_side_join[q], cudaEventDisableTiming)) != cudaSuccess) return bail(cuda_fail(h, e, "cudaEventCreate"));
            }
            h->ev_delta.assign(n_layers, nullptr);
            for (cudaEvent_t& ev : h->ev_delta)
                if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) { ev = nullptr; return bail(cuda_fail(h, e, "cudaEventCreate")); }
            if ((e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming)) != cudaSuccess) return bail(cuda_fail(h, e, "cudaEventCreate"));
        }
        if ((rc = dev_alloc(h, &h->d_s[0], tile, true))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_s[1], tile, true))) return bail(rc);
        if (!h->mirror && (rc = dev_alloc(h, &h->d_dl, tile, true))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_yt, tile, true))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_sp, 1, true))) return bail(rc);
        if ((rc = dev_alloc(h, &h->d_loss, 1, true))) return bail(rc);
        if (cfg->flags & SDNN_FLAG_KEEP_DEBUG)
            if ((rc = dev_alloc(h, &h->d_dbg_delta, L * tile, true))) return bail(rc);
    }
    {   // inference buffers (a training handle can also infer)
        h->compaction = (cfg->flags & SDNN_FLAG_SKIP_DEAD) != 0;
        h->bias_nonpositive.assign(n_layers, 0);
        h->local_pattern.assign(n_layers, 0);
        if ((rc = dev_alloc(h, &h->d_running, 1, true))) return bail(rc);
        if ((rc = alloc_lane(h, h->lane[0], false))) return bail(rc);
        h->cur = &h->lane[0];
    }
    *out = h;
    return SDNN_OK;
}

int sdnn_load_layer(sdnn_t* h, int32_t layer, const int32_t* row_ptr, const int32_t* col_idx, const float* values,
                    const float* bias) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (h->finalized) return fail(h, SDNN_ERR_STATE, "handle already finalized");
    if (layer < 0 || layer >= h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, h->L);
    if (h->loaded[layer]) return fail(h, SDNN_ERR_STATE, "layer %d loaded twice", layer);
    int rc = validate_layer(h, layer, h->N, h->nnz[layer], row_ptr, col_idx, values, bias);
    if (rc) return rc;
    if (h->reorder) {      // the layout of a layer depends on its neighbour's grouping: keep the arrays until sdnn_finalize
        HostLayer& hl = h->pending[layer];
        const int64_t nz = h->nnz[layer];
        hl.rp.assign(row_ptr, row_ptr + h->N + 1);
        hl.col.assign(col_idx, col_idx + nz);
        hl.val.assign(values, values + nz);
        hl.bias.assign(bias, bias + h->N);
        h->loaded[layer] = 1;
        return SDNN_OK;
    }
    rc = upload_layer(h, layer, row_ptr, col_idx, values, bias);
    if (rc) return rc;
    h->loaded[layer] = 1;
    return SDNN_OK;
}

int sdnn_finalize(sdnn_t* h) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (h->finalized) return fail(h, SDNN_ERR_STATE, "handle already finalized");
    for (int l = 0; l < h->L; ++l)
        if (!h->loaded[l]) return fail(h, SDNN_ERR_STATE, "layer %d was never loaded", l);
    if (h->reorder) {
        int rc = build_reordered(h);
        if (rc) return rc;
    }
    CU(h, cudaStreamSynchronize(h->stream));
    h->finalized = true;
    return SDNN_OK;
}

int sdnn_create(sdnn_t** out, int32_t n_layers, int32_t n_neurons, const int32_t* const* row_ptr,
                const int32_t* const* col_idx, const float* const* values, const float* const* bias,
                const sdnn_config* cfg) {
    if (!out) return fail(nullptr, SDNN_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    int rc = validate_cfg(cfg);
    if (rc) return rc;
    if (n_layers < 1 || n_neurons < 1) return fail(nullptr, SDNN_ERR_INVALID_ARG, "n_layers and n_neurons must be >= 1");
    if (!row_ptr || !col_idx || !values || !bias) return fail(nullptr, SDNN_ERR_INVALID_ARG, "NULL array of layer pointers");
    std::vector<int64_t> nnz(n_layers);
    for (int l = 0; l < n_layers; ++l) {
        if (!row_ptr[l]) return fail(nullptr, SDNN_ERR_INVALID_ARG, "layer %d: row_ptr is NULL", l);
        const int32_t last = row_ptr[l][n_neurons];
        if (last < 0) return fail(nullptr, SDNN_ERR_BAD_CSR, "layer %d: row_ptr[N] is negative", l);
        nnz[l] = last;
    }
    // validate everything on the host before any device memory is requested
    for (int l = 0; l < n_layers; ++l)
        if ((rc = validate_layer(nullptr, l, n_neurons, nnz[l], row_ptr[l], col_idx[l], values[l], bias[l]))) return rc;
    sdnn* h = nullptr;
    if ((rc = sdnn_create_deferred(&h, n_layers, n_neurons, nnz.data(), cfg))) return rc;
    for (int l = 0; l < n_layers; ++l)
        if ((rc = sdnn_load_layer(h, l, row_ptr[l], col_idx[l], values[l], bias[l]))) { g_create_error = h->err; sdnn_destroy(h); return rc; }
    if ((rc = sdnn_finalize(h))) { g_create_error = h->err; sdnn_destroy(h); return rc; }
    *out = h;
    return SDNN_OK;
}

int sdnn_train_step(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta, float* loss_out) {
    int rc = check_train_args(h, x0, target, B, eta);
    if (rc) return rc;
    CU(h, cudaSetDevice(h->device));
    return train_step_device(h, x0, target, B, eta, loss_out);
}

int sdnn_train_step_averaged(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta, float* loss_out) {
    int rc = check_train_args(h, x0, target, B, eta);
    if (rc) return rc;
    CU(h, cudaSetDevice(h->device));
    return train_step_device(h, x0, target, B, eta, loss_out, true);
}

int sdnn_train_step_host(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta, float* loss_out) {
    int rc = check_train_args(h, x0, target, B, eta);
    if (rc) return rc;
    CU(h, cudaSetDevice(h->device));
    if ((rc = ensure_stage(h))) return rc;
    const size_t bytes = (size_t)B * h->N * sizeof(float);
    CU(h, cudaMemcpyAsync(h->d_stage_a, x0, bytes, cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(h->d_stage_b, target, bytes, cudaMemcpyHostToDevice, h->stream));
    rc = train_step_device(h, h->d_stage_a, h->d_stage_b, B, eta, loss_out);
    if (rc) return rc;
    CU(h, cudaStreamSynchronize(h->stream));
    return SDNN_OK;
}

int sdnn_infer_batch(sdnn_t* h, const float* x0, int64_t n_inputs, float* y_out, int32_t* nz_count_out,
                     int32_t* nz_index_out, int64_t nz_index_capacity, int64_t* nz_total_out) {
    int rc = check_infer_args(h, x0, n_inputs, nz_index_out, nz_index_capacity);
    if (rc) return rc;
    CU(h, cudaSetDevice(h->device));
    const bool want_sets = nz_count_out || nz_index_out || nz_total_out;
    if (want_sets) CU(h, cudaMemsetAsync(h->d_running, 0, sizeof(long long), h->stream));
    const int T = infer_tile_width(h);
    const int lanes = n_inputs > T ? infer_lanes(h, T) : 1;
    if ((rc = lanes_begin(h, lanes))) return rc;
    int64_t tile_no = 0;
    for (int64_t t0 = 0; t0 < n_inputs; t0 += T, ++tile_no) {
        const int cnt = (int)((n_inputs - t0 < T) ? (n_inputs - t0) : T);
        rc = infer_tile(h, h->lane[tile_no % lanes], x0 + (size_t)t0 * h->N, cnt, y_out ? y_out + (size_t)t0 * h->N : nullptr,
                        nz_count_out ? nz_count_out + t0 : nullptr, nz_index_out, nz_index_capacity, want_sets);
        if (rc) break;
    }
    const int rc_end = lanes_end(h, lanes);
    if (rc || rc_end) return rc ? rc : rc_end;
    if (nz_total_out || nz_index_out) {
        long long total = 0;
        CU(h, cudaMemcpyAsync(&total, h->d_running, sizeof total, cudaMemcpyDeviceToHost, h->stream));
        CU(h, cudaStreamSynchronize(h->stream));
        if (nz_total_out) *nz_total_out = total;
        if (nz_index_out && total > nz_index_capacity)
            return fail(h, SDNN_ERR_INVALID_ARG, "nz_index_capacity %lld too small, %lld ids needed", (long long)nz_index_capacity, total);
    }
    return SDNN_OK;
}

int sdnn_infer_batch_host(sdnn_t* h, const float* x0, int64_t n_inputs, float* y_out, int32_t* nz_count_out,
                          int32_t* nz_index_out, int64_t nz_index_capacity, int64_t* nz_total_out) {
    int rc = check_infer_args(h, x0, n_inputs, nz_index_out, nz_index_capacity);
    if (rc) return rc;
    CU(h, cudaSetDevice(h->device));
    if ((rc = ensure_stage(h))) return rc;
    if (nz_index_out && nz_index_capacity > h->stage_idx_cap) {
        if ((rc = dev_alloc(h, &h->d_stage_idx, (size_t)nz_index_capacity, false))) return rc;   // grows; old block freed at destroy
        h->stage_idx_cap = nz_index_capacity;
    }
    const bool want_sets = nz_count_out || nz_index_out || nz_total_out;
    if (want_sets) CU(h, cudaMemsetAsync(h->d_running, 0, sizeof(long long), h->stream));
    const int T = infer_tile_width(h);
    // two input stages and a copy stream: the copy of tile t+1 runs under the layers of tile t
    if (!h->copy_stream) {
        CU(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
        for (int q = 0; q < 2; ++q) {
            CU(h, cudaEventCreateWithFlags(&h->ev_copied[q], cudaEventDisableTiming));
            CU(h, cudaEventCreateWithFlags(&h->ev_consumed[q], cudaEventDisableTiming));
        }
        if ((rc = dev_alloc(h, &h->d_stage_a2, (size_t)h->cfg.max_batch * h->N, false))) return rc;
    }
    float* stage[2] = {h->d_stage_a, h->d_stage_a2};
    CU(h, cudaEventRecord(h->ev_consumed[0], h->stream));       // the stages may still be read by earlier work on the stream
    CU(h, cudaEventRecord(h->ev_consumed[1], h->stream));
    const int lanes = n_inputs > T ? infer_lanes(h, T) : 1;
    if ((rc = lanes_begin(h, lanes))) return rc;
    h->lane[0].stage_out = h->d_stage_b;
    h->lane[0].stage_cnt = h->d_stage_cnt;
    if (lanes == 2 && !h->lane[1].stage_out) {
        if ((rc = dev_alloc(h, &h->lane[1].stage_out, (size_t)h->cfg.max_batch * h->N, false))) return rc;
        if ((rc = dev_alloc(h, &h->lane[1].stage_cnt, (size_t)h->cfg.max_batch, false))) return rc;
    }
    int64_t tile_no = 0;
    for (int64_t t0 = 0; t0 < n_inputs; t0 += T, ++tile_no) {
        const int cnt = (int)((n_inputs - t0 < T) ? (n_inputs - t0) : T);
        const size_t bytes = (size_t)cnt * h->N * sizeof(float);
        const int q = (int)(tile_no & 1);
        InferLane& ln = h->lane[tile_no % lanes];
        CU(h, cudaStreamWaitEvent(h->copy_stream, h->ev_consumed[q], 0));
        CU(h, cudaMemcpyAsync(stage[q], x0 + (size_t)t0 * h->N, bytes, cudaMemcpyHostToDevice, h->copy_stream));
        CU(h, cudaEventRecord(h->ev_copied[q], h->copy_stream));
        CU(h, cudaStreamWaitEvent(ln.stream, h->ev_copied[q], 0));
        rc = infer_tile(h, ln, stage[q], cnt, y_out ? ln.stage_out : nullptr, nz_count_out ? ln.stage_cnt : nullptr,
                        nz_index_out ? h->d_stage_idx : nullptr, nz_index_capacity, want_sets);
        if (rc) break;
        if (y_out) CU(h, cudaMemcpyAsync(y_out + (size_t)t0 * h->N, ln.stage_out, bytes, cudaMemcpyDeviceToHost, ln.stream));
        if (nz_count_out) CU(h, cudaMemcpyAsync(nz_count_out + t0, ln.stage_cnt, (size_t)cnt * sizeof(int), cudaMemcpyDeviceToHost, ln.stream));
        CU(h, cudaEventRecord(h->ev_consumed[q], ln.stream));
    }
    const int rc_end = lanes_end(h, lanes);
    if (rc || rc_end) return rc ? rc : rc_end;
    long long total = 0;
    if (want_sets) CU(h, cudaMemcpyAsync(&total, h->d_running, sizeof total, cudaMemcpyDeviceToHost, h->stream));
    CU(h, cudaStreamSynchronize(h->stream));
    if (nz_total_out) *nz_total_out = total;
    if (nz_index_out) {
        const long long m = total < nz_index_capacity ? total : nz_index_capacity;
        if (m > 0) CU(h, cudaMemcpy(nz_index_out, h->d_stage_idx, (size_t)m * sizeof(int), cudaMemcpyDeviceToHost));
        if (total > nz_index_capacity)
            return fail(h, SDNN_ERR_INVALID_ARG, "nz_index_capacity %lld too small, %lld ids needed", (long long)nz_index_capacity, total);
    }
    return SDNN_OK;
}

int sdnn_get_weights(sdnn_t* h, int32_t layer, float* values_out, float* bias_out) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (!h->finalized) return fail(h, SDNN_ERR_STATE, "handle is not finalized");
    if (layer < 0 || layer >= h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, h->L);
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    const LayerMem& lm = h->lay[layer];
    const int64_t nnz = h->nnz[layer];
    if (values_out && nnz) {
        std::vector<float> stored((size_t)nnz);
        if (lm.windowed) {
            std::vector<float> tmp((size_t)lm.w_elems);
            CU(h, cudaMemcpy(tmp.data(), lm.w_val, tmp.size() * sizeof(float), cudaMemcpyDeviceToHost));
            for (int r = 0; r < h->N; ++r)
                std::copy(tmp.begin() + lm.w_row_at[r], tmp.begin() + lm.w_row_at[r] + lm.shape.len(r), stored.begin() + lm.shape.start(r));
        } else {
            std::vector<float> tmp((size_t)lm.r_elems);
            CU(h, cudaMemcpy(tmp.data(), lm.r_val, tmp.size() * sizeof(float), cudaMemcpyDeviceToHost));
            sliced_to_csr(h, lm, tmp, stored.data());
        }
        stored_to_caller(lm, stored, values_out, nnz);
    }
    if (bias_out) {
        if (lm.row_src.empty()) {
            CU(h, cudaMemcpy(bias_out, h->d_bias + (size_t)layer * h->N, (size_t)h->N * sizeof(float), cudaMemcpyDeviceToHost));
        } else {
            std::vector<float> tmp((size_t)h->N);
            CU(h, cudaMemcpy(tmp.data(), h->d_bias + (size_t)layer * h->N, tmp.size() * sizeof(float), cudaMemcpyDeviceToHost));
            for (int r = 0; r < h->N; ++r) bias_out[lm.row_src[r]] = tmp[r];
        }
    }
    return SDNN_OK;
}

int sdnn_set_weights(sdnn_t* h, int32_t layer, const float* values, const float* bias) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (!h->finalized) return fail(h, SDNN_ERR_STATE, "handle is not finalized");
    if (layer < 0 || layer >= h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, h->L);
    if (values)
        for (int64_t p = 0; p < h->nnz[layer]; ++p)
            if (!std::isfinite(values[p])) return fail(h, SDNN_ERR_BAD_CSR, "layer %d: non-finite value at entry %lld", layer, (long long)p);
    if (bias)
        for (int i = 0; i < h->N; ++i)
            if (!std::isfinite(bias[i])) return fail(h, SDNN_ERR_BAD_CSR, "layer %d: non-finite bias at row %d", layer, i);
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    const LayerMem& lm = h->lay[layer];
    const int64_t nnz = h->nnz[layer];
    if (values && nnz) {
        std::vector<float> stored, tmp;
        caller_to_stored(lm, values, stored, nnz);
        if (lm.windowed) {
            tmp.assign((size_t)lm.w_elems, 0.0f);
            for (int r = 0; r < h->N; ++r)
                std::copy(stored.begin() + lm.shape.start(r), stored.begin() + lm.shape.start(r) + lm.shape.len(r), tmp.begin() + lm.w_row_at[r]);
            CU(h, cudaMemcpy(lm.w_val, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
        } else {
            csr_to_sliced(h, lm, stored.data(), tmp);
            CU(h, cudaMemcpy(lm.r_val, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
        }
        if (lm.c_val) {
            int rc = refresh_mirror(h, layer, nullptr);
            if (rc) return rc;
            CU(h, cudaStreamSynchronize(h->stream));
        }
    }
    if (bias) {
        if (lm.row_src.empty()) {
            CU(h, cudaMemcpy(h->d_bias + (size_t)layer * h->N, bias, (size_t)h->N * sizeof(float), cudaMemcpyHostToDevice));
        } else {
            std::vector<float> tmp((size_t)h->N);
            for (int r = 0; r < h->N; ++r) tmp[r] = bias[lm.row_src[r]];
            CU(h, cudaMemcpy(h->d_bias + (size_t)layer * h->N, tmp.data(), tmp.size() * sizeof(float), cudaMemcpyHostToDevice));
        }
        bool nonpos = true;
        for (int i = 0; i < h->N && nonpos; ++i) nonpos = !(bias[i] > 0.0f);
        h->bias_nonpositive[layer] = nonpos ? 1 : 0;
    }
    return SDNN_OK;
}

int sdnn_mirror_mismatches(sdnn_t* h, int32_t layer, int64_t* count_out) {
    if (!h || !count_out) return SDNN_ERR_INVALID_ARG;
    if (!h->finalized) return fail(h, SDNN_ERR_STATE, "handle is not finalized");
    if (layer < 0 || layer >= h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, h->L);
    *count_out = 0;
    if (!h->lay[layer].c_val) return SDNN_OK;      // no transposed copy for this layer: nothing can differ
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaMemsetAsync(h->d_mismatch, 0, sizeof(unsigned long long), h->stream));
    int rc = refresh_mirror(h, layer, h->d_mismatch);
    if (rc) return rc;
    unsigned long long v = 0;
    CU(h, cudaMemcpyAsync(&v, h->d_mismatch, sizeof v, cudaMemcpyDeviceToHost, h->stream));
    CU(h, cudaStreamSynchronize(h->stream));
    *count_out = (int64_t)v;
    return SDNN_OK;
}

static int fetch_tile(sdnn_t* h, const float* tile, float* out, int B, int ld, int boundary) {
    // tile [N][ld] on the device -> out [B][N] on the host, neuron i read from the tile row it was given at set-up
    const int N = h->N;
    const std::vector<int>* lab = (boundary < (int)h->labels.size() && !h->labels[boundary].empty()) ? &h->labels[boundary] : nullptr;
    std::vector<float> tmp((size_t)N * ld);
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    CU(h, cudaMemcpy(tmp.data(), tile, tmp.size() * sizeof(float), cudaMemcpyDeviceToHost));
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < N; ++i) out[(size_t)b * N + i] = tmp[(size_t)(lab ? (*lab)[i] : i) * ld + b];
    return SDNN_OK;
}

int sdnn_get_activations(sdnn_t* h, int32_t layer, float* out) {
    if (!h || !out) return SDNN_ERR_INVALID_ARG;
    if (!h->stepped) return fail(h, SDNN_ERR_STATE, "no train step has run");
    if (layer < 0 || layer > h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [0, %d]", layer, h->L);
    return fetch_tile(h, h->d_acts + (size_t)layer * h->N * h->last_ld, out, h->last_b, h->last_ld, layer);
}

int sdnn_get_delta(sdnn_t* h, int32_t layer, float* out) {
    if (!h || !out) return SDNN_ERR_INVALID_ARG;
    if (!h->stepped || !h->d_dbg_delta) return fail(h, SDNN_ERR_STATE, "needs SDNN_FLAG_KEEP_DEBUG and a train step");
    if (layer < 1 || layer > h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [1, %d]", layer, h->L);
    return fetch_tile(h, h->d_dbg_delta + (size_t)(layer - 1) * h->N * h->last_delta_ld, out, h->last_delta_b, h->last_delta_ld, layer);
}

int sdnn_get_gradient(sdnn_t* h, int32_t layer, float* out) {
    if (!h || !out) return SDNN_ERR_INVALID_ARG;
    if (!h->stepped || !h->d_dbg_delta) return fail(h, SDNN_ERR_STATE, "needs SDNN_FLAG_KEEP_DEBUG and a train step");
    if (layer < 1 || layer > h->L) return fail(h, SDNN_ERR_INVALID_ARG, "layer %d outside [1, %d]", layer, h->L);
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    const LayerMem& lm = h->lay[layer - 1];
    if (lm.r_elems && lm.r_grad) {
        std::vector<float> tmp((size_t)lm.r_elems);
        CU(h, cudaMemcpy(tmp.data(), lm.r_grad, tmp.size() * sizeof(float), cudaMemcpyDeviceToHost));
        std::vector<float> stored((size_t)h->nnz[layer - 1]);
        sliced_to_csr(h, lm, tmp, stored.data());
        stored_to_caller(lm, stored, out, h->nnz[layer - 1]);
    }
    return SDNN_OK;
}

int sdnn_get_phase_times(sdnn_t* h, float* fwd_ms, float* bwd_ms) {
    if (!h) return SDNN_ERR_INVALID_ARG;
    if (!h->stepped) return fail(h, SDNN_ERR_STATE, "no train step has run");
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    float a = 0.f, b = 0.f;
    CU(h, cudaEventElapsedTime(&a, h->ev[0], h->ev[1]));
    CU(h, cudaEventElapsedTime(&b, h->ev[1], h->ev[2]));
    if (fwd_ms) *fwd_ms = a;
    if (bwd_ms) *bwd_ms = b;
    return SDNN_OK;
}

int sdnn_get_liveness(sdnn_t* h, int32_t* live_inputs_out) {
    if (!h || !live_inputs_out) return SDNN_ERR_INVALID_ARG;
    if (!h->live_valid) return fail(h, SDNN_ERR_STATE, "liveness is recorded only by inference with SDNN_FLAG_SKIP_DEAD on a net without positive biases");
    CU(h, cudaSetDevice(h->device));
    CU(h, cudaStreamSynchronize(h->stream));
    CU(h, cudaMemcpy(live_inputs_out, h->lane[h->live_lane].live_hist, (size_t)h->L * sizeof(int), cudaMemcpyDeviceToHost));
    return SDNN_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Gather-rate probe (see sdnn_probe_gather_rate in the header).
namespace {

template <int G, int V, bool PAST_L1>
float run_gather_probe_path(const float* table, float* sink, unsigned mask, int per_group, int grid, cudaStream_t st, int reps,
                            cudaEvent_t a, cudaEvent_t b) {
    for (int i = 0; i < 2; ++i) gather_probe_kernel<G, V, PAST_L1><<<grid, 256, 0, st>>>(table, sink, mask, per_group, 17u + i);
    cudaEventRecord(a, st);
    for (int i = 0; i < reps; ++i) gather_probe_kernel<G, V, PAST_L1><<<grid, 256, 0, st>>>(table, sink, mask, per_group, 101u + i);
    cudaEventRecord(b, st);
    cudaEventSynchronize(b);
    float ms = 0.f;
    cudaEventElapsedTime(&ms, a, b);
    return ms / reps;
}
// the faster of the two load paths the layer kernels use: through L1 (read-only path) and past it
template <int G, int V>
float run_gather_probe(const float* table, float* sink, unsigned mask, int per_group, int grid, cudaStream_t st, int reps,
                       cudaEvent_t a, cudaEvent_t b) {
    const float t0 = run_gather_probe_path<G, V, false>(table, sink, mask, per_group, grid, st, reps, a, b);
    if (V != 8) return t0;
    const float t1 = run_gather_probe_path<G, V, true>(table, sink, mask, per_group, grid, st, reps, a, b);
    return (t1 > 0.f && (t0 <= 0.f || t1 < t0)) ? t1 : t0;
}

}  // namespace

extern "C" int sdnn_probe_gather_rate(int32_t row_bytes, int64_t table_rows, double* rows_per_second) {
    if (!rows_per_second) return fail(nullptr, SDNN_ERR_INVALID_ARG, "rows_per_second is NULL");
    *rows_per_second = 0.0;
    if (row_bytes != 16 && row_bytes != 32 && row_bytes != 64 && row_bytes != 128 && row_bytes != 256 && row_bytes != 512 &&
        row_bytes != 1024)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "row_bytes must be 16, 32, 64, 128, 256, 512 or 1024");
    if (table_rows < 1 || (table_rows & (table_rows - 1)) || table_rows * row_bytes > (1LL << 30))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "table_rows must be a power of two with table_rows * row_bytes <= 1 GiB");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float* table = nullptr;
    float* sink = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    const size_t bytes = (size_t)table_rows * row_bytes;
    if (cudaMalloc(&table, bytes) != cudaSuccess || cudaMalloc(&sink, 256) != cudaSuccess || cudaStreamCreate(&st) != cudaSuccess ||
        cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not allocate the probe's table");
    } else {
        cudaMemsetAsync(table, 0, bytes, st);
        // the rate depends on the threads per SM (it peaks between 768 and 2048 depending on the row width): try 2 .. 8
        // CTAs of 256 threads per SM and keep the best, so that the figure is what the path can do, not what one shape does
        const int g = row_bytes == 16 ? 1 : row_bytes / 32;      // 256-bit lanes
        const unsigned mask = (unsigned)(table_rows - 1);
        float ms = 0.f;
        double best = 0.0;
        for (int per_sm = 2; per_sm <= 8; ++per_sm) {
            if (per_sm == 5 || per_sm == 7) continue;
            const int grid = sms * per_sm;
            const int64_t groups = (int64_t)grid * 256 / g;
            const int per_group = (int)std::max<int64_t>(8, ((int64_t)1 << 22) / groups / 8 * 8);
            switch (row_bytes) {
                case 16: ms = run_gather_probe<1, 4>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                case 32: ms = run_gather_probe<1, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                case 64: ms = run_gather_probe<2, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                case 128: ms = run_gather_probe<4, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                case 256: ms = run_gather_probe<8, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                case 512: ms = run_gather_probe<16, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
                default: ms = run_gather_probe<32, 8>(table, sink, mask, per_group, grid, st, 10, a, b); break;
            }
            if (ms > 0.f) best = std::max(best, (double)groups * per_group / (ms * 1e-3));
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess || !(best > 0.0)) rc = cuda_fail(nullptr, e, "gather probe");
        else *rows_per_second = best;
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (table) cudaFree(table);
    if (sink) cudaFree(sink);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Gather rate against rows in flight (see sdnn_probe_gather_inflight in the header).
namespace {
template <int F>
int run_inflight_probe(const float* table, float* sink, unsigned mask, int ctas_per_sm, int sms, cudaStream_t st, cudaEvent_t a,
                       cudaEvent_t b, double* rate) {
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gather_inflight_probe_kernel<F>, 128, 0) != cudaSuccess) { cudaGetLastError(); occ = 0; }
    if (occ < ctas_per_sm) return SDNN_ERR_INVALID_ARG;      // not all resident: the figure would not be what it claims
    const int grid = sms * ctas_per_sm;
    const int64_t lanes_pairs = (int64_t)grid * 64;
    const int batches = (int)std::max<int64_t>(4, ((int64_t)1 << 23) / (lanes_pairs * F));      // launches of about 40 us: ramp and drain are a few per cent
    const int reps = 10;
    for (int i = 0; i < 2; ++i) gather_inflight_probe_kernel<F><<<grid, 128, 0, st>>>(table, sink, mask, batches, 17u + i);
    cudaEventRecord(a, st);
    for (int i = 0; i < reps; ++i) gather_inflight_probe_kernel<F><<<grid, 128, 0, st>>>(table, sink, mask, batches, 101u + i);
    cudaEventRecord(b, st);
    cudaEventSynchronize(b);
    float ms = 0.f;
    cudaEventElapsedTime(&ms, a, b);
    if (!(ms > 0.f)) return SDNN_ERR_CUDA;
    *rate = (double)lanes_pairs * F * batches * reps / (ms * 1e-3);
    return SDNN_OK;
}
}  // namespace

extern "C" int sdnn_probe_gather_inflight(int64_t table_rows, int32_t threads_per_sm, int32_t loads_in_flight, double* rows_per_second) {
    if (!rows_per_second) return fail(nullptr, SDNN_ERR_INVALID_ARG, "rows_per_second is NULL");
    *rows_per_second = 0.0;
    if (table_rows < 1 || (table_rows & (table_rows - 1)) || table_rows * 64 > (1LL << 30))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "table_rows must be a power of two with table_rows * 64 <= 1 GiB");
    if (threads_per_sm < 128 || threads_per_sm > 2048 || threads_per_sm % 128)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "threads_per_sm must be a multiple of 128 between 128 and 2048");
    if (loads_in_flight != 1 && loads_in_flight != 2 && loads_in_flight != 4 && loads_in_flight != 8 && loads_in_flight != 16)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "loads_in_flight must be 1, 2, 4, 8 or 16");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float* table = nullptr;
    float* sink = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    const size_t bytes = (size_t)table_rows * 64;
    if (cudaMalloc(&table, bytes) != cudaSuccess || cudaMalloc(&sink, 256) != cudaSuccess || cudaStreamCreate(&st) != cudaSuccess ||
        cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not allocate the probe's table");
    } else {
        cudaMemsetAsync(table, 0, bytes, st);
        const unsigned mask = (unsigned)(table_rows - 1);
        const int cps = threads_per_sm / 128;
        switch (loads_in_flight) {
            case 1: rc = run_inflight_probe<1>(table, sink, mask, cps, sms, st, a, b, rows_per_second); break;
            case 2: rc = run_inflight_probe<2>(table, sink, mask, cps, sms, st, a, b, rows_per_second); break;
            case 4: rc = run_inflight_probe<4>(table, sink, mask, cps, sms, st, a, b, rows_per_second); break;
            case 8: rc = run_inflight_probe<8>(table, sink, mask, cps, sms, st, a, b, rows_per_second); break;
            default: rc = run_inflight_probe<16>(table, sink, mask, cps, sms, st, a, b, rows_per_second); break;
        }
        cudaError_t e = cudaGetLastError();
        if (rc == SDNN_ERR_INVALID_ARG) rc = fail(nullptr, rc, "that many threads with that many loads in flight do not fit an SM's registers");
        else if (rc != SDNN_OK || e != cudaSuccess) rc = cuda_fail(nullptr, e, "gather in-flight probe");
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (table) cudaFree(table);
    if (sink) cudaFree(sink);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Cost of a layer boundary (see sdnn_probe_layer_boundary in the header).
extern "C" int sdnn_probe_layer_boundary(int32_t ctas_per_sm, int32_t threads, double* barrier_us, double* launch_us) {
    if (!barrier_us || !launch_us) return fail(nullptr, SDNN_ERR_INVALID_ARG, "barrier_us or launch_us is NULL");
    *barrier_us = 0.0; *launch_us = 0.0;
    if (ctas_per_sm < 1 || ctas_per_sm > 4 || threads < 32 || threads > 1024 || threads % 32)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "ctas_per_sm must be 1..4 and threads a multiple of 32 up to 1024");
    int dev = 0, sms = 0, coop = 0, occ = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CU(nullptr, cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    CU(nullptr, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, grid_barrier_probe_kernel, threads, 0));
    if (!coop || occ < ctas_per_sm)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "the device cannot hold that grid resident (a grid barrier needs every CTA running)");
    const int grid = sms * ctas_per_sm, rounds = 1000;
    unsigned* counter = nullptr;
    int* err = nullptr;
    float* data = nullptr;
    cudaStream_t st = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int rc = SDNN_OK;
    if (cudaMalloc(&counter, 4) != cudaSuccess || cudaMalloc(&err, 4) != cudaSuccess ||
        cudaMalloc(&data, (size_t)grid * threads * sizeof(float)) != cudaSuccess || cudaStreamCreate(&st) != cudaSuccess ||
        cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not allocate the probe's buffers");
    } else {
        float best = 0.f;
        int herr = 0;
        for (int rep = 0; rep < 3 && rc == SDNN_OK; ++rep) {      // the barrier: one cooperative launch of `rounds` rounds
            cudaMemsetAsync(counter, 0, 4, st); cudaMemsetAsync(err, 0, 4, st);
            cudaEventRecord(a, st);
            int rr = rounds;
            void* args[] = {&counter, &err, &rr, &data};
            cudaError_t e = cudaLaunchCooperativeKernel((void*)grid_barrier_probe_kernel, dim3(grid), dim3(threads), args, 0, st);
            cudaEventRecord(b, st);
            if (e != cudaSuccess || cudaEventSynchronize(b) != cudaSuccess) { rc = cuda_fail(nullptr, e != cudaSuccess ? e : cudaGetLastError(), "grid barrier probe"); break; }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            if (rep == 0 || ms < best) best = ms;
            cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
            if (herr) rc = fail(nullptr, SDNN_ERR_CUDA, "grid barrier probe: a wait ran out (the grid was not resident as a whole)");
        }
        if (rc == SDNN_OK) *barrier_us = (double)best * 1e3 / rounds;
        if (rc == SDNN_OK) {      // the launch boundary: `rounds` dependent launches, captured into one graph as the library's steps are
            cudaError_t e = cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal);
            for (int r = 0; r < rounds && e == cudaSuccess; ++r) {
                cudaLaunchConfig_t lc = {};
                lc.gridDim = dim3(grid); lc.blockDim = dim3(threads); lc.stream = st;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                at[0].val.programmaticStreamSerializationAllowed = 1;
                lc.attrs = at; lc.numAttrs = 1;
                e = cudaLaunchKernelEx(&lc, launch_chain_probe_kernel, data, r);
            }
            cudaError_t e2 = cudaStreamEndCapture(st, &graph);
            if (e == cudaSuccess) e = e2;
            if (e == cudaSuccess) e = cudaGraphInstantiate(&exec, graph, 0);
            for (int rep = 0; rep < 3 && e == cudaSuccess; ++rep) {
                cudaEventRecord(a, st);
                e = cudaGraphLaunch(exec, st);
                cudaEventRecord(b, st);
                if (e == cudaSuccess) e = cudaEventSynchronize(b);
                float ms = 0.f;
                cudaEventElapsedTime(&ms, a, b);
                if (rep == 0 || ms < best) best = ms;
            }
            if (e != cudaSuccess) rc = cuda_fail(nullptr, e, "launch chain probe");
            else *launch_us = (double)best * 1e3 / rounds;
        }
    }
    if (exec) cudaGraphExecDestroy(exec);
    if (graph) cudaGraphDestroy(graph);
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (counter) cudaFree(counter);
    if (err) cudaFree(err);
    if (data) cudaFree(data);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Scattered 4-byte word probe (see sdnn_probe_word_rate in the header).
extern "C" int sdnn_probe_word_rate(int32_t store, int64_t table_words, double* words_per_second) {
    if (!words_per_second) return fail(nullptr, SDNN_ERR_INVALID_ARG, "words_per_second is NULL");
    *words_per_second = 0.0;
    if (store != 0 && store != 1) return fail(nullptr, SDNN_ERR_INVALID_ARG, "store must be 0 (loads) or 1 (stores)");
    if (table_words < 1024 || (table_words & (table_words - 1)) || table_words > (1LL << 28))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "table_words must be a power of two between 2^10 and 2^28");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float* table = nullptr;
    float* sink = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    const size_t bytes = (size_t)table_words * sizeof(float);
    if (cudaMalloc(&table, bytes) != cudaSuccess || cudaMalloc(&sink, 256) != cudaSuccess || cudaStreamCreate(&st) != cudaSuccess ||
        cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not allocate the probe's table");
    } else {
        cudaMemsetAsync(table, 0, bytes, st);
        const int grid = sms * 8, per_lane = 1024, reps = 10;
        const unsigned mask = (unsigned)(table_words - 1);
        auto launch = [&](unsigned seed) {
            if (store) word_probe_kernel<1><<<grid, 256, 0, st>>>(table, sink, mask, per_lane, seed);
            else word_probe_kernel<0><<<grid, 256, 0, st>>>(table, sink, mask, per_lane, seed);
        };
        launch(17u); launch(18u);
        cudaEventRecord(a, st);
        for (int i = 0; i < reps; ++i) launch(101u + i);
        cudaEventRecord(b, st);
        cudaError_t e = cudaEventSynchronize(b);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess || !(ms > 0.f)) rc = cuda_fail(nullptr, e, "word probe");
        else *words_per_second = (double)grid * 256 * per_lane / (ms / reps * 1e-3);
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (table) cudaFree(table);
    if (sink) cudaFree(sink);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Tensor map of a table of rows for tile::gather4: a two-dimensional tensor [table_rows][row_bytes / 4] of floats in this
// device's own memory, box = one row, no swizzle.  The driver's encoder is looked up at run time (no link against libcuda).
namespace {
int encode_row_map(CUtensorMap* tmap, float* table, int row_bytes, int64_t table_rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        return fail(nullptr, SDNN_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
    }
    const cuuint64_t dims[2] = {(cuuint64_t)(row_bytes / 4), (cuuint64_t)table_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(row_bytes / 4), 1u};
    const cuuint32_t estr[2] = {1u, 1u};
    CUresult cr = reinterpret_cast<EncodeFn>(fn)(tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, table, dims, strides, box, estr,
                                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                                CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(nullptr, SDNN_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)cr);
    return SDNN_OK;
}
}  // namespace

// ---------------------------------------------------------------------------------------------
// Copy-engine gather probe (see sdnn_probe_tma_gather_rate in the header).
extern "C" int sdnn_probe_tma_gather_rate(int32_t row_bytes, int64_t table_rows, int32_t gather4, double* rows_per_second) {
    if (!rows_per_second) return fail(nullptr, SDNN_ERR_INVALID_ARG, "rows_per_second is NULL");
    *rows_per_second = 0.0;
    if (row_bytes != 16 && row_bytes != 32 && row_bytes != 64 && row_bytes != 128 && row_bytes != 256)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "row_bytes must be 16, 32, 64, 128 or 256");
    if (table_rows < 1 || (table_rows & (table_rows - 1)) || table_rows * row_bytes > (1LL << 30))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "table_rows must be a power of two with table_rows * row_bytes <= 1 GiB");
    if (gather4 != 0 && gather4 != 1) return fail(nullptr, SDNN_ERR_INVALID_ARG, "gather4 must be 0 or 1");
    if (gather4 && row_bytes < 32)      // a copy's four rows land in one 128-byte aligned slot of shared memory
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "tile::gather4 needs row_bytes >= 32 here");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float* table = nullptr;
    float* sink = nullptr;
    int* status = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    const size_t bytes = (size_t)table_rows * row_bytes;
    if (cudaMalloc(&table, bytes) != cudaSuccess || cudaMalloc(&sink, 256) != cudaSuccess || cudaMalloc(&status, sizeof(int)) != cudaSuccess ||
        cudaStreamCreate(&st) != cudaSuccess || cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not set up the probe");
    } else {
        cudaMemsetAsync(table, 0, bytes, st);
        cudaMemsetAsync(status, 0, sizeof(int), st);
        CUtensorMap tmap;
        memset(&tmap, 0, sizeof tmap);
        if (gather4) rc = encode_row_map(&tmap, table, row_bytes, table_rows);
        if (rc == SDNN_OK) {
            const unsigned rows_per_copy = gather4 ? 4u : 1u;
            const int issuers = (int)std::min<size_t>(32, 8192 / ((size_t)rows_per_copy * row_bytes));      // lanes of a warp that issue copies
            const size_t smem = (size_t)TMA_WARPS * TMA_STAGES * issuers * rows_per_copy * row_bytes;       // at most 128 KB
            cudaError_t e = gather4 ? cudaFuncSetAttribute(tma_gather_probe_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                    : cudaFuncSetAttribute(tma_gather_probe_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            int occ = 1;
            if (e == cudaSuccess)
                e = gather4 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, tma_gather_probe_kernel<true>, 32 * TMA_WARPS, smem)
                            : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, tma_gather_probe_kernel<false>, 32 * TMA_WARPS, smem);
            if (e != cudaSuccess || occ < 1) rc = cuda_fail(nullptr, e, "copy-engine probe set-up");
            else {
                const int grid = sms * std::min(occ, 4), rounds = 256, reps = 5;
                const unsigned mask = (unsigned)(table_rows - 1);
                auto launch = [&](unsigned seed) {
                    if (gather4) tma_gather_probe_kernel<true><<<grid, 32 * TMA_WARPS, smem, st>>>(table, tmap, sink, status, mask, (unsigned)row_bytes, issuers, rounds, seed);
                    else tma_gather_probe_kernel<false><<<grid, 32 * TMA_WARPS, smem, st>>>(table, tmap, sink, status, mask, (unsigned)row_bytes, issuers, rounds, seed);
                };
                launch(17u); launch(18u);
                cudaEventRecord(a, st);
                for (int i = 0; i < reps; ++i) launch(101u + i);
                cudaEventRecord(b, st);
                e = cudaEventSynchronize(b);
                float ms = 0.f;
                int gave_up = 0;
                if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
                if (e == cudaSuccess) e = cudaMemcpy(&gave_up, status, sizeof(int), cudaMemcpyDeviceToHost);
                if (e == cudaSuccess) e = cudaGetLastError();
                if (e != cudaSuccess || !(ms > 0.f)) rc = cuda_fail(nullptr, e, "copy-engine probe");
                else if (gave_up) rc = fail(nullptr, SDNN_ERR_CUDA, "copy-engine probe: a wait for its copies ran out");
                else *rows_per_second = (double)grid * issuers * TMA_WARPS * rows_per_copy * rounds / (ms / reps * 1e-3);
            }
        }
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (table) cudaFree(table);
    if (sink) cudaFree(sink);
    if (status) cudaFree(status);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Both gather paths at once (see sdnn_probe_mixed_gather in the header).
extern "C" int sdnn_probe_mixed_gather(int32_t row_bytes, int64_t table_rows, int32_t tma_rounds, int32_t lsu_per_group,
                                       double* seconds, double* rows) {
    if (!seconds || !rows) return fail(nullptr, SDNN_ERR_INVALID_ARG, "seconds or rows is NULL");
    *seconds = 0.0; *rows = 0.0;
    if (row_bytes != 64 && row_bytes != 256) return fail(nullptr, SDNN_ERR_INVALID_ARG, "row_bytes must be 64 or 256");
    if (table_rows < 1 || (table_rows & (table_rows - 1)) || table_rows * row_bytes > (1LL << 30))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "table_rows must be a power of two with table_rows * row_bytes <= 1 GiB");
    if (tma_rounds < 0 || tma_rounds > (1 << 16) || lsu_per_group < 0 || lsu_per_group > (1 << 20) || (lsu_per_group & 7) ||
        (tma_rounds == 0 && lsu_per_group == 0))
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "tma_rounds in [0, 65536], lsu_per_group a multiple of 8 in [0, 2^20], not both 0");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    float* table = nullptr;
    float* sink = nullptr;
    int* status = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    const size_t bytes = (size_t)table_rows * row_bytes;
    if (cudaMalloc(&table, bytes) != cudaSuccess || cudaMalloc(&sink, 256) != cudaSuccess || cudaMalloc(&status, sizeof(int)) != cudaSuccess ||
        cudaStreamCreate(&st) != cudaSuccess || cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not set up the probe");
    } else {
        cudaMemsetAsync(table, 0, bytes, st);
        cudaMemsetAsync(status, 0, sizeof(int), st);
        CUtensorMap tmap;
        memset(&tmap, 0, sizeof tmap);
        rc = encode_row_map(&tmap, table, row_bytes, table_rows);
        if (rc == SDNN_OK) {
            const int issuers = (int)std::min<size_t>(32, 8192 / ((size_t)4 * row_bytes));
            const size_t smem = (size_t)TMA_WARPS * TMA_STAGES * issuers * 4 * row_bytes;
            auto k64 = mixed_gather_probe_kernel<2, 8>;
            auto k256 = mixed_gather_probe_kernel<8, 8>;
            cudaError_t e = cudaFuncSetAttribute(row_bytes == 64 ? k64 : k256, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) rc = cuda_fail(nullptr, e, "mixed probe set-up");
            else {
                const int grid = sms, reps = 5;
                const unsigned mask = (unsigned)(table_rows - 1);
                auto launch = [&](unsigned seed) {
                    if (row_bytes == 64) k64<<<grid, 1024, smem, st>>>(table, tmap, sink, status, mask, issuers, tma_rounds, lsu_per_group, seed);
                    else k256<<<grid, 1024, smem, st>>>(table, tmap, sink, status, mask, issuers, tma_rounds, lsu_per_group, seed);
                };
                launch(17u); launch(18u);
                cudaEventRecord(a, st);
                for (int i = 0; i < reps; ++i) launch(101u + i);
                cudaEventRecord(b, st);
                e = cudaEventSynchronize(b);
                float ms = 0.f;
                int gave_up = 0;
                if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
                if (e == cudaSuccess) e = cudaMemcpy(&gave_up, status, sizeof(int), cudaMemcpyDeviceToHost);
                if (e == cudaSuccess) e = cudaGetLastError();
                if (e != cudaSuccess || !(ms > 0.f)) rc = cuda_fail(nullptr, e, "mixed probe");
                else if (gave_up) rc = fail(nullptr, SDNN_ERR_CUDA, "mixed probe: a wait for the copy engine ran out");
                else {
                    const int g = row_bytes / 32;
                    *seconds = ms / reps * 1e-3;
                    *rows = (double)grid * ((double)TMA_WARPS * issuers * 4 * tma_rounds + (double)(1024 - 32 * TMA_WARPS) / g * lsu_per_group);
                }
            }
        }
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (table) cudaFree(table);
    if (sink) cudaFree(sink);
    if (status) cudaFree(status);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Shared-memory / distributed-shared-memory gather probe (see sdnn_probe_smem_gather_rate in the header).
namespace {

template <int G, bool REMOTE>
int run_smem_probe(int cluster, int rows_log2, int cluster_log2, size_t smem, float* sink, cudaStream_t st, cudaEvent_t a, cudaEvent_t b,
                   int sms, double* rows_per_second, int* ctas_out) {
    auto kernel = smem_gather_probe_kernel<G, REMOTE>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess && cluster > 8) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaFuncSetAttribute(smem probe)");
    cudaLaunchConfig_t lc = {};
    lc.blockDim = dim3(1024); lc.dynamicSmemBytes = smem; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    int clusters = sms / cluster;
    if (cluster > 1) {      // how many clusters of this size the device holds at once
        lc.gridDim = dim3(cluster);
        int fit = 0;
        e = cudaOccupancyMaxActiveClusters(&fit, kernel, &lc);
        if (e != cudaSuccess || fit < 1) { cudaGetLastError(); return fail(nullptr, SDNN_ERR_CUDA, "clusters of %d CTAs with %zu bytes of shared memory do not fit this device", cluster, smem); }
        clusters = std::min(clusters, fit);
    }
    const int grid = clusters * cluster;
    lc.gridDim = dim3(grid);
    const int64_t groups = (int64_t)grid * 1024 / G;
    const int per_group = 4096;
    float* snk = sink;
    unsigned rl = (unsigned)rows_log2, cl = (unsigned)cluster_log2;
    for (int i = 0; i < 2; ++i) { unsigned seed = 17u + i; e = cudaLaunchKernelEx(&lc, kernel, snk, rl, cl, per_group, seed); if (e != cudaSuccess) return cuda_fail(nullptr, e, "smem probe launch"); }
    cudaEventRecord(a, st);
    const int reps = 5;
    for (int i = 0; i < reps; ++i) { unsigned seed = 101u + i; cudaLaunchKernelEx(&lc, kernel, snk, rl, cl, per_group, seed); }
    cudaEventRecord(b, st);
    e = cudaEventSynchronize(b);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "smem probe");
    float ms = 0.f;
    cudaEventElapsedTime(&ms, a, b);
    if (!(ms > 0.f)) return fail(nullptr, SDNN_ERR_CUDA, "smem probe: no time measured");
    *rows_per_second = (double)groups * per_group / (ms / reps * 1e-3);
    if (ctas_out) *ctas_out = grid;
    return SDNN_OK;
}

}  // namespace

extern "C" int sdnn_probe_smem_gather_rate(int32_t row_bytes, int32_t cluster_size, double* rows_per_second, int32_t* ctas_out) {
    if (!rows_per_second) return fail(nullptr, SDNN_ERR_INVALID_ARG, "rows_per_second is NULL");
    *rows_per_second = 0.0;
    if (row_bytes != 32 && row_bytes != 64 && row_bytes != 128 && row_bytes != 256)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "row_bytes must be 32, 64, 128 or 256");
    if (cluster_size != 1 && cluster_size != 2 && cluster_size != 4 && cluster_size != 8 && cluster_size != 16)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "cluster_size must be 1, 2, 4, 8 or 16");
    int dev = 0, sms = 0;
    CU(nullptr, cudaGetDevice(&dev));
    CU(nullptr, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const size_t smem = 128u << 10;                      // table bytes per CTA
    int rows_log2 = 0;
    while ((size_t)(2u << rows_log2) * row_bytes <= smem) ++rows_log2;
    int cluster_log2 = 0;
    while ((1 << cluster_log2) < cluster_size) ++cluster_log2;
    float* sink = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st = nullptr;
    int rc = SDNN_OK;
    if (cudaMalloc(&sink, 256) != cudaSuccess || cudaStreamCreate(&st) != cudaSuccess || cudaEventCreate(&a) != cudaSuccess ||
        cudaEventCreate(&b) != cudaSuccess) {
        cudaGetLastError();
        rc = fail(nullptr, SDNN_ERR_OOM, "could not set up the probe");
    } else {
        const bool remote = cluster_size > 1;
#define SDNN_SMEM_PROBE(G) (remote ? run_smem_probe<G, true>(cluster_size, rows_log2, cluster_log2, smem, sink, st, a, b, sms, rows_per_second, ctas_out) \
                                   : run_smem_probe<G, false>(1, rows_log2, 0, smem, sink, st, a, b, sms, rows_per_second, ctas_out))
        switch (row_bytes) {
            case 32: rc = SDNN_SMEM_PROBE(2); break;
            case 64: rc = SDNN_SMEM_PROBE(4); break;
            case 128: rc = SDNN_SMEM_PROBE(8); break;
            default: rc = SDNN_SMEM_PROBE(16); break;
        }
#undef SDNN_SMEM_PROBE
    }
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (st) cudaStreamDestroy(st);
    if (sink) cudaFree(sink);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free inference (see sdnn_infer_noalloc in the header).  The two activation tiles of
// the forward chain live in this file-scope device array instead of memory owned by a handle.
// In host code the array's name is only a stand-in for the symbol, not a device address: the
// address each device gave it is looked up once per device with cudaGetSymbolAddress.
namespace {

static __device__ __align__(256) float g_noalloc_scratch[2 * SDNN_NOALLOC_MAX_TILE_FLOATS];
static __device__ unsigned long long g_noalloc_bad_columns;      // out-of-range column indices met so far (never followed)

// tile geometry of this entry point (plain CSR kernel: 4 batch entries per lane, chunks of 128 columns)
int noalloc_padded_width(int b) {
    if (b <= 4) return 4;
    if (b <= 128) { int w = 4; while (w < b) w <<= 1; return w; }
    return (b + 127) / 128 * 128;
}

constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices] = {};      // per device: address of g_noalloc_scratch on that device
unsigned long long* g_noalloc_bad_ptr[kMaxDevices] = {};

int noalloc_scratch(float** out, unsigned long long** bad_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, SDNN_ERR_INVALID_ARG, "device ordinal %d not supported", dev);
    float* p = g_noalloc_ptr[dev];
    if (!p) {
#pragma omp critical(sdnn_noalloc_setup)
        {
            p = g_noalloc_ptr[dev];
            if (!p) {
                unsigned long long* bad = nullptr;
                e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
                if (e == cudaSuccess) e = cudaGetSymbolAddress(reinterpret_cast<void**>(&bad), g_noalloc_bad_columns);
                if (e == cudaSuccess) { g_noalloc_bad_ptr[dev] = bad; g_noalloc_ptr[dev] = p; } else p = nullptr;
            }
        }
        if (!p) return cuda_fail(nullptr, e, "cudaGetSymbolAddress(scratch)");
    }
    *out = p;
    *bad_out = g_noalloc_bad_ptr[dev];
    return SDNN_OK;
}

template <int G>
void noalloc_forward_g(cudaStream_t st, const int* rp, const int* col, const float* val, const float* bias,
                       const float* xin, float* xout, int n, int ld, int chunks, float clamp, unsigned long long* bad) {
    const int rows_per_block = 8 * (32 / G);
    dim3 grid((n + rows_per_block - 1) / rows_per_block, chunks);
    forward_csr_kernel<G><<<grid, 256, 0, st>>>(rp, col, val, bias, xin, xout, n, ld, clamp, bad);
}

}  // namespace

extern "C" int sdnn_infer_noalloc(int32_t n_layers, int32_t n_neurons, const int32_t* row_ptr, const int32_t* col_idx,
                                  const float* values, const int64_t* layer_offset, const float* bias,
                                  const float* x0, int32_t n_inputs, float* y_out, float clamp, void* cuda_stream) {
    if (n_layers < 1 || n_neurons < 1 || n_inputs < 0) return fail(nullptr, SDNN_ERR_INVALID_ARG, "sizes must be positive");
    if (!row_ptr || !col_idx || !values || !layer_offset || !bias) return fail(nullptr, SDNN_ERR_INVALID_ARG, "NULL network array");
    if (!(clamp > 0.0f) || !std::isfinite(clamp)) return fail(nullptr, SDNN_ERR_INVALID_ARG, "clamp must be finite and > 0");
    if (n_inputs == 0) return SDNN_OK;
    if (!x0 || !y_out) return fail(nullptr, SDNN_ERR_INVALID_ARG, "x0 or y_out is NULL");
    // checked before the batch is rounded up to the tile width, which would not fit 32 bits for batches near 2^31
    if (n_inputs > SDNN_NOALLOC_MAX_TILE_FLOATS)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "problem too large for the built-in scratch: %d inputs, a tile holds %d floats",
                    n_inputs, (int)SDNN_NOALLOC_MAX_TILE_FLOATS);
    const int ld = noalloc_padded_width(n_inputs);
    if (ld <= 0 || (int64_t)n_neurons * ld > (int64_t)SDNN_NOALLOC_MAX_TILE_FLOATS)
        return fail(nullptr, SDNN_ERR_INVALID_ARG,
                    "problem too large for the built-in scratch: n_neurons * padded(n_inputs) = %lld floats, limit %d",
                    (long long)n_neurons * ld, (int)SDNN_NOALLOC_MAX_TILE_FLOATS);
    if ((reinterpret_cast<uintptr_t>(col_idx) | reinterpret_cast<uintptr_t>(values)) & 15)
        return fail(nullptr, SDNN_ERR_INVALID_ARG, "col_idx and values must be 16-byte aligned");
    for (int l = 0; l < n_layers; ++l)
        if (layer_offset[l] < 0 || (layer_offset[l] & 3)) return fail(nullptr, SDNN_ERR_INVALID_ARG, "layer_offset[%d] must be a non-negative multiple of 4", l);

    float* scratch = nullptr;
    unsigned long long* bad = nullptr;
    int rc = noalloc_scratch(&scratch, &bad);
    if (rc) return rc;
    float* tile[2] = {scratch, scratch + SDNN_NOALLOC_MAX_TILE_FLOATS};
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const struct { int g, chunks; } q = {ld <= 128 ? ld / 4 : 32, ld <= 128 ? 1 : ld / 128};
    {
        dim3 grid((n_neurons + 31) / 32, (ld + 31) / 32), block(32, 8);
        transpose_in_kernel<<<grid, block, 0, st>>>(x0, tile[0], n_neurons, n_inputs, ld, ld, nullptr);
    }
    int cur = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int* rp = row_ptr + (size_t)l * (n_neurons + 1);
        const int* col = col_idx + layer_offset[l];
        const float* val = values + layer_offset[l];
        const float* b = bias + (size_t)l * n_neurons;
        switch (q.g) {
            case 1: noalloc_forward_g<1>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
            case 2: noalloc_forward_g<2>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
            case 4: noalloc_forward_g<4>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
            case 8: noalloc_forward_g<8>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
            case 16: noalloc_forward_g<16>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
            default: noalloc_forward_g<32>(st, rp, col, val, b, tile[cur], tile[cur ^ 1], n_neurons, ld, q.chunks, clamp, bad); break;
        }
        cur ^= 1;
    }
    {
        dim3 grid((n_neurons + 31) / 32, (n_inputs + 31) / 32), block(32, 8);
        transpose_out_kernel<<<grid, block, 0, st>>>(tile[cur], y_out, n_neurons, n_inputs, ld);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "kernel launch");
    return SDNN_OK;
}

extern "C" int sdnn_infer_noalloc_bad_columns(int64_t* count_out) {
    if (!count_out) return fail(nullptr, SDNN_ERR_INVALID_ARG, "count_out is NULL");
    unsigned long long v = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_noalloc_bad_columns, sizeof v);      // waits for the work enqueued so far
    if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaMemcpyFromSymbol");
    *count_out = (int64_t)v;
    return SDNN_OK;
}
