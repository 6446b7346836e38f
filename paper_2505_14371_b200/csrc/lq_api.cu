// Host side of liblq: the plan object and the extern "C" entry points declared in lq.h.
// No kernel lives here; this file validates arguments, owns the plan's device tables and
// enqueues the launchers of the other translation units on the caller's stream.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "lq_coding.cuh"

using namespace lq;

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

}  // namespace

// Records a failure reason for lq_last_error() from another translation unit of the library.
int lq::lq_set_error(int code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

namespace {

// Vector loads, stores and asynchronous copies need 16-byte aligned rows (D_pad is a multiple of 32 elements,
// so an aligned base keeps every row and layer aligned); message words and norms are read as 32-bit values.
bool misaligned(const void* p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) != 0; }
#define LQ_ALIGNED(ptr, a)                                                                   \
    do {                                                                                      \
        if (misaligned(ptr, a)) return fail(LQ_EINVAL, #ptr " must be %d-byte aligned", (int)(a)); \
    } while (0)

#define LQ_CUDA(expr)                                                                         \
    do {                                                                                      \
        cudaError_t e_ = (expr);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail(e_ == cudaErrorMemoryAllocation ? LQ_ENOMEM : LQ_ECUDA, "%s: %s", #expr, \
                        cudaGetErrorString(e_));                                              \
    } while (0)

}  // namespace

// The three level tables: `stage` receives lq_set_levels / lq_fit_levels; at the next
// lq_quantize_pack a changed stage is copied into the encode table that is not in use, which
// becomes current, while the other keeps the levels of the previous message.
struct lq_plan {
    PlanDev dev{};
    std::vector<LayerDesc> layers;
    std::vector<Tile> tiles;
    int device = 0;
    uint64_t seed = 0;
    LayerDesc* d_layers = nullptr;
    Tile* d_tiles = nullptr;
    TileJob* d_jobs = nullptr;
    float* d_levels_stage = nullptr;
    float* d_levels_enc[2] = {nullptr, nullptr};
    SearchTables search{};         // derived from d_levels_enc[cur]
    int cur = 0, prev = 0;
    bool stage_dirty = false;
    bool have_message = false;
    bool qoda_ready = false;
    bool stat_pending = false;
    int32_t* d_member_off = nullptr;       // [L + 1] and [L]: the member lists of lq_fit_levels_shared
    int32_t* d_member_layer = nullptr;
    std::vector<int32_t> h_members;        // host staging of both lists (kept alive for the asynchronous copy)
    uint32_t* d_code_enc = nullptr;        // [L][256]   entropy stage, allocated at its first use
    uint16_t* d_code_dec = nullptr;        // [L][kDecEntries]
    uint32_t* d_code_bad = nullptr;        // [1] set by a decode that met an invalid stream
    EncodeScratch code_scratch{nullptr, nullptr};   // allocated with the tables
    std::vector<uint8_t> code_len;         // [L][256] host copy of the word lengths
    double alt_qhat = 0.0;         // > 0: qoda_step follows Eq. (Alt) with this exponent
    double* xsum = nullptr;        // caller-owned running sum of the half iterates (qoda_set_average), or NULL
    const uint32_t* last_packed = nullptr;   // where the last lq_quantize_pack wrote its message
    uint8_t* d_row_mask[2] = {nullptr, nullptr};   // zero-row masks of the last two encoded inputs
    int mask_cur = 0;
    bool masks_known = false;              // d_row_mask[mask_cur] describes the last message of the current worker range
    bool message_intact = false;           // ... and the caller has not said that it rewrote that message (lq_message_modified)
    // optional per-kernel timing (lq_profile_enable): event pairs recorded around each launch
    struct ProfRec { int id; cudaEvent_t a, b; };
    bool profiling = false;
    std::vector<ProfRec> prof_recs;
    std::vector<cudaEvent_t> prof_pool;
};

namespace {

void free_plan(lq_plan* p)
{
    if (!p) return;
    cudaFree(p->d_layers); cudaFree(p->d_tiles); cudaFree(p->d_jobs);
    cudaFree(p->d_levels_stage); cudaFree(p->d_levels_enc[0]); cudaFree(p->d_levels_enc[1]);
    cudaFree(p->search.lut); cudaFree(p->search.ld); cudaFree(p->search.fast);
    cudaFree(p->dev.norm_partial); cudaFree(p->dev.stat_partial); cudaFree(p->dev.sq_diff);
    cudaFree(p->dev.rnorm); cudaFree(p->dev.status); cudaFree(p->dev.scalars); cudaFree(p->d_code_enc); cudaFree(p->d_code_dec); cudaFree(p->d_code_bad); cudaFree(p->code_scratch.lane_bits); cudaFree(p->code_scratch.scan_part); cudaFree(p->d_member_off); cudaFree(p->d_member_layer); cudaFree(p->dev.alt_partial); cudaFree(p->dev.layer_total); cudaFree(p->d_row_mask[0]); cudaFree(p->d_row_mask[1]);
    cudaFree(p->dev.block_live);
    cudaFree(p->dev.energy_partial); cudaFree(p->dev.flag_partial); cudaFree(p->dev.layer_weight);
    for (auto& r : p->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (auto e : p->prof_pool) cudaEventDestroy(e);
    delete p;
}

cudaEvent_t prof_event(lq_plan* p)
{
    cudaEvent_t e = nullptr;
    if (!p->prof_pool.empty()) { e = p->prof_pool.back(); p->prof_pool.pop_back(); }
    else if (cudaEventCreate(&e) != cudaSuccess) e = nullptr;
    return e;
}

// Runs one launcher; when profiling is on, brackets it with two events on the same stream.
template <typename F>
cudaError_t timed(lq_plan* p, int id, cudaStream_t s, F&& launch)
{
    if (!p->profiling || p->prof_recs.size() >= 65536) return launch();
    cudaEvent_t a = prof_event(p), b = prof_event(p);
    if (!a || !b) return launch();
    cudaEventRecord(a, s);
    const cudaError_t e = launch();
    cudaEventRecord(b, s);
    p->prof_recs.push_back({id, a, b});
    return e;
}

// Per block the bitmask of workers that sent anything, if `packed` is the message the plan's last lq_quantize_pack
// wrote for all K <= 32 workers in the layer or global scope (the decoder then leaves all-zero blocks unread);
// otherwise nullptr.
const uint32_t* message_masks(const lq_plan* p, const uint32_t* packed)
{
    const PlanDev& d = p->dev;
    if (!p->have_message || !p->masks_known || !p->message_intact || d.bucket_norm || packed != p->last_packed) return nullptr;
    if (d.worker0 != 0 || d.worker_count != d.num_workers || d.num_workers > 32) return nullptr;
    return d.block_live;
}

template <typename T>
cudaError_t dev_alloc_zero(T** ptr, size_t count)
{
    const size_t bytes = (count ? count : 1) * sizeof(T);
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(ptr), bytes);
    if (e != cudaSuccess) { *ptr = nullptr; return e; }
    return cudaMemset(*ptr, 0, bytes);
}

}  // namespace

extern "C" {

const char* lq_last_error(void) { return g_err; }

const char* lq_error_string(int code)
{
    switch (code) {
        case LQ_OK: return "ok";
        case LQ_EINVAL: return "invalid argument";
        case LQ_ENOMEM: return "out of memory";
        case LQ_ECUDA: return "CUDA runtime error";
        case LQ_ESTATE: return "call out of order";
        default: return "unknown error";
    }
}

int lq_plan_create(lq_plan** out, int32_t num_layers, const int64_t* layer_sizes, const int32_t* bits,
                   int32_t q, int32_t num_workers, uint64_t seed)
{
    if (!out) return fail(LQ_EINVAL, "out is NULL");
    *out = nullptr;
    if (num_layers < 0 || (num_layers > 0 && (!layer_sizes || !bits)))
        return fail(LQ_EINVAL, "num_layers < 0 or NULL layer arrays");
    if (q < 0 || q > 16) return fail(LQ_EINVAL, "q must be 0 (infinity norm) or 1..16, got %d", q);
    if (num_workers < 1 || num_workers > LQ_MAX_WORKERS)
        return fail(LQ_EINVAL, "num_workers must be in [1, %d], got %d", LQ_MAX_WORKERS, num_workers);

    lq_plan* p = new (std::nothrow) lq_plan;
    if (!p) return fail(LQ_ENOMEM, "host allocation failed");
    int64_t elem = 0, word = 0, ntiles = 0, blocks = 0;
    // tile size: as large as possible while (tiles x workers) still fills the GPU several times over
    int tile_blocks = kTileBlocks;
    {
        int64_t total = 0;
        for (int m = 0; m < num_layers; ++m)
            if (layer_sizes[m] > 0) total += (layer_sizes[m] + kBlockCoords - 1) / kBlockCoords;
        while (tile_blocks > kSubBlocks && (total / tile_blocks) * num_workers < 4096) tile_blocks /= 2;
    }
    try {
        p->layers.resize((size_t)num_layers);
        for (int m = 0; m < num_layers; ++m) {
            const int64_t d = layer_sizes[m];
            const int b = bits[m];
            if (d < 0 || d >= ((int64_t)1 << 31)) { delete p; return fail(LQ_EINVAL, "layer %d: size %lld out of [0, 2^31)", m, (long long)d); }
            if (b < 1 || b > LQ_MAX_BITS) { delete p; return fail(LQ_EINVAL, "layer %d: bits %d out of [1, %d]", m, b, LQ_MAX_BITS); }
            LayerDesc& L = p->layers[(size_t)m];
            L.elem_off = elem; L.word_off = word; L.size = d; L.bits = b; L.nlevels = 1 << b;
            L.nblocks = (int32_t)((d + kBlockCoords - 1) / kBlockCoords);
            L.first_tile = (int32_t)ntiles;
            L.ntiles = (L.nblocks + tile_blocks - 1) / tile_blocks;
            L.pad_ = 0;
            L.block_off = blocks;
            blocks += L.nblocks;
            for (int t = 0; t < L.ntiles; ++t) {
                Tile tl;
                tl.layer = m; tl.block0 = t * tile_blocks;
                tl.nblocks = L.nblocks - tl.block0 < tile_blocks ? L.nblocks - tl.block0 : tile_blocks;
                tl.pad_ = 0;
                p->tiles.push_back(tl);
            }
            ntiles += L.ntiles;
            if (ntiles >= ((int64_t)1 << 29)) { delete p; return fail(LQ_EINVAL, "too many tiles"); }
            elem += (d + 31) / 32 * 32;
            word += (int64_t)L.nblocks * 32 * (b + 1);
        }
    } catch (const std::bad_alloc&) {
        delete p;
        return fail(LQ_ENOMEM, "host allocation failed");
    }
    if (elem == 0) elem = 32;
    p->seed = seed;
    PlanDev& d = p->dev;
    d.num_layers = num_layers; d.num_tiles = (int32_t)ntiles; d.num_workers = num_workers; d.q = q;
    d.worker0 = 0; d.worker_count = num_workers;
    d.sub_tiles = tile_blocks / kSubBlocks;
    d.sub_shift = 0;
    while ((1 << d.sub_shift) < d.sub_tiles) ++d.sub_shift;
    d.padded_elems = elem; d.packed_words = word; d.total_blocks = blocks;
    d.seed_lo = (uint32_t)seed; d.seed_hi = (uint32_t)(seed >> 32);
    for (int r = 0; r < 8; ++r) {
        d.rk0[r] = d.seed_lo + (uint32_t)(r + 2) * 0x9E3779B9u;
        d.rk1[r] = d.seed_hi + (uint32_t)(r + 2) * 0xBB67AE85u;
    }

    cudaError_t e = cudaGetDevice(&p->device);
    const size_t KL = (size_t)num_workers * (size_t)(num_layers ? num_layers : 1);
    const size_t KT = (size_t)num_workers * (size_t)(ntiles ? ntiles : 1);
    const size_t lev = (size_t)(num_layers ? num_layers : 1) * kLevelStride;
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_layers, p->layers.size());
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_tiles, p->tiles.size());
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_jobs, p->tiles.size());
    if (e == cudaSuccess && !p->tiles.empty()) {
        // the encoder's launch order: tiles sorted by their relative position inside their layer, so that every
        // layer is under way from the first wave of CTAs to the last
        std::vector<int32_t> order;
        try { order.resize(p->tiles.size()); } catch (const std::bad_alloc&) { free_plan(p); return fail(LQ_ENOMEM, "host allocation failed"); }
        for (size_t i = 0; i < order.size(); ++i) order[i] = (int32_t)i;
        const std::vector<LayerDesc>& Ls = p->layers;
        const std::vector<Tile>& Ts = p->tiles;
        std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
            const LayerDesc& La = Ls[(size_t)Ts[(size_t)a].layer];
            const LayerDesc& Lb = Ls[(size_t)Ts[(size_t)b].layer];
            // (2 i + 1) / (2 n) compared exactly by cross-multiplication
            const int64_t ka = (2 * (int64_t)(a - La.first_tile) + 1) * Lb.ntiles;
            const int64_t kb = (2 * (int64_t)(b - Lb.first_tile) + 1) * La.ntiles;
            return ka != kb ? ka < kb : a < b;
        });
        std::vector<TileJob> jobs;
        try { jobs.resize(order.size()); } catch (const std::bad_alloc&) { free_plan(p); return fail(LQ_ENOMEM, "host allocation failed"); }
        for (size_t i = 0; i < order.size(); ++i) {
            const Tile& T = Ts[(size_t)order[i]];
            const LayerDesc& L = Ls[(size_t)T.layer];
            TileJob& J = jobs[i];
            J.tile = order[i]; J.layer = T.layer; J.block0 = T.block0; J.nblocks = T.nblocks; J.bits = L.bits; J.pad_ = 0;
            J.size = L.size; J.elem_off = L.elem_off; J.word_off = L.word_off; J.block_off = L.block_off; J.pad2_ = 0;
        }
        e = cudaMemcpy(p->d_jobs, jobs.data(), jobs.size() * sizeof(TileJob), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_levels_stage, lev);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_levels_enc[0], lev);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_levels_enc[1], lev);
    const size_t nl = (size_t)(num_layers ? num_layers : 1);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->search.lut, nl * kLutEntries);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->search.ld, nl * kMaxLevels);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->search.fast, nl);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.norm_partial, KT * (size_t)d.sub_tiles);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.stat_partial, KT);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.sq_diff, KL);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.rnorm, KL);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.status, KL);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.layer_total, KL);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.block_live, (size_t)(blocks ? blocks : 1));
    if (e == cudaSuccess) e = dev_alloc_zero(&d.energy_partial, KT);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.flag_partial, KT);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.layer_weight, KL);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_member_off, nl + 1);
    if (e == cudaSuccess) e = dev_alloc_zero(&p->d_member_layer, nl);
    if (e == cudaSuccess) e = dev_alloc_zero(&d.alt_partial, 2 * (size_t)(ntiles ? ntiles : 1) * (size_t)d.sub_tiles);
    for (int i = 0; i < 2; ++i)
        if (e == cudaSuccess) e = dev_alloc_zero(&p->d_row_mask[i], (size_t)num_workers * (size_t)(blocks ? blocks : 1));
    d.row_mask = p->d_row_mask[0]; d.row_mask_prev = nullptr;
    if (e == cudaSuccess) e = dev_alloc_zero(&d.scalars, 1);
    if (e == cudaSuccess && !p->layers.empty())
        e = cudaMemcpy(p->d_layers, p->layers.data(), p->layers.size() * sizeof(LayerDesc), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !p->tiles.empty())
        e = cudaMemcpy(p->d_tiles, p->tiles.data(), p->tiles.size() * sizeof(Tile), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        // uniform levels j / (2^b - 1), rounded once from fp64
        std::vector<float> host(lev, 0.0f);
        for (int m = 0; m < num_layers; ++m) {
            const int n = p->layers[(size_t)m].nlevels;
            for (int j = 0; j < n; ++j)
                host[(size_t)m * kLevelStride + j] = (float)((double)j / (double)(n - 1));
        }
        for (float* t : {p->d_levels_stage, p->d_levels_enc[0], p->d_levels_enc[1]})
            if (e == cudaSuccess) e = cudaMemcpy(t, host.data(), lev * sizeof(float), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) {
        QodaScalars s0{};
        s0.t = 1; s0.eta = 1.0f; s0.gamma = 1.0f; s0.eta_cur = 1.0f;
        e = cudaMemcpy(d.scalars, &s0, sizeof s0, cudaMemcpyHostToDevice);
    }
    if (e != cudaSuccess) {
        const int code = e == cudaErrorMemoryAllocation ? LQ_ENOMEM : LQ_ECUDA;
        free_plan(p);
        return fail(code, "plan setup: %s", cudaGetErrorString(e));
    }
    d.layers = p->d_layers; d.tiles = p->d_tiles; d.jobs = p->d_jobs;
    e = launch_build_search(d, p->d_levels_enc[0], p->search, nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free_plan(p);
        return fail(LQ_ECUDA, "plan setup: %s", cudaGetErrorString(e));
    }
    *out = p;
    return LQ_OK;
}

int lq_plan_destroy(lq_plan* plan)
{
    if (!plan) return LQ_OK;
    cudaDeviceSynchronize();
    free_plan(plan);
    return LQ_OK;
}

int64_t lq_plan_padded_elems(const lq_plan* plan) { return plan ? plan->dev.padded_elems : (int64_t)fail(LQ_EINVAL, "plan is NULL"); }
int64_t lq_plan_packed_words(const lq_plan* plan) { return plan ? plan->dev.packed_words : (int64_t)fail(LQ_EINVAL, "plan is NULL"); }

int lq_plan_layer_info(const lq_plan* plan, int32_t layer, int64_t* elem_off, int64_t* word_off, int32_t* num_levels)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    if (layer < 0 || layer >= plan->dev.num_layers) return fail(LQ_EINVAL, "layer %d out of range", layer);
    const LayerDesc& L = plan->layers[(size_t)layer];
    if (elem_off) *elem_off = L.elem_off;
    if (word_off) *word_off = L.word_off;
    if (num_levels) *num_levels = L.nlevels;
    return LQ_OK;
}

int lq_set_levels(lq_plan* plan, int32_t layer, const float* host_levels, int32_t n)
{
    if (!plan || !host_levels) return fail(LQ_EINVAL, "NULL argument");
    if (layer < 0 || layer >= plan->dev.num_layers) return fail(LQ_EINVAL, "layer %d out of range", layer);
    const LayerDesc& L = plan->layers[(size_t)layer];
    if (n != L.nlevels) return fail(LQ_EINVAL, "layer %d has %d levels, got %d", layer, L.nlevels, n);
    if (host_levels[0] != 0.0f || host_levels[n - 1] != 1.0f)
        return fail(LQ_EINVAL, "levels must start at 0 and end at 1");
    for (int j = 1; j < n; ++j) {
        // gaps below 2^-100 are refused: they could not be told apart from rounding noise anyway
        if (!(host_levels[j] - host_levels[j - 1] >= 7.888609052210118e-31f))
            return fail(LQ_EINVAL, "levels must be strictly increasing (index %d)", j);
    }
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(plan->d_levels_stage + (size_t)layer * kLevelStride, host_levels,
                       (size_t)n * sizeof(float), cudaMemcpyHostToDevice));
    plan->stage_dirty = true;
    return LQ_OK;
}

int lq_get_levels(const lq_plan* plan, int32_t layer, float* host_levels, int32_t n)
{
    if (!plan || !host_levels) return fail(LQ_EINVAL, "NULL argument");
    if (layer < 0 || layer >= plan->dev.num_layers) return fail(LQ_EINVAL, "layer %d out of range", layer);
    const LayerDesc& L = plan->layers[(size_t)layer];
    if (n != L.nlevels) return fail(LQ_EINVAL, "layer %d has %d levels, got %d", layer, L.nlevels, n);
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(host_levels, plan->d_levels_stage + (size_t)layer * kLevelStride,
                       (size_t)n * sizeof(float), cudaMemcpyDeviceToHost));
    return LQ_OK;
}

int lq_layer_norms(lq_plan* plan, const float* grads, float* norms, void* stream)
{
    if (!plan || !grads || !norms) return fail(LQ_EINVAL, "NULL argument");
    LQ_ALIGNED(grads, 16); LQ_ALIGNED(norms, 4);
    if (plan->dev.bucket_norm)
        return fail(LQ_EINVAL, "lq_layer_norms: in bucket scope the norms are written by lq_quantize_pack");
    if (plan->dev.num_layers == 0) return LQ_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const PlanDev& d = plan->dev;
    LQ_CUDA(timed(plan, LQ_KERNEL_NORM_PARTIAL, s, [&] { return launch_norm_partial(d, grads, false, s); }));
    LQ_CUDA(timed(plan, LQ_KERNEL_NORM_FINALIZE, s, [&] { return launch_norm_finalize(d, norms, s); }));
    return LQ_OK;
}

int lq_quantize_pack(lq_plan* plan, const float* grads, uint32_t step, uint32_t* packed, float* norms,
                     uint32_t* hist, const uint32_t* prev_packed, const float* prev_norms, void* stream)
{
    if (!plan || !grads || !packed || !norms) return fail(LQ_EINVAL, "NULL argument");
    if ((prev_packed == nullptr) != (prev_norms == nullptr))
        return fail(LQ_EINVAL, "prev_packed and prev_norms must both be given or both be NULL");
    if (prev_packed == packed) return fail(LQ_EINVAL, "prev_packed must not alias packed");
    if (prev_packed && plan->have_message && !plan->masks_known)
        return fail(LQ_ESTATE, "the worker range changed since the plan's last message: the first message of the new "
                    "range has no previous message (pass prev_packed = NULL)");
    LQ_ALIGNED(grads, 16); LQ_ALIGNED(packed, 4); LQ_ALIGNED(norms, 4); LQ_ALIGNED(hist, 4);
    LQ_ALIGNED(prev_packed, 4); LQ_ALIGNED(prev_norms, 4);
    if (plan->dev.num_layers == 0) return LQ_OK;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t lev_bytes = (size_t)plan->dev.num_layers * kLevelStride * sizeof(float);
    if (plan->stage_dirty) {
        const int next = plan->have_message ? 1 - plan->cur : plan->cur;
        LQ_CUDA(cudaMemcpyAsync(plan->d_levels_enc[next], plan->d_levels_stage, lev_bytes,
                                cudaMemcpyDeviceToDevice, s));
        plan->prev = plan->cur;
        plan->cur = next;
        plan->stage_dirty = false;
        LQ_CUDA(launch_build_search(plan->dev, plan->d_levels_enc[next], plan->search, s));
    } else {
        plan->prev = plan->cur;
    }
    // the masks written now describe this message; the ones of the last call describe prev_packed
    // (they describe prev_packed only if that is the very message the last call wrote, untouched since; for any
    // other previous message every row is taken as possibly nonzero)
    plan->dev.row_mask_prev = (plan->have_message && plan->masks_known && plan->message_intact && prev_packed == plan->last_packed)
                                  ? plan->d_row_mask[plan->mask_cur] : nullptr;
    plan->mask_cur = plan->have_message ? 1 - plan->mask_cur : plan->mask_cur;
    plan->dev.row_mask = plan->d_row_mask[plan->mask_cur];
    const PlanDev& d = plan->dev;
    const float* lc = plan->d_levels_enc[plan->cur];
    const float* lp = plan->d_levels_enc[plan->prev];
    if (d.bucket_norm) {                 // one pass: the norms come out of the encoder itself
        LQ_CUDA(timed(plan, LQ_KERNEL_QUANTIZE_PACK, s, [&] {
            return launch_quantize_bucketed(d, grads, step, packed, norms, hist, prev_packed, prev_norms, lc, lp,
                                            plan->search, s);
        }));
        LQ_CUDA(timed(plan, LQ_KERNEL_STAT_FINALIZE, s, [&] { return launch_bucket_finalize(d, s); }));
        plan->have_message = true;
        plan->masks_known = true;          // (no masks in this scope: the flag also marks an unbroken stream of messages)
        plan->message_intact = true;
        plan->stat_pending = true;
        return LQ_OK;
    }
    LQ_CUDA(timed(plan, LQ_KERNEL_NORM_PARTIAL, s, [&] { return launch_norm_partial(d, grads, true, s); }));
    LQ_CUDA(timed(plan, LQ_KERNEL_NORM_FINALIZE, s, [&] { return launch_norm_finalize(d, norms, s); }));
    LQ_CUDA(timed(plan, LQ_KERNEL_QUANTIZE_PACK, s, [&] {
        // under Eq. (Alt) nothing consumes the statistic of Eq. (general_stepsize): it is left out (and reads 0)
        return launch_quantize(d, grads, step, packed, norms, hist, prev_packed, prev_norms, lc, lp,
                               plan->search, plan->alt_qhat <= 0.0, s);
    }));
    LQ_CUDA(timed(plan, LQ_KERNEL_STAT_FINALIZE, s, [&] { return launch_stat_finalize(d, s); }));
    plan->have_message = true;
    plan->masks_known = true;
    plan->message_intact = true;
    plan->last_packed = packed;
    plan->stat_pending = true;
    return LQ_OK;
}

int lq_fit_levels(lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples, void* stream)
{
    if (!plan || !hist || !norms) return fail(LQ_EINVAL, "NULL argument");
    if (num_samples < 1 || num_samples > LQ_MAX_WORKERS)
        return fail(LQ_EINVAL, "num_samples must be in [1, %d]", LQ_MAX_WORKERS);
    cudaStream_t s = (cudaStream_t)stream;
    LQ_CUDA(timed(plan, LQ_KERNEL_FIT, s, [&] {
        return launch_fit(plan->dev, hist, plan->dev.bucket_norm ? plan->dev.layer_weight : norms, num_samples,
                          plan->d_levels_stage, s);
    }));
    plan->stage_dirty = true;
    return LQ_OK;
}

int lq_fit_levels_shared(lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples,
                         const int32_t* layer_type, void* stream)
{
    if (!plan || !hist || !norms || !layer_type) return fail(LQ_EINVAL, "NULL argument");
    if (num_samples < 1 || num_samples > LQ_MAX_WORKERS)
        return fail(LQ_EINVAL, "num_samples must be in [1, %d]", LQ_MAX_WORKERS);
    const int L = plan->dev.num_layers;
    if (L == 0) return LQ_OK;
    // member lists: layers grouped by type id, types in order of first appearance
    std::vector<int32_t> ids, off(1, 0), members;
    try {
        for (int m = 0; m < L; ++m) {
            bool seen = false;
            for (int32_t id : ids) if (id == layer_type[m]) { seen = true; break; }
            if (!seen) ids.push_back(layer_type[m]);
        }
        for (int32_t id : ids) {
            int first = -1;
            for (int m = 0; m < L; ++m) {
                if (layer_type[m] != id) continue;
                if (first < 0) first = m;
                else if (plan->layers[(size_t)m].nlevels != plan->layers[(size_t)first].nlevels)
                    return fail(LQ_EINVAL, "layers %d and %d share type %d but not their code width", first, m, id);
                members.push_back(m);
            }
            off.push_back((int32_t)members.size());
        }
        plan->h_members = off;
        plan->h_members.insert(plan->h_members.end(), members.begin(), members.end());
    } catch (const std::bad_alloc&) {
        return fail(LQ_ENOMEM, "host allocation failed");
    }
    cudaStream_t s = (cudaStream_t)stream;
    const int num_types = (int)ids.size();
    LQ_CUDA(cudaMemcpyAsync(plan->d_member_off, plan->h_members.data(), off.size() * sizeof(int32_t),
                            cudaMemcpyHostToDevice, s));
    LQ_CUDA(cudaMemcpyAsync(plan->d_member_layer, plan->h_members.data() + off.size(), members.size() * sizeof(int32_t),
                            cudaMemcpyHostToDevice, s));
    LQ_CUDA(timed(plan, LQ_KERNEL_FIT, s, [&] {
        return launch_fit_shared(plan->dev, hist, plan->dev.bucket_norm ? plan->dev.layer_weight : norms, num_samples,
                                 plan->d_levels_stage, plan->d_member_off,
                                 plan->d_member_layer, num_types, s);
    }));
    plan->stage_dirty = true;
    return LQ_OK;
}

int lq_decode_aggregate(const lq_plan* plan, const uint32_t* packed, const float* norms, float* gbar, void* stream)
{
    if (!plan || !packed || !norms || !gbar) return fail(LQ_EINVAL, "NULL argument");
    LQ_ALIGNED(packed, 4); LQ_ALIGNED(norms, 4); LQ_ALIGNED(gbar, 16);
    cudaStream_t s = (cudaStream_t)stream;
    lq_plan* mp = const_cast<lq_plan*>(plan);      // the profiler's bookkeeping is not plan state
    LQ_CUDA(timed(mp, LQ_KERNEL_DECODE, s, [&] {
        return launch_decode(plan->dev, packed, norms, plan->d_levels_enc[plan->cur], nullptr, nullptr,
                             nullptr, nullptr, gbar, 0, nullptr, s);
    }));
    return LQ_OK;
}

int qoda_init(lq_plan* plan, const float* X1, float* Y, float* Xhalf, void* stream)
{
    if (!plan || !X1 || !Y || !Xhalf) return fail(LQ_EINVAL, "NULL argument");
    LQ_ALIGNED(X1, 16); LQ_ALIGNED(Y, 16); LQ_ALIGNED(Xhalf, 16);
    LQ_CUDA(launch_qoda_init(plan->dev, X1, Y, Xhalf, (cudaStream_t)stream));
    if (plan->xsum)
        LQ_CUDA(cudaMemsetAsync(plan->xsum, 0, (size_t)plan->dev.padded_elems * sizeof(double), (cudaStream_t)stream));
    plan->qoda_ready = true;
    plan->stat_pending = false;
    return LQ_OK;
}

int qoda_step(lq_plan* plan, const uint32_t* packed, const float* norms, const float* X1, float* Y,
              float* Xhalf, float* X_opt, float* gbar_opt, void* stream)
{
    if (!plan || !packed || !norms || !X1 || !Y || !Xhalf) return fail(LQ_EINVAL, "NULL argument");
    LQ_ALIGNED(packed, 4); LQ_ALIGNED(norms, 4); LQ_ALIGNED(X1, 16); LQ_ALIGNED(Y, 16); LQ_ALIGNED(Xhalf, 16);
    LQ_ALIGNED(X_opt, 16); LQ_ALIGNED(gbar_opt, 16);
    if (!plan->qoda_ready) return fail(LQ_ESTATE, "qoda_step before qoda_init");
    if (!plan->stat_pending) return fail(LQ_ESTATE, "qoda_step needs a new lq_quantize_pack message");
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t* live = message_masks(plan, packed);
    if (live)                        // folds the K workers' zero-row masks into one word per block
        LQ_CUDA(timed(plan, LQ_KERNEL_BLOCK_LIVE, s, [&] { return launch_block_live(plan->dev, s); }));
    if (plan->xsum)                  // X_{t+1/2}, before this step overwrites it
        LQ_CUDA(timed(plan, LQ_KERNEL_AVERAGE, s, [&] { return launch_average(plan->dev, Xhalf, plan->xsum, s); }));
    if (plan->alt_qhat > 0.0) {
        const double qh = plan->alt_qhat;
        LQ_CUDA(timed(plan, LQ_KERNEL_QODA_SCALARS, s, [&] { return launch_alt_scalars(plan->dev, qh, s); }));
        LQ_CUDA(timed(plan, LQ_KERNEL_DECODE, s, [&] {
            return launch_decode(plan->dev, packed, norms, plan->d_levels_enc[plan->cur], X1, Y, Xhalf, X_opt,
                                 gbar_opt, 2, live, s);
        }));
        LQ_CUDA(timed(plan, LQ_KERNEL_ALT_FINALIZE, s, [&] { return launch_alt_finalize(plan->dev, s); }));
    } else {
        LQ_CUDA(timed(plan, LQ_KERNEL_QODA_SCALARS, s, [&] { return launch_qoda_scalars(plan->dev, s); }));
        LQ_CUDA(timed(plan, LQ_KERNEL_DECODE, s, [&] {
            return launch_decode(plan->dev, packed, norms, plan->d_levels_enc[plan->cur], X1, Y, Xhalf, X_opt,
                                 gbar_opt, 1, live, s);
        }));
    }
    plan->stat_pending = false;
    return LQ_OK;
}

int qoda_set_average(lq_plan* plan, double* xsum, void* stream)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    LQ_ALIGNED(xsum, 16);
    plan->xsum = xsum;
    if (xsum) LQ_CUDA(cudaMemsetAsync(xsum, 0, (size_t)plan->dev.padded_elems * sizeof(double), (cudaStream_t)stream));
    return LQ_OK;
}

int lq_set_norm_scope(lq_plan* plan, int32_t scope)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    if (scope != LQ_NORM_PER_LAYER && scope != LQ_NORM_GLOBAL && scope != LQ_NORM_BUCKET)
        return fail(LQ_EINVAL, "unknown norm scope %d", scope);
    const int bucket = scope == LQ_NORM_BUCKET ? 1 : 0;
    if (bucket != plan->dev.bucket_norm && plan->have_message)
        return fail(LQ_ESTATE, "the bucket scope can only be entered or left before the first lq_quantize_pack");
    plan->dev.global_norm = scope == LQ_NORM_GLOBAL ? 1 : 0;
    plan->dev.bucket_norm = bucket;
    return LQ_OK;
}

int lq_message_modified(lq_plan* plan)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    plan->message_intact = false;
    return LQ_OK;
}

int lq_set_worker_range(lq_plan* plan, int32_t first_worker, int32_t count)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    if (first_worker < 0 || count < 1 || first_worker > plan->dev.num_workers - count)
        return fail(LQ_EINVAL, "worker range [%d, %d) is not inside [0, %d)", first_worker, first_worker + count,
                    plan->dev.num_workers);
    if (first_worker != plan->dev.worker0 || count != plan->dev.worker_count)
        plan->masks_known = false;         // the stored zero-row masks describe another set of workers' last input
    plan->dev.worker0 = first_worker;
    plan->dev.worker_count = count;
    return LQ_OK;
}

int lq_side_data_export(const lq_plan* plan, double* sq_diff, float* layer_weight, uint32_t* flags, void* stream)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    LQ_ALIGNED(sq_diff, 8); LQ_ALIGNED(layer_weight, 4); LQ_ALIGNED(flags, 4);
    const size_t KL = (size_t)plan->dev.num_workers * (size_t)plan->dev.num_layers;
    cudaStream_t s = (cudaStream_t)stream;
    if (sq_diff) LQ_CUDA(cudaMemcpyAsync(sq_diff, plan->dev.sq_diff, KL * sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (layer_weight) LQ_CUDA(cudaMemcpyAsync(layer_weight, plan->dev.layer_weight, KL * sizeof(float), cudaMemcpyDeviceToDevice, s));
    if (flags) LQ_CUDA(cudaMemcpyAsync(flags, plan->dev.status, KL * sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    return LQ_OK;
}

int lq_side_data_import(lq_plan* plan, const double* sq_diff, const float* layer_weight, const uint32_t* flags, void* stream)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    LQ_ALIGNED(sq_diff, 8); LQ_ALIGNED(layer_weight, 4); LQ_ALIGNED(flags, 4);
    const size_t KL = (size_t)plan->dev.num_workers * (size_t)plan->dev.num_layers;
    cudaStream_t s = (cudaStream_t)stream;
    if (sq_diff) LQ_CUDA(cudaMemcpyAsync(plan->dev.sq_diff, sq_diff, KL * sizeof(double), cudaMemcpyDeviceToDevice, s));
    if (layer_weight) LQ_CUDA(cudaMemcpyAsync(plan->dev.layer_weight, layer_weight, KL * sizeof(float), cudaMemcpyDeviceToDevice, s));
    if (flags) LQ_CUDA(cudaMemcpyAsync(plan->dev.status, flags, KL * sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    return LQ_OK;
}

int64_t lq_plan_norm_count(const lq_plan* plan)
{
    if (!plan) return (int64_t)fail(LQ_EINVAL, "plan is NULL");
    return plan->dev.bucket_norm ? plan->dev.total_blocks * 8 : (int64_t)plan->dev.num_layers;
}

int lq_layer_weights(const lq_plan* plan, float* host_weights)
{
    if (!plan || !host_weights) return fail(LQ_EINVAL, "NULL argument");
    if (!plan->dev.bucket_norm) return fail(LQ_ESTATE, "lq_layer_weights: the plan is not in bucket scope");
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(host_weights, plan->dev.layer_weight,
                       (size_t)plan->dev.num_workers * (size_t)plan->dev.num_layers * sizeof(float), cudaMemcpyDeviceToHost));
    return LQ_OK;
}

int lq_level_probabilities(const lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples,
                           int32_t staged, double* probs, void* stream)
{
    if (!plan || !hist || !norms || !probs) return fail(LQ_EINVAL, "NULL argument");
    if (num_samples < 1 || num_samples > LQ_MAX_WORKERS)
        return fail(LQ_EINVAL, "num_samples must be in [1, %d]", LQ_MAX_WORKERS);
    const float* levels = staged ? plan->d_levels_stage : plan->d_levels_enc[plan->cur];
    LQ_CUDA(launch_level_probabilities(plan->dev, hist, plan->dev.bucket_norm ? plan->dev.layer_weight : norms,
                                       num_samples, levels, probs, (cudaStream_t)stream));
    return LQ_OK;
}

int lq_symbol_counts(const lq_plan* plan, const uint32_t* packed, uint32_t* counts, void* stream)
{
    if (!plan || !packed || !counts) return fail(LQ_EINVAL, "NULL argument");
    LQ_CUDA(launch_symbol_counts(plan->dev, packed, counts, (cudaStream_t)stream));
    return LQ_OK;
}

int qoda_set_alt_rates(lq_plan* plan, double q_hat)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    if (!(q_hat >= 0.0 && q_hat <= 0.25)) return fail(LQ_EINVAL, "q_hat must be in (0, 1/4], or 0 to switch back; got %g", q_hat);
    plan->alt_qhat = q_hat;
    return LQ_OK;
}

int qoda_get_alt_scalars(const lq_plan* plan, double* lambda, double* mu, double* gamma)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    QodaScalars h;
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(&h, plan->dev.scalars, sizeof h, cudaMemcpyDeviceToHost));
    if (lambda) *lambda = h.lambda;
    if (mu) *mu = h.mu;
    if (gamma) *gamma = (double)h.gamma;
    return LQ_OK;
}

int qoda_get_scalars(const lq_plan* plan, int64_t* t, double* S, double* eta)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    QodaScalars h;
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(&h, plan->dev.scalars, sizeof h, cudaMemcpyDeviceToHost));
    if (t) *t = (int64_t)h.t;
    if (S) *S = h.S;
    if (eta) *eta = (double)h.eta;
    return LQ_OK;
}

int lq_get_statistics(const lq_plan* plan, double* host_sq_diff, uint32_t* host_flags)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    const size_t KL = (size_t)plan->dev.num_workers * (size_t)plan->dev.num_layers;
    LQ_CUDA(cudaDeviceSynchronize());
    if (host_sq_diff && KL)
        LQ_CUDA(cudaMemcpy(host_sq_diff, plan->dev.sq_diff, KL * sizeof(double), cudaMemcpyDeviceToHost));
    if (host_flags && KL)
        LQ_CUDA(cudaMemcpy(host_flags, plan->dev.status, KL * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    return LQ_OK;
}

int lq_profile_enable(lq_plan* plan, int32_t enable)
{
    if (!plan) return fail(LQ_EINVAL, "plan is NULL");
    plan->profiling = enable != 0;
    return LQ_OK;
}

int lq_profile_read(lq_plan* plan, double* total_ms, int64_t* launches)
{
    if (!plan || !total_ms || !launches) return fail(LQ_EINVAL, "NULL argument");
    for (int i = 0; i < LQ_NUM_KERNELS; ++i) { total_ms[i] = 0.0; launches[i] = 0; }
    LQ_CUDA(cudaDeviceSynchronize());
    for (auto& r : plan->prof_recs) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess && r.id >= 0 && r.id < LQ_NUM_KERNELS) {
            total_ms[r.id] += (double)ms;
            launches[r.id] += 1;
        }
        plan->prof_pool.push_back(r.a);
        plan->prof_pool.push_back(r.b);
    }
    plan->prof_recs.clear();
    return LQ_OK;
}

}  // extern "C"

namespace {

// Uploads the tables of one layer's code.
int upload_code(lq_plan* plan, int layer, const uint8_t* len, int n)
{
    std::vector<uint32_t> code(kMaxLevels, 0), enc(kMaxLevels, 0);
    std::vector<uint16_t> dec((size_t)kDecEntries);
    if (!canonical_codes_host(len, n, kCodeMaxLen, code.data()))
        return fail(LQ_EINVAL, "layer %d: lengths must lie in [1, %d] and satisfy Kraft's inequality", layer, kCodeMaxLen);
    build_code_tables_host(len, code.data(), n, enc.data(), dec.data());
    LQ_CUDA(cudaMemcpy(plan->d_code_enc + (size_t)layer * kMaxLevels, enc.data(), kMaxLevels * sizeof(uint32_t),
                       cudaMemcpyHostToDevice));
    LQ_CUDA(cudaMemcpy(plan->d_code_dec + (size_t)layer * kDecEntries, dec.data(), dec.size() * sizeof(uint16_t),
                       cudaMemcpyHostToDevice));
    std::copy(len, len + n, plan->code_len.begin() + (size_t)layer * kMaxLevels);
    return LQ_OK;
}

// First use of the entropy stage: tables for every layer, initialised to the flat code (b bits per index).
int ensure_codes(lq_plan* plan)
{
    if (plan->d_code_enc) return LQ_OK;
    const size_t L = (size_t)(plan->dev.num_layers ? plan->dev.num_layers : 1);
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(dev_alloc_zero(&plan->d_code_enc, L * kMaxLevels));
    LQ_CUDA(dev_alloc_zero(&plan->d_code_dec, L * (size_t)kDecEntries));
    LQ_CUDA(dev_alloc_zero(&plan->d_code_bad, 1));
    {
        const size_t K = (size_t)plan->dev.num_workers, nb = (size_t)(plan->dev.total_blocks ? plan->dev.total_blocks : 1);
        LQ_CUDA(dev_alloc_zero(&plan->code_scratch.lane_bits, K * nb * 32));
        LQ_CUDA(dev_alloc_zero(&plan->code_scratch.scan_part, K * ((nb + 1023) / 1024)));
    }
    try { plan->code_len.assign(L * kMaxLevels, 0); } catch (const std::bad_alloc&) { return fail(LQ_ENOMEM, "host allocation failed"); }
    for (int m = 0; m < plan->dev.num_layers; ++m) {
        const LayerDesc& Ld = plan->layers[(size_t)m];
        uint8_t flat[kMaxLevels];
        for (int j = 0; j < Ld.nlevels; ++j) flat[j] = (uint8_t)Ld.bits;
        const int rc = upload_code(plan, m, flat, Ld.nlevels);
        if (rc != LQ_OK) return rc;
    }
    return LQ_OK;
}

}  // namespace

extern "C" {

int lq_code_build(const double* weights, int32_t n, uint8_t* lengths)
{
    if (!weights || !lengths) return fail(LQ_EINVAL, "NULL argument");
    if (n < 1 || n > kMaxLevels) return fail(LQ_EINVAL, "n must be in [1, %d]", kMaxLevels);
    try {
        if (!huffman_lengths_host(weights, n, kCodeMaxLen, lengths)) return fail(LQ_EINVAL, "weights must be non-negative numbers");
    } catch (const std::bad_alloc&) { return fail(LQ_ENOMEM, "host allocation failed"); }
    return LQ_OK;
}

int lq_code_universal(int32_t n, uint8_t* lengths)
{
    if (!lengths) return fail(LQ_EINVAL, "NULL argument");
    if (n < 1 || n > kMaxLevels) return fail(LQ_EINVAL, "n must be in [1, %d]", kMaxLevels);
    for (int j = 0; j < n; ++j) {
        // length of the recursive code of j + 1: the closing 0, then the binary forms of the value, of its bit
        // count minus one, and so on down to 1
        int len = 1;
        for (unsigned v = (unsigned)j + 1u; v > 1u;) {
            int nb = 0;
            for (unsigned t = v; t; t >>= 1) ++nb;
            len += nb;
            v = (unsigned)nb - 1u;
        }
        if (len > kCodeMaxLen)
            return fail(LQ_EINVAL, "the recursive code of level index %d has %d bits, more than %d: use it with at "
                        "most 63 levels (b <= 5)", j, len, kCodeMaxLen);
        lengths[j] = (uint8_t)len;
    }
    return LQ_OK;
}

int lq_code_set(lq_plan* plan, int32_t layer, const uint8_t* lengths, int32_t n)
{
    if (!plan || !lengths) return fail(LQ_EINVAL, "NULL argument");
    if (layer < 0 || layer >= plan->dev.num_layers) return fail(LQ_EINVAL, "layer %d out of range", layer);
    if (n != plan->layers[(size_t)layer].nlevels) return fail(LQ_EINVAL, "layer %d has %d levels, got %d", layer, plan->layers[(size_t)layer].nlevels, n);
    const int rc = ensure_codes(plan);
    if (rc != LQ_OK) return rc;
    LQ_CUDA(cudaDeviceSynchronize());
    return upload_code(plan, layer, lengths, n);
}

int lq_code_get(lq_plan* plan, int32_t layer, uint8_t* lengths, int32_t n)
{
    if (!plan || !lengths) return fail(LQ_EINVAL, "NULL argument");
    if (layer < 0 || layer >= plan->dev.num_layers) return fail(LQ_EINVAL, "layer %d out of range", layer);
    if (n != plan->layers[(size_t)layer].nlevels) return fail(LQ_EINVAL, "layer %d has %d levels, got %d", layer, plan->layers[(size_t)layer].nlevels, n);
    const int rc = ensure_codes(plan);
    if (rc != LQ_OK) return rc;
    std::copy(plan->code_len.begin() + (size_t)layer * kMaxLevels, plan->code_len.begin() + (size_t)layer * kMaxLevels + n, lengths);
    return LQ_OK;
}

int64_t lq_plan_blocks(const lq_plan* plan) { return plan ? plan->dev.total_blocks : (int64_t)fail(LQ_EINVAL, "plan is NULL"); }

int lq_entropy_encode(lq_plan* plan, const uint32_t* packed, uint32_t* stream_words, int64_t capacity_words,
                      uint32_t* block_offsets, uint16_t* run_offsets, void* stream)
{
    LQ_ALIGNED(run_offsets, 2);
    if (!plan || !packed || !stream_words || !block_offsets) return fail(LQ_EINVAL, "NULL argument");
    if (capacity_words < 0) return fail(LQ_EINVAL, "capacity_words < 0");
    LQ_ALIGNED(packed, 4); LQ_ALIGNED(stream_words, 4); LQ_ALIGNED(block_offsets, 4);
    const int rc = ensure_codes(plan);
    if (rc != LQ_OK) return rc;
    LQ_CUDA(launch_entropy_encode(plan->dev, packed, plan->d_code_enc, block_offsets, stream_words, capacity_words,
                                  run_offsets, plan->code_scratch, (cudaStream_t)stream));
    return LQ_OK;
}

int lq_entropy_decode(lq_plan* plan, const uint32_t* stream_words, int64_t capacity_words,
                      const uint32_t* block_offsets, const uint16_t* run_offsets, uint32_t* packed, void* stream)
{
    LQ_ALIGNED(run_offsets, 2);
    if (!plan || !packed || !stream_words || !block_offsets) return fail(LQ_EINVAL, "NULL argument");
    if (capacity_words < 0) return fail(LQ_EINVAL, "capacity_words < 0");
    LQ_ALIGNED(packed, 4); LQ_ALIGNED(stream_words, 4); LQ_ALIGNED(block_offsets, 4);
    const int rc = ensure_codes(plan);
    if (rc != LQ_OK) return rc;
    LQ_CUDA(launch_entropy_decode(plan->dev, stream_words, capacity_words, block_offsets, run_offsets, plan->d_code_dec,
                                  packed, plan->d_code_bad, (cudaStream_t)stream));
    return LQ_OK;
}

int lq_entropy_status(lq_plan* plan, uint32_t* host_flag)
{
    if (!plan || !host_flag) return fail(LQ_EINVAL, "NULL argument");
    *host_flag = 0;
    if (!plan->d_code_bad) return LQ_OK;
    LQ_CUDA(cudaDeviceSynchronize());
    LQ_CUDA(cudaMemcpy(host_flag, plan->d_code_bad, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    LQ_CUDA(cudaMemset(plan->d_code_bad, 0, sizeof(uint32_t)));
    return LQ_OK;
}

}  // extern "C"
