// Host side of the C ABI declared in include/lpmm.h: argument validation, arena layout, the
// device-side tensor table and the launch sequence of one step. No device memory is allocated here.
#include <cmath>
#include <cstddef>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/lpmm.h"
#include "lpmm_internal.h"

using namespace lpmm;

namespace {

thread_local int32_t g_last_cuda_error = 0;

lpmm_status cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int32_t)e;
    return LPMM_ERR_CUDA;
}
#define LPMM_CUDA(call)                                   \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) return cuda_fail(e__);    \
    } while (0)

constexpr size_t kAlign = 256;
size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct TensorLayout {
    int32_t kind;       // K_* of lpmm_internal.h
    int64_t rows, cols, numel;
    size_t m_codes, m_scale, v_codes, v_bscale, m32, v32;  // byte offsets into the arena (0 = unused)
    int64_t rc_index;   // float index of this tensor's [r | c] inside each rank-1 scale buffer
    int32_t c_off;
    int32_t n_outer = 1;            // leading axes (Alg. 4 in general form: ndim - 1)
    int32_t outer_dim[3] = {0, 0, 0};
    int32_t outer_off[3] = {0, 0, 0};
    int32_t rc_len = 0;             // floats of this tensor's share of every rank-1 scale buffer (all axes, padded)
    int32_t nd = 0;                 // three or four axes: their number, extents and offsets inside the tensor's share
    int32_t nd_dim[4] = {0, 0, 0, 0};
    int32_t nd_off[4] = {0, 0, 0, 0};
    bool p1_tiled = false;          // K_RANK1_FLAT matrix whose maxima pass runs on the tiled kernel (cols % 8 == 0)
    int32_t nd_split = 0;           // > 0: composite tensor on the tiled path, axes [0, nd_split) are its rows
    size_t exp_old = 0, exp_new = 0, exp_rcp = 0;   // composite: per-step expanded statistics (arena offsets)
    int32_t exp_len = 0;
    size_t fact_rowpart = 0, fact_colpart = 0, fact_blockpart = 0;   // K_FACT: scratch for the partial sums of g^2
    int32_t fact_nstrips = 0, fact_tiles_y = 0;
};

struct Layout {
    std::vector<TensorLayout> t;
    size_t descs = 0, params = 0, params16 = 0, grads = 0, tiles1 = 0, tiles2 = 0, tiles3 = 0, tiles4 = 0, tiles5 = 0, tiles6 = 0, tiles7 = 0;
    size_t tsync = 0, work = 0;       // fused schedule: per-tensor progress counters, work list
    int64_t work_items = 0;           // capacity of the work list
    size_t rc[3] = {0, 0, 0}, rcp = 0;
    int64_t rc_floats = 0;
    size_t total = 0;
    size_t states_end = 0;            // end of the schedule-independent part (the work list comes after it)
    uint64_t shape_hash = 0;          // of everything the layout depends on (checked by lpmm_state_attach)
    std::vector<size_t> guards;       // checking build: offsets of the 256-byte guard zones
};

// The first 256 bytes of the arena: device status word, the tile counters of a launch, and a description of the
// layout that lpmm_state_attach compares with what the caller claims the arena holds.
constexpr uint32_t kArenaMagic = 0x4d4d504cu;    // "LPMM"
#ifdef LPMM_DEBUG
constexpr uint32_t kArenaLayoutVersion = 0x80000002u;   // the checking build's arenas carry guard zones: another layout
#else
constexpr uint32_t kArenaLayoutVersion = 2u;     // bump whenever offsets or the meaning of a region change
#endif
struct ArenaHeader {
    uint32_t status;          // byte 0: device status word (0 = ok)
    uint32_t pad0[3];
    int32_t tile_counter[2];  // byte 16: next tile of the running launch, finished CTAs
    uint32_t pad1[2];
    uint32_t magic;           // byte 32
    uint32_t version;
    uint64_t total_bytes;
    uint64_t shape_hash;
    int32_t n_tensors;
    int32_t m_block;
    int32_t v_mode;
    int32_t pad2;
    uint64_t pad3[7];
    unsigned long long wait_stats[2];   // byte 128: fused schedule, {waits that had to poll, their summed nanoseconds}
    int32_t tile_counter_aux[2];        // byte 144: the same pair as tile_counter for a launch that runs beside another one
};
static_assert(sizeof(ArenaHeader) <= 256, "header block");

// Resident CTAs of the step kernels on a B200 (148 SMs x 2): the device-independent figure the tile sizes are planned
// with, so that lpmm_state_bytes can size the work list without a device.
constexpr int kPlanResidentCtas = 296;

bool uses_rc(int32_t k) { return k == K_RANK1_FAST || k == K_RANK1_FLAT || k == K_FACT; }

int public_kind(int32_t k) {
    if (k == K_FP32) return LPMM_KIND_FP32;
    if (k == K_BLOCK || k == K_BLOCK_TILED) return LPMM_KIND_BLOCK;
    if (k == K_FACT) return LPMM_KIND_FACTORED;
    return LPMM_KIND_RANK1;
}

int32_t choose_kind(const lpmm_config& cfg, const lpmm_shape& s);
int64_t folded_cols(const lpmm_config& cfg, int64_t numel);
bool fused_eligible(const lpmm_config& cfg);

lpmm_status validate_config(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n) {
    if (!cfg || !shapes || n <= 0) return LPMM_ERR_INVALID_ARG;
    if (cfg->min_quant_numel < 0) return LPMM_ERR_INVALID_ARG;
    if (cfg->v_mode != LPMM_V_RANK1 && cfg->v_mode != LPMM_V_BLOCK && cfg->v_mode != LPMM_V_FACTORED) return LPMM_ERR_INVALID_ARG;
    if (cfg->bits != 4) return LPMM_ERR_UNSUPPORTED;
    if ((cfg->m_block != 128 && cfg->m_block != 2048) || cfg->v_block != 128) return LPMM_ERR_UNSUPPORTED;
    if (cfg->update_math != LPMM_UPDATE_FAST && cfg->update_math != LPMM_UPDATE_IEEE) return LPMM_ERR_INVALID_ARG;
    if (cfg->schedule != LPMM_SCHEDULE_AUTO && cfg->schedule != LPMM_SCHEDULE_TWO_PASS && cfg->schedule != LPMM_SCHEDULE_FUSED &&
        cfg->schedule != LPMM_SCHEDULE_OVERLAP)
        return LPMM_ERR_INVALID_ARG;
    if (cfg->overlap_groups < 0 || cfg->overlap_groups > 4096) return LPMM_ERR_INVALID_ARG;
    if (cfg->schedule == LPMM_SCHEDULE_FUSED && !fused_eligible(*cfg)) return LPMM_ERR_UNSUPPORTED;
    for (int32_t te : {cfg->tile_elems, cfg->tile_elems_maxima})
        if (te != 0 && (te < 2048 || te > (1 << 22) || (te & (te - 1)) != 0)) return LPMM_ERR_INVALID_ARG;
    if (cfg->l2_keep_mbytes < 0 || cfg->lead_melems < 0 || cfg->gap_items < 0) return LPMM_ERR_INVALID_ARG;
    if (cfg->no_l2_hints != 0 && cfg->no_l2_hints != 1) return LPMM_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i) {
        const lpmm_shape& s = shapes[i];
        if (s.rows <= 0 || s.cols <= 0) return LPMM_ERR_INVALID_ARG;
        if (s.ndim < 1) return LPMM_ERR_INVALID_ARG;
        if (s.ndim > LPMM_MAX_NDIM) return LPMM_ERR_UNSUPPORTED;
        if (s.ndim == 1 && s.cols != 1) return LPMM_ERR_INVALID_ARG;
        if (s.ndim >= 3) {   // rows, cols restate dims
            int64_t lead = 1;
            for (int32_t a = 0; a < s.ndim; ++a) {
                if (s.dims[a] <= 0 || s.dims[a] > (int64_t)1 << 30) return LPMM_ERR_INVALID_ARG;
                if (a + 1 < s.ndim) {
                    if (lead > ((int64_t)1 << 40) / s.dims[a]) return LPMM_ERR_INVALID_ARG;
                    lead *= s.dims[a];
                }
            }
            if (lead != s.rows || s.dims[s.ndim - 1] != s.cols) return LPMM_ERR_INVALID_ARG;
            if (cfg->v_mode == LPMM_V_FACTORED) return LPMM_ERR_UNSUPPORTED;   // Sec. 4.3 factorizes matrices
        }
        if ((s.flags & LPMM_FORCE_QUANT) && (s.flags & LPMM_FORCE_FP32)) return LPMM_ERR_INVALID_ARG;
        if (s.rows > (int64_t)1 << 40 || s.cols > (int64_t)1 << 40 || s.rows > ((int64_t)1 << 40) / s.cols)
            return LPMM_ERR_INVALID_ARG;  // numel overflow guard
        if (s.rows + s.cols > (int64_t)1 << 30) return LPMM_ERR_UNSUPPORTED;
        if (s.ndim >= 3) {
            int64_t stats = 0;
            for (int32_t a = 0; a < s.ndim; ++a) stats += s.dims[a] + 3;
            if (stats > (int64_t)1 << 30) return LPMM_ERR_UNSUPPORTED;
        }
        // the factorized second moment is built for the tiled path only: whole first-moment blocks inside a row
        if (cfg->v_mode == LPMM_V_FACTORED && choose_kind(*cfg, s) == K_RANK1_FLAT) return LPMM_ERR_UNSUPPORTED;
    }
    return LPMM_OK;
}

// A long 1-D tensor (a flattened parameter group, say) is block-wise in both moments, and its blocks do not care
// how the elements are folded into rows: folded into rows of `cols` elements it can take the tiled update path.
// Returns that row length, or 0 when the tensor stays on the element-indexed path.
int64_t folded_cols(const lpmm_config& cfg, int64_t numel) {
    if (numel < 65536) return 0;
    if (cfg.m_block == 2048) return (numel % 2048 == 0) ? 2048 : 0;
    for (int64_t c = 1024; c >= 128; c /= 2)
        if (numel % c == 0) return c;
    return 0;
}

int32_t choose_kind(const lpmm_config& cfg, const lpmm_shape& s) {
    const int64_t numel = s.rows * s.cols;
    if (s.flags & LPMM_FORCE_FP32) return K_FP32;
    if (!(s.flags & LPMM_FORCE_QUANT) && numel <= cfg.min_quant_numel) return K_FP32;  // App. D.1
    if (s.ndim == 1 || s.rows == 1 || s.cols == 1)   // Sec. 4.2
        return (cfg.v_mode != LPMM_V_FACTORED && folded_cols(cfg, numel) > 0) ? K_BLOCK_TILED : K_BLOCK;
    if (cfg.v_mode == LPMM_V_BLOCK) {   // block-wise second moment on a matrix: tiled when whole blocks lie inside a row
        const bool tiled = s.ndim == 2 && s.cols % 128 == 0 && s.cols % cfg.m_block == 0 && s.cols <= ((int64_t)1 << 24);
        return tiled ? K_BLOCK_TILED : K_BLOCK;
    }
    // the tiled path needs whole first-moment blocks inside a row (and, for B2048, one block per tile width)
    // the tiled path keeps 32-bit element offsets inside a tile: rows of at most 2^24 elements
    if (s.ndim >= 3) return K_RANK1_FLAT;     // Alg. 4 with more than two axes: element-indexed path
    if (s.cols % cfg.m_block != 0 || s.cols > ((int64_t)1 << 24)) return K_RANK1_FLAT;   // (refused in the factorized mode)
    return (cfg.v_mode == LPMM_V_FACTORED) ? K_FACT : K_RANK1_FAST;
}

// Which schedule a state runs: the fused one needs the default quantizers (rank-1 second moments, B128 first moments).
bool fused_eligible(const lpmm_config& cfg) { return cfg.v_mode == LPMM_V_RANK1 && cfg.m_block == 128; }
// AUTO goes by measurement (B200): the fused launch wins where launch overhead and the gaps between the three kernels
// matter (1024x4096 + bias: 44 vs 51 us; the 181-tensor Transformer-base list, 60.5 M: 0.228 vs 0.254 ms); from one
// 8192x8192 matrix (64 Mi) upwards the two-pass schedule is ahead (0.250 vs 0.258 ms; LLaMA-7B list 17.2 vs 18.3 ms).
constexpr int64_t kAutoFusedMaxElems = (int64_t)63 << 20;
bool wants_fused(const lpmm_config& cfg, int64_t total_elems) {
    if (!fused_eligible(cfg)) return false;
    if (cfg.schedule == LPMM_SCHEDULE_FUSED) return true;
    return cfg.schedule == LPMM_SCHEDULE_AUTO && total_elems <= kAutoFusedMaxElems;
}

struct TileSizes { int64_t update, maxima, flat; };   // flat: the element-indexed tensors' tiles (a launch of their own)

// Elements per tile of the update pass and of the maxima pass (powers of two). Tiles are handed out on demand, so the
// aim is >= 6 tiles per resident CTA (the tail is what is balanced). Two-pass schedule, measured optima of the update
// pass: 32 Ki for 60-70 M parameters, 64-128 Ki for 355 M, 256 Ki for 6.7 G; the maxima pass gains from taller tiles
// (each tile ends with a flush of its column maxima and starts with an empty load pipeline), up to 1 Mi. The fused
// schedule wants shorter tiles (an update tile can only start when the tensor's last maxima tile has finished), but
// every tile costs about 2 us of start-up: 128 Ki / 256 Ki measured best on the 6.7 G list.
TileSizes choose_tile_sizes(const lpmm_config& cfg, int64_t total_elems, int64_t flat_elems, bool fused) {
    const int64_t cap2 = fused ? 131072 : 262144, cap1 = fused ? 262144 : (1 << 20);
    const int64_t hard2 = fused ? 262144 : ((int64_t)1 << 22);   // fused: an update tile has at most 1024 rows of 256 columns
    const int64_t target = total_elems / (6LL * kPlanResidentCtas);
    TileSizes ts;
    ts.update = 2048;
    while (ts.update * 2 <= target && ts.update < cap2) ts.update *= 2;
    if (fused && ts.update < 8192) ts.update = 8192;   // (one 1024x4096 matrix: 41.7 us with 8 Ki / 16 Ki tiles, 45.3 with 2 Ki / 4 Ki)
    if (cfg.tile_elems > 0) ts.update = cfg.tile_elems < hard2 ? cfg.tile_elems : hard2;
    ts.maxima = ts.update;
    while (ts.maxima * 2 <= target && ts.maxima < cap1) ts.maxima *= 2;
    if (fused && ts.maxima < cap1 && ts.maxima * 2 <= 2 * target) ts.maxima *= 2;
    if (fused && ts.maxima < 16384) ts.maxima = 16384;
    if (cfg.tile_elems_maxima > 0) ts.maxima = cfg.tile_elems_maxima;
    if (ts.maxima < ts.update) ts.maxima = ts.update;
    // the element-indexed tensors are sized by their own total: their kernel is a separate launch, and a few long tiles
    // would leave most of the GPU idle behind a chain of dependent chunks
    const int64_t target_flat = (fused ? total_elems : flat_elems) / (6LL * kPlanResidentCtas);
    ts.flat = 2048;
    while (ts.flat * 2 <= target_flat && ts.flat < ts.update) ts.flat *= 2;
    return ts;
}

struct TilePlan {
    int32_t wx = 0, tiles_x = 0, tile_rows = 0, tile_rows1 = 0, flat_chunks = 1;
    int64_t tiles_update = 0;   // tiles of the update pass (tiled or element-indexed, by kind)
    int64_t tiles_maxima = 0;   // tiles of the maxima pass (rank-1 kinds and the factorized kind; else 0)
    int64_t tiles_flat = 0;     // element-indexed tiles (what the SGDM step uses for every tensor)
};

TilePlan plan_tensor(const lpmm_config& cfg, const TensorLayout& t, const TileSizes& ts) {
    TilePlan p;
    const bool tiled = t.kind == K_RANK1_FAST || t.kind == K_FACT || t.kind == K_BLOCK_TILED;
    if (tiled || t.p1_tiled) {
        p.wx = (cfg.m_block == 2048) ? 8 : (t.cols % 1024 == 0) ? 4 : (t.cols % 512 == 0) ? 2 : 1;
        const int64_t tile_cols = (int64_t)kWarpElems * p.wx;
        int64_t tr = ts.update / tile_cols;
        // at least four rows per warp: the maxima pass works in trips of four rows (shorter tiles repeat rows)
        if (tr < 4 * (kWarps / p.wx)) tr = 4 * (kWarps / p.wx);
        p.tile_rows = (int32_t)tr;
        p.tiles_x = (int32_t)((t.cols + tile_cols - 1) / tile_cols);
        p.tiles_update = (int64_t)p.tiles_x * ((t.rows + tr - 1) / tr);
        int64_t tr1 = ts.maxima / tile_cols;
        if (tr1 < tr) tr1 = tr;
        p.tile_rows1 = (int32_t)tr1;
        if (t.kind != K_BLOCK_TILED) p.tiles_maxima = (int64_t)p.tiles_x * ((t.rows + tr1 - 1) / tr1);
        if (!tiled) p.tiles_update = 0;   // (set below: the update pass of such a tensor is element-indexed)
    }
    int64_t chunks = (tiled || t.kind == K_FP32 ? ts.update : ts.flat) / (kWarps * kWarpElems);
    if (chunks < 1) chunks = 1;
    if (chunks > 16) chunks = 16;
    p.flat_chunks = (int32_t)chunks;
    const int64_t per_tile = chunks * kWarps * kWarpElems;
    p.tiles_flat = (t.numel + per_tile - 1) / per_tile;
    if (!tiled) {
        p.tiles_update = p.tiles_flat;
        if (t.kind == K_RANK1_FLAT && !t.p1_tiled) p.tiles_maxima = p.tiles_flat;
    }
    return p;
}

// End of a sub-buffer that stops at byte `end`: the next 256-byte boundary. The checking build (-DLPMM_DEBUG) puts a
// guard zone of 256 bytes behind every sub-buffer, filled with a pattern at initialisation and never written by any
// kernel: lpmm_state_check_guards() finds a stray write that crossed a sub-buffer's end.
#ifdef LPMM_DEBUG
constexpr bool kGuards = true;
#else
constexpr bool kGuards = false;
#endif
constexpr unsigned char kGuardByte = 0xC5;
size_t region_end(Layout* L, size_t end) {
    size_t e = align_up(end);
    if (kGuards) { L->guards.push_back(e); e += kAlign; }
    return e;
}

uint64_t fnv1a(uint64_t h, const void* data, size_t bytes) {
    const unsigned char* p = static_cast<const unsigned char*>(data);
    for (size_t i = 0; i < bytes; ++i) { h ^= p[i]; h *= 1099511628211ull; }
    return h;
}

void compute_layout(const lpmm_config& cfg, const lpmm_shape* shapes, int32_t n, Layout* L) {
    L->t.resize(n);
    L->guards.clear();
    {
        uint64_t h = 1469598103934665603ull;
        const int64_t c[5] = {cfg.bits, cfg.m_block, cfg.v_block, cfg.v_mode, cfg.min_quant_numel};
        h = fnv1a(h, c, sizeof(c));
        for (int32_t i = 0; i < n; ++i) {
            const lpmm_shape& s = shapes[i];
            const int64_t v[4] = {s.rows, s.cols, s.ndim, (int64_t)s.flags};
            h = fnv1a(h, v, sizeof(v));
            if (s.ndim >= 3) h = fnv1a(h, s.dims, sizeof(int64_t) * s.ndim);
        }
        L->shape_hash = h;
    }
    size_t off = kAlign;  // header block
    L->descs = off;  off = region_end(L, off + sizeof(TensorDesc) * n);
    L->params = off; off = region_end(L, off + sizeof(void*) * n);
    L->params16 = off; off = region_end(L, off + sizeof(void*) * n);
    L->grads = off;  off = region_end(L, off + sizeof(void*) * n);
    L->tiles1 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles2 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles3 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles4 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles5 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles6 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tiles7 = off; off = region_end(L, off + sizeof(int32_t) * (n + 1));
    L->tsync = off;  off = region_end(L, off + sizeof(TensorSync) * n);
    int64_t rc = 0;
    for (int32_t i = 0; i < n; ++i) {
        TensorLayout& t = L->t[i];
        t = TensorLayout{};
        t.rows = shapes[i].rows; t.cols = shapes[i].cols; t.numel = t.rows * t.cols;
        t.kind = choose_kind(cfg, shapes[i]);
        if (t.kind == K_BLOCK_TILED && (shapes[i].ndim == 1 || t.rows == 1 || t.cols == 1)) {   // folded, see folded_cols()
            t.cols = folded_cols(cfg, t.numel);
            t.rows = t.numel / t.cols;
        }
        if (uses_rc(t.kind)) {
            t.rc_index = rc;
            if (shapes[i].ndim >= 3) {   // one vector of statistics per axis, each padded to 4 floats
                t.n_outer = shapes[i].ndim - 1;
                int64_t o = 0;
                for (int32_t a = 0; a < t.n_outer; ++a) {
                    t.outer_dim[a] = (int32_t)shapes[i].dims[a];
                    t.outer_off[a] = (int32_t)o;
                    o += (shapes[i].dims[a] + 3) / 4 * 4;
                }
                t.c_off = (int32_t)o;
                t.nd = shapes[i].ndim;
                for (int32_t a = 0; a < t.nd; ++a) {
                    t.nd_dim[a] = (int32_t)shapes[i].dims[a];
                    t.nd_off[a] = a + 1 < t.nd ? t.outer_off[a] : t.c_off;
                }
            } else {
                t.n_outer = 1;
                t.outer_dim[0] = (int32_t)t.rows;
                t.c_off = (int32_t)((t.rows + 3) / 4 * 4);
            }
            t.rc_len = (int32_t)(t.c_off + (t.cols + 3) / 4 * 4);
            t.p1_tiled = t.kind == K_RANK1_FLAT && shapes[i].ndim == 2 && t.cols % 8 == 0 && t.cols >= 128 &&
                         t.cols <= ((int64_t)1 << 24);
            rc += t.rc_len;
            rc = (rc + 63) / 64 * 64;  // 256-byte granules so r and c always start 16-byte aligned
        }
    }
    L->rc_floats = rc;
    L->rc[0] = off; off = region_end(L, off + sizeof(float) * rc);
    L->rc[1] = off; off = region_end(L, off + sizeof(float) * rc);
    L->rc[2] = off; off = region_end(L, off + sizeof(float) * rc);
    L->rcp = off;   off = region_end(L, off + sizeof(float) * rc);
    int64_t total_elems = 0, flat_elems = 0;
    for (int32_t i = 0; i < n; ++i) total_elems += L->t[i].numel;
    // Tensors with three or four axes whose trailing axes multiply to whole first-moment blocks go to the tiled path as
    // "composite" matrices (leading axes = rows, trailing axes = columns) with per-step expanded statistics. (Not under
    // the fused schedule, whose element-indexed tiles handle them.)
    if (!wants_fused(cfg, total_elems)) {
        for (int32_t i = 0; i < n; ++i) {
            TensorLayout& t = L->t[i];
            if (t.kind != K_RANK1_FLAT || t.nd < 3) continue;
            int32_t best = 0;
            int64_t best_cols = 0;
            for (int32_t sp = t.nd - 1; sp >= 1; --sp) {
                int64_t c = 1;
                for (int32_t a = sp; a < t.nd; ++a) c *= t.nd_dim[a];
                if (c % 128 != 0 || c % cfg.m_block != 0 || c > ((int64_t)1 << 24)) continue;
                if (best == 0 || (best_cols < 1024 && c > best_cols)) { best = sp; best_cols = c; }   // the narrowest one that fills a tile
            }
            bool whole_blocks = best != 0;
            if (!whole_blocks && cfg.m_block == 128) {
                // no split makes rows of whole first-moment blocks: rows of whole lanes (cols % 8 == 0, at least 256) still get
                // the tiled maxima pass and the stepped interior loop of the element-indexed update
                for (int32_t sp = t.nd - 1; sp >= 1; --sp) {
                    int64_t c = 1;
                    for (int32_t a = sp; a < t.nd; ++a) c *= t.nd_dim[a];
                    if (c % 8 != 0 || c < 256 || c > ((int64_t)1 << 24)) continue;
                    if (best == 0 || (best_cols < 1024 && c > best_cols)) { best = sp; best_cols = c; }
                }
            }
            if (best == 0) continue;
            if (whole_blocks) t.kind = K_RANK1_FAST;
            else t.p1_tiled = true;
            t.nd_split = best;
            t.cols = best_cols;
            t.rows = t.numel / best_cols;
            t.n_outer = 1;
            t.c_off = (int32_t)((t.rows + 3) / 4 * 4);
            t.exp_len = (int32_t)(t.c_off + (t.cols + 3) / 4 * 4);
            t.exp_old = off; off = region_end(L, off + sizeof(float) * (size_t)t.exp_len);
            t.exp_new = off; off = region_end(L, off + sizeof(float) * (size_t)t.exp_len);
            t.exp_rcp = off; off = region_end(L, off + sizeof(float) * (size_t)t.exp_len);
        }
    }
    for (int32_t i = 0; i < n; ++i)
        if (L->t[i].kind == K_RANK1_FLAT || L->t[i].kind == K_BLOCK) flat_elems += L->t[i].numel;
    for (int32_t i = 0; i < n; ++i) {
        TensorLayout& t = L->t[i];
        if (t.kind == K_FP32) {
            t.m32 = off; off = region_end(L, off + sizeof(float) * t.numel);
            t.v32 = off; off = region_end(L, off + sizeof(float) * t.numel);
        } else {
            const size_t code_bytes = (size_t)((t.numel + 1) / 2);
            const size_t nblk = (size_t)((t.numel + 127) / 128);
            const size_t nblk_m = (size_t)((t.numel + cfg.m_block - 1) / cfg.m_block);
            t.m_codes = off; off = region_end(L, off + code_bytes);
            if (t.kind != K_FACT) { t.v_codes = off; off = region_end(L, off + code_bytes); }
            t.m_scale = off; off = region_end(L, off + sizeof(float) * nblk_m);
            if (t.kind == K_BLOCK || t.kind == K_BLOCK_TILED) { t.v_bscale = off; off = region_end(L, off + sizeof(float) * nblk); }
        }
    }
    if (cfg.v_mode == LPMM_V_FACTORED) {   // scratch of the sums pass (same tile plan as build_tables)
        const TileSizes ts = choose_tile_sizes(cfg, total_elems, flat_elems, false);
        for (int32_t i = 0; i < n; ++i) {
            TensorLayout& t = L->t[i];
            if (t.kind != K_FACT) continue;
            const TilePlan p = plan_tensor(cfg, t, ts);
            t.fact_nstrips = (int32_t)((t.cols + kWarpElems - 1) / kWarpElems);
            t.fact_tiles_y = (int32_t)((t.rows + p.tile_rows1 - 1) / p.tile_rows1);
            t.fact_rowpart = off; off = region_end(L, off + sizeof(float) * (size_t)t.rows * t.fact_nstrips);
            t.fact_colpart = off; off = region_end(L, off + sizeof(float) * (size_t)t.fact_tiles_y * t.cols);
            t.fact_blockpart = off; off = region_end(L, off + sizeof(double) * (size_t)((t.rc_len + 31) / 32));
        }
    }
    L->states_end = off;   // everything a checkpoint must keep lies below this offset
    if (wants_fused(cfg, total_elems)) {   // the work list: one item per tile of either pass
        const TileSizes ts = choose_tile_sizes(cfg, total_elems, flat_elems, true);
        int64_t items = 0;
        for (int32_t i = 0; i < n; ++i) {
            const TilePlan p = plan_tensor(cfg, L->t[i], ts);
            items += p.tiles_update + p.tiles_maxima;
        }
        L->work_items = items;
        L->work = off; off = region_end(L, off + sizeof(uint2) * (size_t)items);
    }
    L->total = off;
}

}  // namespace

struct lpmm_state {
    lpmm_config cfg;
    int32_t n;
    Layout L;
    char* arena;
    size_t arena_bytes;
    int32_t phase;
    int32_t grid1, grid2, total1, total2;
    std::vector<int32_t> tiles4;           // prefix sums of the folded 1-D tensors' tiles (their own update launch)
    int32_t last_launches;
    bool ptrs_valid;
    std::vector<void*> params, grads;  // what the device-side pointer arrays currently hold
    std::vector<void*> params16;       // likewise for the optional bfloat16 copies (empty until first used)
    bool params_a32 = false, grads_a32 = false;   // all current parameter / gradient pointers are 32-byte aligned
    size_t stage_bytes;
    std::vector<size_t> stage_off;
    bool fused = false;                    // the state runs the fused schedule (one launch per step)
    int32_t work_total = 0;                // items of the work list
    bool new_rc_clean = false;             // the scale buffer that receives the next step's maxima is known to be zero
    uint32_t epoch = 0;                    // fused launches made on this state (the per-tensor counters count along)
    int32_t sms, occ1, occ2;
    int32_t p1_ctas;                       // which instantiation of the maxima pass (2 or 3 CTAs per SM)
    std::vector<int32_t> tiles7;           // prefix sums of the update tiles of the element-indexed tensors
    std::vector<int32_t> tiles6;           // prefix sums of the composite tensors' 256-entry chunks of expanded statistics
    std::vector<int32_t> tiles5;           // prefix sums of the factorized tensors' 32-statistic chunks (finalize kernel)
    std::vector<int32_t> tiles1, tiles2, tiles3;   // host copies of the tile prefix sums (3: element-indexed tiles of every tensor)
    cudaStream_t aux = nullptr;            // overlapped schedule: the stream of the maxima passes (lazily created)
    std::vector<cudaEvent_t> ov_events;    // overlapped schedule: per group {maxima done, update done}, then the fork event
    std::vector<int32_t> group_cut;        // overlapped schedule: first tensor of every group, then n
    cudaStream_t copy_in, copy_out;        // lazily created by the host-buffer entry point
    std::vector<cudaEvent_t> host_events;
    bool profile;                          // record events around each kernel of a step
    std::vector<cudaEvent_t> prof_events;  // ring of 4 per recorded step: start, after pass 1, after rcp, after pass 2
    size_t prof_used = 0;                  // events of the ring in use since the last read
};

namespace {

constexpr size_t kProfRingSteps = 256;     // steps that can be recorded between two reads

// The work list of the fused schedule, built by a small simulation of the hand-out. Two streams are merged: the
// maxima tiles of the rank-1 tensors in table order, and the update tiles of the same tensors in the same order (inside
// a tensor: last rows first - the maxima pass read them last, so they are the likeliest to be in L2).
//   - An update tile may only be listed once its tensor's maxima tiles are all listed, and then at least `gap` items
//     later, so that the maxima tiles still running when it is handed out have time to finish (else the CTA waits).
//   - The maxima stream runs ahead until `lead` elements of update work are ready, and no further: what it has read
//     should still be in L2 when the update pass comes for it. While both streams have something to list they alternate.
//   - A maxima tile is flagged "keep" when it lies in the last `keep` bytes (gradient + codes) of its tensor's maxima
//     pass: only what can still be in L2 when the update pass arrives asks for it.
// The update tiles of everything else (fp32 and block-wise tensors: no dependencies) come last.
void build_work_list(const lpmm_state* st, const std::vector<TilePlan>& plans, std::vector<uint2>* work) {
    const lpmm_config& cfg = st->cfg;
    const int32_t n = st->n;
    std::vector<int32_t> rank1;
    for (int32_t i = 0; i < n; ++i)
        if (plans[i].tiles_maxima > 0) rank1.push_back(i);
    const int64_t keep_bytes = (cfg.l2_keep_mbytes > 0 ? (int64_t)cfg.l2_keep_mbytes : 48) << 20;
    const int64_t lead_elems = (cfg.lead_melems > 0 ? (int64_t)cfg.lead_melems : 30) << 20;
    const int64_t gap = cfg.gap_items > 0 ? cfg.gap_items : 2 * kPlanResidentCtas;
    work->clear();
    auto tile_elems1 = [&](int32_t t) {
        const TilePlan& p = plans[t];
        return (p.wx > 0) ? (int64_t)p.tile_rows1 * kWarpElems * p.wx : (int64_t)p.flat_chunks * kWarps * kWarpElems;
    };
    size_t k1 = 0, k2 = 0;             // tensors (positions in rank1) the two streams are at
    int64_t i1 = 0, i2 = 0;            // next tile inside them
    int64_t ready = 0;                 // elements of update work whose maxima tiles are all listed
    std::vector<int64_t> complete_at(rank1.size(), -1);   // list position of a tensor's last maxima tile
    bool turn_update = true;
    while (k1 < rank1.size() || k2 < rank1.size()) {
        const bool have1 = k1 < rank1.size();
        const bool want1 = have1 && ready < lead_elems;
        bool can2 = k2 < rank1.size() && complete_at[k2] >= 0;
        if (can2 && i2 == 0 && (int64_t)work->size() - complete_at[k2] < gap && have1) can2 = false;   // too early (unless nothing else is left)
        bool emit_update;
        if (want1 && can2) { emit_update = turn_update; turn_update = !turn_update; }
        else if (want1) emit_update = false;
        else if (can2) emit_update = true;
        else emit_update = !have1;     // neither wanted nor allowed: run the maxima stream further ahead if it has anything
        if (emit_update) {
            const int32_t t = rank1[k2];
            const int64_t n2 = plans[t].tiles_update;
            work->push_back(make_uint2((uint32_t)t | kWorkUpdate, (uint32_t)(n2 - 1 - i2)));
            ready -= st->L.t[t].numel / n2;
            if (++i2 == n2) { ++k2; i2 = 0; }
        } else {
            const int32_t t = rank1[k1];
            const int64_t n1 = plans[t].tiles_maxima;
            // bytes of gradient (counted at 2 per element) and codes from this tile to the end of the tensor's pass
            const int64_t after = (n1 - i1) * tile_elems1(t) * 5 / 2;
            work->push_back(make_uint2((uint32_t)t | (after <= keep_bytes ? kWorkKeep : 0u), (uint32_t)i1));
            if (++i1 == n1) {
                complete_at[k1] = (int64_t)work->size() - 1;
                ready += st->L.t[t].numel;
                ++k1; i1 = 0;
            }
        }
    }
    for (int32_t i = 0; i < n; ++i) {
        if (plans[i].tiles_maxima > 0 || st->L.t[i].kind == K_BLOCK_TILED) continue;
        for (int64_t j = 0; j < plans[i].tiles_update; ++j) work->push_back(make_uint2((uint32_t)i | kWorkUpdate, (uint32_t)j));
    }
}

// Fills descriptors and tile tables, and uploads them. Tile sizes adapt to the amount of work so that
// small parameter sets still spread over the whole GPU.
lpmm_status build_tables(lpmm_state* st, cudaStream_t s) {
    int dev = 0, sms = 0, occ1 = 1, occ2 = 1;
    LPMM_CUDA(cudaGetDevice(&dev));
    LPMM_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    {   // the tiled maxima path wants two CTAs per SM, the other pass-1 paths three: go by the elements of each
        int64_t tiled = 0, other = 0;
        for (int32_t i = 0; i < st->n; ++i) {
            const TensorLayout& t = st->L.t[i];
            if (t.kind == K_RANK1_FAST) tiled += t.numel;
            else if (t.kind == K_RANK1_FLAT || t.kind == K_FACT) other += t.numel;
        }
        st->p1_ctas = tiled >= other ? 2 : 3;
    }
    LPMM_CUDA(step_kernel_occupancy(st->p1_ctas, &occ1, &occ2));
    if (occ1 < 1) occ1 = 1;
    if (occ2 < 1) occ2 = 1;
    const int32_t n = st->n;
    int64_t total_elems = 0;
    for (int32_t i = 0; i < n; ++i) total_elems += st->L.t[i].numel;
    st->fused = wants_fused(st->cfg, total_elems) && st->L.work_items > 0 && st->L.work_items <= 0x7fffffffLL;
    int64_t flat_elems = 0;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t k = st->L.t[i].kind;
        if (k == K_RANK1_FLAT || k == K_BLOCK) flat_elems += st->L.t[i].numel;
    }
    const TileSizes ts = choose_tile_sizes(st->cfg, total_elems, flat_elems, st->fused);

    std::vector<TensorDesc> descs(n);
    std::vector<TilePlan> plans(n);
    std::vector<int32_t> t1(n + 1, 0), t2(n + 1, 0), t3(n + 1, 0), t4(n + 1, 0), t5(n + 1, 0), t6(n + 1, 0), t7(n + 1, 0);
    // In a state whose matrices are not block-wise, folded 1-D tensors leave the main update launch (0 tiles there)
    // and get one of their own with the block-wise kernel (table 4).
    const bool own_launch = st->cfg.v_mode != LPMM_V_BLOCK;
    char* A = st->arena;
    for (int32_t i = 0; i < n; ++i) {
        const TensorLayout& t = st->L.t[i];
        TensorDesc& d = descs[i];
        std::memset(&d, 0, sizeof(d));
        d.rows = t.rows; d.cols = t.cols; d.numel = t.numel; d.kind = t.kind; d.c_off = t.c_off;
        d.n_outer = t.n_outer;
        for (int a = 0; a < 3; ++a) { d.outer_dim[a] = t.outer_dim[a]; d.outer_off[a] = t.outer_off[a]; }
        d.m_shift = (st->cfg.m_block == 2048) ? 11 : 7;
        d.dbg_status = reinterpret_cast<uint32_t*>(A);
        d.p1_tiled = t.p1_tiled ? 1 : 0;
        if (t.kind == K_FP32) {
            d.m32 = reinterpret_cast<float*>(A + t.m32);
            d.v32 = reinterpret_cast<float*>(A + t.v32);
        } else {
            d.m_codes = reinterpret_cast<uint8_t*>(A + t.m_codes);
            d.v_codes = (t.kind == K_FACT) ? nullptr : reinterpret_cast<uint8_t*>(A + t.v_codes);
            d.m_scale = reinterpret_cast<float*>(A + t.m_scale);
            if (t.kind == K_BLOCK || t.kind == K_BLOCK_TILED) d.v_bscale = reinterpret_cast<float*>(A + t.v_bscale);
            if (uses_rc(t.kind)) {
                d.rc[0] = reinterpret_cast<float*>(A + st->L.rc[0]) + t.rc_index;
                d.rc[1] = reinterpret_cast<float*>(A + st->L.rc[1]) + t.rc_index;
                d.rc[2] = reinterpret_cast<float*>(A + st->L.rc[2]) + t.rc_index;
                d.rcp_new = reinterpret_cast<float*>(A + st->L.rcp) + t.rc_index;
                d.rc_floats = t.rc_len;
            }
            if (t.nd_split > 0) {
                d.exp_old = reinterpret_cast<float*>(A + t.exp_old);
                d.exp_new = reinterpret_cast<float*>(A + t.exp_new);
                d.rcp_new = reinterpret_cast<float*>(A + t.exp_rcp);
                d.exp_len = t.exp_len;
                d.nd = t.nd; d.nd_split = t.nd_split;
                for (int a = 0; a < 4; ++a) { d.nd_dim[a] = t.nd_dim[a]; d.nd_off[a] = t.nd_off[a]; }
            }
            if (t.kind == K_FACT) {
                d.fact_rowpart = reinterpret_cast<float*>(A + t.fact_rowpart);
                d.fact_colpart = reinterpret_cast<float*>(A + t.fact_colpart);
                d.fact_blockpart = reinterpret_cast<double*>(A + t.fact_blockpart);
                d.fact_nstrips = t.fact_nstrips;
                d.fact_tiles_y = t.fact_tiles_y;
            }
        }
        const TilePlan p = plan_tensor(st->cfg, t, ts);
        plans[i] = p;
        d.wx = p.wx; d.tiles_x = p.tiles_x; d.tile_rows = p.tile_rows; d.tile_rows1 = p.tile_rows1;
        d.flat_chunks = p.flat_chunks;
        if (p.tiles_update > 0x7fffffffLL || p.tiles_maxima > 0x7fffffffLL || p.tiles_flat > 0x7fffffffLL) return LPMM_ERR_UNSUPPORTED;
        d.tiles1 = (int32_t)p.tiles_maxima;
        d.tiles2 = (int32_t)p.tiles_update;
        if (t3[i] + p.tiles_flat > 0x7fffffffLL) return LPMM_ERR_UNSUPPORTED;
        t3[i + 1] = t3[i] + (int32_t)p.tiles_flat;
        if (t2[i] + p.tiles_update > 0x7fffffffLL) return LPMM_ERR_UNSUPPORTED;
        const bool moved = own_launch && t.kind == K_BLOCK_TILED;
        const bool on_tiled_path = t.kind == K_RANK1_FAST || t.kind == K_FACT || t.kind == K_BLOCK_TILED || t.kind == K_FP32;
        t2[i + 1] = t2[i] + ((moved || !on_tiled_path) ? 0 : (int32_t)p.tiles_update);
        t7[i + 1] = t7[i] + (on_tiled_path ? 0 : (int32_t)p.tiles_update);
        t4[i + 1] = t4[i] + (moved ? (int32_t)p.tiles_update : 0);
        if (t1[i] + p.tiles_maxima > 0x7fffffffLL) return LPMM_ERR_UNSUPPORTED;
        t1[i + 1] = t1[i] + (int32_t)p.tiles_maxima;
        t5[i + 1] = t5[i] + (t.kind == K_FACT ? (d.rc_floats + 31) / 32 : 0);
        t6[i + 1] = t6[i] + (t.nd_split > 0 ? (t.exp_len + 255) / 256 : 0);
        if (t.kind == K_FACT && (int64_t)d.tile_rows1 * d.fact_tiles_y < t.rows) return LPMM_ERR_UNSUPPORTED;   // (layout and plan disagree)
    }
    st->total1 = t1[n];
    st->total2 = t2[n];
    st->grid1 = st->total1 < sms * occ1 ? st->total1 : sms * occ1;
    st->grid2 = st->total2 < sms * occ2 ? st->total2 : sms * occ2;
    st->sms = sms; st->occ1 = occ1; st->occ2 = occ2;
    st->tiles1 = t1;
    st->tiles2 = t2;
    st->tiles3 = t3;
    st->tiles4 = t4;
    st->tiles5 = t5;
    st->tiles6 = t6;
    st->tiles7 = t7;
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles7, t7.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles6, t6.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles5, t5.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    {   // overlapped schedule: consecutive groups of about equal size, each with at least one maxima tile
        int32_t groups = st->cfg.overlap_groups > 0 ? st->cfg.overlap_groups : 8;
        st->group_cut.assign(1, 0);
        const int64_t per_group = total_elems / groups + 1;
        int64_t acc = 0;
        for (int32_t i = 0; i < n; ++i) {
            acc += st->L.t[i].numel;
            if (acc >= per_group && i + 1 < n && t1[i + 1] > t1[st->group_cut.back()]) { st->group_cut.push_back(i + 1); acc = 0; }
        }
        if (t1[n] == t1[st->group_cut.back()] && st->group_cut.size() > 1) st->group_cut.pop_back();   // no maxima work in the tail
        st->group_cut.push_back(n);
    }
    if (st->fused) {
        std::vector<uint2> work;
        build_work_list(st, plans, &work);
        if ((int64_t)work.size() > st->L.work_items) return LPMM_ERR_ARENA_TOO_SMALL;   // cannot happen: same plan as the layout
        st->work_total = (int32_t)work.size();
        LPMM_CUDA(cudaMemcpyAsync(A + st->L.work, work.data(), sizeof(uint2) * work.size(), cudaMemcpyHostToDevice, s));
        LPMM_CUDA(cudaStreamSynchronize(s));   // `work` is about to go out of scope
    }
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles4, t4.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles3, t3.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.descs, descs.data(), sizeof(TensorDesc) * n, cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles1, t1.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    LPMM_CUDA(cudaMemcpyAsync(A + st->L.tiles2, t2.data(), sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, s));
    // the vectors above are pageable memory: the runtime stages such copies before returning
    return LPMM_OK;
}

lpmm_status make_state(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n, void* d_arena, size_t arena_bytes,
                       bool fresh, int32_t phase, lpmm_state** out, void* stream) {
    if (!out) return LPMM_ERR_INVALID_ARG;
    *out = nullptr;
    lpmm_status v = validate_config(cfg, shapes, n);
    if (v != LPMM_OK) return v;
    if (!d_arena) return LPMM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d_arena) % kAlign != 0) return LPMM_ERR_ALIGNMENT;
    if (phase < 0 || phase > 2) return LPMM_ERR_INVALID_ARG;
    lpmm_state* st = new (std::nothrow) lpmm_state();
    if (!st) return LPMM_ERR_INVALID_ARG;
    st->cfg = *cfg;
    st->n = n;
    compute_layout(*cfg, shapes, n, &st->L);
    if (arena_bytes < st->L.total) { delete st; return LPMM_ERR_ARENA_TOO_SMALL; }
    st->arena = static_cast<char*>(d_arena);
    st->arena_bytes = arena_bytes;
    st->phase = phase;
    st->last_launches = 0;
    st->profile = false;
    st->copy_in = nullptr;
    st->copy_out = nullptr;
    st->ptrs_valid = false;
    st->params.assign(n, nullptr);
    st->grads.assign(n, nullptr);
    st->stage_off.resize(n);
    size_t so = 0;
    for (int32_t i = 0; i < n; ++i) { st->stage_off[i] = so; so = align_up(so + 4 * (size_t)st->L.t[i].numel); }
    st->stage_bytes = so;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    lpmm_status rc = LPMM_OK;
    if (fresh) {
        // s_0 = 0 (Alg. 1): every scale 0, second-moment codes 0, fp32 states 0 ...
        cudaError_t e = cudaMemsetAsync(d_arena, 0, st->L.total, s);
        // ... and first-moment codes = 7, the zero entry of the signed table (an odd tail keeps nibble 0).
        for (int32_t i = 0; i < n && e == cudaSuccess; ++i) {
            const TensorLayout& t = st->L.t[i];
            if (t.kind == K_FP32) continue;
            e = cudaMemsetAsync(st->arena + t.m_codes, 0x77, (size_t)(t.numel / 2), s);
            if (e == cudaSuccess && (t.numel & 1))
                e = cudaMemsetAsync(st->arena + t.m_codes + t.numel / 2, 0x07, 1, s);
        }
        for (size_t k = 0; k < st->L.guards.size() && e == cudaSuccess; ++k)
            e = cudaMemsetAsync(st->arena + st->L.guards[k], kGuardByte, kAlign, s);
        if (e != cudaSuccess) rc = cuda_fail(e);
    } else {
        // An attached arena must describe itself as what the caller says it is ...
        ArenaHeader hd;
        cudaError_t e = cudaMemcpyAsync(&hd, d_arena, sizeof(hd), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) {
            rc = cuda_fail(e);
        } else if (hd.magic != kArenaMagic || hd.version != kArenaLayoutVersion || hd.total_bytes != st->L.states_end ||
                   hd.shape_hash != st->L.shape_hash || hd.n_tensors != n || hd.m_block != cfg->m_block ||
                   hd.v_mode != cfg->v_mode) {
            rc = LPMM_ERR_INVALID_ARG;
        } else {
            // ... and keeps its states; the status word, the tile counters, the progress counters and the scale buffer
            // that receives the next step's maxima start clean.
            e = cudaMemsetAsync(d_arena, 0, 32, s);
            if (e == cudaSuccess) e = cudaMemsetAsync(st->arena + offsetof(ArenaHeader, wait_stats), 0, 16, s);
            if (e == cudaSuccess) e = cudaMemsetAsync(st->arena + st->L.tsync, 0, sizeof(TensorSync) * n, s);
            for (int k = 1; k <= 2 && e == cudaSuccess && st->L.rc_floats > 0; ++k)
                e = cudaMemsetAsync(st->arena + st->L.rc[(phase + k) % 3], 0, sizeof(float) * (size_t)st->L.rc_floats, s);
            if (e != cudaSuccess) rc = cuda_fail(e);
        }
    }
    if (rc == LPMM_OK && fresh) {
        ArenaHeader hd;
        std::memset(&hd, 0, sizeof(hd));
        hd.magic = kArenaMagic; hd.version = kArenaLayoutVersion; hd.total_bytes = st->L.states_end;
        hd.shape_hash = st->L.shape_hash; hd.n_tensors = n; hd.m_block = cfg->m_block; hd.v_mode = cfg->v_mode;
        const cudaError_t e = cudaMemcpyAsync(d_arena, &hd, sizeof(hd), cudaMemcpyHostToDevice, s);   // pageable: staged before return
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    st->new_rc_clean = true;
    if (rc == LPMM_OK) rc = build_tables(st, s);
    if (rc != LPMM_OK) { delete st; return rc; }
    *out = st;
    return LPMM_OK;
}

bool finite_nonneg(float x) { return std::isfinite(x) && x >= 0.0f; }

// Polls of a device-side wait before it gives up (each poll is an L2 round trip plus a short sleep: about two
// seconds in all, far beyond any legitimate wait, which is bounded by the duration of one tile).
constexpr uint32_t kSpinLimit = 1u << 22;

}  // namespace

extern "C" {

lpmm_status lpmm_state_bytes(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n, size_t* arena_bytes) {
    if (!arena_bytes) return LPMM_ERR_INVALID_ARG;
    lpmm_status v = validate_config(cfg, shapes, n);
    if (v != LPMM_OK) return v;
    Layout L;
    compute_layout(*cfg, shapes, n, &L);
    *arena_bytes = L.total;
    return LPMM_OK;
}

lpmm_status lpmm_state_init(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n,
                            void* d_arena, size_t arena_bytes, lpmm_state** out, void* stream) {
    return make_state(cfg, shapes, n, d_arena, arena_bytes, true, 0, out, stream);
}

lpmm_status lpmm_state_attach(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n,
                              void* d_arena, size_t arena_bytes, int32_t phase, lpmm_state** out, void* stream) {
    return make_state(cfg, shapes, n, d_arena, arena_bytes, false, phase, out, stream);
}

}  // extern "C" (reopened below)

namespace {

lpmm_status check_step_args(const lpmm_state* st, const void* p, const void* g, int32_t grad_dtype, float lr, float beta1,
                            float beta2, float eps, float weight_decay, int64_t step) {
    if (!st || !p || !g) return LPMM_ERR_INVALID_ARG;
    if (grad_dtype != LPMM_F32 && grad_dtype != LPMM_BF16) return LPMM_ERR_INVALID_ARG;
    if (step < 1) return LPMM_ERR_INVALID_ARG;
    if (!finite_nonneg(lr) || !finite_nonneg(eps) || !finite_nonneg(weight_decay)) return LPMM_ERR_INVALID_ARG;
    if (!finite_nonneg(beta1) || !finite_nonneg(beta2) || beta1 >= 1.0f || beta2 >= 1.0f) return LPMM_ERR_INVALID_ARG;
    return LPMM_OK;
}

// Makes the device-side pointer arrays hold these parameter / gradient pointers (uploads only on change).
lpmm_status set_pointers(lpmm_state* st, void* const* d_params, const void* const* d_grads, cudaStream_t s) {
    const int32_t n = st->n;
    bool changed = !st->ptrs_valid;
    for (int32_t i = 0; i < n; ++i) {
        if (!d_params[i] || !d_grads[i]) return LPMM_ERR_INVALID_ARG;
        if (!aligned16(d_params[i]) || !aligned16(d_grads[i])) return LPMM_ERR_ALIGNMENT;
        if (d_params[i] != st->params[i] || d_grads[i] != st->grads[i]) changed = true;
    }
    if (changed) {
        bool pa = true, ga = true;
        for (int32_t i = 0; i < n; ++i) {
            st->params[i] = d_params[i]; st->grads[i] = const_cast<void*>(d_grads[i]);
            pa = pa && (reinterpret_cast<uintptr_t>(d_params[i]) & 31u) == 0;
            ga = ga && (reinterpret_cast<uintptr_t>(d_grads[i]) & 31u) == 0;
        }
        st->params_a32 = pa; st->grads_a32 = ga;
        st->ptrs_valid = false;
        LPMM_CUDA(cudaMemcpyAsync(st->arena + st->L.params, st->params.data(), sizeof(void*) * n, cudaMemcpyHostToDevice, s));
        LPMM_CUDA(cudaMemcpyAsync(st->arena + st->L.grads, st->grads.data(), sizeof(void*) * n, cudaMemcpyHostToDevice, s));
        st->ptrs_valid = true;
    }
    return LPMM_OK;
}

StepArgs make_args(const lpmm_state* st, float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step) {
    StepArgs a;
    a.descs = reinterpret_cast<const TensorDesc*>(st->arena + st->L.descs);
    a.params = reinterpret_cast<float* const*>(st->arena + st->L.params);
    a.params_bf16 = nullptr;
    a.grads = reinterpret_cast<const void* const*>(st->arena + st->L.grads);
    a.n_tensors = st->n;
    a.sel.old_i = st->phase;
    a.sel.new_i = (st->phase + 1) % 3;
    a.sel.zero_i = (st->phase + 2) % 3;
    a.epoch = 0;
    a.l2_hints = st->cfg.no_l2_hints ? 0 : 1;
    a.wait_stats = reinterpret_cast<unsigned long long*>(st->arena + offsetof(ArenaHeader, wait_stats));
    a.work = reinterpret_cast<const uint2*>(st->arena + st->L.work);
    a.tsync = reinterpret_cast<TensorSync*>(st->arena + st->L.tsync);
    a.spin_limit = kSpinLimit;
    a.aligned32 = 0;   // set by the callers that know the gradient type
    a.dev_status = reinterpret_cast<uint32_t*>(st->arena);
    a.tile_counter = reinterpret_cast<int32_t*>(st->arena + 16);   // header block: [status | .. | counters]
    a.h.lr = lr; a.h.beta1 = beta1; a.h.beta2 = beta2; a.h.eps = eps;
    a.h.omb1 = 1.0f - beta1;
    a.h.omb2 = 1.0f - beta2;
    const double bc1 = 1.0 - std::pow((double)beta1, (double)step);   // Eq. 1: 1 - beta^t
    const double bc2 = 1.0 - std::pow((double)beta2, (double)step);
    a.h.bc1 = (float)bc1;
    a.h.bc2 = (float)bc2;
    a.h.decay = 1.0f - lr * weight_decay;
    a.h.one = 1.0f;
    a.h.step_size = (float)((double)lr / bc1);
    a.h.rbc2 = (float)(1.0 / bc2);
    const double step_size = (double)lr / bc1;
    a.h.upd_c1 = step_size > 0.0 ? (float)(-std::sqrt(1.0 / bc2) / step_size) : 0.0f;
    a.h.upd_e1 = step_size > 0.0 ? (float)(-(double)eps / step_size) : 0.0f;
    a.h2 = make_hyper2(a.h);
    return a;
}

// The approximate update flushes a denormal v^ before the square root (only safe with a real eps) and divides its
// constants by the step size (only possible when that is a normal number): otherwise Eq. 1 is evaluated as written.
bool wants_ieee_update(const lpmm_state* st, const Hyper& h) {
    if (st->cfg.update_math == LPMM_UPDATE_IEEE) return true;
    if (h.eps < 1e-30f || h.step_size < 1e-30f) return true;
    return !(std::isfinite(h.upd_c1) && std::isfinite(h.upd_e1));
}

// Enqueues the maxima pass of tensors [t0, t1) and what follows it (clearing of the new r, c before; their
// reciprocals, or the factorized statistics, after). grid_cap: most CTAs to launch. aux: the launch may run beside
// another step kernel and uses the second pair of tile counters. ev (2 events or nullptr) brackets the maxima kernel.
lpmm_status enqueue_maxima(lpmm_state* st, StepArgs a, int32_t t0, int32_t t1, bool bf16, int32_t grid_cap, bool aux,
                           cudaStream_t s, cudaEvent_t* ev, int32_t* launches) {
    a.aligned32 = (st->params_a32 && (bf16 || st->grads_a32)) ? 1 : 0;
    if (aux) a.tile_counter = reinterpret_cast<int32_t*>(st->arena + offsetof(ArenaHeader, tile_counter_aux));
    const int32_t p1_begin = st->tiles1[t0], p1_end = st->tiles1[t1];
    if (p1_end <= p1_begin) {
        if (ev) { LPMM_CUDA(cudaEventRecord(ev[0], s)); LPMM_CUDA(cudaEventRecord(ev[1], s)); }
        return LPMM_OK;
    }
    // the rank-1 scale region of these tensors is one contiguous range of the scale buffers
    int64_t rc_begin = -1, rc_end = 0;
    for (int32_t i = t0; i < t1; ++i) {
        const TensorLayout& t = st->L.t[i];
        if (!uses_rc(t.kind)) continue;
        if (rc_begin < 0) rc_begin = t.rc_index;
        rc_end = (t.rc_index + t.rc_len + 63) / 64 * 64;
    }
    float* rc_new = reinterpret_cast<float*>(st->arena + st->L.rc[(st->phase + 1) % 3]) + rc_begin;
    const bool factored = st->cfg.v_mode == LPMM_V_FACTORED;    // (its sums are written, not accumulated: nothing to clear)
    if (!factored) LPMM_CUDA(cudaMemsetAsync(rc_new, 0, sizeof(float) * (size_t)(rc_end - rc_begin), s));
    const bool composite = st->tiles6[t1] > st->tiles6[t0];
    StepArgs nd_args = a;
    if (composite) {   // expanded current statistics of the composite tensors; their expanded accumulators start at zero
        nd_args.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles6);
        nd_args.tile_begin = st->tiles6[t0];
        nd_args.tile_end = st->tiles6[t1];
        LPMM_CUDA(launch_nd_stats(nd_args, 0, s));
        *launches += 1;
    }
    if (ev) LPMM_CUDA(cudaEventRecord(ev[0], s));
    a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles1);
    a.tile_begin = p1_begin;
    a.tile_end = p1_end;
    const int32_t tiles = p1_end - p1_begin;
    LPMM_CUDA(launch_pass1(a, bf16, st->p1_ctas, tiles < grid_cap ? tiles : grid_cap, s));
    if (ev) LPMM_CUDA(cudaEventRecord(ev[1], s));
    if (factored) {   // partial sums -> statistics' moving averages, sum(R), row factors R_i / sum(R): one small kernel
        a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles5);
        a.tile_begin = st->tiles5[t0];
        a.tile_end = st->tiles5[t1];
        LPMM_CUDA(launch_factor_finalize(a, s));
        *launches += 2;
    } else {
        LPMM_CUDA(launch_rcp(rc_new, reinterpret_cast<float*>(st->arena + st->L.rcp) + rc_begin, rc_end - rc_begin, s));
        *launches += 2;
        if (composite) {   // row / column maxima -> per-axis maxima (Alg. 4), then their expanded reciprocals
            LPMM_CUDA(launch_nd_stats(nd_args, 1, s));
            LPMM_CUDA(launch_nd_stats(nd_args, 2, s));
            *launches += 2;
        }
    }
    return LPMM_OK;
}

// Enqueues the update pass of tensors [t0, t1) (and the folded 1-D tensors' own launch).
lpmm_status enqueue_update(lpmm_state* st, StepArgs a, int32_t t0, int32_t t1, bool bf16, bool ieee_update,
                           cudaStream_t s, int32_t* launches) {
    a.aligned32 = (st->params_a32 && (bf16 || st->grads_a32)) ? 1 : 0;
    a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles2);
    a.tile_begin = st->tiles2[t0];
    a.tile_end = st->tiles2[t1];
    const int32_t cap = st->sms * st->occ2, tiles = a.tile_end - a.tile_begin;
    LPMM_CUDA(launch_pass2(a, bf16, ieee_update, st->cfg.m_block == 2048 ? 11 : 7,
                           st->cfg.v_mode == LPMM_V_FACTORED ? 1 : (st->cfg.v_mode == LPMM_V_BLOCK ? 2 : 0),
                           tiles < cap ? tiles : cap, s));
    if (tiles > 0) *launches += 1;
    if (st->tiles7[t1] > st->tiles7[t0]) {   // the element-indexed tensors: a kernel (and launch) of their own
        a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles7);
        a.tile_begin = st->tiles7[t0];
        a.tile_end = st->tiles7[t1];
        const int32_t tiles7 = a.tile_end - a.tile_begin;
        LPMM_CUDA(launch_pass2(a, bf16, ieee_update, st->cfg.m_block == 2048 ? 11 : 7, 3, tiles7 < cap ? tiles7 : cap, s));
        *launches += 1;
    }
    if (st->tiles4[t1] > st->tiles4[t0]) {   // folded 1-D tensors of a state that is not block-wise
        a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles4);
        a.tile_begin = st->tiles4[t0];
        a.tile_end = st->tiles4[t1];
        const int32_t tiles4 = a.tile_end - a.tile_begin;
        LPMM_CUDA(launch_pass2(a, bf16, ieee_update, st->cfg.m_block == 2048 ? 11 : 7, 2, tiles4 < cap ? tiles4 : cap, s));
        *launches += 1;
    }
    return LPMM_OK;
}

// Enqueues the kernels of one step for tensors [t0, t1) one after the other. ev (4 events or nullptr) brackets them.
lpmm_status enqueue_range(lpmm_state* st, StepArgs a, int32_t t0, int32_t t1, bool bf16, bool ieee_update,
                          cudaStream_t s, cudaEvent_t* ev, int32_t* launches) {
    lpmm_status rc = enqueue_maxima(st, a, t0, t1, bf16, st->sms * st->occ1, false, s, ev, launches);
    if (rc != LPMM_OK) return rc;
    if (ev) LPMM_CUDA(cudaEventRecord(ev[2], s));
    rc = enqueue_update(st, a, t0, t1, bf16, ieee_update, s, launches);
    if (rc != LPMM_OK) return rc;
    if (ev) LPMM_CUDA(cudaEventRecord(ev[3], s));
    return LPMM_OK;
}

// The overlapped two-pass schedule: the tensor list is cut into groups; the maxima pass of group k + 1 runs on a second
// stream beside the update pass of group k (the two kernels share every SM, one CTA each: the maxima pass is bound by
// instruction issue, the update pass by DRAM). Nothing waits on the device; the order is kept by events:
//   aux:  maxima(0) | maxima(1) after update(-)... each maxima(k+1) starts when update(k-1) has finished
//   main: update(k) after maxima(k)
lpmm_status enqueue_overlapped(lpmm_state* st, const StepArgs& a, bool bf16, bool ieee_update, cudaStream_t s, int32_t* launches) {
    if (!st->aux) LPMM_CUDA(cudaStreamCreateWithFlags(&st->aux, cudaStreamNonBlocking));
    const std::vector<int32_t>& cut = st->group_cut;
    const size_t groups = cut.size() - 1;
    while (st->ov_events.size() < 2 * groups + 1) {
        cudaEvent_t e;
        LPMM_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        st->ov_events.push_back(e);
    }
    cudaEvent_t ev_fork = st->ov_events[2 * groups];
    LPMM_CUDA(cudaEventRecord(ev_fork, s));              // earlier work on the caller's stream comes first
    LPMM_CUDA(cudaStreamWaitEvent(st->aux, ev_fork, 0));
    lpmm_status rc = enqueue_maxima(st, a, cut[0], cut[1], bf16, st->sms * st->occ1, true, st->aux, nullptr, launches);
    if (rc != LPMM_OK) return rc;
    LPMM_CUDA(cudaEventRecord(st->ov_events[0], st->aux));
    for (size_t k = 0; k < groups; ++k) {
        cudaEvent_t ev_m = st->ov_events[2 * k], ev_u = st->ov_events[2 * k + 1];
        if (k + 1 < groups) {    // the next group's maxima pass: beside this group's update pass, one CTA per SM
            if (k > 0) LPMM_CUDA(cudaStreamWaitEvent(st->aux, st->ov_events[2 * (k - 1) + 1], 0));
            rc = enqueue_maxima(st, a, cut[k + 1], cut[k + 2], bf16, st->sms, true, st->aux, nullptr, launches);
            if (rc != LPMM_OK) return rc;
            LPMM_CUDA(cudaEventRecord(st->ov_events[2 * (k + 1)], st->aux));
        }
        LPMM_CUDA(cudaStreamWaitEvent(s, ev_m, 0));
        rc = enqueue_update(st, a, cut[k], cut[k + 1], bf16, ieee_update, s, launches);
        if (rc != LPMM_OK) return rc;
        LPMM_CUDA(cudaEventRecord(ev_u, s));
    }
    return LPMM_OK;   // the caller's stream ends after the last update; the second stream has nothing left in flight
}

// Makes the device-side array of bfloat16-copy pointers hold d_params16 (uploads only on change).
lpmm_status set_pointers16(lpmm_state* st, void* const* d_params16, cudaStream_t s) {
    const int32_t n = st->n;
    bool changed = st->params16.empty();
    if (changed) st->params16.assign(n, nullptr);
    for (int32_t i = 0; i < n; ++i) {
        if (!d_params16[i]) return LPMM_ERR_INVALID_ARG;
        if (!aligned16(d_params16[i])) return LPMM_ERR_ALIGNMENT;
        if (d_params16[i] != st->params16[i]) changed = true;
    }
    if (changed) {
        for (int32_t i = 0; i < n; ++i) st->params16[i] = d_params16[i];
        const cudaError_t e = cudaMemcpyAsync(st->arena + st->L.params16, st->params16.data(), sizeof(void*) * n, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) { st->params16.clear(); return cuda_fail(e); }
    }
    return LPMM_OK;
}

lpmm_status adamw4_step_impl(lpmm_state* st, void* const* d_params, void* const* d_params16, const void* const* d_grads,
                             int32_t grad_dtype, float lr, float beta1, float beta2, float eps,
                             float weight_decay, int64_t step, void* stream) {
    lpmm_status rc = check_step_args(st, d_params, d_grads, grad_dtype, lr, beta1, beta2, eps, weight_decay, step);
    if (rc != LPMM_OK) return rc;
    if (d_params16 && st->cfg.v_mode == LPMM_V_FACTORED) return LPMM_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = set_pointers(st, d_params, d_grads, s);
    if (rc != LPMM_OK) return rc;
    if (d_params16) {
        rc = set_pointers16(st, d_params16, s);
        if (rc != LPMM_OK) return rc;
    }
    StepArgs a = make_args(st, lr, beta1, beta2, eps, weight_decay, step);
    if (d_params16) a.params_bf16 = reinterpret_cast<uint16_t* const*>(st->arena + st->L.params16);
    // Per-kernel timing: the next four events of the ring made by lpmm_state_profile (a full ring records nothing more).
    cudaEvent_t* ev = nullptr;
    if (st->profile && st->prof_used + 4 <= st->prof_events.size()) {
        ev = &st->prof_events[st->prof_used];
        st->prof_used += 4;
    }
    const bool ieee_update = wants_ieee_update(st, a.h);
    const bool bf16 = grad_dtype == LPMM_BF16;
    int32_t launches = 0;
    if (st->fused && !d_params16) {
        // One launch over the work list: maxima tiles and update tiles of every tensor, ordered by counters in the arena.
        if (!st->new_rc_clean && st->L.rc_floats > 0)
            LPMM_CUDA(cudaMemsetAsync(st->arena + st->L.rc[(st->phase + 1) % 3], 0, sizeof(float) * (size_t)st->L.rc_floats, s));
        a.aligned32 = (st->params_a32 && (bf16 || st->grads_a32)) ? 1 : 0;
        a.tile_begin = 0;
        a.tile_end = st->work_total;
        a.tile_start = nullptr;
        a.epoch = ++st->epoch;
        if (ev) { LPMM_CUDA(cudaEventRecord(ev[0], s)); LPMM_CUDA(cudaEventRecord(ev[1], s)); LPMM_CUDA(cudaEventRecord(ev[2], s)); }
        const int32_t cap = st->sms * st->occ2;
        LPMM_CUDA(launch_fused(a, bf16, ieee_update, st->work_total < cap ? st->work_total : cap, s));
        launches = 1;
        if (st->tiles4[st->n] > 0) {   // folded 1-D tensors: the block-wise form of the tiled update kernel
            a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles4);
            a.tile_end = st->tiles4[st->n];
            LPMM_CUDA(launch_pass2(a, bf16, ieee_update, 7, 2, a.tile_end < cap ? a.tile_end : cap, s));
            launches += 1;
        }
        if (ev) LPMM_CUDA(cudaEventRecord(ev[3], s));
        st->new_rc_clean = true;       // the maxima tiles have cleared the buffer the next step reduces into
    } else if (st->cfg.schedule == LPMM_SCHEDULE_OVERLAP && st->group_cut.size() > 2) {
        if (ev) { LPMM_CUDA(cudaEventRecord(ev[0], s)); LPMM_CUDA(cudaEventRecord(ev[1], s)); LPMM_CUDA(cudaEventRecord(ev[2], s)); }
        rc = enqueue_overlapped(st, a, bf16, ieee_update, s, &launches);
        if (rc != LPMM_OK) return rc;
        if (ev) LPMM_CUDA(cudaEventRecord(ev[3], s));
        st->new_rc_clean = false;
    } else {
        rc = enqueue_range(st, a, 0, st->n, bf16, ieee_update, s, ev, &launches);
        if (rc != LPMM_OK) return rc;
        st->new_rc_clean = false;
    }
    st->phase = (st->phase + 1) % 3;
    st->last_launches = launches;
    return LPMM_OK;
}

}  // namespace

extern "C" {

lpmm_status lpmm_adamw4_step(lpmm_state* st, void* const* d_params, const void* const* d_grads,
                             int32_t grad_dtype, float lr, float beta1, float beta2, float eps,
                             float weight_decay, int64_t step, void* stream) {
    return adamw4_step_impl(st, d_params, nullptr, d_grads, grad_dtype, lr, beta1, beta2, eps, weight_decay, step, stream);
}

lpmm_status lpmm_adamw4_step_bf16w(lpmm_state* st, void* const* d_params, void* const* d_params_bf16,
                                   const void* const* d_grads, int32_t grad_dtype, float lr, float beta1, float beta2,
                                   float eps, float weight_decay, int64_t step, void* stream) {
    if (!d_params_bf16) return LPMM_ERR_INVALID_ARG;
    return adamw4_step_impl(st, d_params, d_params_bf16, d_grads, grad_dtype, lr, beta1, beta2, eps, weight_decay, step, stream);
}

lpmm_status lpmm_sgdm4_step(lpmm_state* st, void* const* d_params, const void* const* d_grads,
                            int32_t grad_dtype, float lr, float beta, void* stream) {
    lpmm_status rc = check_step_args(st, d_params, d_grads, grad_dtype, lr, beta, 0.0f, 0.0f, 0.0f, 1);
    if (rc != LPMM_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = set_pointers(st, d_params, d_grads, s);
    if (rc != LPMM_OK) return rc;
    StepArgs a = make_args(st, lr, beta, 0.0f, 0.0f, 0.0f, 1);
    a.h2.neg_step = make_float2(-lr, -lr);
    a.aligned32 = (st->params_a32 && (grad_dtype == LPMM_BF16 || st->grads_a32)) ? 1 : 0;
    a.tile_start = reinterpret_cast<const int32_t*>(st->arena + st->L.tiles3);
    a.tile_begin = 0;
    a.tile_end = st->tiles3[st->n];
    const int32_t cap = st->sms * 3;
    LPMM_CUDA(launch_sgdm(a, grad_dtype == LPMM_BF16, a.tile_end < cap ? a.tile_end : cap, s));
    st->last_launches = 1;
    return LPMM_OK;
}

lpmm_status lpmm_stage_bytes(const lpmm_state* st, size_t* bytes) {
    if (!st || !bytes) return LPMM_ERR_INVALID_ARG;
    *bytes = st->stage_bytes;
    return LPMM_OK;
}

lpmm_status lpmm_adamw4_step_host(lpmm_state* st, void* const* h_params, const void* const* h_grads,
                                  int32_t grad_dtype, float lr, float beta1, float beta2, float eps,
                                  float weight_decay, int64_t step,
                                  void* d_param_stage, void* d_grad_stage, size_t stage_bytes, void* stream) {
    lpmm_status rc = check_step_args(st, h_params, h_grads, grad_dtype, lr, beta1, beta2, eps, weight_decay, step);
    if (rc != LPMM_OK) return rc;
    if (!d_param_stage || !d_grad_stage) return LPMM_ERR_INVALID_ARG;
    if (stage_bytes < st->stage_bytes) return LPMM_ERR_ARENA_TOO_SMALL;
    if (!aligned16(d_param_stage) || !aligned16(d_grad_stage)) return LPMM_ERR_ALIGNMENT;
    const int32_t n = st->n;
    for (int32_t i = 0; i < n; ++i) if (!h_params[i] || !h_grads[i]) return LPMM_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!st->copy_in) LPMM_CUDA(cudaStreamCreateWithFlags(&st->copy_in, cudaStreamNonBlocking));
    if (!st->copy_out) LPMM_CUDA(cudaStreamCreateWithFlags(&st->copy_out, cudaStreamNonBlocking));

    // Tensors are cut into consecutive groups of roughly equal size. Group k+1 is copied in and group k-1 is
    // copied out (the link is full duplex) while group k is updated: three streams chained by events.
    std::vector<int32_t> cut(1, 0);
    {
        int64_t total = 0;
        for (int32_t i = 0; i < n; ++i) total += st->L.t[i].numel;
        const int64_t per_group = total / 32 + 1;
        int64_t acc = 0;
        for (int32_t i = 0; i < n; ++i) {
            acc += st->L.t[i].numel;
            if (acc >= per_group || i == n - 1) { cut.push_back(i + 1); acc = 0; }
        }
    }
    const size_t groups = cut.size() - 1;
    const size_t need_events = 2 * groups + 2;
    while (st->host_events.size() < need_events) {
        cudaEvent_t e;
        LPMM_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        st->host_events.push_back(e);
    }
    cudaEvent_t ev_start = st->host_events[2 * groups], ev_end = st->host_events[2 * groups + 1];

    const size_t gsz = (grad_dtype == LPMM_BF16) ? 2 : 4;
    std::vector<void*> dp(n);
    std::vector<const void*> dg(n);
    for (int32_t i = 0; i < n; ++i) {
        dp[i] = static_cast<char*>(d_param_stage) + st->stage_off[i];
        dg[i] = static_cast<char*>(d_grad_stage) + st->stage_off[i];
    }
    rc = set_pointers(st, dp.data(), dg.data(), s);
    if (rc != LPMM_OK) return rc;
    const StepArgs a = make_args(st, lr, beta1, beta2, eps, weight_decay, step);
    const bool ieee_update = wants_ieee_update(st, a.h);

    LPMM_CUDA(cudaEventRecord(ev_start, s));                       // earlier work on the caller's stream comes first
    LPMM_CUDA(cudaStreamWaitEvent(st->copy_in, ev_start, 0));
    LPMM_CUDA(cudaStreamWaitEvent(st->copy_out, ev_start, 0));
    int32_t launches = 0;
    for (size_t k = 0; k < groups; ++k) {
        cudaEvent_t ev_in = st->host_events[2 * k], ev_done = st->host_events[2 * k + 1];
        for (int32_t i = cut[k]; i < cut[k + 1]; ++i) {
            const size_t numel = (size_t)st->L.t[i].numel;
            LPMM_CUDA(cudaMemcpyAsync(dp[i], h_params[i], 4 * numel, cudaMemcpyHostToDevice, st->copy_in));
            LPMM_CUDA(cudaMemcpyAsync(const_cast<void*>(dg[i]), h_grads[i], gsz * numel, cudaMemcpyHostToDevice, st->copy_in));
        }
        LPMM_CUDA(cudaEventRecord(ev_in, st->copy_in));
        LPMM_CUDA(cudaStreamWaitEvent(s, ev_in, 0));
        rc = enqueue_range(st, a, cut[k], cut[k + 1], grad_dtype == LPMM_BF16, ieee_update, s, nullptr, &launches);
        if (rc != LPMM_OK) return rc;
        LPMM_CUDA(cudaEventRecord(ev_done, s));
        LPMM_CUDA(cudaStreamWaitEvent(st->copy_out, ev_done, 0));
        for (int32_t i = cut[k]; i < cut[k + 1]; ++i)
            LPMM_CUDA(cudaMemcpyAsync(h_params[i], dp[i], 4 * (size_t)st->L.t[i].numel, cudaMemcpyDeviceToHost, st->copy_out));
    }
    LPMM_CUDA(cudaEventRecord(ev_end, st->copy_out));
    LPMM_CUDA(cudaStreamWaitEvent(s, ev_end, 0));                  // the caller's stream ends after the last copy-out
    st->new_rc_clean = false;
    st->phase = (st->phase + 1) % 3;
    st->last_launches = launches;
    return LPMM_OK;
}

lpmm_status lpmm_quantize(const float* d_x, int64_t rows, int64_t cols, int32_t norm, int32_t map,
                          int32_t block, uint32_t flags, uint8_t* d_codes, float* d_scale0, float* d_scale1,
                          void* stream) {
    if (!d_x || !d_codes || !d_scale0 || rows <= 0 || cols <= 0) return LPMM_ERR_INVALID_ARG;
    if (norm != LPMM_NORM_BLOCK && norm != LPMM_NORM_RANK1) return LPMM_ERR_INVALID_ARG;
    if (map != LPMM_MAP_DE_SIGNED && map != LPMM_MAP_LINEAR_NOZERO) return LPMM_ERR_INVALID_ARG;
    if (flags & ~LPMM_Q_GIVEN_SCALES) return LPMM_ERR_INVALID_ARG;
    if (rows > ((int64_t)1 << 40) / cols) return LPMM_ERR_INVALID_ARG;
    if (norm == LPMM_NORM_RANK1) {
        if (!d_scale1) return LPMM_ERR_INVALID_ARG;
        if (map != LPMM_MAP_LINEAR_NOZERO) return LPMM_ERR_UNSUPPORTED;
    } else if (block != 128 && block != 2048) {
        return LPMM_ERR_UNSUPPORTED;
    }
    LPMM_CUDA(launch_quantize(d_x, rows, cols, norm, map, block, (flags & LPMM_Q_GIVEN_SCALES) != 0, d_codes,
                              d_scale0, d_scale1, static_cast<cudaStream_t>(stream)));
    return LPMM_OK;
}

lpmm_status lpmm_quantize_rank1_noalloc(const float* d_x, int64_t rows, int64_t cols, uint8_t* d_codes,
                                        float* d_scale0, float* d_scale1, void* stream) {
    if (!d_x || !d_codes || !d_scale0 || !d_scale1 || rows <= 0 || cols <= 0) return LPMM_ERR_INVALID_ARG;
    if (rows > ((int64_t)1 << 40) / cols) return LPMM_ERR_INVALID_ARG;
    if ((rows + 3) / 4 * 4 + cols > LPMM_NOALLOC_MAX_SCALES) return LPMM_ERR_TOO_LARGE;
    LPMM_CUDA(launch_quantize_rank1_noalloc(d_x, rows, cols, d_codes, d_scale0, d_scale1,
                                            static_cast<cudaStream_t>(stream)));
    return LPMM_OK;
}

lpmm_status lpmm_dequantize(const uint8_t* d_codes, const float* d_scale0, const float* d_scale1,
                            int64_t rows, int64_t cols, int32_t norm, int32_t map, int32_t block,
                            float* d_out, void* stream) {
    if (!d_codes || !d_scale0 || !d_out || rows <= 0 || cols <= 0) return LPMM_ERR_INVALID_ARG;
    if (norm != LPMM_NORM_BLOCK && norm != LPMM_NORM_RANK1) return LPMM_ERR_INVALID_ARG;
    if (map != LPMM_MAP_DE_SIGNED && map != LPMM_MAP_LINEAR_NOZERO) return LPMM_ERR_INVALID_ARG;
    if (rows > ((int64_t)1 << 40) / cols) return LPMM_ERR_INVALID_ARG;
    if (norm == LPMM_NORM_RANK1) {
        if (!d_scale1) return LPMM_ERR_INVALID_ARG;
        if (map != LPMM_MAP_LINEAR_NOZERO) return LPMM_ERR_UNSUPPORTED;
    } else if (block != 128 && block != 2048) {
        return LPMM_ERR_UNSUPPORTED;
    }
    LPMM_CUDA(launch_dequantize(d_codes, d_scale0, d_scale1, rows, cols, norm, map, block, d_out,
                                static_cast<cudaStream_t>(stream)));
    return LPMM_OK;
}

lpmm_status lpmm_state_view(const lpmm_state* st, int32_t tensor, int32_t* kind,
                            const uint8_t** m_codes, const float** m_scale,
                            const uint8_t** v_codes, const float** v_scale0, const float** v_scale1,
                            const float** m32, const float** v32) {
    if (!st || tensor < 0 || tensor >= st->n) return LPMM_ERR_INVALID_ARG;
    const TensorLayout& t = st->L.t[tensor];
    const char* A = st->arena;
    const bool q = (t.kind != K_FP32);
    const bool r1 = uses_rc(t.kind);
    if (kind) *kind = public_kind(t.kind);
    if (m_codes) *m_codes = q ? reinterpret_cast<const uint8_t*>(A + t.m_codes) : nullptr;
    if (m_scale) *m_scale = q ? reinterpret_cast<const float*>(A + t.m_scale) : nullptr;
    if (v_codes) *v_codes = (q && t.kind != K_FACT) ? reinterpret_cast<const uint8_t*>(A + t.v_codes) : nullptr;
    const float* rc = reinterpret_cast<const float*>(A + st->L.rc[st->phase]) + t.rc_index;
    if (v_scale0) *v_scale0 = r1 ? rc : ((t.kind == K_BLOCK || t.kind == K_BLOCK_TILED) ? reinterpret_cast<const float*>(A + t.v_bscale) : nullptr);
    if (v_scale1) *v_scale1 = r1 ? rc + (t.nd >= 3 ? t.nd_off[t.nd - 1] : t.c_off) : nullptr;
    if (m32) *m32 = q ? nullptr : reinterpret_cast<const float*>(A + t.m32);
    if (v32) *v32 = q ? nullptr : reinterpret_cast<const float*>(A + t.v32);
    return LPMM_OK;
}

lpmm_status lpmm_state_view_axis(const lpmm_state* st, int32_t tensor, int32_t axis, const float** mu, int64_t* extent) {
    if (!st || tensor < 0 || tensor >= st->n || !mu || !extent) return LPMM_ERR_INVALID_ARG;
    const TensorLayout& t = st->L.t[tensor];
    if (!uses_rc(t.kind) || axis < 0 || axis >= (t.nd >= 3 ? t.nd : 2)) return LPMM_ERR_INVALID_ARG;
    const float* rc = reinterpret_cast<const float*>(st->arena + st->L.rc[st->phase]) + t.rc_index;
    if (t.nd >= 3) { *mu = rc + t.nd_off[axis]; *extent = t.nd_dim[axis]; }
    else if (axis == 0) { *mu = rc; *extent = t.rows; }
    else { *mu = rc + t.c_off; *extent = t.cols; }
    return LPMM_OK;
}

lpmm_status lpmm_state_profile(lpmm_state* st, int32_t enable) {
    if (!st) return LPMM_ERR_INVALID_ARG;
    if (enable) {   // the events are made here, once, so that a recorded step creates nothing
        while (st->prof_events.size() < 4 * kProfRingSteps) {
            cudaEvent_t e;
            LPMM_CUDA(cudaEventCreate(&e));
            st->prof_events.push_back(e);
        }
    }
    st->profile = (enable != 0);
    return LPMM_OK;
}

lpmm_status lpmm_state_profile_read(lpmm_state* st, double* pass1_ms, double* rcp_ms, double* pass2_ms, int32_t* steps) {
    if (!st) return LPMM_ERR_INVALID_ARG;
    double t[3] = {0.0, 0.0, 0.0};
    const size_t n = st->prof_used / 4;
    lpmm_status rc = LPMM_OK;
    for (size_t i = 0; i < n && rc == LPMM_OK; ++i) {
        cudaEvent_t* e = &st->prof_events[4 * i];
        cudaError_t err = cudaEventSynchronize(e[3]);
        for (int k = 0; k < 3 && err == cudaSuccess; ++k) {
            float ms = 0.0f;
            err = cudaEventElapsedTime(&ms, e[k], e[k + 1]);
            t[k] += ms;
        }
        if (err != cudaSuccess) rc = cuda_fail(err);
    }
    st->prof_used = 0;
    if (pass1_ms) *pass1_ms = t[0];
    if (rcp_ms) *rcp_ms = t[1];
    if (pass2_ms) *pass2_ms = t[2];
    if (steps) *steps = (int32_t)n;
    return rc;
}

lpmm_status lpmm_state_device_status(lpmm_state* st, int32_t* status, void* stream) {
    if (!st || !status) return LPMM_ERR_INVALID_ARG;
    uint32_t word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    LPMM_CUDA(cudaMemcpyAsync(&word, st->arena, sizeof(word), cudaMemcpyDeviceToHost, s));
    LPMM_CUDA(cudaStreamSynchronize(s));
    *status = (int32_t)word;
    return LPMM_OK;
}

lpmm_status lpmm_state_selftest_wait(lpmm_state* st, int32_t* ctas_gave_up, int32_t* status_word, void* stream) {
    if (!st || !ctas_gave_up || !status_word) return LPMM_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ArenaHeader* hd = reinterpret_cast<ArenaHeader*>(st->arena);
    // pad1[0] counts the CTAs that gave up; pad1[1] is the flag they wait on, which nothing ever sets
    LPMM_CUDA(cudaMemsetAsync(hd->pad1, 0, sizeof(hd->pad1), s));
    LPMM_CUDA(launch_wait_selftest(&hd->pad1[1], 1u, 2000u, &hd->status,
                                   reinterpret_cast<int32_t*>(&hd->pad1[0]), s));
    uint32_t words[8] = {0};
    LPMM_CUDA(cudaMemcpyAsync(words, st->arena, sizeof(words), cudaMemcpyDeviceToHost, s));
    LPMM_CUDA(cudaStreamSynchronize(s));
    *status_word = (int32_t)words[0];
    *ctas_gave_up = (int32_t)words[6];
    LPMM_CUDA(cudaMemsetAsync(st->arena, 0, 32, s));     // the state stays usable: status word and counters back to zero
    return LPMM_OK;
}

lpmm_status lpmm_state_wait_stats(lpmm_state* st, int64_t* waits, int64_t* wait_ns, void* stream) {
    if (!st || !waits || !wait_ns) return LPMM_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long w[2] = {0, 0};
    char* p = st->arena + offsetof(ArenaHeader, wait_stats);
    LPMM_CUDA(cudaMemcpyAsync(w, p, sizeof(w), cudaMemcpyDeviceToHost, s));
    LPMM_CUDA(cudaStreamSynchronize(s));
    LPMM_CUDA(cudaMemsetAsync(p, 0, sizeof(w), s));
    *waits = (int64_t)w[0];
    *wait_ns = (int64_t)w[1];
    return LPMM_OK;
}

lpmm_status lpmm_state_check_guards(lpmm_state* st, int64_t* zones, int64_t* damaged, void* stream) {
    if (!st || !zones || !damaged) return LPMM_ERR_INVALID_ARG;
    if (!kGuards) return LPMM_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ArenaHeader* hd = reinterpret_cast<ArenaHeader*>(st->arena);
    LPMM_CUDA(cudaMemsetAsync(hd->pad1, 0, sizeof(hd->pad1), s));
    for (size_t k = 0; k < st->L.guards.size(); ++k)
        LPMM_CUDA(launch_guard_check(reinterpret_cast<const unsigned char*>(st->arena + st->L.guards[k]), (int)kAlign, kGuardByte, &hd->pad1[0], s));
    uint32_t bad = 0;
    LPMM_CUDA(cudaMemcpyAsync(&bad, &hd->pad1[0], sizeof(bad), cudaMemcpyDeviceToHost, s));
    LPMM_CUDA(cudaStreamSynchronize(s));
    LPMM_CUDA(cudaMemsetAsync(hd->pad1, 0, sizeof(hd->pad1), s));
    *zones = (int64_t)st->L.guards.size();
    *damaged = (int64_t)bad;
    return LPMM_OK;
}

int32_t lpmm_build_is_checking(void) { return kGuards ? 1 : 0; }

lpmm_status lpmm_state_selftest_check(lpmm_state* st, int32_t* status_word, void* stream) {
    if (!st || !status_word) return LPMM_ERR_INVALID_ARG;
    if (!kGuards) return LPMM_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    LPMM_CUDA(launch_check_selftest(reinterpret_cast<uint32_t*>(st->arena), s));
    LPMM_CUDA(cudaMemcpyAsync(&word, st->arena, sizeof(word), cudaMemcpyDeviceToHost, s));
    LPMM_CUDA(cudaStreamSynchronize(s));
    LPMM_CUDA(cudaMemsetAsync(st->arena, 0, 4, s));
    *status_word = (int32_t)word;
    return LPMM_OK;
}

int32_t lpmm_state_phase(const lpmm_state* st) { return st ? st->phase : -1; }

int32_t lpmm_state_schedule(const lpmm_state* st) {
    if (!st) return -1;
    if (st->fused) return LPMM_SCHEDULE_FUSED;
    return (st->cfg.schedule == LPMM_SCHEDULE_OVERLAP && st->group_cut.size() > 2) ? LPMM_SCHEDULE_OVERLAP : LPMM_SCHEDULE_TWO_PASS;
}

int32_t lpmm_state_last_launches(const lpmm_state* st) { return st ? st->last_launches : 0; }

void lpmm_state_destroy(lpmm_state* st) {
    if (!st) return;
    for (cudaEvent_t e : st->prof_events) cudaEventDestroy(e);
    for (cudaEvent_t e : st->host_events) cudaEventDestroy(e);
    for (cudaEvent_t e : st->ov_events) cudaEventDestroy(e);
    if (st->aux) cudaStreamDestroy(st->aux);
    if (st->copy_in) cudaStreamDestroy(st->copy_in);
    if (st->copy_out) cudaStreamDestroy(st->copy_out);
    delete st;
}

const char* lpmm_status_string(lpmm_status s) {
    switch (s) {
        case LPMM_OK: return "ok";
        case LPMM_ERR_INVALID_ARG: return "invalid argument";
        case LPMM_ERR_UNSUPPORTED: return "unsupported configuration";
        case LPMM_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
        case LPMM_ERR_ARENA_TOO_SMALL: return "arena or staging buffer too small";
        case LPMM_ERR_CUDA: return "CUDA runtime error";
        case LPMM_ERR_TOO_LARGE: return "size exceeds the fixed capacity of the allocation-free entry point";
        default: return "unknown status";
    }
}

int32_t lpmm_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
