// C-ABI entry points of the G-KV library: configuration checks, the host-side schedule state, the
// workspace layout, TMA descriptor encoding and the kernel launches.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "gkv_common.cuh"
#include "gkv_internal.h"

using namespace gkv;

namespace {

constexpr int kMaxCapacity = 4096;
constexpr int kMaxPromptShared = 8192;   // up to here a prompt's scores stay in shared memory during the selection
constexpr int kMaxPrompt = 1 << 20;      // longest prompt gkv_compress_prompt takes (a stated bound, not a structural one)
constexpr uint64_t kAlign = 256;

uint64_t align_up(uint64_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

gkv_status check_config(const gkv_config* c) {
    if (!c) return GKV_ERR_INVALID_ARG;
    if (c->n_layers <= 0 || c->batch <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->head_dim <= 0)
        return GKV_ERR_INVALID_ARG;
    if (c->budget <= 0 || c->buffer <= 0 || c->window <= 0 || c->interval <= 0) return GKV_ERR_INVALID_ARG;
    if (c->window >= c->budget || c->interval > c->buffer || c->interval < c->window) return GKV_ERR_INVALID_ARG;
    if (!(c->alpha >= 0.f && c->alpha <= 1.f)) return GKV_ERR_INVALID_ARG;
    if (c->mode < GKV_MODE_MAX || c->mode > GKV_MODE_LOCAL) return GKV_ERR_INVALID_ARG;
    if (c->n_q_heads % c->n_kv_heads != 0) return GKV_ERR_INVALID_ARG;
    if (c->max_prompt < 0) return GKV_ERR_INVALID_ARG;
    if (c->max_prompt > kMaxPrompt) return GKV_ERR_UNSUPPORTED;
    // beyond the cache sizes only the tensor-core scoring kernel passes its window sums through in chunks
    if (c->max_prompt > kMaxPromptShared && c->n_kv_heads > 0 &&
        score_tc_rows_per_cta(c->n_q_heads / c->n_kv_heads, c->window) == 0)
        return GKV_ERR_UNSUPPORTED;
    if ((uint64_t)c->batch * c->n_kv_heads * (uint64_t)c->max_prompt >= (1ull << 31)) return GKV_ERR_UNSUPPORTED;
    if (c->pool_kernel < 0 || (c->pool_kernel > 1 && (c->pool_kernel & 1) == 0)) return GKV_ERR_INVALID_ARG;
    if (c->use_redundancy) {
        if (!(c->redundancy_lambda >= 0.f && c->redundancy_lambda <= 1.f)) return GKV_ERR_INVALID_ARG;
        if (!(c->redundancy_threshold > 0.f) || !(c->redundancy_eps >= 0.f) || c->redundancy_recent < 0)
            return GKV_ERR_INVALID_ARG;
    }
    if (c->policy != GKV_POLICY_SCORE && c->policy != GKV_POLICY_STREAMING) return GKV_ERR_INVALID_ARG;
    if (c->policy == GKV_POLICY_STREAMING &&
        (c->n_sink < 0 || c->n_sink > c->budget - c->window || c->use_redundancy || c->pool_kernel > 1))
        return GKV_ERR_INVALID_ARG;
    if (c->head_dim != kHeadDim) return GKV_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > kMaxGroup) return GKV_ERR_UNSUPPORTED;
    if (c->budget + c->buffer > kMaxCapacity) return GKV_ERR_UNSUPPORTED;
    const uint64_t rows = (uint64_t)c->n_layers * c->batch * c->n_kv_heads * (uint64_t)(c->budget + c->buffer);
    if (rows >= (1ull << 31)) return GKV_ERR_UNSUPPORTED;  // TMA row coordinate is a signed 32-bit integer
    return GKV_OK;
}

void layout_workspace(const gkv_config* c, int sm_count, WorkspaceLayout* w) {
    const uint64_t L = c->n_layers, B = c->batch, H = c->n_kv_heads;
    const uint64_t C = c->budget + c->buffer;
    const uint64_t upl = B * H;
    uint64_t off = 0;
    w->status = off;    off = align_up(off + 64 * sizeof(int32_t));
    w->seq_done = off;  off = align_up(off + L * B * sizeof(int32_t));
    (void)sm_count;   // the decode kernel keeps nothing else here: split units merge in shared memory, logits stay in TMEM
    w->kept = off;     off = align_up(off + upl * c->budget * sizeof(int32_t));
    w->fscratch = off; off = align_up(off + upl * C * sizeof(float));
    const uint64_t red = c->use_redundancy ? 1 : 0;   // the redundancy term's scratch exists only when it is on
    w->prompt_sums = off; off = align_up(off + upl * (uint64_t)c->max_prompt * sizeof(float));
    w->prompt_len = off;  off = align_up(off + (c->max_prompt > 0 ? B : 0) * sizeof(int32_t));
    const uint64_t long_arrays = c->max_prompt > kMaxPromptShared ? ((c->pool_kernel > 1 || c->use_redundancy) ? 2 : 1) : 0;
    w->prompt_f = off;    off = align_up(off + long_arrays * upl * (uint64_t)c->max_prompt * sizeof(float));
    const uint64_t sel = (c->use_redundancy || c->pool_kernel > 1) ? 1 : 0;
    w->fsel = off;     off = align_up(off + sel * upl * C * sizeof(float));
    // per cached row of every layer, or per token of a prompt being compressed, whichever is more
    const uint64_t red_rows = L * upl * C > upl * (uint64_t)c->max_prompt ? L * upl * C : upl * (uint64_t)c->max_prompt;
    w->inv_norm = off; off = align_up(off + red * red_rows * sizeof(float));
    w->cbar = off;     off = align_up(off + red * red_rows * sizeof(float));
    w->total = off;
}

void fill_sizes(const gkv_config* c, int sm_count, gkv_sizes* s, WorkspaceLayout* wl) {
    const uint64_t L = c->n_layers, B = c->batch, H = c->n_kv_heads, Hq = c->n_q_heads;
    const uint64_t C = c->budget + c->buffer;
    const uint64_t rows = L * B * H * C;
    s->k = rows * kHeadDim * 2;
    s->v = s->k;
    s->f = rows * 4;
    s->sacc = rows * 4;
    s->pos = c->track_positions ? rows * 4 : 0;
    s->len = 2 * L * B * 4;
    WorkspaceLayout tmp;
    layout_workspace(c, sm_count, &tmp);
    s->workspace = tmp.total;
    if (wl) *wl = tmp;
    // staging for the host-buffer calls: q, k_new, v_new, out for all layers, or q_window + kept
    const uint64_t dec = L * B * (Hq + 2 * H + Hq) * kHeadDim * 2;
    const uint64_t evi = L * B * Hq * (uint64_t)c->window * kHeadDim * 2 + L * B * H * (uint64_t)c->budget * 4;
    s->staging = align_up(dec > evi ? dec : evi) + 4 * kAlign;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once (no link-time dependency on libcuda).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess && sym)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// 2-D view of a buffer of 128-element bf16 rows: [rows][128], boxes of box_rows rows x 64 elements,
// 128-byte swizzle (K and V: 64-row boxes; 16-row and 128-row boxes for the kernels that want them).
gkv_status encode_map(CUtensorMap* map, void* base, uint64_t rows, uint32_t box_rows = kTileKeys) {
    const EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return GKV_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kRowBytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? GKV_OK : GKV_ERR_CUDA;
}

// 3-D view of the window queries [heads][w][128] bf16 for the tensor-core scoring kernel: one box = box_rows
// consecutive window rows of `g` consecutive heads x 64 elements (128-byte swizzle), so a block of window rows of all
// the heads of a KV head arrives with one copy, head after head.
gkv_status encode_query_map(CUtensorMap* map, const void* base, uint64_t heads, uint32_t w, uint32_t box_rows, uint32_t g) {
    const EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return GKV_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)w, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)kRowBytes, (cuuint64_t)kRowBytes * w};
    const cuuint32_t box[3] = {64, box_rows, g};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? GKV_OK : GKV_ERR_CUDA;
}

bool layer_ok(const gkv_ctx* ctx, int32_t layer) { return layer >= -1 && layer < ctx->cfg.n_layers; }
void layer_range(const gkv_ctx* ctx, int32_t layer, int* l0, int* nl) {
    if (layer < 0) { *l0 = 0; *nl = ctx->cfg.n_layers; }
    else { *l0 = layer; *nl = 1; }
}
template <typename T>
T* ws_ptr(const gkv_ctx* ctx, uint64_t off) { return reinterpret_cast<T*>(static_cast<uint8_t*>(ctx->buf.workspace) + off); }

// All layers of a multi-layer call must be in the same schedule state.
bool uniform(const std::vector<int32_t>& v, int l0, int nl) {
    for (int i = 1; i < nl; ++i)
        if (v[l0 + i] != v[l0]) return false;
    return true;
}

EvictLaunch make_evict(gkv_ctx* ctx, int l0, int nl, int32_t* kept_out) {
    EvictLaunch p;
    const gkv_config& c = ctx->cfg;
    p.k_cache = static_cast<__nv_bfloat16*>(ctx->buf.k);
    p.v_cache = static_cast<__nv_bfloat16*>(ctx->buf.v);
    p.f = static_cast<float*>(ctx->buf.f);
    p.sacc = static_cast<float*>(ctx->buf.sacc);
    p.pos = c.track_positions ? static_cast<int32_t*>(ctx->buf.pos) : nullptr;
    p.len = static_cast<int32_t*>(ctx->buf.len);
    p.seq_done = ws_ptr<int32_t>(ctx, ctx->ws.seq_done);
    p.kept_out = kept_out;
    p.kept_ws = ws_ptr<int32_t>(ctx, ctx->ws.kept);
    p.f_ws = ws_ptr<float>(ctx, ctx->ws.fscratch);
    p.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
    p.work = p.status + 34;       // (the decode kernel's counters are words 32 and 33)
    p.sm_count = ctx->sm_count;
    p.layer0 = l0; p.n_layers = nl; p.L_total = c.n_layers; p.batch = c.batch; p.h_kv = c.n_kv_heads;
    p.C = ctx->C; p.b = c.budget; p.w = c.window; p.alpha = c.alpha; p.mode = c.mode;
    p.evict_log = ctx->evict_log;
    p.cbar = c.use_redundancy ? ws_ptr<float>(ctx, ctx->ws.cbar) : nullptr;
    p.fsel_ws = ws_ptr<float>(ctx, ctx->ws.fsel);
    p.lambda = c.redundancy_lambda;
    p.pool_kernel = c.pool_kernel;
    p.policy = c.policy; p.n_sink = c.n_sink;
    return p;
}

// Redundancy level of every cached key of the layers [l0, l0 + nl): key norms, then the thresholded
// cosine-similarity sums (two launches).
gkv_status launch_redundancy_for(gkv_ctx* ctx, int l0, int nl, cudaStream_t s) {
    RedundancyLaunch rp;
    const gkv_config& c = ctx->cfg;
    rp.k_cache = static_cast<const __nv_bfloat16*>(ctx->buf.k);
    rp.len = static_cast<const int32_t*>(ctx->buf.len);
    rp.inv_norm = ws_ptr<float>(ctx, ctx->ws.inv_norm);
    rp.cbar = ws_ptr<float>(ctx, ctx->ws.cbar);
    rp.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
    rp.layer0 = l0; rp.n_layers = nl; rp.batch = c.batch; rp.h_kv = c.n_kv_heads; rp.C = ctx->C;
    rp.recent = c.redundancy_recent; rp.tau = c.redundancy_threshold; rp.eps = c.redundancy_eps;
    if (launch_keynorm(rp, s) != cudaSuccess || launch_redundancy(rp, ctx->tm_k, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    ctx->launches += 2;
    return GKV_OK;
}

// tcgen05 kernel for windows that split into 16-, 32- or 64-row slices; the mma.sync kernel covers the rest.
gkv_status dispatch_score(gkv_ctx* ctx, const ScoreLaunch& sp, const CUtensorMap& tm_k, const CUtensorMap& tm_k128, cudaStream_t s) {
    const gkv_config& c = ctx->cfg;
    const int wk = score_tc_rows_per_cta(ctx->g, c.window);
    if (wk > 0 && (reinterpret_cast<uintptr_t>(sp.q_win) & 15) == 0) {
        CUtensorMap tm_q;
        const uint64_t q_heads = (uint64_t)sp.n_layers * c.batch * c.n_q_heads;
        if (encode_query_map(&tm_q, sp.q_win, q_heads, (uint32_t)c.window, (uint32_t)score_tc_q_box_rows(wk), (uint32_t)ctx->g) != GKV_OK) return GKV_ERR_CUDA;
        if (launch_score_tc(sp, tm_k128, tm_q, wk, s) != cudaSuccess) return GKV_ERR_CUDA;
    } else if (sp.C > kMaxPromptShared) {
        return GKV_ERR_INVALID_ARG;   // a long prompt with misaligned window queries: the other kernel holds all sums on chip
    } else if (launch_score(sp, tm_k, s) != cudaSuccess) {
        return GKV_ERR_CUDA;
    }
    ctx->launches += 1;
    return GKV_OK;
}

gkv_status launch_score_for(gkv_ctx* ctx, int l0, int nl, const void* q_window, cudaStream_t s) {
    ScoreLaunch sp;
    const gkv_config& c = ctx->cfg;
    sp.q_win = static_cast<const __nv_bfloat16*>(q_window);
    sp.sacc = static_cast<float*>(ctx->buf.sacc);
    sp.len = static_cast<const int32_t*>(ctx->buf.len);
    sp.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
    sp.layer0 = l0; sp.n_layers = nl; sp.batch = c.batch; sp.h_q = c.n_q_heads; sp.h_kv = c.n_kv_heads;
    sp.g = ctx->g; sp.C = ctx->C; sp.w = c.window; sp.sm_count = ctx->sm_count;
    sp.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kHeadDim));
    return dispatch_score(ctx, sp, ctx->tm_k, ctx->tm_k128, s);
}

// Shared validation of an eviction request. Returns GKV_OK with *noop set when len <= b.
gkv_status evict_precheck(gkv_ctx* ctx, int32_t layer, bool need_window_sums, int* l0, int* nl, bool* noop) {
    if (!ctx || !layer_ok(ctx, layer)) return GKV_ERR_INVALID_ARG;
    layer_range(ctx, layer, l0, nl);
    if (!uniform(ctx->len, *l0, *nl) || !uniform(ctx->n_hist, *l0, *nl) || !uniform(ctx->since_evict, *l0, *nl) ||
        !uniform(ctx->sacc_valid, *l0, *nl))
        return GKV_ERR_STATE;
    const int len = ctx->len[*l0];
    *noop = len <= ctx->cfg.budget;
    if (*noop) return GKV_OK;
    if (need_window_sums && ctx->cfg.policy != GKV_POLICY_STREAMING) {
        const bool fused_ready = ctx->cfg.fuse_window_scores && ctx->since_evict[*l0] == ctx->cfg.interval;
        if (!fused_ready && !ctx->sacc_valid[*l0]) return GKV_ERR_STATE;
    }
    return GKV_OK;
}

void after_evict(gkv_ctx* ctx, int l0, int nl, bool noop) {
    for (int i = l0; i < l0 + nl; ++i) {
        if (!noop) {
            ctx->len[i] = ctx->cfg.budget;
            ctx->n_hist[i] = ctx->cfg.budget - ctx->cfg.window;
        }
        ctx->since_evict[i] = 0;
        ctx->sacc_valid[i] = 0;
        ctx->stage_next[i] = 0;
        ctx->cbar_valid[i] = 0;
    }
}

// A compression call that evicts nothing: the window sums restart and the eviction log (if any) reads "nothing".
gkv_status reset_sacc(gkv_ctx* ctx, int l0, int nl, cudaStream_t s) {
    const size_t per_layer = (size_t)ctx->units_per_layer * ctx->C * sizeof(float);
    if (cudaMemsetAsync(static_cast<uint8_t*>(ctx->buf.sacc) + l0 * per_layer, 0, nl * per_layer, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    if (ctx->evict_log) {
        const size_t log_layer = (size_t)ctx->units_per_layer * ctx->cfg.buffer * sizeof(int32_t);
        if (cudaMemsetAsync(reinterpret_cast<uint8_t*>(ctx->evict_log) + l0 * log_layer, 0xFF, nl * log_layer, s) != cudaSuccess)
            return GKV_ERR_CUDA;
    }
    return GKV_OK;
}

// Self-test of the bounded wait: one warp waits, with a short limit, on an mbarrier that nobody arrives on. The wait
// runs out, the kernel latches the status word the way every kernel of the library does, and returns.
__global__ void gkv_selftest_wait_kernel(int32_t* status, uint32_t spins) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0 && !mbar_wait_bounded(smem_u32(&bar), 0, spins)) {
        if (atomicCAS(status, 0, kStatusTimeout) == 0) {
            status[1] = 90;
            status[2] = blockIdx.x;
        }
    }
}

}  // namespace

extern "C" {

gkv_status gkv_selftest_bounded_wait(gkv_ctx* ctx, int32_t spins, void* stream) {
    if (!ctx || spins < 1 || spins > (1 << 16)) return GKV_ERR_INVALID_ARG;
    gkv_selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ws_ptr<int32_t>(ctx, ctx->ws.status), (uint32_t)spins);
    if (cudaGetLastError() != cudaSuccess) return GKV_ERR_CUDA;
    ctx->launches += 1;
    return GKV_OK;
}

gkv_status gkv_query_sizes(const gkv_config* cfg, gkv_sizes* out) {
    if (!out) return GKV_ERR_INVALID_ARG;
    const gkv_status st = check_config(cfg);
    if (st != GKV_OK) return st;
    int sm = 0, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    (void)cudaGetLastError();  // no device (size queries on a CPU-only host) is not an error here
    fill_sizes(cfg, sm, out, nullptr);
    return GKV_OK;
}

gkv_status gkv_init(gkv_ctx** out, const gkv_config* cfg, const gkv_buffers* b, void* stream) {
    if (!out || !b) return GKV_ERR_INVALID_ARG;
    *out = nullptr;
    gkv_status st = check_config(cfg);
    if (st != GKV_OK) return st;
    if (!b->k || !b->v || !b->f || !b->sacc || !b->len || !b->workspace) return GKV_ERR_INVALID_ARG;
    if (cfg->track_positions && !b->pos) return GKV_ERR_INVALID_ARG;
    const void* ptrs[] = {b->k, b->v, b->f, b->sacc, b->len, b->workspace, b->pos, b->staging};
    for (const void* p : ptrs)
        if (p && (reinterpret_cast<uintptr_t>(p) % kAlign) != 0) return GKV_ERR_INVALID_ARG;

    gkv_ctx* ctx = new (std::nothrow) gkv_ctx();
    if (!ctx) return GKV_ERR_CUDA;
    ctx->cfg = *cfg;
    ctx->buf = *b;
    ctx->C = cfg->budget + cfg->buffer;
    ctx->g = cfg->n_q_heads / cfg->n_kv_heads;
    ctx->units_per_layer = cfg->batch * cfg->n_kv_heads;
    ctx->launches = 0;
    ctx->evict_log = nullptr;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bool ok = cudaGetDevice(&ctx->device) == cudaSuccess &&
              cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) == cudaSuccess;
    if (ok) {
        fill_sizes(cfg, ctx->sm_count, &ctx->sizes, &ctx->ws);
        ok = cudaMemsetAsync(b->k, 0, ctx->sizes.k, s) == cudaSuccess &&
             cudaMemsetAsync(b->v, 0, ctx->sizes.v, s) == cudaSuccess &&
             cudaMemsetAsync(b->f, 0, ctx->sizes.f, s) == cudaSuccess &&
             cudaMemsetAsync(b->sacc, 0, ctx->sizes.sacc, s) == cudaSuccess &&
             cudaMemsetAsync(b->len, 0, ctx->sizes.len, s) == cudaSuccess &&
             cudaMemsetAsync(b->workspace, 0, ctx->sizes.workspace, s) == cudaSuccess &&
             (!cfg->track_positions || cudaMemsetAsync(b->pos, 0, ctx->sizes.pos, s) == cudaSuccess);
    }
    if (ok) ok = decode_kernel_setup() == cudaSuccess && score_kernel_setup() == cudaSuccess && score_tc_kernel_setup() == cudaSuccess &&
                 redundancy_kernel_setup() == cudaSuccess;
    if (ok) {
        const uint64_t rows = (uint64_t)cfg->n_layers * ctx->units_per_layer * ctx->C;
        ok = encode_map(&ctx->tm_k, b->k, rows) == GKV_OK && encode_map(&ctx->tm_v, b->v, rows) == GKV_OK &&
             encode_map(&ctx->tm_k128, b->k, rows, kScoreTcKeyBoxRows) == GKV_OK && encode_map(&ctx->tm_k16, b->k, rows, 16) == GKV_OK && encode_map(&ctx->tm_v16, b->v, rows, 16) == GKV_OK;
    }
    if (!ok) {
        (void)cudaGetLastError();
        delete ctx;
        return GKV_ERR_CUDA;
    }
    ctx->len.assign(cfg->n_layers, 0);
    ctx->n_hist.assign(cfg->n_layers, 0);
    ctx->since_evict.assign(cfg->n_layers, 0);
    ctx->sacc_valid.assign(cfg->n_layers, 0);
    ctx->stage_next.assign(cfg->n_layers, 0);
    ctx->cbar_valid.assign(cfg->n_layers, 0);
    *out = ctx;
    return GKV_OK;
}

gkv_status gkv_set_state(gkv_ctx* ctx, int32_t layer, int32_t len, int32_t n_hist, int32_t since_evict,
                         int32_t window_scores_valid, void* stream) {
    if (!ctx || !layer_ok(ctx, layer)) return GKV_ERR_INVALID_ARG;
    if (len < 0 || len > ctx->C || n_hist < 0 || n_hist > len || since_evict < 0) return GKV_ERR_INVALID_ARG;
    int l0, nl;
    layer_range(ctx, layer, &l0, &nl);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int B = ctx->cfg.batch, L = ctx->cfg.n_layers;
    int32_t* dl = static_cast<int32_t*>(ctx->buf.len);
    // a copy from pageable host memory has staged its source when the call returns, so `h` may be reused
    std::vector<int32_t> h((size_t)nl * B);
    for (auto& x : h) x = len;
    if (cudaMemcpyAsync(dl + (size_t)l0 * B, h.data(), h.size() * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    for (auto& x : h) x = n_hist;
    if (cudaMemcpyAsync(dl + (size_t)L * B + (size_t)l0 * B, h.data(), h.size() * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    for (int i = l0; i < l0 + nl; ++i) {
        ctx->len[i] = len;
        ctx->n_hist[i] = n_hist;
        ctx->since_evict[i] = since_evict;
        ctx->sacc_valid[i] = window_scores_valid ? 1 : 0;
        ctx->stage_next[i] = 0;
        ctx->cbar_valid[i] = 0;
    }
    return GKV_OK;
}

gkv_status gkv_decode_attn(gkv_ctx* ctx, int32_t layer, const void* q, const void* k_new, const void* v_new,
                           void* out, void* stream) {
    if (!ctx || !layer_ok(ctx, layer) || !q || !k_new || !v_new || !out) return GKV_ERR_INVALID_ARG;
    // 16-byte vector accesses and, for q, bulk copies
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
         reinterpret_cast<uintptr_t>(out)) % 16 != 0)
        return GKV_ERR_INVALID_ARG;
    int l0, nl;
    layer_range(ctx, layer, &l0, &nl);
    if (!uniform(ctx->len, l0, nl) || !uniform(ctx->since_evict, l0, nl)) return GKV_ERR_STATE;
    const gkv_config& c = ctx->cfg;
    if (ctx->len[l0] >= ctx->C) return GKV_ERR_CAPACITY;
    if (c.fuse_window_scores && ctx->since_evict[l0] >= c.interval) return GKV_ERR_STATE;

    DecodeLaunch p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.k_cache = static_cast<__nv_bfloat16*>(ctx->buf.k);
    p.v_cache = static_cast<__nv_bfloat16*>(ctx->buf.v);
    p.sacc = static_cast<float*>(ctx->buf.sacc);
    p.len = static_cast<int32_t*>(ctx->buf.len);
    p.seq_done = ws_ptr<int32_t>(ctx, ctx->ws.seq_done);
    p.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
    p.layer0 = l0; p.n_layers = nl; p.batch = c.batch; p.h_q = c.n_q_heads; p.h_kv = c.n_kv_heads;
    p.g = ctx->g; p.C = ctx->C;
    p.accum = (c.fuse_window_scores && ctx->since_evict[l0] >= c.interval - c.window) ? 1 : 0;
    p.sm_count = ctx->sm_count;
    p.work_next = p.status + 32;
    decode_plan(&p, 0);
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kHeadDim));
    const DecodeMaps maps = {ctx->tm_k, ctx->tm_v, ctx->tm_k16, ctx->tm_v16};
    if (launch_decode(p, maps, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    ctx->launches += 1;
    for (int i = l0; i < l0 + nl; ++i) {
        ctx->len[i] += 1;
        ctx->since_evict[i] += 1;
        ctx->stage_next[i] = 0;
        ctx->cbar_valid[i] = 0;
        // window sums written by hand are stale once further tokens are decoded without accumulation
        if (!p.accum) ctx->sacc_valid[i] = 0;
    }
    return GKV_OK;
}

gkv_status gkv_evict(gkv_ctx* ctx, int32_t layer, const void* q_window, int32_t* kept_idx_out, void* stream) {
    int l0, nl;
    bool noop;
    gkv_status st = evict_precheck(ctx, layer, q_window == nullptr, &l0, &nl, &noop);
    if (st != GKV_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (noop) {
        st = reset_sacc(ctx, l0, nl, s);
        if (st != GKV_OK) return st;
        after_evict(ctx, l0, nl, true);
        return GKV_OK;
    }
    if (q_window && ctx->cfg.policy != GKV_POLICY_STREAMING) {
        st = launch_score_for(ctx, l0, nl, q_window, s);
        if (st != GKV_OK) return st;
    }
    if (ctx->cfg.use_redundancy) {
        st = launch_redundancy_for(ctx, l0, nl, s);
        if (st != GKV_OK) return st;
    }
    const EvictLaunch p = make_evict(ctx, l0, nl, kept_idx_out);
    if (launch_evict_fused(p, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    ctx->launches += 1;
    after_evict(ctx, l0, nl, false);
    return GKV_OK;
}

gkv_status gkv_evict_stage(gkv_ctx* ctx, int32_t layer, int32_t stage, const void* q_window, int32_t* kept_idx_out,
                           void* stream) {
    int l0, nl;
    bool noop;
    if (!ctx || stage < GKV_STAGE_SCORE || stage > GKV_STAGE_REDUNDANCY) return GKV_ERR_INVALID_ARG;
    if (stage == GKV_STAGE_REDUNDANCY && !ctx->cfg.use_redundancy) return GKV_ERR_INVALID_ARG;
    gkv_status st = evict_precheck(ctx, layer, false, &l0, &nl, &noop);
    if (st != GKV_OK) return st;
    if (nl != 1) return GKV_ERR_UNSUPPORTED;  // the staged scratch holds one layer
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int& next = ctx->stage_next[l0];
    if (noop) {
        if (stage == GKV_STAGE_COMPACT) {
            st = reset_sacc(ctx, l0, nl, s);
            if (st != GKV_OK) return st;
            after_evict(ctx, l0, nl, true);
        }
        return GKV_OK;
    }
    if (stage == GKV_STAGE_SCORE) {
        if (!q_window || next != 0) return next != 0 ? GKV_ERR_STATE : GKV_ERR_INVALID_ARG;
        st = launch_score_for(ctx, l0, nl, q_window, s);
        if (st != GKV_OK) return st;
        ctx->sacc_valid[l0] = 1;
        next = GKV_STAGE_MERGE;
        return GKV_OK;
    }
    if (stage == GKV_STAGE_REDUNDANCY) {
        if (next != 0 && next != GKV_STAGE_MERGE) return GKV_ERR_STATE;
        st = launch_redundancy_for(ctx, l0, nl, s);
        if (st != GKV_OK) return st;
        ctx->cbar_valid[l0] = 1;
        return GKV_OK;
    }
    const EvictLaunch p = make_evict(ctx, l0, nl, stage == GKV_STAGE_SELECT ? kept_idx_out : nullptr);
    cudaError_t e;
    if (stage == GKV_STAGE_MERGE) {
        if (next != 0 && next != GKV_STAGE_MERGE) return GKV_ERR_STATE;
        const bool fused_ready = ctx->cfg.fuse_window_scores && ctx->since_evict[l0] == ctx->cfg.interval;
        if (!fused_ready && !ctx->sacc_valid[l0] && ctx->cfg.policy != GKV_POLICY_STREAMING) return GKV_ERR_STATE;
        if (ctx->cfg.use_redundancy && !ctx->cbar_valid[l0]) return GKV_ERR_STATE;   // REDUNDANCY stage first
        e = launch_evict_merge(p, s);
        if (e == cudaSuccess) next = GKV_STAGE_SELECT;
    } else if (stage == GKV_STAGE_SELECT) {
        if (next != GKV_STAGE_SELECT) return GKV_ERR_STATE;
        e = launch_evict_select(p, s);
        if (e == cudaSuccess) next = GKV_STAGE_COMPACT;
    } else {
        if (next != GKV_STAGE_COMPACT) return GKV_ERR_STATE;
        e = launch_evict_compact(p, ctx->sm_count, s);
        if (e == cudaSuccess) after_evict(ctx, l0, nl, false);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    ctx->launches += 1;
    return GKV_OK;
}

// Device alias of a host pointer when the memory is page-locked and mapped into the device's address space
// (cudaHostAlloc / cudaHostRegister, torch's pin_memory()); NULL for pageable memory.
static void* mapped_alias(const void* host_ptr) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return (at.type == cudaMemoryTypeHost) ? at.devicePointer : nullptr;
}

gkv_status gkv_decode_attn_host(gkv_ctx* ctx, int32_t layer, const void* q_host, const void* k_new_host,
                                const void* v_new_host, void* out_host, void* stream) {
    if (!ctx || !layer_ok(ctx, layer) || !q_host || !k_new_host || !v_new_host || !out_host) return GKV_ERR_INVALID_ARG;
    {
        // Zero copy: with page-locked, mapped host buffers the kernel itself reads q / k_new / v_new and writes out
        // across the bus, so the transfers of one unit overlap the attention of the others instead of being
        // serialised before and after the launch.
        void *aq = mapped_alias(q_host), *ak = mapped_alias(k_new_host), *av = mapped_alias(v_new_host), *ao = mapped_alias(out_host);
        if (aq && ak && av && ao) return gkv_decode_attn(ctx, layer, aq, ak, av, ao, stream);
    }
    if (!ctx->buf.staging) return GKV_ERR_INVALID_ARG;
    int l0, nl;
    layer_range(ctx, layer, &l0, &nl);
    const gkv_config& c = ctx->cfg;
    // the checks gkv_decode_attn would fail on, before any copy is queued
    if (!uniform(ctx->len, l0, nl) || !uniform(ctx->since_evict, l0, nl)) return GKV_ERR_STATE;
    if (ctx->len[l0] >= ctx->C) return GKV_ERR_CAPACITY;
    if (c.fuse_window_scores && ctx->since_evict[l0] >= c.interval) return GKV_ERR_STATE;
    const size_t qb = (size_t)nl * c.batch * c.n_q_heads * kHeadDim * 2;
    const size_t kb = (size_t)nl * c.batch * c.n_kv_heads * kHeadDim * 2;
    uint8_t* st = static_cast<uint8_t*>(ctx->buf.staging);
    uint8_t *dq = st, *dk = st + align_up(qb), *dv = dk + align_up(kb), *dout = dv + align_up(kb);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    const gkv_status r = gkv_decode_attn(ctx, layer, dq, dk, dv, dout, stream);
    if (r != GKV_OK) return r;
    if (cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GKV_ERR_CUDA;
    return GKV_OK;
}

gkv_status gkv_evict_host(gkv_ctx* ctx, int32_t layer, const void* q_window_host, int32_t* kept_idx_out_host,
                          void* stream) {
    if (!ctx || !layer_ok(ctx, layer)) return GKV_ERR_INVALID_ARG;
    if (!ctx->buf.staging) return GKV_ERR_INVALID_ARG;
    int l0, nl;
    layer_range(ctx, layer, &l0, &nl);
    const gkv_config& c = ctx->cfg;
    const size_t qb = (size_t)nl * c.batch * c.n_q_heads * c.window * kHeadDim * 2;
    const size_t kb = (size_t)nl * c.batch * c.n_kv_heads * c.budget * 4;
    uint8_t* st = static_cast<uint8_t*>(ctx->buf.staging);
    uint8_t *dq = st, *dkept = st + align_up(qb);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (q_window_host && cudaMemcpyAsync(dq, q_window_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    const bool will_evict = ctx->len[l0] > c.budget;
    const gkv_status r = gkv_evict(ctx, layer, q_window_host ? dq : nullptr,
                                   kept_idx_out_host ? reinterpret_cast<int32_t*>(dkept) : nullptr, stream);
    if (r != GKV_OK) return r;
    if (kept_idx_out_host && will_evict &&
        cudaMemcpyAsync(kept_idx_out_host, dkept, kb, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return GKV_ERR_CUDA;
    return GKV_OK;
}

gkv_status gkv_compress_prompt(gkv_ctx* ctx, int32_t layer, const void* k_prompt, const void* v_prompt,
                               const void* q_window, const int32_t* prompt_len_host, int32_t* kept_idx_out, void* stream) {
    if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers || !k_prompt || !v_prompt || !prompt_len_host)
        return GKV_ERR_INVALID_ARG;
    const gkv_config& c = ctx->cfg;
    if (c.max_prompt <= 0) return GKV_ERR_STATE;
    if ((reinterpret_cast<uintptr_t>(k_prompt) & 15) || (reinterpret_cast<uintptr_t>(v_prompt) & 15)) return GKV_ERR_INVALID_ARG;
    int longest = 0;
    bool any_long = false;
    for (int i = 0; i < c.batch; ++i) {
        const int n = prompt_len_host[i];
        if (n < 1 || n > c.max_prompt) return GKV_ERR_INVALID_ARG;
        any_long |= n > c.budget;
        const int rows = n > c.budget ? c.budget : n;
        if (rows > longest) longest = rows;
    }
    const bool scored = c.policy != GKV_POLICY_STREAMING;
    if (any_long && scored && !q_window) return GKV_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t* d_len = ws_ptr<int32_t>(ctx, ctx->ws.prompt_len);
    // a copy from pageable host memory has staged its source when the call returns
    if (cudaMemcpyAsync(d_len, prompt_len_host, sizeof(int32_t) * c.batch, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    float* sums = ws_ptr<float>(ctx, ctx->ws.prompt_sums);
    if (any_long && scored) {
        CUtensorMap tm_kp, tm_kp128;
        const uint64_t rows = (uint64_t)c.batch * c.n_kv_heads * c.max_prompt;
        if (encode_map(&tm_kp, const_cast<void*>(k_prompt), rows) != GKV_OK ||
            encode_map(&tm_kp128, const_cast<void*>(k_prompt), rows, kScoreTcKeyBoxRows) != GKV_OK)
            return GKV_ERR_CUDA;
        ScoreLaunch sp;
        sp.q_win = static_cast<const __nv_bfloat16*>(q_window);
        sp.sacc = sums;
        sp.len = d_len;
        sp.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
        sp.layer0 = 0; sp.n_layers = 1; sp.batch = c.batch; sp.h_q = c.n_q_heads; sp.h_kv = c.n_kv_heads;
        sp.g = ctx->g; sp.C = c.max_prompt; sp.w = c.window; sp.sm_count = ctx->sm_count;
        sp.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kHeadDim));
        const gkv_status st = dispatch_score(ctx, sp, tm_kp, tm_kp128, s);
        if (st != GKV_OK) {
            (void)cudaGetLastError();
            return st;
        }
        if (c.use_redundancy) {
            // redundancy level of every prompt key, in the scratch the cached layers' levels use as well
            RedundancyLaunch rp;
            rp.k_cache = static_cast<const __nv_bfloat16*>(k_prompt);
            rp.len = d_len;
            rp.inv_norm = ws_ptr<float>(ctx, ctx->ws.inv_norm);
            rp.cbar = ws_ptr<float>(ctx, ctx->ws.cbar);
            rp.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
            rp.layer0 = 0; rp.n_layers = 1; rp.batch = c.batch; rp.h_kv = c.n_kv_heads; rp.C = c.max_prompt;
            rp.recent = c.redundancy_recent; rp.tau = c.redundancy_threshold; rp.eps = c.redundancy_eps;
            if (launch_keynorm(rp, s) != cudaSuccess || launch_redundancy(rp, tm_kp, s) != cudaSuccess) {
                (void)cudaGetLastError();
                return GKV_ERR_CUDA;
            }
            ctx->launches += 2;
            for (int i = 0; i < c.n_layers; ++i) ctx->cbar_valid[i] = 0;
        }
    }
    PromptLaunch p;
    p.k_src = static_cast<const __nv_bfloat16*>(k_prompt);
    p.v_src = static_cast<const __nv_bfloat16*>(v_prompt);
    p.k_cache = static_cast<__nv_bfloat16*>(ctx->buf.k);
    p.v_cache = static_cast<__nv_bfloat16*>(ctx->buf.v);
    p.f = static_cast<float*>(ctx->buf.f);
    p.sacc = static_cast<float*>(ctx->buf.sacc);
    p.pos = c.track_positions ? static_cast<int32_t*>(ctx->buf.pos) : nullptr;
    p.len = static_cast<int32_t*>(ctx->buf.len);
    p.sums = sums;
    p.f_long = c.max_prompt > kMaxPromptShared ? ws_ptr<float>(ctx, ctx->ws.prompt_f) : nullptr;
    p.cbar = (c.use_redundancy && any_long) ? ws_ptr<float>(ctx, ctx->ws.cbar) : nullptr;
    p.lambda = c.redundancy_lambda;
    p.prompt_len = d_len;
    p.seq_done = ws_ptr<int32_t>(ctx, ctx->ws.seq_done);
    p.kept_out = kept_idx_out;
    p.status = ws_ptr<int32_t>(ctx, ctx->ws.status);
    p.layer = layer; p.L_total = c.n_layers; p.batch = c.batch; p.h_kv = c.n_kv_heads; p.C = ctx->C;
    p.P_max = c.max_prompt; p.b = c.budget; p.w = c.window; p.pool_kernel = c.pool_kernel;
    p.policy = c.policy; p.n_sink = c.n_sink;
    if (launch_prompt_compress(p, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    ctx->launches += 1;
    ctx->len[layer] = longest;                       // host counters follow the longest sequence of the layer
    ctx->n_hist[layer] = any_long ? c.budget - c.window : 0;
    ctx->since_evict[layer] = 0;
    ctx->sacc_valid[layer] = 0;
    ctx->stage_next[layer] = 0;
    ctx->cbar_valid[layer] = 0;
    return GKV_OK;
}

gkv_status gkv_set_eviction_log(gkv_ctx* ctx, int32_t* log_device) {
    if (!ctx) return GKV_ERR_INVALID_ARG;
    if (log_device && (reinterpret_cast<uintptr_t>(log_device) & 3) != 0) return GKV_ERR_INVALID_ARG;
    ctx->evict_log = log_device;
    return GKV_OK;
}

gkv_status gkv_get_redundancy(gkv_ctx* ctx, int32_t layer, float* out_device, void* stream) {
    if (!ctx || !out_device || layer < 0 || layer >= ctx->cfg.n_layers) return GKV_ERR_INVALID_ARG;
    if (!ctx->cfg.use_redundancy) return GKV_ERR_STATE;
    const size_t per_layer = (size_t)ctx->units_per_layer * ctx->C;
    if (cudaMemcpyAsync(out_device, ws_ptr<float>(ctx, ctx->ws.cbar) + layer * per_layer, per_layer * sizeof(float),
                        cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return GKV_ERR_CUDA;
    }
    return GKV_OK;
}

gkv_status gkv_get_state(const gkv_ctx* ctx, int32_t layer, int32_t* len, int32_t* n_hist, int32_t* since_evict) {
    if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers) return GKV_ERR_INVALID_ARG;
    if (len) *len = ctx->len[layer];
    if (n_hist) *n_hist = ctx->n_hist[layer];
    if (since_evict) *since_evict = ctx->since_evict[layer];
    return GKV_OK;
}

int64_t gkv_launch_count(const gkv_ctx* ctx) { return ctx ? ctx->launches : 0; }

gkv_status gkv_poll_device_status(gkv_ctx* ctx, void* stream) {
    if (!ctx) return GKV_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t h[4] = {0, 0, 0, 0};
    int32_t* d = ws_ptr<int32_t>(ctx, ctx->ws.status);
    if (cudaMemcpyAsync(h, d, sizeof h, cudaMemcpyDeviceToHost, s) != cudaSuccess) return GKV_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return GKV_ERR_CUDA;
    if (h[0] != 0) {
        // A kernel that gave up may have left its completion and work counters part-way (they are returned to zero
        // by the last CTA of a launch that runs to its end): clear them together with the latch.
        if (cudaMemsetAsync(d, 0, ctx->ws.kept - ctx->ws.status, s) != cudaSuccess) return GKV_ERR_CUDA;
        return h[0] == kStatusBounds ? GKV_ERR_INTERNAL : GKV_ERR_TIMEOUT;
    }
    return GKV_OK;
}

gkv_status gkv_decode_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t window_step,
                                  int32_t sm_count, gkv_decode_plan_t* out) {
    if (!out) return GKV_ERR_INVALID_ARG;
    const gkv_status st = check_config(cfg);
    if (st != GKV_OK) return st;
    if (n_layers_in_launch != 1 && n_layers_in_launch != cfg->n_layers) return GKV_ERR_INVALID_ARG;
    DecodeLaunch d = {};
    d.n_layers = n_layers_in_launch; d.batch = cfg->batch; d.h_kv = cfg->n_kv_heads; d.C = cfg->budget + cfg->buffer;
    d.accum = window_step ? 1 : 0;
    d.sm_count = sm_count;
    decode_plan(&d, 0);
    int ctas = 0;
    size_t smem = 0;
    decode_plan_resources(d, &ctas, &smem);
    out->grid = d.grid; out->splits = d.splits; out->stages = d.stages; out->ctas_per_sm = ctas;
    out->smem_bytes = (int32_t)smem; out->tmem_cols = d.accum ? d.tmem_cols : 0;
    return GKV_OK;
}

gkv_status gkv_evict_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t sm_count, gkv_evict_plan_t* out) {
    if (!out) return GKV_ERR_INVALID_ARG;
    const gkv_status st = check_config(cfg);
    if (st != GKV_OK) return st;
    if (n_layers_in_launch != 1 && n_layers_in_launch != cfg->n_layers) return GKV_ERR_INVALID_ARG;
    EvictLaunch p = {};
    p.n_layers = n_layers_in_launch; p.batch = cfg->batch; p.h_kv = cfg->n_kv_heads;
    p.C = cfg->budget + cfg->buffer; p.b = cfg->budget; p.w = cfg->window;
    p.sm_count = sm_count;
    p.pool_kernel = cfg->pool_kernel;
    // only whether these are set matters for the shared-memory layout
    p.pos = cfg->track_positions ? reinterpret_cast<int32_t*>(1) : nullptr;
    p.cbar = cfg->use_redundancy ? reinterpret_cast<const float*>(1) : nullptr;
    int stages = 0, grid = 0, ctas = 0;
    size_t smem = 0;
    evict_plan(p, &stages, &grid, &smem, &ctas);
    out->grid = grid; out->stages = stages; out->ctas_per_sm = ctas; out->smem_bytes = (int32_t)smem;
    return GKV_OK;
}

gkv_status gkv_score_launch_plan(const gkv_config* cfg, int32_t n_layers_in_launch, int32_t sm_count, gkv_score_plan_t* out) {
    if (!out) return GKV_ERR_INVALID_ARG;
    const gkv_status st = check_config(cfg);
    if (st != GKV_OK) return st;
    if (n_layers_in_launch != 1 && n_layers_in_launch != cfg->n_layers) return GKV_ERR_INVALID_ARG;
    const int g = cfg->n_q_heads / cfg->n_kv_heads;
    const int wk = score_tc_rows_per_cta(g, cfg->window);
    *out = {};
    if (wk == 0) return GKV_OK;   // this window goes to the other scoring kernel: tensor_core stays 0
    ScoreLaunch p = {};
    p.n_layers = n_layers_in_launch; p.batch = cfg->batch; p.h_q = cfg->n_q_heads; p.h_kv = cfg->n_kv_heads;
    p.g = g; p.C = cfg->budget + cfg->buffer; p.w = cfg->window; p.sm_count = sm_count;
    ScoreTcPlan plan;
    score_tc_plan(p, wk, &plan);
    out->tensor_core = 1; out->grid = plan.grid; out->items = plan.items; out->rows_per_item = plan.rows;
    out->stages = plan.stages; out->query_buffers = plan.q_bufs; out->smem_bytes = (int32_t)plan.smem;
    return GKV_OK;
}

gkv_status gkv_memory_model(const gkv_config* cfg, int64_t seq_len, int32_t elem_bytes, gkv_memory_model_t* out) {
    if (!cfg || !out || seq_len <= 0 || elem_bytes <= 0) return GKV_ERR_INVALID_ARG;
    if (cfg->n_layers <= 0 || cfg->batch <= 0 || cfg->n_kv_heads <= 0 || cfg->head_dim <= 0 || cfg->budget <= 0 ||
        cfg->interval <= 0 || cfg->window < 0 || cfg->window >= cfg->budget)
        return GKV_ERR_INVALID_ARG;
    // K and V: layers x head_dim x kv_heads x tokens x elem_bytes x 2, times the batch
    const uint64_t per_token = (uint64_t)cfg->n_layers * cfg->head_dim * cfg->n_kv_heads * elem_bytes * 2ull;
    out->full_kv = per_token * (uint64_t)seq_len * cfg->batch;
    out->compressed_kv = per_token * (uint64_t)(cfg->budget + cfg->interval) * cfg->batch;
    out->score_cache = (uint64_t)cfg->n_layers * cfg->n_kv_heads * (uint64_t)(cfg->budget - cfg->window) *
                       elem_bytes * cfg->batch;
    return GKV_OK;
}

const char* gkv_strerror(gkv_status status) {
    switch (status) {
        case GKV_OK: return "ok";
        case GKV_ERR_INVALID_ARG: return "invalid argument";
        case GKV_ERR_STATE: return "call not allowed in the current schedule state";
        case GKV_ERR_CAPACITY: return "cache full: evict before decoding further";
        case GKV_ERR_CUDA: return "CUDA call failed";
        case GKV_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case GKV_ERR_UNSUPPORTED: return "configuration not supported by this library";
        case GKV_ERR_SCRATCH_LIMIT: return "problem exceeds the library's built-in scratch array";
        case GKV_ERR_INTERNAL: return "checked build: a kernel computed a row index out of range (access skipped)";
        default: return "unknown status";
    }
}

void gkv_destroy(gkv_ctx* ctx) { delete ctx; }

}  // extern "C"
