// Local score recomputed from the observation window on the 5th-generation tensor cores
// (Section 3: Eq. 1 window attention, max over the query heads of a KV head, Eq. 2 mean over the
// window). Writes w * S into the window-sum buffer, like the decode kernel's step-by-step sums.
//
// The softmax of Eq. 1 needs every row's normaliser before the max over heads can be taken, so the
// keys of a unit are streamed twice, and the two passes use the two orientations of the product so
// that every reduction is a loop inside one thread:
//   pass 1   D[q row][key] = Q K^T   (M = 128 query rows, N = 128 keys per tile): the thread that
//            owns a TMEM lane owns a query row and keeps its online (max, sum) over the keys;
//   pass 2   D[key][q row] = K Q^T   (M = 128 keys, N = g * wk query rows): the thread that owns a
//            lane owns a key, and the max over heads and the sum over window rows run over columns.
// A work item is one unit (layer, sequence, KV head) and wk <= 64 window rows of all g heads
// (g * wk <= 256 rows; wider windows take several items that add into the same sums).
//
// The kernel is persistent: one CTA per SM walks over the items, and the copy and tensor roles run
// on across item boundaries, so the next item's window queries and first key tiles are in flight,
// and its first products issued, while the softmax warps finish the item before. Warp 0 streams K
// tiles by TMA (a ring that continues across items; pass 2 walks the tiles backwards, so what it
// reads is still in L2) and the window queries (two buffers), warp 1 issues tcgen05.mma into two
// 256-column TMEM accumulators, warps 2-17 (four groups of four, one TMEM lane quarter per warp)
// read the accumulators back with tcgen05.ld and do the softmax arithmetic.
//
// Pass 1 is bound by the exponentials (one per logit; the special-function unit does 16 a clock and
// SM, the tensor core 8192 flop): half of them are evaluated on the FMA pipe instead, as
// 2^x = 2^round(x) * P(x - round(x)) with a cubic P (relative error < 8e-5; pass 1 only feeds the
// row sums, and the scores are compared at 1e-3). With at most 64 query rows the rows are loaded
// twice (lanes 64-127 of the accumulator repeat lanes 0-63) and the two copies split the keys of a
// tile, so that no lane idles.
// Window token k sees the keys t <= n - w + k (its own key included).
#include "gkv_common.cuh"
#include "gkv_internal.h"
#include "gkv_tcgen05.cuh"

namespace gkv {

constexpr int kTcGroups = 4;                                 // softmax warp groups (4 warps each)
constexpr int kTcSoftmaxThreads = kTcGroups * 128;
constexpr int kTcThreads = 64 + kTcSoftmaxThreads;
constexpr int kTcTileKeys = 128;
constexpr int kTcMaxStages = 6;                              // K ring depth is chosen per launch from the shared memory left
constexpr int kTcKStageBytes = kTcTileKeys * kRowBytes;      // 32 KB: d-low half then d-high half
constexpr int kTcMaxRows = 256;
constexpr int kTcAccCols = 256;                              // TMEM columns of one accumulator
constexpr uint32_t kTcTmemCols = 512;
constexpr int kTcChunkKeys = 8192;                           // keys whose window sums are held in shared memory at a time

struct __align__(8) ScoreTcTail {
    uint64_t q_full[2];
    uint64_t q_empty[2];
    uint64_t k_full[kTcMaxStages];
    uint64_t k_empty[kTcMaxStages];
    uint64_t d_full[2];
    uint64_t d_empty[2];
    uint64_t drain;
    uint64_t chunk_bar;   // the softmax warps meet here when the window sums move on to the next chunk of keys
    uint32_t tmem_base;
    int abort_flag;
    int issued;           // K tiles whose copies have been started (all items)
    int q_issued;         // items whose window queries have been started
    int abort_seen;       // the abort flag as one softmax thread saw it between two barriers
};

__device__ __forceinline__ void tc_abort(ScoreTcTail* tail, int32_t* status, int where) {
    if (atomicExch(&tail->abort_flag, 1) == 0 && atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kTcSoftmaxThreads) : "memory"); }

// 2^x for a pair of x <= 0 on the FMA pipe: t = x + 1.5 * 2^23 rounds x to the nearest integer in the low mantissa
// bits of t; f = x - round(x) lies in [-0.5, 0.5]; a cubic in f (relative error < 8e-5) is scaled by adding the
// integer to the exponent field. x is clamped at -125 first (the result, ~2e-38, stands for 0).
__device__ __forceinline__ float2 exp2_fma_pair(float xa, float xb) {
    constexpr float kMagic = 12582912.f;
    const float2 x = make_float2(fmaxf(xa, -125.f), fmaxf(xb, -125.f));
    const float2 one = make_float2(1.f, 1.f);
    const float2 t = fma_f32x2(x, one, make_float2(kMagic, kMagic));
    const float2 r = fma_f32x2(t, one, make_float2(-kMagic, -kMagic));
    const float2 f = fma_f32x2(r, make_float2(-1.f, -1.f), x);
    float2 pl = fma_f32x2(f, make_float2(0.05520550534129143f, 0.05520550534129143f), make_float2(0.24261397123336792f, 0.24261397123336792f));
    pl = fma_f32x2(pl, f, make_float2(0.6932547688484192f, 0.6932547688484192f));
    pl = fma_f32x2(pl, f, make_float2(0.9999276995658875f, 0.9999276995658875f));
    float2 y;
    y.x = __int_as_float(__float_as_int(pl.x) + (__float_as_int(t.x) << 23));
    y.y = __int_as_float(__float_as_int(pl.y) + (__float_as_int(t.y) << 23));
    return y;
}

// Online (max, sum) of one query row over N more keys whose raw logits are z[0..N): `m_raw` is the running maximum
// of the unscaled logits, `l` the sum of 2^((z - m_raw) * scale). Half of the exponentials go to the special-function
// unit, half to the FMA pipe.
template <int N>
__device__ __forceinline__ void row_update(float (&z)[N], int key0, int last_vis, bool need_mask, float scale,
                                           float& m_raw, float& l) {
    if (need_mask) {
#pragma unroll
        for (int j = 0; j < N; ++j)
            if (key0 + j > last_vis) z[j] = -INFINITY;
    }
    float c0 = fmaxf(z[0], z[1]), c1 = fmaxf(z[2], z[3]), c2 = fmaxf(z[4], z[5]), c3 = fmaxf(z[6], z[7]);
#pragma unroll
    for (int j = 8; j < N; j += 8) {
        c0 = fmaxf(c0, fmaxf(z[j], z[j + 1]));
        c1 = fmaxf(c1, fmaxf(z[j + 2], z[j + 3]));
        c2 = fmaxf(c2, fmaxf(z[j + 4], z[j + 5]));
        c3 = fmaxf(c3, fmaxf(z[j + 6], z[j + 7]));
    }
    const float mn = fmaxf(m_raw, fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)));
    if (mn == -INFINITY) return;
    const float neg = -mn * scale;
    float s0 = 0.f, s1 = 0.f;
    float2 sp = make_float2(0.f, 0.f);
    const float2 sc2 = make_float2(scale, scale), ng2 = make_float2(neg, neg);
#pragma unroll
    for (int j = 0; j < N; j += 4) {
        s0 += fast_exp2(fmaf(z[j], scale, neg));
        s1 += fast_exp2(fmaf(z[j + 1], scale, neg));
        const float2 a = fma_f32x2(make_float2(z[j + 2], z[j + 3]), sc2, ng2);
        const float2 e = exp2_fma_pair(a.x, a.y);
        sp = fma_f32x2(e, make_float2(1.f, 1.f), sp);
    }
    l = l * fast_exp2(fmaf(m_raw, scale, neg)) + ((s0 + s1) + (sp.x + sp.y));
    m_raw = mn;
}

// What one work item covers (every role derives it the same way).
struct ScoreItem {
    int unit_local, k0, head, ls, n, T, row0;
    long unit;
};
__device__ __forceinline__ ScoreItem score_item(const ScoreLaunch& p, int item, int n_cta, int wk) {
    ScoreItem d;
    d.unit_local = item / n_cta;
    d.k0 = (item - d.unit_local * n_cta) * wk;         // first window row of this item
    d.head = d.unit_local % p.h_kv;
    d.ls = d.unit_local / p.h_kv;                       // layer_local * batch + seq
    const int lseq_global = p.layer0 * p.batch + d.ls;
    d.unit = (long)lseq_global * p.h_kv + d.head;
    d.n = p.len[lseq_global];
    d.T = (d.n + kTcTileKeys - 1) / kTcTileKeys;
    d.row0 = (int)(d.unit * p.C);
    return d;
}

// WK = window rows handled by one item (16, 32 or 64); the item's local query row of (head h, window
// row k0 + kk) is h * WK + kk.
template <int WK>
__global__ void __launch_bounds__(kTcThreads, 1)
gkv_score_tc_kernel(const ScoreLaunch p, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_q, int n_cta, int stages, int q_bufs) {
    constexpr int HW = WK / kTcGroups;   // window rows one softmax group handles in pass 2
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int R = p.g * WK;                          // query rows of an item, a multiple of 16
    const int MT = (R + 127) >> 7;                   // 128-row tiles of pass 1
    // the rows are loaded twice and the copies split a tile's keys (whole warps per copy: a warp reads one column range)
    const bool dup = 2 * R <= 128 && R % 32 == 0;
    const int q_half = MT * 128 * 128;               // bytes of one d-half of a Q buffer (d-low, then d-high)
    const int q_bytes = 2 * q_half;
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + (size_t)q_bufs * q_bytes;
    float* s_c = reinterpret_cast<float*>(k_smem + stages * kTcKStageBytes);      // [256] m + log2 l of every local row
    float* s_pm = s_c + kTcMaxRows;                                               // [groups][128] partial row maxima
    float* s_pl = s_pm + kTcGroups * 128;                                         // [groups][128] partial row sums
    // [2][c_pad] window sums of this item's rows: two groups add into each plane, so every sum has two addends and
    // the result does not depend on the order in which the groups arrive. Caches hold at most kTcChunkKeys rows and
    // fit whole; a longer key range (a prompt being compressed) passes through in chunks of kTcChunkKeys keys, each
    // written out when pass 2, which walks the tiles from the last to the first, leaves it.
    float* s_sum = s_pl + kTcGroups * 128;
    const int c_pad = min((p.C + 63) & ~63, kTcChunkKeys);
    ScoreTcTail* tail = reinterpret_cast<ScoreTcTail*>(s_sum + 2 * c_pad);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total_items = p.n_layers * p.batch * p.h_kv * n_cta;

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tail->q_full[b]), 1);
            mbar_init(smem_u32(&tail->q_empty[b]), 1);
            mbar_init(smem_u32(&tail->d_full[b]), 1);
            mbar_init(smem_u32(&tail->d_empty[b]), kTcSoftmaxThreads / 32);   // one arrival per softmax warp
        }
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->k_full[s]), 1);
            mbar_init(smem_u32(&tail->k_empty[s]), 1);
        }
        mbar_init(smem_u32(&tail->drain), 1);
        mbar_init(smem_u32(&tail->chunk_bar), kTcSoftmaxThreads / 32);
        tail->abort_flag = 0;
        tail->issued = 0;
        tail->q_issued = 0;
        fence_mbar_init();
    }
    if (warp == 1) {   // whole warp: the CTA takes all of the SM's tensor memory (one CTA per SM by shared memory)
        tmem_alloc(smem_u32(&tail->tmem_base), kTcTmemCols);
        tmem_relinquish_alloc_permit();
        tmem_fence_before_sync();
    }
    for (int t = tid; t < 2 * c_pad; t += kTcThreads) s_sum[t] = 0.f;
    // rows of the Q tiles that no copy fills take part in the pass-1 products: make them zeros (both buffers, once)
    {
        const int filled = dup ? 2 * R : R;
        const int per_half = (MT * 128 - filled) * 8;          // 16-byte pieces per d-half
        for (int e = tid; e < q_bufs * 2 * per_half; e += kTcThreads) {
            const int qb = e / (2 * per_half);
            const int rem = e - qb * 2 * per_half;
            const int half = rem / per_half;
            const int r = rem - half * per_half;
            *reinterpret_cast<uint4*>(q_smem + (size_t)qb * q_bytes + (size_t)half * q_half + (size_t)filled * 128 + r * 16) = make_uint4(0, 0, 0, 0);
        }
    }
    fence_proxy_async_smem();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&tail->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_q);
            int s = 0, round = 0, issued = 0;
            bool ok = true;
            for (int item = blockIdx.x, j = 0; ok && item < total_items; item += gridDim.x, ++j) {
                const ScoreItem d = score_item(p, item, n_cta, WK);
                const int qb = j % q_bufs;
                const int total = 2 * d.T;
                // The item's first K tiles go out before its window queries: the ring slots they need are freed by the
                // item before, while the query buffer may have to wait for that item's last product.
                const int pre = min(stages, total);
                for (int i = 0; i <= total; ++i) {
                    if (i == pre) {
                        // the buffer's previous queries (item j - q_bufs) have been through their last product
                        if (j >= q_bufs && !tc_wait(smem_u32(&tail->q_empty[qb]), ((j / q_bufs) - 1) & 1, &tail->abort_flag)) {
                            tc_abort(tail, p.status, 20);
                            ok = false;
                            break;
                        }
                        const uint32_t qbar = smem_u32(&tail->q_full[qb]);
                        mbar_arrive_expect_tx(qbar, (uint32_t)(dup ? 2 * R : R) * kRowBytes);
                        const int qrow0 = (d.ls * p.h_q + d.head * p.g) * p.w + d.k0;
                        uint8_t* qdst = q_smem + (size_t)qb * q_bytes;
                        for (int c = 0; c < (dup ? 2 : 1); ++c)
                            for (int h = 0; h < p.g; ++h) {
                                tma_load_2d(smem_u32(qdst + (size_t)(c * R + h * WK) * 128), &tm_q, 0, qrow0 + h * p.w, qbar);
                                tma_load_2d(smem_u32(qdst + q_half + (size_t)(c * R + h * WK) * 128), &tm_q, 64, qrow0 + h * p.w, qbar);
                            }
                        *(volatile int*)&tail->q_issued = j + 1;
                    }
                    if (i == total) break;
                    if (round > 0 && !tc_wait(smem_u32(&tail->k_empty[s]), (round - 1) & 1, &tail->abort_flag)) {
                        tc_abort(tail, p.status, 21);
                        ok = false;
                        break;
                    }
                    const int tile = (i < d.T) ? i : total - 1 - i;   // pass 2 walks back: the tiles read last are still in L2
                    const uint32_t bar = smem_u32(&tail->k_full[s]);
                    const uint32_t dst = smem_u32(k_smem + (size_t)s * kTcKStageBytes);
                    const int y = d.row0 + tile * kTcTileKeys;
                    mbar_arrive_expect_tx(bar, kTcKStageBytes);
                    tma_load_2d(dst, &tm_k, 0, y, bar);
                    tma_load_2d(dst + kBoxBytes, &tm_k, 0, y + 64, bar);
                    tma_load_2d(dst + 2 * kBoxBytes, &tm_k, 64, y, bar);
                    tma_load_2d(dst + 3 * kBoxBytes, &tm_k, 64, y + 64, bar);
                    *(volatile int*)&tail->issued = ++issued;
                    if (++s == stages) { s = 0; ++round; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t k_lo = umma_desc_lo(smem_u32(k_smem));
            const uint32_t idesc1 = umma_idesc_bf16_m128(kTcTileKeys), idesc2 = umma_idesc_bf16_m128(R);
            int s = 0, round = 0, ai = 0;            // ring position and accumulator turn, carried across items
            bool ok = true;
            for (int item = blockIdx.x, j = 0; ok && item < total_items; item += gridDim.x, ++j) {
                const ScoreItem d = score_item(p, item, n_cta, WK);
                const int qb = j % q_bufs;
                if (!tc_wait(smem_u32(&tail->q_full[qb]), (j / q_bufs) & 1, &tail->abort_flag)) {
                    tc_abort(tail, p.status, 22);
                    break;
                }
                const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem + (size_t)qb * q_bytes));
                const int total = 2 * d.T;
                for (int i = 0; i < total; ++i, ++ai) {
                    const int buf = ai & 1;
                    if (ai >= 2 && !tc_wait(smem_u32(&tail->d_empty[buf]), ((ai >> 1) - 1) & 1, &tail->abort_flag)) {
                        tc_abort(tail, p.status, 23);
                        ok = false;
                        break;
                    }
                    if (!tc_wait(smem_u32(&tail->k_full[s]), round & 1, &tail->abort_flag)) {
                        tc_abort(tail, p.status, 24);
                        ok = false;
                        break;
                    }
                    tmem_fence_after_sync();
                    const uint32_t ks_lo = k_lo + (uint32_t)s * (kTcKStageBytes >> 4);
                    const uint32_t dcol = tmem_base + (uint32_t)buf * kTcAccCols;
                    if (i < d.T) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(dcol, umma_desc(q_lo + umma_kstep(ks, q_half)), umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)),
                                      idesc1, ks > 0);
                        if (MT == 2) {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)
                                umma_bf16(dcol + 128, umma_desc(q_lo + ((128 * 128) >> 4) + umma_kstep(ks, q_half)),
                                          umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)), idesc1, ks > 0);
                        }
                    } else {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(dcol, umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)), umma_desc(q_lo + umma_kstep(ks, q_half)),
                                      idesc2, ks > 0);
                    }
                    umma_commit(smem_u32(&tail->k_empty[s]));
                    umma_commit(smem_u32(&tail->d_full[buf]));
                    if (++s == stages) { s = 0; ++round; }
                }
                if (ok) umma_commit(smem_u32(&tail->q_empty[qb]));   // the item's last product has read its queries
            }
            // everything issued has completed before the accumulators are given back
            umma_commit(smem_u32(&tail->drain));
            mbar_wait_bounded(smem_u32(&tail->drain), 0);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int wg = (warp - 2) >> 2;               // group of four consecutive warps
        const int q4 = warp & 3;                      // TMEM lane quarter this warp may touch
        const int L = q4 * 32 + lane;                 // TMEM lane = accumulator row of this thread
        const int stid = (warp - 2) * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const float scale = p.scale_log2;
        bool ok = true;
        int ai = 0;                                   // accumulator turn, carried across items
        uint32_t chunk_phase = 0;

        // pass-1 role of this thread. Two 128-row tiles: two groups per tile, 64 keys each. One tile: all four
        // groups, 32 keys each; with the rows loaded twice, 16 keys for each copy.
        const int copy = dup ? (L >= R ? 1 : 0) : 0;
        const int rl = (MT == 2) ? (wg >> 1) * 128 + L : L - copy * R;                    // local query row
        const bool valid = (MT == 2) ? rl < R : L < (dup ? 2 * R : R);
        const int col0 = (MT == 2) ? (wg & 1) * 64 : wg * 32 + copy * 16;
        const uint32_t t_p1 = t_lane + (uint32_t)((MT == 2) ? (wg >> 1) * 128 + col0 : col0);

        for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
            const ScoreItem d = score_item(p, item, n_cta, WK);
            const int n = d.n, T = d.T, k0 = d.k0, total = 2 * T;
            // ---- pass 1: online (max, sum) of the row this thread owns over its share of the tile's keys
            const int last_vis = n - p.w + k0 + (rl % WK);    // last key the row's token sees
            float m_raw = -INFINITY, l = 0.f;                 // maximum in unscaled logits, sum relative to it
            for (int i = 0; i < T; ++i, ++ai) {
                const int buf = ai & 1;
                ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[buf]), (ai >> 1) & 1, &tail->abort_flag));
                if (!ok) { tc_abort(tail, p.status, 25); break; }
                tmem_fence_after_sync();
                const int key_base = i * kTcTileKeys + col0;
                const bool need_mask = i * kTcTileKeys + kTcTileKeys - 1 > n - p.w + k0;
                if (MT == 2) {
#pragma unroll 1
                    for (int ch = 0; ch < 2; ++ch) {
                        float z[32];
                        tmem_ld<32>(t_p1 + (uint32_t)(buf * kTcAccCols + ch * 32), z);
                        if (valid) row_update<32>(z, key_base + ch * 32, last_vis, need_mask, scale, m_raw, l);
                    }
                } else if (dup) {
                    float z[16];
                    tmem_ld<16>(t_p1 + (uint32_t)(buf * kTcAccCols), z);
                    if (valid) row_update<16>(z, key_base, last_vis, need_mask, scale, m_raw, l);
                } else {
                    float z[32];
                    tmem_ld<32>(t_p1 + (uint32_t)(buf * kTcAccCols), z);
                    if (valid) row_update<32>(z, key_base, last_vis, need_mask, scale, m_raw, l);
                }
                tmem_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[buf]));
            }
            // (a warp whose wait gave up still walks through every barrier below; all leave together at a point
            // where one thread's view of the abort flag decides for everybody)
            // combine the partials of a row and publish c = m + log2 l (scaled, log2 domain)
            s_pm[wg * 128 + L] = m_raw * scale;
            s_pl[wg * 128 + L] = l;
            softmax_bar_sync();
            if ((MT == 2) ? (wg & 1) == 0 : (wg == 0 && L < R)) {
                const int first = (MT == 2) ? wg : 0, count = (MT == 2) ? 2 : kTcGroups;   // groups that shared this row
                float mm = -INFINITY, ll = 0.f;
                for (int c = 0; c <= (dup ? 1 : 0); ++c)
                    for (int q = first; q < first + count; ++q) mm = fmaxf(mm, s_pm[q * 128 + L + c * R]);
                for (int c = 0; c <= (dup ? 1 : 0); ++c)
                    for (int q = first; q < first + count; ++q) {
                        const float mq = s_pm[q * 128 + L + c * R];
                        ll += (mq == -INFINITY) ? 0.f : s_pl[q * 128 + L + c * R] * fast_exp2(mq - mm);
                    }
                s_c[(MT == 2) ? rl : L] = mm + log2f(ll);
            }
            if (stid == 0) tail->abort_seen = *(volatile int*)&tail->abort_flag;
            softmax_bar_sync();
            if (*(volatile int*)&tail->abort_seen) break;

            // ---- pass 2: this thread owns key `tile * 128 + L`; group wg covers window rows k0 + wg*HW .. + HW - 1
            float* out = p.sacc + (size_t)d.unit * p.C;
            // window sums of keys [lo, lo + c_pad) leave shared memory (which is zeroed for the next chunk or item)
            auto flush_chunk = [&](int lo) {
                const int hi = min(lo + c_pad, p.C);
                for (int t = lo + stid; t < hi; t += kTcSoftmaxThreads) {
                    const float v = s_sum[t - lo] + s_sum[c_pad + t - lo];
                    s_sum[t - lo] = 0.f;
                    s_sum[c_pad + t - lo] = 0.f;
                    if (n_cta == 1) out[t] = (t < n) ? v : 0.f;
                    else if (t < n) atomicAdd(&out[t], v);   // buffer zeroed by the host
                }
            };
            int chunk_lo = T > 0 ? ((T - 1) * kTcTileKeys / c_pad) * c_pad : 0;
            for (int i = T; ok && i < total; ++i, ++ai) {
                const int buf = ai & 1;
                const int tile_lo = ((total - 1 - i) * kTcTileKeys / c_pad) * c_pad;
                if (tile_lo != chunk_lo) {
                    // Every softmax warp has added its part of the chunk; then the chunk is written and cleared; then all
                    // go on. mbarrier waits, not bar.sync: a warp that gives up (abort flag) must not leave the others at
                    // a barrier it will never reach.
                    for (int step = 0; ok && step < 2; ++step) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&tail->chunk_bar));
                        ok = __all_sync(0xffffffffu, tc_wait(smem_u32(&tail->chunk_bar), chunk_phase & 1, &tail->abort_flag));
                        ++chunk_phase;
                        if (ok && step == 0) flush_chunk(chunk_lo);
                    }
                    if (!ok) { tc_abort(tail, p.status, 27); break; }
                    chunk_lo = tile_lo;
                }
                ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[buf]), (ai >> 1) & 1, &tail->abort_flag));
                if (!ok) { tc_abort(tail, p.status, 26); break; }
                tmem_fence_after_sync();
                float v[HW];
#pragma unroll
                for (int jj = 0; jj < HW; ++jj) v[jj] = -INFINITY;
                for (int h = 0; h < p.g; ++h) {
                    float z[HW];
                    tmem_ld<HW>(t_lane + (uint32_t)(buf * kTcAccCols + h * WK + wg * HW), z);
                    const float4* c4 = reinterpret_cast<const float4*>(s_c + h * WK + wg * HW);
#pragma unroll
                    for (int jj = 0; jj < HW; jj += 4) {
                        const float4 c = c4[jj >> 2];
                        v[jj] = fmaxf(v[jj], fmaf(z[jj], scale, -c.x));
                        v[jj + 1] = fmaxf(v[jj + 1], fmaf(z[jj + 1], scale, -c.y));
                        v[jj + 2] = fmaxf(v[jj + 2], fmaf(z[jj + 2], scale, -c.z));
                        v[jj + 3] = fmaxf(v[jj + 3], fmaf(z[jj + 3], scale, -c.w));
                    }
                }
                tmem_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[buf]));
                const int key = (total - 1 - i) * kTcTileKeys + L;
                if (key < n) {
                    const int first_k = key - (n - p.w) - k0 - wg * HW;   // rows jj < first_k decoded before this key existed
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int jj = 0; jj < HW; jj += 2) {
                        s0 += (jj >= first_k) ? fast_exp2(v[jj]) : 0.f;
                        s1 += (jj + 1 >= first_k) ? fast_exp2(v[jj + 1]) : 0.f;
                    }
                    atomicAdd(&s_sum[(wg >> 1) * c_pad + key - chunk_lo], s0 + s1);
                }
            }
            softmax_bar_sync();
            if (stid == 0) tail->abort_seen = *(volatile int*)&tail->abort_flag;
            if (ok && !*(volatile int*)&tail->abort_flag) {
                flush_chunk(chunk_lo);   // the chunk of the first tile, walked last
                // rows past the chunk that holds the last key were never in shared memory
                if (n_cta == 1)
                    for (int t = (T > 0 ? ((T - 1) * kTcTileKeys / c_pad + 1) * c_pad : 0) + stid; t < p.C; t += kTcSoftmaxThreads) out[t] = 0.f;
            }
            softmax_bar_sync();      // the sums are clear and the row constants free before the next item uses them
            if (*(volatile int*)&tail->abort_seen) break;
        }
    }

    __syncthreads();
    if (*(volatile int*)&tail->abort_flag && tid == 0) {
        // give copies still in flight a bounded time to land before the CTA exits
        const int q_issued = *(volatile int*)&tail->q_issued;
        for (int j = max(0, q_issued - q_bufs); j < q_issued; ++j)
            mbar_wait_bounded(smem_u32(&tail->q_full[j % q_bufs]), (j / q_bufs) & 1);
        const int issued = *(volatile int*)&tail->issued;
        for (int i = max(0, issued - stages); i < issued; ++i)
            mbar_wait_bounded(smem_u32(&tail->k_full[i % stages]), (i / stages) & 1);
    }
    __syncthreads();
    if (warp == 1) {
        tmem_fence_after_sync();
        tmem_dealloc(tmem_base, kTcTmemCols);
    }
}

static size_t score_tc_smem_bytes(int C, int rows, int stages, int q_bufs) {
    const int mt = (rows + 127) >> 7;
    return 1024 + (size_t)q_bufs * mt * 128 * kRowBytes + (size_t)stages * kTcKStageBytes +
           sizeof(float) * (kTcMaxRows + 2 * kTcGroups * 128 + 2 * min((C + 63) & ~63, kTcChunkKeys)) + sizeof(ScoreTcTail);
}

// Window rows per item for this shape, or 0 when the shape is left to the mma.sync kernel.
int score_tc_rows_per_cta(int g, int w) {
    if (w % 16 != 0 || g < 1 || g > kMaxGroup) return 0;
    for (int wk = 64; wk >= 16; wk >>= 1)
        if (wk <= w && w % wk == 0 && g * wk <= kTcMaxRows) return wk;
    return 0;
}

cudaError_t score_tc_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(gkv_score_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gkv_score_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gkv_score_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_score_tc(const ScoreLaunch& p, const CUtensorMap& tm_k, const CUtensorMap& tm_q, int wk, cudaStream_t s) {
    const int n_cta = p.w / wk;
    const int units = p.n_layers * p.batch * p.h_kv;
    const int items = units * n_cta;
    // two buffers for the window queries when at least three K stages still fit beside them, then the deepest K ring
    const int rows = p.g * wk;
    const int q_bufs = score_tc_smem_bytes(p.C, rows, 3, 2) <= 227 * 1024 ? 2 : 1;
    int stages = 2;
    while (stages < kTcMaxStages && score_tc_smem_bytes(p.C, rows, stages + 1, q_bufs) <= 227 * 1024) ++stages;
    const size_t smem = score_tc_smem_bytes(p.C, rows, stages, q_bufs);
    if (n_cta > 1) {
        const size_t off = (size_t)p.layer0 * p.batch * p.h_kv * p.C;
        cudaError_t e = cudaMemsetAsync(p.sacc + off, 0, sizeof(float) * (size_t)units * p.C, s);
        if (e != cudaSuccess) return e;
    }
    // persistent: one CTA per SM (shared memory and tensor memory allow no more), rounds filled equally
    const int sm = p.sm_count > 0 ? p.sm_count : 148;
    int grid = items < sm ? items : sm;
    if (items > sm) {
        const int rounds = (items + sm - 1) / sm;
        grid = (items + rounds - 1) / rounds;
    }
    if (wk == 16) gkv_score_tc_kernel<16><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else if (wk == 32) gkv_score_tc_kernel<32><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else gkv_score_tc_kernel<64><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    return cudaGetLastError();
}

}  // namespace gkv
