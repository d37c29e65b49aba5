// Local score recomputed from the observation window on the 5th-generation tensor cores
// (Section 3: Eq. 1 window attention, max over the query heads of a KV head, Eq. 2 mean over the
// window). Writes w * S into the window-sum buffer, like the decode kernel's step-by-step sums.
//
// The softmax of Eq. 1 needs every row's normaliser before the max over heads can be taken, so the
// keys of a unit are streamed twice, and the two passes use the two orientations of the product so
// that every reduction is a loop inside one thread:
//   pass 1   D[q row][key] = Q K^T   (M = 128 query rows, N = 128 keys per tile): the thread that
//            owns a TMEM lane owns a query row and keeps its online (max, sum) over the keys;
//   pass 2   D[key][q row] = K Q^T   (M = 128 keys, N = up to 128 query rows): the thread that owns a
//            lane owns a key, and the max over heads and the sum over window rows run over columns.
// A work item is one unit (layer, sequence, KV head) and wk <= 64 window rows of all g heads
// (g * wk <= 256 rows; wider windows take several items that add into the same sums).
//
// The kernel is persistent: one CTA per SM walks over the items, and the copy and tensor roles run
// on across item boundaries, so the next item's window queries and first key tiles are in flight,
// and its first products issued, while the softmax warps finish the item before. Warp 0 streams K
// tiles by TMA (a ring that continues across items; pass 2 walks the tiles backwards, so what it
// reads is still in L2) and the window queries (two buffers). The products are cut into turns of
// 128 x 128 (eight tcgen05.mma) that go round four 128-column TMEM accumulators; the turns of even
// number are issued by one thread (warp 1) and read back by one set of eight softmax warps, those
// of odd number by a second thread (warp 18) and the other set (warps 2-17: two sets of two groups
// of four warps, one TMEM lane quarter per warp). One thread needs longer to issue a turn (two
// waits, eight instructions, two commits) than the tensor core to execute it, and a set's
// tcgen05.ld latency is exposed once per turn: with two independent issuer / reader pairs, each
// with two accumulators of its own, one pair's waits and loads run under the other's work.
//
// Pass 1 is bound by the instructions of the exponentials (one per logit; the special-function unit
// does 16 a clock and SM): a quarter of them are evaluated on the FMA pipe instead, as
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
constexpr int kTcIssuerB = 2 + kTcSoftmaxThreads / 32;       // the warp after the softmax warps: second tcgen05.mma issuer
constexpr int kTcThreads = 64 + kTcSoftmaxThreads + 32;
constexpr int kTcTileKeys = 128;
constexpr int kTcMaxStages = 6;                              // K ring depth is chosen per launch from the shared memory left
constexpr int kTcKStageBytes = kTcTileKeys * kRowBytes;      // 32 KB: d-low half then d-high half
constexpr int kTcMaxRows = 256;
constexpr int kTcAccCols = 128;                              // TMEM columns of one accumulator (four of them)
constexpr uint32_t kTcTmemCols = 512;
constexpr int kTcChunkKeys = 8192;                           // keys whose window sums are held in shared memory at a time

struct __align__(8) ScoreTcTail {
    uint64_t q_full[2];
    uint64_t q_empty[2];
    uint64_t k_full[kTcMaxStages];
    uint64_t k_empty[kTcMaxStages];
    uint64_t d_full[4];
    uint64_t d_empty[4];
    uint64_t drain[2];
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
// Maximum of three (one instruction; NaN operands are dropped like in fmaxf).
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
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
// of the unscaled logits, `l` the sum of 2^((z - m_raw) * scale). Three quarters of the exponentials go to the
// special-function unit, a quarter to the FMA pipe.
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
        c0 = max3(c0, z[j], z[j + 1]);
        c1 = max3(c1, z[j + 2], z[j + 3]);
        c2 = max3(c2, z[j + 4], z[j + 5]);
        c3 = max3(c3, z[j + 6], z[j + 7]);
    }
    const float mn = fmaxf(max3(m_raw, c0, c1), fmaxf(c2, c3));
    if (mn == -INFINITY) return;
    const float neg = -mn * scale;
    float s0 = 0.f, s1 = 0.f;
    float2 sp = make_float2(0.f, 0.f);
    const float2 sc2 = make_float2(scale, scale), ng2 = make_float2(neg, neg);
#pragma unroll
    for (int j = 0; j < N; j += 8) {
        s0 += fast_exp2(fmaf(z[j], scale, neg));
        s1 += fast_exp2(fmaf(z[j + 1], scale, neg));
        s0 += fast_exp2(fmaf(z[j + 2], scale, neg));
        s1 += fast_exp2(fmaf(z[j + 3], scale, neg));
        s0 += fast_exp2(fmaf(z[j + 4], scale, neg));
        s1 += fast_exp2(fmaf(z[j + 5], scale, neg));
        const float2 a = fma_f32x2(make_float2(z[j + 6], z[j + 7]), sc2, ng2);
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

// Window rows of one block of the query tile (see the kernel's comment on the row order).
__host__ __device__ constexpr int score_tc_block_rows(int wk) { return wk == 64 ? 16 : 8; }

// WK = window rows handled by one item (16, 32 or 64).
//
// Order of the item's query rows in shared memory (row index of the pass-1 accumulators and of s_c, column index of
// the pass-2 accumulators): blocks of PW consecutive window rows of one head, the heads of a block of window rows next
// to each other: row = (wrb * g + h) * PW + jj for window row k0 + wrb * PW + jj of head h. So the columns that a
// pass-2 thread needs for the max over heads of a few window rows are contiguous and come with few tensor-memory
// loads, and the rows split into halves by window row, not by head.
//
// A turn is one 128 x 128 product (eight instructions) into one of four 128-column accumulators: in pass 1 a row
// tile (of MT) times a key tile, in pass 2 a key tile times a column chunk (of MT: all the rows, or with more than 128
// rows the rows of one half of the window). Turn t uses accumulator t % 4; turns of parity 0 belong to issuer 0 and
// softmax set 0, those of parity 1 to issuer 1 and set 1, so each pair works through its own two accumulators and the
// pairs share nothing but the K ring and the tensor core. With two row tiles set `rt` always gets row tile `rt` and
// the column chunk of window half `rt`.
// LONG: the keys do not fit the shared-memory window sums at once (a prompt of more than kTcChunkKeys tokens).
template <int WK, bool LONG>
__global__ void __launch_bounds__(kTcThreads, 1)
gkv_score_tc_kernel(const ScoreLaunch p, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_q, int n_cta, int stages, int q_bufs) {
    constexpr int PW = score_tc_block_rows(WK);      // window rows of a block
    constexpr int NB = WK / PW;                      // blocks of window rows: 2 or 4
    constexpr int HB = 32 / PW;                      // heads whose block columns one 32-column tensor-memory load covers
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int R = p.g * WK;                          // query rows of an item, a multiple of 16
    const int MT = (R + 127) >> 7;                   // 128-row tiles of pass 1 = column chunks of pass 2 = turns per key tile
    const int mt_shift = MT - 1;                     // MT is 1 or 2
    const int N2 = R >> mt_shift;                    // columns of a pass-2 product
    // the rows are loaded twice and the copies split a tile's keys (whole warps per copy: a warp reads one column range)
    const bool dup = 2 * R <= 128 && R % 32 == 0;
    const int q_half = MT * 128 * 128;               // bytes of one d-half of a Q buffer (d-low, then d-high)
    const int q_bytes = 2 * q_half;
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + (size_t)q_bufs * q_bytes;
    float* s_c = reinterpret_cast<float*>(k_smem + stages * kTcKStageBytes);      // [256] m + log2 l of every local row
    float* s_pm = s_c + kTcMaxRows;                                               // [groups][128] partial row maxima
    float* s_pl = s_pm + kTcGroups * 128;                                         // [groups][128] partial row sums
    // [MT][c_pad] window sums of this item's rows: a plane per softmax set that adds to a key (one set with one column
    // chunk, both with two), and within a plane the set's two groups add, so every sum is a + b (+ c + d in a fixed
    // order at the end) and the result does not depend on the order in which the groups arrive. Caches hold at most
    // kTcChunkKeys rows and fit whole; a longer key range (a prompt being compressed) passes through in chunks of
    // kTcChunkKeys keys, each written out when pass 2, which walks the tiles from the last to the first, leaves it.
    float* s_sum = s_pl + kTcGroups * 128;
    const int c_pad = LONG ? kTcChunkKeys : min((p.C + 63) & ~63, kTcChunkKeys);   // LONG: a chunk is 64 key tiles
    ScoreTcTail* tail = reinterpret_cast<ScoreTcTail*>(s_sum + MT * c_pad);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total_items = p.n_layers * p.batch * p.h_kv * n_cta;

    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tail->q_full[b]), 1);
            mbar_init(smem_u32(&tail->q_empty[b]), 2);                        // one commit from either issuer
        }
        for (int b = 0; b < 4; ++b) {
            mbar_init(smem_u32(&tail->d_full[b]), 1);
            mbar_init(smem_u32(&tail->d_empty[b]), kTcSoftmaxThreads / 64);   // one arrival per warp of the set that reads it
        }
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->k_full[s]), 1);
            mbar_init(smem_u32(&tail->k_empty[s]), MT);                       // one commit per turn that read the tile
        }
        mbar_init(smem_u32(&tail->drain[0]), 1);
        mbar_init(smem_u32(&tail->drain[1]), 1);
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
    for (int t = tid; t < MT * c_pad; t += kTcThreads) s_sum[t] = 0.f;
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
                        const int qhead0 = d.ls * p.h_q + d.head * p.g;   // first query head of the unit
                        uint8_t* qdst = q_smem + (size_t)qb * q_bytes;
                        // one box = a block of window rows of all g heads (the query map is [heads][w][d])
                        for (int c = 0; c < (dup ? 2 : 1); ++c)
                            for (int wrb = 0; wrb < NB; ++wrb) {
                                const uint32_t dst = smem_u32(qdst + (size_t)(c * R + wrb * p.g * PW) * 128);
                                tma_load_3d(dst, &tm_q, 0, d.k0 + wrb * PW, qhead0, qbar);
                                tma_load_3d(dst + q_half, &tm_q, 64, d.k0 + wrb * PW, qhead0, qbar);
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
                    tma_load_2d(dst, &tm_k, 0, y, bar);                      // 128-row boxes: d-low half, d-high half
                    tma_load_2d(dst + kTcKStageBytes / 2, &tm_k, 64, y, bar);
                    *(volatile int*)&tail->issued = ++issued;
                    if (++s == stages) { s = 0; ++round; }
                }
            }
        }
    } else if (warp == 1 || warp == kTcIssuerB) {
        // ------------------------------------------------------------------ MMA issuers
        // Two threads, one per turn parity. Issuing the eight instructions of a product, with its two waits before and
        // its two commits after, takes one thread longer than the tensor core needs for them; with two threads one
        // product's instructions are queued while the other's execute. The two never touch the same accumulator, and a
        // commit covers the instructions of the thread that makes it, so a ring slot is released by every turn that read
        // it (the barrier counts them) and the query buffer by both threads.
        if (lane == 0) {
            const int me = warp == 1 ? 0 : 1;
            const uint32_t k_lo = umma_desc_lo(smem_u32(k_smem));
            const uint32_t idesc1 = umma_idesc_bf16_m128(kTcTileKeys), idesc2 = umma_idesc_bf16_m128(N2);
            const int lstep = 2 >> mt_shift;            // K tiles between two turns of one issuer: 2 with one turn per tile, else 1
            int s = (me >> mt_shift) % stages, round = (me >> mt_shift) / stages;   // ring position of this issuer's next turn
            int t0 = 0;                                 // turn of the item's first product (always even)
            bool ok = true;
            for (int item = blockIdx.x, j = 0; ok && item < total_items; item += gridDim.x, ++j) {
                const ScoreItem d = score_item(p, item, n_cta, WK);
                const int qb = j % q_bufs;
                if (!tc_wait(smem_u32(&tail->q_full[qb]), (j / q_bufs) & 1, &tail->abort_flag)) {
                    tc_abort(tail, p.status, 22);
                    break;
                }
                const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem + (size_t)qb * q_bytes));
                // this issuer's operand of the query tile: pass 1 row tile `me` (of two) or the only one; pass 2 the column
                // chunk `me` (rows me * N2 ...) or all rows
                const uint32_t q_off1 = (uint32_t)((MT == 2 ? me * 128 : 0) * 128) >> 4, q_off2 = (uint32_t)((MT == 2 ? me * N2 : 0) * 128) >> 4;
                uint64_t q_desc[8];
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) q_desc[ks] = umma_desc(q_lo + umma_kstep(ks, q_half));
                const int half_turns = d.T << mt_shift, total = 2 * half_turns;
                for (int i = me; i < total; i += 2) {
                    const int turn = t0 + i;
                    const int acc = turn & 3, use = turn >> 2;   // accumulator of this turn and how often it has been used
                    const uint32_t dcol = tmem_base + (uint32_t)(acc * kTcAccCols);
                    if (use > 0 && !tc_wait(smem_u32(&tail->d_empty[acc]), (use - 1) & 1, &tail->abort_flag)) {
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
                    const uint64_t k_desc = umma_desc(k_lo + (uint32_t)s * (kTcKStageBytes >> 4));
                    if (i < half_turns) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(dcol, q_desc[ks] + q_off1, k_desc + umma_kstep(ks, kTcKStageBytes / 2), idesc1, ks > 0);
                    } else {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(dcol, k_desc + umma_kstep(ks, kTcKStageBytes / 2), q_desc[ks] + q_off2, idesc2, ks > 0);
                    }
                    umma_commit(smem_u32(&tail->k_empty[s]));
                    umma_commit(smem_u32(&tail->d_full[acc]));
                    s += lstep;
                    while (s >= stages) { s -= stages; ++round; }
                }
                if (ok) umma_commit(smem_u32(&tail->q_empty[qb]));   // this issuer's last product of the item has read its queries
                t0 += total;
            }
            // everything this thread issued has completed before the accumulators are given back
            umma_commit(smem_u32(&tail->drain[me]));
            mbar_wait_bounded(smem_u32(&tail->drain[me]), 0);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps
        // Two sets of two groups: set 0 takes the turns of parity 0, set 1 those of parity 1, so one set's
        // tensor-memory reads run under the other set's arithmetic.
        const int wg = (warp - 2) >> 2;               // group of four consecutive warps
        const int set = wg >> 1, sub = wg & 1;
        const int q4 = warp & 3;                      // TMEM lane quarter this warp may touch
        const int L = q4 * 32 + lane;                 // TMEM lane = accumulator row of this thread
        const int stid = (warp - 2) * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const float scale = p.scale_log2;
        bool ok = true;
        int t0 = 0;                                   // turn of the item's first product

        // pass-1 role of this thread: a row of the set's row tile, and 64 of a turn's 128 keys (32 for each copy when
        // the rows are loaded twice)
        const int copy = dup ? (L >= R ? 1 : 0) : 0;
        const int rl = (MT == 2 ? set * 128 : 0) + L - copy * R;                          // local query row
        const bool valid = (MT == 2) ? rl < R : L < (dup ? 2 * R : R);
        const int col0 = sub * 64 + copy * 32;
        const int nch1 = dup ? 1 : 2;                                                     // 32-key pieces per turn
        const int blk = rl / PW;
        const int row_k = (blk / p.g) * PW + (rl - blk * PW);                             // window row (within the item) of row rl
        // pass-2 role: the blocks of window rows whose columns this thread reduces for its key. One column chunk: the set
        // takes every other key tile and its two groups half of the window each; two chunks: the set takes the chunk of
        // its half of the window, its two groups a quarter each.
        const int nb2 = MT == 2 ? 1 : NB / 2;
        const int wrb0 = MT == 2 ? set * (NB / 2) + sub : sub * (NB / 2);
        const int colb0 = (MT == 2 ? sub : wrb0) * p.g * PW;                              // column of block wrb0 in the accumulator
        const int plane = MT == 2 ? set * c_pad : 0;     // this set's plane of the window sums

        for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
            const ScoreItem d = score_item(p, item, n_cta, WK);
            const int n = d.n, T = d.T, k0 = d.k0, half_turns = T << mt_shift, total = 2 * half_turns;
            // ---- pass 1: online (max, sum) of the row this thread owns over its share of its set's turns
            const int last_vis = n - p.w + k0 + row_k;        // last key the row's token sees
            float m_raw = -INFINITY, l = 0.f;                 // maximum in unscaled logits, sum relative to it
            for (int i = set; i < half_turns; i += 2) {
                const int turn = t0 + i, acc = turn & 3;
                const uint32_t t_acc = t_lane + (uint32_t)(acc * kTcAccCols);
                ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[acc]), (turn >> 2) & 1, &tail->abort_flag));
                if (!ok) { tc_abort(tail, p.status, 25); break; }
                tmem_fence_after_sync();
                const int kt = i >> mt_shift;
                const int key_base = kt * kTcTileKeys + col0;
                const bool need_mask = kt * kTcTileKeys + kTcTileKeys - 1 > n - p.w + k0;
#pragma unroll 1
                for (int ch = 0; ch < nch1; ++ch) {
                    float z[32];
                    tmem_ld<32>(t_acc + (uint32_t)(col0 + ch * 32), z);
                    if (valid) row_update<32>(z, key_base + ch * 32, last_vis, need_mask, scale, m_raw, l);
                }
                tmem_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[acc]));
            }
            // (a warp whose wait gave up still walks through every barrier below; all leave together at a point
            // where one thread's view of the abort flag decides for everybody)
            // combine the partials of a row and publish c = m + log2 l (scaled, log2 domain)
            s_pm[wg * 128 + L] = m_raw * scale;
            s_pl[wg * 128 + L] = l;
            softmax_bar_sync();
            if ((MT == 2) ? sub == 0 : (wg == 0 && L < R)) {
                // the groups that shared this row: with two row tiles, the two groups of the set; else all four
                const int first = (MT == 2) ? set * 2 : 0, count = (MT == 2) ? 2 : kTcGroups;
                float mm = -INFINITY, ll = 0.f;
                for (int c = 0; c <= (dup ? 1 : 0); ++c)
                    for (int q = first; q < first + count; ++q) mm = fmaxf(mm, s_pm[q * 128 + L + c * R]);
                for (int c = 0; c <= (dup ? 1 : 0); ++c)
                    for (int q = first; q < first + count; ++q) {
                        const float mq = s_pm[q * 128 + L + c * R];
                        ll += (mq == -INFINITY) ? 0.f : s_pl[q * 128 + L + c * R] * fast_exp2(mq - mm);
                    }
                if (rl < R) s_c[rl] = mm + log2f(ll);
            }
            if (stid == 0) tail->abort_seen = *(volatile int*)&tail->abort_flag;
            softmax_bar_sync();
            if (*(volatile int*)&tail->abort_seen) break;

            // ---- pass 2: this thread owns key `tile * 128 + L` of its set's turns
            // window sums of keys [lo, lo + c_pad) leave shared memory (which is zeroed for the next chunk or item)
            auto flush_chunk = [&](int lo) {
                float* out = p.sacc + (size_t)d.unit * p.C;
                const int hi = min(lo + c_pad, p.C);
                for (int t = lo + stid; t < hi; t += kTcSoftmaxThreads) {
                    float v = s_sum[t - lo];
                    s_sum[t - lo] = 0.f;
                    if (MT == 2) {
                        v += s_sum[c_pad + t - lo];
                        s_sum[c_pad + t - lo] = 0.f;
                    }
                    if (n_cta == 1) out[t] = (t < n) ? v : 0.f;
                    else if (t < n) atomicAdd(&out[t], v);   // buffer zeroed by the host
                }
            };
            int chunk_lo = 0;
            if constexpr (LONG) chunk_lo = T > 0 ? (((T - 1) * kTcTileKeys) & ~(kTcChunkKeys - 1)) : 0;
            for (int i = half_turns + ((half_turns ^ set) & 1); ok && i < total; i += 2) {   // this set's turns of pass 2
                const int turn = t0 + i, acc = turn & 3;
                const int tile = T - 1 - ((i - half_turns) >> mt_shift);
                if constexpr (LONG) {
                const int tile_lo = (tile * kTcTileKeys) & ~(kTcChunkKeys - 1);
                if (tile_lo != chunk_lo) {
                    // Every softmax warp has added its part of the chunk; then the chunk is written and cleared; then all
                    // go on. mbarrier waits, not bar.sync: a warp that gives up (abort flag) must not leave the others at
                    // a barrier it will never reach. (A chunk is 64 tiles, so both sets cross every boundary once.)
                    for (int step = 0; ok && step < 2; ++step) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&tail->chunk_bar));
                        // two phases of the barrier per boundary: its parity is `step` every time
                        ok = __all_sync(0xffffffffu, tc_wait(smem_u32(&tail->chunk_bar), (uint32_t)step, &tail->abort_flag));
                        if (ok && step == 0) flush_chunk(chunk_lo);
                    }
                    if (!ok) { tc_abort(tail, p.status, 27); break; }
                    chunk_lo = tile_lo;
                }
                }
                const uint32_t t_acc = t_lane + (uint32_t)(acc * kTcAccCols);
                ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[acc]), (turn >> 2) & 1, &tail->abort_flag));
                if (!ok) { tc_abort(tail, p.status, 26); break; }
                tmem_fence_after_sync();
                const int key = tile * kTcTileKeys + L;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll 1
                for (int b = 0; b < nb2; ++b) {
                    const int wrb = wrb0 + b;
                    float v[PW];
#pragma unroll
                    for (int jj = 0; jj < PW; ++jj) v[jj] = -INFINITY;
                    for (int h0 = 0; h0 < p.g; h0 += HB) {
                        float z[32];
                        tmem_ld<32>(t_acc + (uint32_t)(colb0 + (b * p.g + h0) * PW), z);
                        const float4* c4 = reinterpret_cast<const float4*>(s_c + (wrb * p.g + h0) * PW);
#pragma unroll
                        for (int hh = 0; hh < HB; hh += 2) {
                            if (h0 + hh + 1 < p.g) {          // two heads per maximum
#pragma unroll
                                for (int jj = 0; jj < PW; jj += 4) {
                                    const float4 c = c4[(hh * PW + jj) >> 2], e = c4[((hh + 1) * PW + jj) >> 2];
                                    v[jj] = max3(v[jj], fmaf(z[hh * PW + jj], scale, -c.x), fmaf(z[(hh + 1) * PW + jj], scale, -e.x));
                                    v[jj + 1] = max3(v[jj + 1], fmaf(z[hh * PW + jj + 1], scale, -c.y), fmaf(z[(hh + 1) * PW + jj + 1], scale, -e.y));
                                    v[jj + 2] = max3(v[jj + 2], fmaf(z[hh * PW + jj + 2], scale, -c.z), fmaf(z[(hh + 1) * PW + jj + 2], scale, -e.z));
                                    v[jj + 3] = max3(v[jj + 3], fmaf(z[hh * PW + jj + 3], scale, -c.w), fmaf(z[(hh + 1) * PW + jj + 3], scale, -e.w));
                                }
                            } else if (h0 + hh < p.g) {
#pragma unroll
                                for (int jj = 0; jj < PW; jj += 4) {
                                    const float4 c = c4[(hh * PW + jj) >> 2];
                                    v[jj] = fmaxf(v[jj], fmaf(z[hh * PW + jj], scale, -c.x));
                                    v[jj + 1] = fmaxf(v[jj + 1], fmaf(z[hh * PW + jj + 1], scale, -c.y));
                                    v[jj + 2] = fmaxf(v[jj + 2], fmaf(z[hh * PW + jj + 2], scale, -c.z));
                                    v[jj + 3] = fmaxf(v[jj + 3], fmaf(z[hh * PW + jj + 3], scale, -c.w));
                                }
                            }
                        }
                    }
                    if (b == nb2 - 1) {   // the last read of this turn: the accumulator goes back before the exponentials
                        tmem_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[acc]));
                    }
                    const int fk = key - (n - p.w) - k0 - wrb * PW;   // rows before it decoded before this key existed
#pragma unroll
                    for (int jj = 0; jj < PW; jj += 2) {
                        s0 += (jj >= fk) ? fast_exp2(v[jj]) : 0.f;
                        s1 += (jj + 1 >= fk) ? fast_exp2(v[jj + 1]) : 0.f;
                    }
                }
                if (key < n) atomicAdd(&s_sum[plane + key - chunk_lo], s0 + s1);   // two addends per key and plane (the set's two groups)
            }
            softmax_bar_sync();
            if (stid == 0) tail->abort_seen = *(volatile int*)&tail->abort_flag;
            if (ok && !*(volatile int*)&tail->abort_flag) {
                flush_chunk(chunk_lo);   // the chunk of the first tile, walked last
                // rows past the chunk that holds the last key were never in shared memory
                if (n_cta == 1) {
                    float* out = p.sacc + (size_t)d.unit * p.C;
                    for (int t = (T > 0 ? ((T - 1) * kTcTileKeys / c_pad + 1) * c_pad : 0) + stid; t < p.C; t += kTcSoftmaxThreads) out[t] = 0.f;
                }
            }
            softmax_bar_sync();      // the sums are clear and the row constants free before the next item uses them
            if (*(volatile int*)&tail->abort_seen) break;
            t0 += total;
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
           sizeof(float) * (kTcMaxRows + 2 * kTcGroups * 128 + mt * min((C + 63) & ~63, kTcChunkKeys)) + sizeof(ScoreTcTail);
}

// Rows of one box of the window-query tensor map (the kernel loads the queries block by block).
int score_tc_q_box_rows(int wk) { return score_tc_block_rows(wk); }

// Window rows per item for this shape, or 0 when the shape is left to the mma.sync kernel.
int score_tc_rows_per_cta(int g, int w) {
    if (w % 16 != 0 || g < 1 || g > kMaxGroup) return 0;
    for (int wk = 64; wk >= 16; wk >>= 1)
        if (wk <= w && w % wk == 0 && g * wk <= kTcMaxRows) return wk;
    return 0;
}

cudaError_t score_tc_kernel_setup() {
    const void* kernels[6] = {(const void*)gkv_score_tc_kernel<16, false>, (const void*)gkv_score_tc_kernel<32, false>,
                              (const void*)gkv_score_tc_kernel<64, false>, (const void*)gkv_score_tc_kernel<16, true>,
                              (const void*)gkv_score_tc_kernel<32, true>,  (const void*)gkv_score_tc_kernel<64, true>};
    for (const void* k : kernels) {
        const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Launch shape of the kernel for window rows per item `wk`: items, query rows per item, query buffers, ring depth,
// shared memory and grid.
void score_tc_plan(const ScoreLaunch& p, int wk, ScoreTcPlan* out) {
    const int n_cta = p.w / wk;
    const int units = p.n_layers * p.batch * p.h_kv;
    const int items = units * n_cta;
    // two buffers for the window queries when at least three K stages still fit beside them, then the deepest K ring
    const int rows = p.g * wk;
    const int q_bufs = score_tc_smem_bytes(p.C, rows, 3, 2) <= 227 * 1024 ? 2 : 1;
    int stages = 2;
    while (stages < kTcMaxStages && score_tc_smem_bytes(p.C, rows, stages + 1, q_bufs) <= 227 * 1024) ++stages;
    // With one turn per key tile the two issuers take alternate tiles. The ring depth must then be even, so that a ring
    // slot always belongs to the same issuer: a thread that saw only every other phase of a slot's barrier could pass a
    // parity wait two phases early. (With two turns per tile both issuers wait for every tile.)
    if (rows <= 128) stages &= ~1;
    // persistent: one CTA per SM (shared memory and tensor memory allow no more), rounds filled equally
    const int sm = p.sm_count > 0 ? p.sm_count : 148;
    int grid = items < sm ? items : sm;
    if (items > sm) {
        const int rounds = (items + sm - 1) / sm;
        grid = (items + rounds - 1) / rounds;
    }
    out->items = items; out->items_per_unit = n_cta; out->rows = rows; out->q_bufs = q_bufs; out->stages = stages;
    out->grid = grid; out->smem = score_tc_smem_bytes(p.C, rows, stages, q_bufs);
}

cudaError_t launch_score_tc(const ScoreLaunch& p, const CUtensorMap& tm_k, const CUtensorMap& tm_q, int wk, cudaStream_t s) {
    ScoreTcPlan plan;
    score_tc_plan(p, wk, &plan);
    const int n_cta = plan.items_per_unit, units = p.n_layers * p.batch * p.h_kv, stages = plan.stages, q_bufs = plan.q_bufs;
    const int grid = plan.grid;
    const size_t smem = plan.smem;
    if (n_cta > 1) {
        const size_t off = (size_t)p.layer0 * p.batch * p.h_kv * p.C;
        cudaError_t e = cudaMemsetAsync(p.sacc + off, 0, sizeof(float) * (size_t)units * p.C, s);
        if (e != cudaSuccess) return e;
    }
    const bool chunked = p.C > kTcChunkKeys;
    if (wk == 16 && !chunked) gkv_score_tc_kernel<16, false><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else if (wk == 32 && !chunked) gkv_score_tc_kernel<32, false><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else if (!chunked) gkv_score_tc_kernel<64, false><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else if (wk == 16) gkv_score_tc_kernel<16, true><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else if (wk == 32) gkv_score_tc_kernel<32, true><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    else gkv_score_tc_kernel<64, true><<<grid, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages, q_bufs);
    return cudaGetLastError();
}

}  // namespace gkv
