// GQA decode attention over the compressed cache, with the append of the current token and the
// optional accumulation of the window score (the every-step half of the G-KV path).
//
// A work item is one unit = (layer, sequence, KV head), or one piece of a unit split over the keys. The kernel
// is persistent: the grid holds as many CTAs as are resident at once, and each CTA takes items from a device-wide
// counter until none is left. A producer warp streams 64-key K and V tiles (TMA, 128-byte swizzle) through a ring of stages that
// runs on across item boundaries, so the first tiles of the next item are already in flight while the
// consumers finish the current one; four consumer warps each own 16 keys of every tile and keep their
// own online-softmax state, so the tile loop has no CTA-wide barrier, and every barrier of the per-item
// epilogue is among the consumer warps only. Both products run on mma.sync m16n8k16 with the KEYS on
// the M side and the g <= 8 query heads of the group on the N side (S^T = K Q^T, O^T = V^T P^T): no
// padded rows, each K/V byte is read from shared memory exactly once, and the P^T operand comes from
// the S^T accumulator by an 8x8 register transpose (movmatrix).
#include "gkv_common.cuh"
#include "gkv_internal.h"

namespace gkv {

constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 6;
constexpr int kPartFloats = 16 + kHeadDim * 8;  // M[8], L[8], acc[128][8]

struct __align__(16) DecodeSmemTail {
    uint64_t full_bar[kMaxStages];
    uint64_t empty_bar[kMaxStages];
    float m[kConsumerWarps][8];
    float l[kConsumerWarps][8];
    float fin_m[8];
    float fin_l[8];
    float fin_c[8];     // fin_m + log2 fin_l of the whole unit: what a window step subtracts from its parked logits
    float wgt[kConsumerWarps][8];
    uint64_t q_full;    // the item's query rows have landed in q_rows (one bulk copy by the producer lane)
    uint64_t q_empty;   // the four consumer warps have the item's query fragments in registers
    // Key split. First CTA of the cluster: the others arrive here when their partial results are in rx. Other CTAs
    // (window steps): the first CTA arrives here when it has stored the unit's fin_c into this CTA's shared memory.
    uint64_t cl_bar;
    // The group's g query rows, contiguous as in global memory, and the current token's k and v rows.
    alignas(16) uint8_t q_rows[8 * 256];
    alignas(16) uint8_t new_rows[2 * 256];
    // Scratch slot of the per-item epilogue: the cross-warp merge of the output accumulators (64 dims x 8 heads fp32
    // at a time; with key split the splits' statistics and weights), then the bf16 output rows on their way out.
    alignas(16) uint8_t scratch[8 * 256];
    int item_ids[8];   // work items in the order the producer took them (a ring: the producer is < 8 items ahead)
    int cur_item;      // the item the consumers are on, or -1: no more
    int abort_flag;
    int abort_seen;   // the abort flag as consumer thread 0 saw it between two barriers of the epilogue
    int issued;
    int q_issued;     // bulk copies of query rows started (the last one may be in flight at an abort)
    int is_last;
    uint32_t tmem_base;
};

__device__ __forceinline__ void latch_timeout(int32_t* status, int where) {
    if (atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}
// Bounded wait that also gives up as soon as another role of the CTA has raised the abort flag.
__device__ __forceinline__ bool decode_wait(uint32_t bar, uint32_t parity, const int* abort_flag) {
    for (uint32_t i = 0; i < kWaitSpins; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*(volatile const int*)abort_flag) return false;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

// Shared memory for the unit's window sums on window steps without key split.
__host__ __device__ constexpr size_t decode_sum_bytes(int C, int accum_mode) {
    return accum_mode == 1 ? (size_t)((C + 63) & ~63) * sizeof(float) : 0;
}

// What one work item covers.
struct DecodeItem {
    int unit_local, split, head, layer_local, seq, lseq_global;
    long unit;
    int len_old, n, tiles_total, t_begin, t_end, slot_end, row0;
};
__device__ __forceinline__ DecodeItem decode_item(const DecodeLaunch& p, int item) {
    DecodeItem d;
    d.unit_local = item / p.splits;
    d.split = item - d.unit_local * p.splits;
    d.head = d.unit_local % p.h_kv;
    const int ls = d.unit_local / p.h_kv;             // layer_local * batch + seq
    d.layer_local = ls / p.batch;
    d.seq = ls - d.layer_local * p.batch;
    d.lseq_global = (p.layer0 + d.layer_local) * p.batch + d.seq;
    d.unit = (long)d.lseq_global * p.h_kv + d.head;
    d.len_old = p.len[d.lseq_global];
    d.n = d.len_old + 1;                              // keys attended (current token included)
    d.tiles_total = (d.n + kTileKeys - 1) / kTileKeys;
    const int tps = (d.tiles_total + p.splits - 1) / p.splits;
    d.t_begin = min(d.split * tps, d.tiles_total);
    d.t_end = min(d.t_begin + tps, d.tiles_total);
    d.slot_end = max(d.t_end, d.t_begin + 1);         // ring slots the item takes: its tiles, or one empty slot
    d.row0 = (int)(d.unit * p.C);                     // first cache row of this unit in the 2-D view
    return d;
}

// ACCUM = 0: plain step. ACCUM = 1: window step (the logits are parked in TMEM until the unit's normaliser is known).
template <int ACCUM>
__global__ void __launch_bounds__(kDecodeThreads, 3)
gkv_decode_kernel(const DecodeLaunch p, const __grid_constant__ DecodeMaps maps) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the swizzled TMA boxes
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint8_t* stage_base = smem;
    float* s_sum = reinterpret_cast<float*>(smem + (size_t)stages * kStageBytes);   // [C] window sums, window steps only
    DecodeSmemTail* tail = reinterpret_cast<DecodeSmemTail*>(smem + (size_t)stages * kStageBytes + decode_sum_bytes(p.C, ACCUM));
    // Window steps keep the scaled logits [key][head] on chip until the row's
    // normaliser is final. They live in tensor memory, not shared memory: a consumer thread parks
    // the 4 values it owns of every tile in 4 columns of its own TMEM lane and reads them back
    // itself in the epilogue, so shared memory (and with it the number of resident CTAs) is nearly the
    // same as on plain steps.
    constexpr bool use_tmem = ACCUM == 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total_items = p.n_layers * p.batch * p.h_kv * p.splits;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->full_bar[s]), 1);
            mbar_init(smem_u32(&tail->empty_bar[s]), kConsumerWarps);
        }
        mbar_init(smem_u32(&tail->q_full), 1);
        mbar_init(smem_u32(&tail->q_empty), kConsumerWarps);
        if (p.splits > 1) mbar_init(smem_u32(&tail->cl_bar), (blockIdx.x % p.splits == 0) ? (uint32_t)p.splits - 1 : 1u);
        tail->q_issued = 0;
        tail->abort_flag = 0;
        tail->abort_seen = 0;
        tail->cur_item = -1;
        tail->issued = 0;
        tail->is_last = 0;
        fence_mbar_init();
    }
    if (use_tmem && warp == kConsumerWarps) {   // whole warp; p.tmem_cols x resident CTAs <= 512, so this never waits
        tmem_alloc(smem_u32(&tail->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish_alloc_permit();
        tmem_fence_before_sync();
    }
    __syncthreads();
    // Key split: the CTAs of a unit form a cluster (launched so); none may reach into another's shared memory or
    // barriers before all have initialised theirs.
    if (p.splits > 1) cluster_sync_all();
    if (use_tmem) tmem_fence_after_sync();
    const uint32_t tmem_warp = use_tmem ? (*(volatile uint32_t*)&tail->tmem_base + ((uint32_t)(warp & 3) << 21)) : 0u;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            prefetch_tensormap(&maps.k64);
            prefetch_tensormap(&maps.v64);
            prefetch_tensormap(&maps.k16);
            prefetch_tensormap(&maps.v16);
            int s = 0, round = 0;                       // ring position, carried across items
            bool ok = true;
            // Work items are handed out first come, first served: a CTA's first item is its own index, every further
            // one comes from a device-wide counter. (CTAs do not run at the same speed -- per-item times differ by
            // several per cent with the SM's place on the chip -- and a fixed share would leave the fast ones idle
            // at the end.) The item's number travels to the consumers in a small ring, written before the arrive on
            // the item's first slot; the list ends with an empty slot that carries -1.
            int item = blockIdx.x;
            for (int k = 0; ok; ++k) {
                const bool more = item < total_items;
                tail->item_ids[k & 7] = more ? item : -1;
                DecodeItem d;
                if (more) {
                    d = decode_item(p, item);
                    // The group's query rows, one bulk copy, started the moment the item is known: about two tiles
                    // before the consumers get to it, so the rows' latency -- microseconds when q is mapped host
                    // memory and the bus is busy -- is over by then. The buffer is free once the consumers have
                    // the previous item's fragments in registers, which they take at the start of an item.
                    if (k > 0 && !decode_wait(smem_u32(&tail->q_empty), (k - 1) & 1, &tail->abort_flag)) {
                        if (!*(volatile int*)&tail->abort_flag) latch_timeout(p.status, 4);
                        tail->abort_flag = 1;
                        break;
                    }
                    const uint32_t qbar = smem_u32(&tail->q_full);
                    const bool appends = d.len_old / kTileKeys >= d.t_begin && d.len_old / kTileKeys < d.t_end;
                    mbar_arrive_expect_tx(qbar, (uint32_t)p.g * 256u + (appends ? 512u : 0u));
                    bulk_load(smem_u32(tail->q_rows),
                              p.q + ((size_t)(d.layer_local * p.batch + d.seq) * p.h_q + (size_t)d.head * p.g) * kHeadDim,
                              (uint32_t)p.g * 256u, qbar);
                    if (appends) {   // this item holds the tile that the current token's row goes into
                        const size_t src = ((size_t)(d.layer_local * p.batch + d.seq) * p.h_kv + d.head) * kHeadDim;
                        bulk_load(smem_u32(tail->new_rows), p.k_new + src, 256u, qbar);
                        bulk_load(smem_u32(tail->new_rows + 256), p.v_new + src, 256u, qbar);
                    }
                    *(volatile int*)&tail->q_issued = k + 1;
                } else {
                    d.t_begin = d.t_end = 0; d.slot_end = 1; d.n = 0; d.row0 = 0;
                }
                for (int it = d.t_begin; it < d.slot_end; ++it) {
                    if (round > 0 && !decode_wait(smem_u32(&tail->empty_bar[s]), (round - 1) & 1, &tail->abort_flag)) {
                        if (!*(volatile int*)&tail->abort_flag) latch_timeout(p.status, 1);
                        tail->abort_flag = 1;
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&tail->full_bar[s]);
                    const uint32_t dst = smem_u32(stage_base + (size_t)s * kStageBytes);
                    const int y = d.row0 + it * kTileKeys;
                    const int rows_left = d.n - it * kTileKeys;     // keys of this tile that exist
                    if (it >= d.t_end) {
                        // A split without a tile still passes one empty slot through the ring. The consumers wait for
                        // it, so they cannot complete the item -- and with it perhaps the sequence, whose length is
                        // then rewritten -- before this lane has read the item's length.
                        mbar_arrive(bar);
                    } else if (rows_left > kTileKeys - 16) {
                        mbar_arrive_expect_tx(bar, kStageBytes);
                        tma_load_2d(dst, &maps.k64, 0, y, bar);
                        tma_load_2d(dst + kBoxBytes, &maps.k64, 64, y, bar);
                        tma_load_2d(dst + kTileBytes, &maps.v64, 0, y, bar);
                        tma_load_2d(dst + kTileBytes + kBoxBytes, &maps.v64, 64, y, bar);
                    } else {
                        // ragged last tile: only the 16-row pieces that hold keys (a 16-row piece of a 128-byte-swizzled
                        // 64-row box is 2 KB at row offset 16 * piece; the swizzle pattern repeats every 8 rows)
                        const int pieces = (rows_left + 15) >> 4;
                        mbar_arrive_expect_tx(bar, (uint32_t)pieces * 4 * 2048);
                        for (int pc = 0; pc < pieces; ++pc) {
                            const uint32_t o = (uint32_t)pc * 2048;
                            tma_load_2d(dst + o, &maps.k16, 0, y + pc * 16, bar);
                            tma_load_2d(dst + kBoxBytes + o, &maps.k16, 64, y + pc * 16, bar);
                            tma_load_2d(dst + kTileBytes + o, &maps.v16, 0, y + pc * 16, bar);
                            tma_load_2d(dst + kTileBytes + kBoxBytes + o, &maps.v16, 64, y + pc * 16, bar);
                        }
                    }
                    *(volatile int*)&tail->issued = *(volatile int*)&tail->issued + 1;
                    if (++s == stages) { s = 0; ++round; }
                }
                if (!more) break;
                // a split launch has one CTA per item (the cluster's ranks are the unit's pieces)
                item = (p.splits > 1) ? total_items : (int)gridDim.x + atomicAdd(p.work_next, 1);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int r_in = lane & 7, mat = lane >> 3;
        const int hq = lane >> 2;                     // head whose Q row this lane holds (B operand)
        const int krow = warp * 16 + (mat & 1) * 8 + r_in;   // K ldmatrix: row this lane addresses
        const int kch = mat >> 1;                             //   and which 16-byte chunk of the k step
        const int vrow = warp * 16 + (mat >> 1) * 8 + r_in;   // V ldmatrix (transposed)
        const int vch = mat & 1;
        const int h0 = (lane & 3) * 2;                // heads of this lane's accumulator columns: h0, h0 + 1
        int s = 0, round = 0;                         // ring position, carried across items

        for (int k = 0;; ++k) {
            // One thread waits for the first slot of the next item (the tile loop waits on it again and passes at
            // once) and reads the item's number; the barrier hands it to the other consumers, and it is also the point
            // where the previous item's use of the scratch slot, the statistics and the window sums has ended.
            if (tid == 0) {
                int next = -1;
                bool timed_out = false;
                if (decode_wait(smem_u32(&tail->full_bar[s]), round & 1, &tail->abort_flag)) {
                    next = *(volatile int*)&tail->item_ids[k & 7];
                    if (next >= 0 && !decode_wait(smem_u32(&tail->q_full), k & 1, &tail->abort_flag)) {
                        next = -1;
                        timed_out = true;
                    }
                } else {
                    timed_out = true;
                }
                if (timed_out) {
                    if (!*(volatile int*)&tail->abort_flag) latch_timeout(p.status, 3);
                    tail->abort_flag = 1;
                }
                tail->cur_item = next;
            }
            consumer_bar_sync();
            const int item = *(volatile int*)&tail->cur_item;
            if (item < 0) break;
            const DecodeItem d = decode_item(p, item);
            const int n = d.n, len_old = d.len_old;

            // The group's g query rows are in q_rows (thread 0 has seen the copy complete; the wait below passes at
            // once and makes the copied bytes visible to this thread). Fragment order: B[k = d][n = head].
            uint32_t qf[8][2];
            (void)decode_wait(smem_u32(&tail->q_full), k & 1, &tail->abort_flag);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                if (hq < p.g) {
                    const uint8_t* row = tail->q_rows + hq * 256 + ks * 32 + (lane & 3) * 4;
                    qf[ks][0] = *reinterpret_cast<const uint32_t*>(row);
                    qf[ks][1] = *reinterpret_cast<const uint32_t*>(row + 16);
                } else {
                    qf[ks][0] = qf[ks][1] = 0u;
                }
            }
            // The current token's row lands in the last tile; the warp that will append it takes its 16 bytes per lane
            // now (lanes 0-15 of the k row, 16-31 of the v row).
            uint4 new_row = make_uint4(0u, 0u, 0u, 0u);
            if (warp == ((len_old & (kTileKeys - 1)) >> 4) && (len_old / kTileKeys) >= d.t_begin && (len_old / kTileKeys) < d.t_end)
                new_row = *reinterpret_cast<const uint4*>(tail->new_rows + (lane >> 4) * 256 + (lane & 15) * 16);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->q_empty));
            // Window steps: the unit's current window sums start their way into shared memory now and are needed only
            // in the epilogue; the updated sums go back with plain coalesced stores. (One atomic per key is measurably
            // slower: the L2 atomic units saturate at ~4 M reductions a launch.)
            if (ACCUM == 1) {
                const float* gsum = p.sacc + (size_t)d.unit * p.C;
                const int k_hi = min(d.t_end * kTileKeys, n);      // this item's keys: [t_begin * 64, k_hi)
                for (int t = d.t_begin * kTileKeys + tid; t < k_hi; t += kConsumerThreads) cp_async_4(smem_u32(s_sum + t), gsum + t);
                cp_async_commit();
            }

            // per-thread softmax / output state (heads h0, h0 + 1)
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
            float acc[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

            for (int it = d.t_begin; it < d.slot_end; ++it) {   // an empty slot has key0 >= n: nothing to compute
                if (!decode_wait(smem_u32(&tail->full_bar[s]), round & 1, &tail->abort_flag)) {
                    if (!*(volatile int*)&tail->abort_flag) latch_timeout(p.status, 2);
                    tail->abort_flag = 1;
                    break;
                }
                uint8_t* kt = stage_base + (size_t)s * kStageBytes;
                uint8_t* vt = kt + kTileBytes;
                const int key0 = it * kTileKeys + warp * 16;
                if (key0 < n) {
                    // append: the warp that owns row len_old overwrites it (in the tile and in the cache)
                    if (len_old >= key0 && len_old < key0 + 16) {
                        const int lr = len_old - it * kTileKeys;          // row inside the tile
                        const int c = lane & 15;
                        const size_t dstg = ((size_t)d.unit * p.C + len_old) * kHeadDim + c * 8;
                        if (lane < 16) {
                            *reinterpret_cast<uint4*>(kt + tile_off(lr, c)) = new_row;
                            *reinterpret_cast<uint4*>(p.k_cache + dstg) = new_row;
                        } else {
                            *reinterpret_cast<uint4*>(vt + tile_off(lr, c)) = new_row;
                            *reinterpret_cast<uint4*>(p.v_cache + dstg) = new_row;
                        }
                        fence_proxy_async_smem();
                    }
                    // rows past the end of the cache may hold anything: zero the V rows so 0 * x stays 0
                    if (key0 + 16 > n) {
                        const int first = n - it * kTileKeys;             // first invalid row of the tile
                        for (int e = lane; e < (warp * 16 + 16 - first) * 16; e += 32) {
                            const int lr = first + (e >> 4);
                            *reinterpret_cast<uint4*>(vt + tile_off(lr, e & 15)) = make_uint4(0, 0, 0, 0);
                        }
                    }
                    __syncwarp();

                    // S^T[16 keys x 8 heads] = K_tile Q^T, two accumulators to halve the dependent chain
                    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
                    const uint32_t kaddr = smem_u32(kt);
#pragma unroll
                    for (int ks = 0; ks < 8; ks += 2) {
                        uint32_t a[4], a2[4];
                        ldmatrix_x4(kaddr + tile_off(krow, ks * 2 + kch), a);
                        ldmatrix_x4(kaddr + tile_off(krow, ks * 2 + 2 + kch), a2);
                        mma_bf16_16816(sa, a, qf[ks][0], qf[ks][1]);
                        mma_bf16_16816(sb, a2, qf[ks + 1][0], qf[ks + 1][1]);
                    }
                    const int key_a = key0 + (lane >> 2), key_b = key_a + 8;
                    float s0 = (sa[0] + sb[0]) * p.scale_log2, s1 = (sa[1] + sb[1]) * p.scale_log2;
                    float s2 = (sa[2] + sb[2]) * p.scale_log2, s3 = (sa[3] + sb[3]) * p.scale_log2;
                    if (key_a >= n) s0 = s1 = -INFINITY;
                    if (key_b >= n) s2 = s3 = -INFINITY;
                    if (ACCUM == 1) tmem_st4(tmem_warp + 4u * (uint32_t)it, s0, s1, s2, s3);
                    // tile maximum per head over the warp's 16 keys (lanes sharing lane & 3)
                    float t0 = fmaxf(s0, s2), t1 = fmaxf(s1, s3);
#pragma unroll
                    for (int o = 4; o < 32; o <<= 1) {
                        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, o));
                        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, o));
                    }
                    const float mn0 = fmaxf(m0, t0), mn1 = fmaxf(m1, t1);
                    const float sc0 = fast_exp2(m0 - mn0), sc1 = fast_exp2(m1 - mn1);
                    m0 = mn0; m1 = mn1;
                    const float p0 = fast_exp2(s0 - mn0), p1 = fast_exp2(s1 - mn1);
                    const float p2 = fast_exp2(s2 - mn0), p3 = fast_exp2(s3 - mn1);
                    l0 = l0 * sc0 + p0 + p2;
                    l1 = l1 * sc1 + p1 + p3;
                    if (__any_sync(0xffffffffu, (sc0 != 1.f) | (sc1 != 1.f))) {
#pragma unroll
                        for (int dt = 0; dt < 8; ++dt) {
                            acc[dt][0] *= sc0; acc[dt][1] *= sc1; acc[dt][2] *= sc0; acc[dt][3] *= sc1;
                        }
                    }
                    // P^T operand: transpose the two 8x8 (key x head) blocks in registers
                    const uint32_t b0 = movmatrix_trans(pack_bf16x2(p0, p1));
                    const uint32_t b1 = movmatrix_trans(pack_bf16x2(p2, p3));
                    const uint32_t vaddr = smem_u32(vt);
#pragma unroll
                    for (int dt = 0; dt < 8; ++dt) {
                        uint32_t a[4];
                        ldmatrix_x4_trans(vaddr + tile_off(vrow, dt * 2 + vch), a);
                        mma_bf16_16816(acc[dt], a, b0, b1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tail->empty_bar[s]));
                if (++s == stages) { s = 0; ++round; }
            }

            // ---------------------------------------------------------------- per-item epilogue (consumer warps only)
            if (use_tmem) tmem_wait_st();
            if (ACCUM == 1) cp_async_wait_all();
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, o);
                l1 += __shfl_xor_sync(0xffffffffu, l1, o);
            }
            if ((lane >> 2) == 0) {
                tail->m[warp][h0] = m0; tail->m[warp][h0 + 1] = m1;
                tail->l[warp][h0] = l0; tail->l[warp][h0 + 1] = l1;
            }
            consumer_bar_sync();   // [E1] statistics of the four warps are in
            // One thread samples the abort flag between two barriers, so that the four warps take the same decision
            // even when the producer raises the flag at this very moment.
            if (tid == 32) tail->abort_seen = *(volatile int*)&tail->abort_flag;
            // per head: the combined (max, sum) and each warp's weight
            if (tid < 8) {
                const int h = tid;
                float mm = tail->m[0][h];
#pragma unroll
                for (int w = 1; w < kConsumerWarps; ++w) mm = fmaxf(mm, tail->m[w][h]);
                float ll = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) {
                    const float wm = tail->m[w][h];
                    const float wgt = (wm == -INFINITY) ? 0.f : fast_exp2(wm - mm);
                    tail->wgt[w][h] = wgt;
                    ll += wgt * tail->l[w][h];
                }
                tail->fin_m[h] = mm;
                tail->fin_l[h] = ll;
                if (ACCUM != 0) tail->fin_c[h] = (h < p.g) ? mm + log2f(ll) : INFINITY;
            }
            consumer_bar_sync();   // [E2]
            if (*(volatile int*)&tail->abort_seen) break;   // all four warps leave together
            // Cross-warp merge of the accumulators, 64 dims at a time through the 2 KB scratch slot: warp 0 stores its
            // weighted part, warps 1..3 add theirs one after the other (fixed order: the result does not depend on
            // timing); then thread tid reads the 8 heads of dim tid.
            float o[8];
            {
                const float w0 = tail->wgt[warp][h0], w1 = tail->wgt[warp][h0 + 1];
                float* s_o = reinterpret_cast<float*>(tail->scratch);     // [64 dims][8 heads]
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int k = 0; k < kConsumerWarps; ++k) {
                        if (warp == k) {
#pragma unroll
                            for (int dq = 0; dq < 4; ++dq) {
                                const int dt = half * 4 + dq;
                                float2* lo = reinterpret_cast<float2*>(s_o + (dq * 16 + (lane >> 2)) * 8 + h0);
                                float2* hi = reinterpret_cast<float2*>(s_o + (dq * 16 + (lane >> 2) + 8) * 8 + h0);
                                float2 a = make_float2(acc[dt][0] * w0, acc[dt][1] * w1);
                                float2 b = make_float2(acc[dt][2] * w0, acc[dt][3] * w1);
                                if (k > 0) { const float2 pa = *lo, pb = *hi; a.x += pa.x; a.y += pa.y; b.x += pb.x; b.y += pb.y; }
                                *lo = a; *hi = b;
                            }
                        }
                        consumer_bar_sync();
                    }
                    if ((tid >> 6) == half) {
                        const float4 x = *reinterpret_cast<const float4*>(s_o + (tid & 63) * 8);
                        const float4 y = *reinterpret_cast<const float4*>(s_o + (tid & 63) * 8 + 4);
                        o[0] = x.x; o[1] = x.y; o[2] = x.z; o[3] = x.w; o[4] = y.x; o[5] = y.y; o[6] = y.z; o[7] = y.w;
                    }
                    consumer_bar_sync();   // the slot is read before the next half (or the next use) overwrites it
                }
            }

            bool do_final = true;          // this CTA writes the output (always true without split)
            if (p.splits > 1) {
                // (Lifetime of the shared memory that other CTAs of the cluster write: rx and cl_bar of the first CTA;
                // on window steps also fin_c and cl_bar of the others. Every CTA of a split launch arrives on the
                // cluster barrier as its last act, and the CTAs that own remotely written memory also wait on it, so
                // they stay resident until every peer has passed its last remote store -- by order, also when a bounded
                // wait has expired somewhere, since every wait in this kernel is bounded and every CTA gets to the end.)
                // The pieces of a unit are the CTAs of one cluster. Every CTA stores its (max, sum) per head and its
                // accumulators into slot `rank` of the receive buffer in the shared memory of the cluster's first CTA
                // (distributed shared memory: no trip through L2, no completion counter in global memory), then
                // arrives on that CTA's mbarrier and is done. The first CTA waits for the others and merges.
                float* rx = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(tail) + sizeof(DecodeSmemTail));   // [splits][kPartFloats]
                const uint32_t slot = cluster_map_shared(smem_u32(rx + (size_t)d.split * kPartFloats), 0);
                if (tid < 8) {
                    st_cluster_f32(slot + 4u * tid, tail->fin_m[tid]);
                    st_cluster_f32(slot + 4u * (8 + tid), tail->fin_l[tid]);
                }
                st_cluster_f32x4(slot + 4u * (16 + tid * 8), o[0], o[1], o[2], o[3]);
                st_cluster_f32x4(slot + 4u * (16 + tid * 8 + 4), o[4], o[5], o[6], o[7]);
                fence_acq_rel_cluster();
                consumer_bar_sync();
                do_final = d.split == 0;
                if (!do_final && tid == 0) mbar_arrive_cluster(cluster_map_shared(smem_u32(&tail->cl_bar), 0));
                // The first CTA waits for the others' partial results; on a window step the others wait for the first
                // CTA to hand them the unit's normaliser (they hold the logits of their own keys).
                if (do_final || ACCUM != 0) {
                    if (tid == 0) {
                        bool ok = false;
                        for (uint32_t i = 0; i < kWaitSpins && !ok; ++i) {
                            ok = mbar_try_wait_cluster(smem_u32(&tail->cl_bar), 0);
                            if (!ok && *(volatile int*)&tail->abort_flag) break;
                            if (!ok && i > 64) __nanosleep(64);
                        }
                        if (!ok) {
                            if (!*(volatile int*)&tail->abort_flag) latch_timeout(p.status, 5);
                            tail->abort_flag = 1;
                        }
                        tail->is_last = ok;
                    }
                    consumer_bar_sync();
                    if (!tail->is_last) break;   // all four warps: the cluster did not deliver
                    fence_acq_rel_cluster();
                }
                if (do_final) {
                    // (1) per head the global max, the pieces' weights and the global sum, (2) per dim the weighted sum
                    // of the pieces' accumulators
                    float* s_stat = reinterpret_cast<float*>(tail->scratch);   // [splits <= 8][16]: M[8] (then the weights), L[8]
                    for (int idx = tid; idx < p.splits * 16; idx += kConsumerThreads)
                        s_stat[idx] = rx[(size_t)(idx >> 4) * kPartFloats + (idx & 15)];
                    consumer_bar_sync();
                    if (tid < 8) {
                        const int h = tid;
                        float mm = -INFINITY;
                        for (int sp = 0; sp < p.splits; ++sp) mm = fmaxf(mm, s_stat[sp * 16 + h]);
                        float ll = 0.f;
                        for (int sp = 0; sp < p.splits; ++sp) {
                            const float wm = s_stat[sp * 16 + h];
                            const float wgt = (wm == -INFINITY) ? 0.f : fast_exp2(wm - mm);
                            s_stat[sp * 16 + h] = wgt;   // over the maximum it came from: only this thread reads that word
                            ll += wgt * s_stat[sp * 16 + 8 + h];
                        }
                        tail->fin_m[h] = mm;
                        tail->fin_l[h] = ll;
                        if (ACCUM != 0) {
                            const float c = (h < p.g) ? mm + log2f(ll) : INFINITY;
                            tail->fin_c[h] = c;
                            for (int r = 1; r < p.splits; ++r) st_cluster_f32(cluster_map_shared(smem_u32(&tail->fin_c[h]), (uint32_t)r), c);
                            fence_acq_rel_cluster();
                        }
                    }
                    consumer_bar_sync();
                    if (ACCUM != 0 && tid == 0)
                        for (int r = 1; r < p.splits; ++r) mbar_arrive_cluster(cluster_map_shared(smem_u32(&tail->cl_bar), (uint32_t)r));
#pragma unroll
                    for (int h = 0; h < 8; ++h) o[h] = 0.f;
#pragma unroll 4
                    for (int sp = 0; sp < p.splits; ++sp) {
                        const float4* a4 = reinterpret_cast<const float4*>(rx + (size_t)sp * kPartFloats + 16 + tid * 8);
                        const float4 a = a4[0], b = a4[1];
                        const float4 wa = *reinterpret_cast<const float4*>(s_stat + sp * 16);
                        const float4 wb = *reinterpret_cast<const float4*>(s_stat + sp * 16 + 4);
                        o[0] = fmaf(wa.x, a.x, o[0]); o[1] = fmaf(wa.y, a.y, o[1]); o[2] = fmaf(wa.z, a.z, o[2]); o[3] = fmaf(wa.w, a.w, o[3]);
                        o[4] = fmaf(wb.x, b.x, o[4]); o[5] = fmaf(wb.y, b.y, o[5]); o[6] = fmaf(wb.z, b.z, o[6]); o[7] = fmaf(wb.w, b.w, o[7]);
                    }
                    consumer_bar_sync();   // weights read before the slot turns into the output rows
                }
            }

            if (do_final) {
                // out = o / L as bf16, transposed through the scratch slot so that it leaves in 16-byte pieces, 256
                // contiguous bytes per head: one row per half warp.
#pragma unroll
                for (int h = 0; h < 8; ++h)
                    if (h < p.g)
                        *reinterpret_cast<__nv_bfloat16*>(tail->scratch + h * 256 + tid * 2) = __float2bfloat16_rn(o[h] / tail->fin_l[h]);
                consumer_bar_sync();
                if (tid < p.g * 16) {
                    const int h = tid >> 4, c = tid & 15;
                    __nv_bfloat16* orow = p.out + ((size_t)(d.layer_local * p.batch + d.seq) * p.h_q + (size_t)d.head * p.g + h) * kHeadDim;
                    *reinterpret_cast<uint4*>(orow + c * 8) = *reinterpret_cast<const uint4*>(tail->scratch + h * 256 + c * 16);
                }
            }
            if (ACCUM != 0) {
                // Sacc[t] += max over the group of the final weights = exp2(max_h (z_h[t] - M_h - log2 L_h)), for the keys
                // of this item's tiles: their logits are in this CTA's TMEM, and each key is owned by exactly one thread.
                const float c0 = tail->fin_c[h0], c1 = tail->fin_c[h0 + 1];
                float* gsum = p.sacc + (size_t)d.unit * p.C;
                // four tiles per TMEM access; columns of tiles that are not this item's hold other data and are skipped
                for (int it4 = d.t_begin & ~3; it4 < d.t_end; it4 += 4) {
                    float z[16];
                    tmem_ld16(tmem_warp + 4u * (uint32_t)it4, z);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (it4 + u < d.t_begin || it4 + u >= d.t_end) continue;   // the same for the whole warp
                        float va = fmaxf(z[4 * u] - c0, z[4 * u + 1] - c1), vb = fmaxf(z[4 * u + 2] - c0, z[4 * u + 3] - c1);
                        va = fmaxf(va, __shfl_xor_sync(0xffffffffu, va, 1));
                        vb = fmaxf(vb, __shfl_xor_sync(0xffffffffu, vb, 1));
                        va = fmaxf(va, __shfl_xor_sync(0xffffffffu, va, 2));
                        vb = fmaxf(vb, __shfl_xor_sync(0xffffffffu, vb, 2));
                        const int key = (it4 + u) * kTileKeys + warp * 16 + (lane >> 2) + ((lane & 1) ? 8 : 0);
                        if ((lane & 2) == 0 && key < n) s_sum[key] += fast_exp2((lane & 1) ? vb : va);
                    }
                }
                consumer_bar_sync();   // every key's sum is final (its prefetch landed before [E1])
                const int k_hi = min(d.t_end * kTileKeys, n);
                for (int t = d.t_begin * kTileKeys + tid; t < k_hi; t += kConsumerThreads) gsum[t] = s_sum[t];
            }

            // The last item of a (layer, sequence) publishes the new length.
            if (tid == 0) {
                const int per_seq = p.h_kv * p.splits;
                const int prev = atomicAdd(&p.seq_done[d.lseq_global], 1);
                if (prev == per_seq - 1) {
                    p.seq_done[d.lseq_global] = 0;
                    p.len[d.lseq_global] = n;
                }
            }
        }
    }

    if (use_tmem && warp < kConsumerWarps) tmem_fence_before_sync();
    __syncthreads();   // producer and consumers
    if (*(volatile int*)&tail->abort_flag && tid == 0) {
        // Give copies that are still in flight a bounded time to land before the CTA exits: the last `stages` tiles
        // issued (an earlier one on the same stage completed before its successor could be issued).
        const int issued = *(volatile int*)&tail->issued;
        for (int j = max(0, issued - stages); j < issued; ++j)
            mbar_wait_bounded(smem_u32(&tail->full_bar[j % stages]), (j / stages) & 1);
        const int q_issued = *(volatile int*)&tail->q_issued;
        if (q_issued > 0) mbar_wait_bounded(smem_u32(&tail->q_full), (q_issued - 1) & 1);
    }
    if (ACCUM == 1) cp_async_wait_all();
    __syncthreads();
    if (p.splits > 1) {
        // closing cluster barrier: all arrive (does not block); only owners of remotely written shared memory wait
        cluster_arrive_all();
        if (blockIdx.x % p.splits == 0 || ACCUM != 0) cluster_wait_all();
    }
    // The last CTA to get here puts the two counters back to zero for the next launch (every CTA has taken its last
    // number from work_next before it counts itself done).
    if (tid == 0) {
        const int prev = atomicAdd(p.work_next + 1, 1);
        if (prev == (int)gridDim.x - 1) {
            p.work_next[0] = 0;
            p.work_next[1] = 0;
        }
    }
    if (use_tmem && warp == kConsumerWarps) {
        tmem_fence_after_sync();
        tmem_dealloc(*(volatile uint32_t*)&tail->tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
constexpr int kMaxSplits = 8;   // a unit's pieces are one thread-block cluster (portable size limit)

static size_t decode_smem_bytes(int C, int accum, int stages, int splits) {
    const size_t rx = splits > 1 ? (size_t)splits * kPartFloats * sizeof(float) : 0;   // the cluster's receive buffer
    return 1024 + (size_t)stages * kStageBytes + decode_sum_bytes(C, accum ? 1 : 0) + sizeof(DecodeSmemTail) + rx;
}

// TMEM columns a window-step CTA allocates for its logits: 4 per 64-key tile, a power of two >= 32.
int decode_tmem_cols(int C) {
    const int need = 4 * ((C + kTileKeys - 1) / kTileKeys);
    int cols = 32;
    while (cols < need) cols <<= 1;
    return cols;   // C <= 4096 -> at most 256
}

// Key split of `units` units that would leave most of the device idle: about two CTAs per SM, so that all pieces
// run at once (measured on 4..256 units of 18 tiles: 2 and 3 per SM are equal, 4 and more cost a second wave and
// 30-50 % more time), at most kMaxSplits pieces per unit; the tiles are then spread evenly (no piece without a
// tile at full length).
int decode_pick_splits(int units, int C, int sm_count) {
    const int max_tiles = (C + kTileKeys - 1) / kTileKeys;
    if (units <= 0 || units >= 2 * sm_count) return 1;
    int s_max = (2 * sm_count) / units;
    if (s_max > kMaxSplits) s_max = kMaxSplits;
    if (s_max < 1) s_max = 1;
    const int tiles_per_split = (max_tiles + s_max - 1) / s_max;
    return (max_tiles + tiles_per_split - 1) / tiles_per_split;
}

// CTAs of a given shape that one SM holds (shared memory decides; 160 threads x 128 registers allow 3).
// Window steps hold TMEM: resident CTAs x columns must stay within the SM's 512 columns, so that no CTA
// ever waits for its allocation.
static int decode_ctas_per_sm(int C, int accum, int stages, int splits) {
    const size_t cap = 227 * 1024;
    const int cta_cap = accum ? min(3, 512 / decode_tmem_cols(C)) : 3;
    int ctas = (int)(cap / (decode_smem_bytes(C, accum, stages, splits) + 1024));  // 1 KB per-CTA reservation
    return ctas > cta_cap ? cta_cap : ctas;
}

// Resident CTAs per SM matter more than ring depth: with four consumer warps per CTA the per-warp
// dependent chain (ldmatrix -> mma -> shuffles -> exp2 -> mma) needs >= 8-12 warps per SM to hide, so take
// the stage count that allows the most CTAs per SM (up to 3), then the deepest ring that still fits.
static int decode_pick_stages(int C, int accum, int splits) {
    const size_t cap = 227 * 1024;
    int best = 2, best_score = -1;
    for (int st = 2; st <= kMaxStages; ++st) {
        if (decode_smem_bytes(C, accum, st, splits) > cap) break;
        const int score = decode_ctas_per_sm(C, accum, st, splits) * 100 + st;
        if (score > best_score) {
            best_score = score;
            best = st;
        }
    }
    return best;
}

// Work plan of a launch. The grid is persistent (at most the CTAs the device holds at once) and hands out items
// first come, first served. Units are whole items; only a launch so small that whole units would leave most SMs
// idle is split over the keys, so that about two CTAs per SM run: then the grid is one CTA per piece and the
// pieces of a unit form a thread-block cluster. (Splitting the last units of a large launch into pieces of a few
// tiles, to even out the end, was measured and lost: a piece's epilogue costs as much time as three tiles.)
// `max_pieces` > 0 bounds the number of pieces.
void decode_plan(DecodeLaunch* p, int max_pieces) {
    const int sm = p->sm_count > 0 ? p->sm_count : 148;
    const int units = p->n_layers * p->batch * p->h_kv;
    p->tmem_cols = decode_tmem_cols(p->C);
    p->splits = decode_pick_splits(units, p->C, sm);
    if (max_pieces > 0 && (long)units * p->splits > max_pieces) p->splits = 1;   // whole units still fit one wave
    p->stages = decode_pick_stages(p->C, p->accum, p->splits);
    const int resident = decode_ctas_per_sm(p->C, p->accum, p->stages, p->splits) * sm;
    const long items = (long)units * p->splits;
    p->grid = (int)((p->splits > 1 || items < resident) ? items : resident);
    // A few rounds of whole units with a nearly empty last one (say 512 units on 444 CTAs): that round would run at
    // a fraction of the memory bandwidth. A smaller grid with the same number of full rounds is faster (512 units:
    // 256 CTAs x 2 items, 58 -> 52.5 us); with many rounds or a well-filled last one it is not (measured 1.4 to
    // 7 rounds: within +-1.5 %).
    if (p->splits == 1 && items > resident) {
        const long rounds = (items + resident - 1) / resident;
        if (rounds <= 6 && (items % resident) * 4 < resident) p->grid = (int)((items + rounds - 1) / rounds);
    }
}

void decode_plan_resources(const DecodeLaunch& p, int* ctas_per_sm, size_t* smem_bytes) {
    *ctas_per_sm = decode_ctas_per_sm(p.C, p.accum, p.stages, p.splits);
    *smem_bytes = decode_smem_bytes(p.C, p.accum, p.stages, p.splits);
}

cudaError_t decode_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(gkv_decode_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gkv_decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

// `p` must have been through decode_plan().
cudaError_t launch_decode(const DecodeLaunch& p, const DecodeMaps& maps, cudaStream_t s) {
    const size_t smem = decode_smem_bytes(p.C, p.accum, p.stages, p.splits);
    if (p.splits == 1) {
        if (!p.accum) gkv_decode_kernel<0><<<p.grid, kDecodeThreads, smem, s>>>(p, maps);
        else gkv_decode_kernel<1><<<p.grid, kDecodeThreads, smem, s>>>(p, maps);
        return cudaGetLastError();
    }
    // key split: clusters of p.splits CTAs, one per unit (grid = units x splits)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(kDecodeThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (!p.accum) return cudaLaunchKernelEx(&cfg, gkv_decode_kernel<0>, p, maps);
    return cudaLaunchKernelEx(&cfg, gkv_decode_kernel<1>, p, maps);
}

}  // namespace gkv
