// GQA decode attention over the compressed cache, with the append of the current token and the
// optional accumulation of the window score (the every-step half of the G-KV path).
//
// One CTA = one (unit, split), unit = (layer, sequence, KV head). A producer warp streams 64-key
// K and V tiles (TMA, 128-byte swizzle) through a ring of stages; four consumer warps each own 16
// keys of every tile and keep their own online-softmax state, so the main loop has no CTA-wide
// barrier. Both products run on mma.sync m16n8k16 with the KEYS on the M side and the g <= 8 query
// heads of the group on the N side (S^T = K Q^T, O^T = V^T P^T): no padded rows, each K/V byte
// is read from shared memory exactly once, and the P^T operand comes from the S^T accumulator by
// an 8x8 register transpose (movmatrix).
#include "gkv_common.cuh"
#include "gkv_internal.h"

namespace gkv {

constexpr int kConsumerWarps = 4;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 6;
constexpr int kPartFloats = 16 + kHeadDim * 8;  // M[8], L[8], acc[128][8]
constexpr int kQRowBytes = 272;                 // 256 bytes of a query row + 16 of padding

struct __align__(16) DecodeSmemTail {
    uint64_t full_bar[kMaxStages];
    uint64_t empty_bar[kMaxStages];
    float m[kConsumerWarps][8];
    float l[kConsumerWarps][8];
    float fin_m[8];
    float fin_l[8];
    float wgt[kConsumerWarps][8];
    alignas(16) uint8_t q_rows[8 * 272];   // the group's query rows, 272 bytes apart
    int abort_flag;
    int issued;
    int is_last;
    uint32_t tmem_base;
};

__device__ __forceinline__ void latch_timeout(int32_t* status, int where) {
    if (atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}

// Shared memory for the unit's window sums on window steps without key split.
__host__ __device__ constexpr size_t decode_sum_bytes(int C, int accum_mode) {
    return accum_mode == 1 ? (size_t)((C + 63) & ~63) * sizeof(float) : 0;
}

// ACCUM = 0: plain step. ACCUM = 1: window step, one CTA per unit, logits parked in TMEM.
// ACCUM = 2: window step with the keys split over several CTAs, logits in the workspace.
template <int ACCUM>
__global__ void __launch_bounds__(kDecodeThreads)
gkv_decode_kernel(const DecodeLaunch p, const __grid_constant__ DecodeMaps maps) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the swizzled TMA boxes
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint8_t* stage_base = smem;
    float* s_sum = reinterpret_cast<float*>(smem + (size_t)stages * kStageBytes);   // [C] window sums, ACCUM == 1 only
    DecodeSmemTail* tail = reinterpret_cast<DecodeSmemTail*>(smem + (size_t)stages * kStageBytes + decode_sum_bytes(p.C, ACCUM));
    // Window steps without key split keep the scaled logits [key][head] on chip until the row's
    // normaliser is final. They live in tensor memory, not shared memory: a consumer thread parks
    // the 4 values it owns of every tile in 4 columns of its own TMEM lane and reads them back
    // itself in the epilogue, so shared memory (and with it the number of resident CTAs) is the
    // same as on plain steps.
    constexpr bool use_tmem = ACCUM == 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit_local = blockIdx.x / p.splits;
    const int split = blockIdx.x - unit_local * p.splits;
    const int head = unit_local % p.h_kv;
    const int ls = unit_local / p.h_kv;              // layer_local * batch + seq
    const int layer_local = ls / p.batch;
    const int seq = ls - layer_local * p.batch;
    const int layer = p.layer0 + layer_local;
    const int lseq_global = layer * p.batch + seq;
    const long unit = (long)lseq_global * p.h_kv + head;

    const int len_old = p.len[lseq_global];
    const int n = len_old + 1;                        // keys attended (current token included)
    const int tiles_total = (n + kTileKeys - 1) / kTileKeys;
    const int tps = (tiles_total + p.splits - 1) / p.splits;
    const int t_begin = min(split * tps, tiles_total);
    const int t_end = min(t_begin + tps, tiles_total);
    const int row0 = (int)(unit * p.C);               // first cache row of this unit in the 2-D view

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->full_bar[s]), 1);
            mbar_init(smem_u32(&tail->empty_bar[s]), kConsumerWarps);
        }
        tail->abort_flag = 0;
        tail->issued = t_begin;
        tail->is_last = 0;
        fence_mbar_init();
    }
    if (use_tmem && warp == kConsumerWarps) {   // whole warp; p.tmem_cols x resident CTAs <= 512, so this never waits
        tmem_alloc(smem_u32(&tail->tmem_base), (uint32_t)p.tmem_cols);
        tmem_relinquish_alloc_permit();
        tmem_fence_before_sync();
    }
    __syncthreads();
    if (use_tmem) tmem_fence_after_sync();
    const uint32_t tmem_warp = use_tmem ? (*(volatile uint32_t*)&tail->tmem_base + ((uint32_t)(warp & 3) << 21)) : 0u;

    // Window steps: the unit's current window sums start their way into shared memory now and are
    // needed only in the epilogue; the updated sums go back with plain coalesced stores. (One
    // atomic per key is measurably slower: the L2 atomic units saturate at ~4 M reductions a launch.)
    if (ACCUM == 1 && warp < kConsumerWarps) {
        const float* gsum = p.sacc + (size_t)unit * p.C;
        for (int t = tid; t < n; t += kConsumerWarps * 32) cp_async_4(smem_u32(s_sum + t), gsum + t);
        cp_async_commit();
    }

    // per-thread softmax / output state of a consumer warp (heads h0 = 2*(lane&3), h0+1)
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            prefetch_tensormap(&maps.k64);
            prefetch_tensormap(&maps.v64);
            if (n & (kTileKeys - 1)) {
                prefetch_tensormap(&maps.k16);
                prefetch_tensormap(&maps.v16);
            }
            for (int it = t_begin; it < t_end; ++it) {
                const int j = it - t_begin;
                const int s = j % stages;
                if (j >= stages) {
                    if (!mbar_wait_bounded(smem_u32(&tail->empty_bar[s]), ((j / stages) - 1) & 1)) {
                        latch_timeout(p.status, 1);
                        tail->abort_flag = 1;
                        break;
                    }
                }
                if (*(volatile int*)&tail->abort_flag) break;
                const uint32_t bar = smem_u32(&tail->full_bar[s]);
                const uint32_t dst = smem_u32(stage_base + (size_t)s * kStageBytes);
                const int y = row0 + it * kTileKeys;
                const int rows_left = n - it * kTileKeys;       // keys of this tile that exist
                if (rows_left > kTileKeys - 16) {
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
                *(volatile int*)&tail->issued = it + 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int r_in = lane & 7, mat = lane >> 3;
        const int hq = lane >> 2;                     // head whose Q row this lane holds (B operand)
        // Q^T fragments: B[k = d][n = head], two packed bf16 pairs per 16-wide k step
        // The group's g query rows come in once per CTA with 16-byte loads (warp w fetches heads w and w + 4, one
        // row per half warp) and are re-read from shared memory in fragment order: one bus or L2 transaction per
        // 16 bytes instead of four copies of it in 4-byte pieces. Rows are 272 bytes apart: conflict-free reads.
        uint32_t qf[8][2];
        {
            const int hl = warp + (lane >> 4) * kConsumerWarps;          // head this half warp fetches
            if (hl < p.g) {
                const __nv_bfloat16* qrow =
                    p.q + ((size_t)(layer_local * p.batch + seq) * p.h_q + (size_t)head * p.g + hl) * kHeadDim;
                *reinterpret_cast<uint4*>(tail->q_rows + hl * kQRowBytes + (lane & 15) * 16) =
                    *reinterpret_cast<const uint4*>(qrow + (lane & 15) * 8);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");   // the four consumer warps only
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                if (hq < p.g) {
                    const uint8_t* row = tail->q_rows + hq * kQRowBytes + ks * 32 + (lane & 3) * 4;
                    qf[ks][0] = *reinterpret_cast<const uint32_t*>(row);
                    qf[ks][1] = *reinterpret_cast<const uint32_t*>(row + 16);
                } else {
                    qf[ks][0] = qf[ks][1] = 0u;
                }
            }
        }
        // The current token's row lands in the last tile; the warp that will append it fetches its 16 bytes per lane
        // now (lanes 0-15 of k_new, 16-31 of v_new), so that the load's latency -- a bus round trip when the inputs
        // are mapped host memory -- is long over when the row is needed.
        uint4 new_row = make_uint4(0u, 0u, 0u, 0u);
        if (warp == ((len_old & (kTileKeys - 1)) >> 4) && (len_old / kTileKeys) >= t_begin && (len_old / kTileKeys) < t_end) {
            const size_t src = ((size_t)(layer_local * p.batch + seq) * p.h_kv + head) * kHeadDim + (lane & 15) * 8;
            new_row = *reinterpret_cast<const uint4*>((lane < 16 ? p.k_new : p.v_new) + src);
        }
        const int krow = warp * 16 + (mat & 1) * 8 + r_in;   // K ldmatrix: row this lane addresses
        const int kch = mat >> 1;                             //   and which 16-byte chunk of the k step
        const int vrow = warp * 16 + (mat >> 1) * 8 + r_in;   // V ldmatrix (transposed)
        const int vch = mat & 1;

        for (int it = t_begin; it < t_end; ++it) {
            const int j = it - t_begin;
            const int s = j % stages;
            if (!mbar_wait_bounded(smem_u32(&tail->full_bar[s]), (j / stages) & 1)) {
                latch_timeout(p.status, 2);
                tail->abort_flag = 1;
                break;
            }
            if (*(volatile int*)&tail->abort_flag) break;
            uint8_t* kt = stage_base + (size_t)s * kStageBytes;
            uint8_t* vt = kt + kTileBytes;
            const int key0 = it * kTileKeys + warp * 16;
            if (key0 < n) {
                // append: the warp that owns row len_old overwrites it (in the tile and in the cache)
                if (len_old >= key0 && len_old < key0 + 16) {
                    const int lr = len_old - it * kTileKeys;          // row inside the tile
                    const int c = lane & 15;
                    const size_t dstg = ((size_t)unit * p.C + len_old) * kHeadDim + c * 8;
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
                if (ACCUM != 0) {
                    const int h0 = (lane & 3) * 2;
                    if (ACCUM == 1) {
                        tmem_st4(tmem_warp + 4u * (uint32_t)it, s0, s1, s2, s3);
                    } else {
                        float* g_log = p.logits + (size_t)unit_local * p.C * 8;
                        if (key_a < n) *reinterpret_cast<float2*>(g_log + key_a * 8 + h0) = make_float2(s0, s1);
                        if (key_b < n) *reinterpret_cast<float2*>(g_log + key_b * 8 + h0) = make_float2(s2, s3);
                    }
                }
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
        }
    }

    if (use_tmem && warp < kConsumerWarps) {
        tmem_wait_st();
        tmem_fence_before_sync();
    }
    __syncthreads();  // [A] every consumer is done with the stage buffers
    if (*(volatile int*)&tail->abort_flag) {
        // Give copies that are still in flight a bounded time to land before the CTA exits.
        if (tid == 0) {
            const int issued = *(volatile int*)&tail->issued;
            for (int it = max(t_begin, issued - stages); it < issued; ++it) {
                const int j = it - t_begin;
                mbar_wait_bounded(smem_u32(&tail->full_bar[j % stages]), (j / stages) & 1);
            }
        }
        if (ACCUM == 1) cp_async_wait_all();
        if (use_tmem && warp == kConsumerWarps) {
            __syncwarp();
            tmem_fence_after_sync();
            tmem_dealloc(*(volatile uint32_t*)&tail->tmem_base, (uint32_t)p.tmem_cols);
        }
        return;
    }

    float* s_acc = reinterpret_cast<float*>(stage_base);  // [warp][128 dims][8 heads], aliases stage 0
    if (warp < kConsumerWarps) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, o);
            l1 += __shfl_xor_sync(0xffffffffu, l1, o);
        }
        const int h0 = (lane & 3) * 2;
        if ((lane >> 2) == 0) {
            tail->m[warp][h0] = m0; tail->m[warp][h0 + 1] = m1;
            tail->l[warp][h0] = l0; tail->l[warp][h0 + 1] = l1;
        }
        float* dst = s_acc + warp * (kHeadDim * 8);
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            const int dim = dt * 16 + (lane >> 2);
            *reinterpret_cast<float2*>(dst + dim * 8 + h0) = make_float2(acc[dt][0], acc[dt][1]);
            *reinterpret_cast<float2*>(dst + (dim + 8) * 8 + h0) = make_float2(acc[dt][2], acc[dt][3]);
        }
    }
    __syncthreads();  // [B]

    // CTA-level state: per head the combined (max, sum) of the four warps and each warp's weight ...
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
    }
    __syncthreads();
    // ... and per thread (one of the 128 dims) the merged accumulator of the 8 heads
    float o[8];
    if (tid < kHeadDim) {
#pragma unroll
        for (int h = 0; h < 8; ++h) {
            float oo = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) oo += tail->wgt[w][h] * s_acc[w * (kHeadDim * 8) + tid * 8 + h];
            o[h] = oo;
        }
    }

    const int n_keys_all = n;
    bool do_final = true;          // this CTA writes the output (always true without split)
    if (p.splits > 1) {
        float* mine = p.part + ((size_t)unit_local * p.splits + split) * kPartFloats;
        if (tid < kHeadDim) {
            if (tid < 8) { mine[tid] = tail->fin_m[tid]; mine[8 + tid] = tail->fin_l[tid]; }
            float4* d4 = reinterpret_cast<float4*>(mine + 16 + tid * 8);
            d4[0] = make_float4(o[0], o[1], o[2], o[3]);
            d4[1] = make_float4(o[4], o[5], o[6], o[7]);
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int prev = atomicAdd(&p.unit_done[unit], 1);
            tail->is_last = (prev == p.splits - 1);
            if (prev == p.splits - 1) p.unit_done[unit] = 0;   // self-reset for the next launch
        }
        __syncthreads();
        do_final = tail->is_last != 0;
        if (do_final) {
            // The last CTA of the unit merges the partials. All loads of a phase are independent, so the merge
            // costs a few L2 round trips, not one per split: (1) every split's (max, sum) into shared memory,
            // (2) per head the global max, the splits' weights and the global sum, (3) per dim the weighted sum
            // of the splits' accumulators.
            __threadfence();
            const float* base = p.part + (size_t)unit_local * p.splits * kPartFloats;
            float* s_stat = s_acc;                 // [splits][16]: M[8], L[8]   (the accumulators are in registers now)
            float* s_w = s_acc + 32 * 16;          // [splits][8] weights
            for (int idx = tid; idx < p.splits * 16; idx += kDecodeThreads)
                s_stat[idx] = __ldcg(base + (size_t)(idx >> 4) * kPartFloats + (idx & 15));
            __syncthreads();
            if (tid < 8) {
                const int h = tid;
                float mm = -INFINITY;
                for (int sp = 0; sp < p.splits; ++sp) mm = fmaxf(mm, s_stat[sp * 16 + h]);
                float ll = 0.f;
                for (int sp = 0; sp < p.splits; ++sp) {
                    const float wm = s_stat[sp * 16 + h];
                    const float wgt = (wm == -INFINITY) ? 0.f : fast_exp2(wm - mm);
                    s_w[sp * 8 + h] = wgt;
                    ll += wgt * s_stat[sp * 16 + 8 + h];
                }
                tail->fin_m[h] = mm;
                tail->fin_l[h] = ll;
            }
            __syncthreads();
            if (tid < kHeadDim) {
#pragma unroll
                for (int h = 0; h < 8; ++h) o[h] = 0.f;
#pragma unroll 4
                for (int sp = 0; sp < p.splits; ++sp) {
                    const float4* a4 = reinterpret_cast<const float4*>(base + (size_t)sp * kPartFloats + 16 + tid * 8);
                    const float4 a = __ldcg(a4), b = __ldcg(a4 + 1);
                    const float4 wa = *reinterpret_cast<const float4*>(s_w + sp * 8);
                    const float4 wb = *reinterpret_cast<const float4*>(s_w + sp * 8 + 4);
                    o[0] = fmaf(wa.x, a.x, o[0]); o[1] = fmaf(wa.y, a.y, o[1]); o[2] = fmaf(wa.z, a.z, o[2]); o[3] = fmaf(wa.w, a.w, o[3]);
                    o[4] = fmaf(wb.x, b.x, o[4]); o[5] = fmaf(wb.y, b.y, o[5]); o[6] = fmaf(wb.z, b.z, o[6]); o[7] = fmaf(wb.w, b.w, o[7]);
                }
            }
        }
    }

    if (do_final) {
        // out = o / L as bf16, transposed through shared memory (the query rows' slot is free by now) so that it
        // leaves in 16-byte pieces, 256 contiguous bytes per head: one row per half warp.
        if (tid < kHeadDim) {
#pragma unroll
            for (int h = 0; h < 8; ++h)
                if (h < p.g)
                    *reinterpret_cast<__nv_bfloat16*>(tail->q_rows + h * kQRowBytes + tid * 2) = __float2bfloat16_rn(o[h] / tail->fin_l[h]);
        }
        __syncthreads();
        if (tid < p.g * 16) {
            const int h = tid >> 4, c = tid & 15;
            __nv_bfloat16* orow = p.out + ((size_t)(layer_local * p.batch + seq) * p.h_q + (size_t)head * p.g + h) * kHeadDim;
            *reinterpret_cast<uint4*>(orow + c * 8) = *reinterpret_cast<const uint4*>(tail->q_rows + h * kQRowBytes + c * 16);
        }
        if (ACCUM != 0) {
            if (ACCUM == 1) cp_async_wait_all();
            __syncthreads();
            // Sacc[t] += max over the group of the final weights = exp2(max_h (z_h[t] - M_h - log2 L_h)).
            float* sacc = p.sacc + (size_t)unit * p.C;
            if (ACCUM == 1) {
                if (warp < kConsumerWarps) {
                    const int h0 = (lane & 3) * 2;
                    const float c0 = (h0 < p.g) ? tail->fin_m[h0] + log2f(tail->fin_l[h0]) : INFINITY;
                    const float c1 = (h0 + 1 < p.g) ? tail->fin_m[h0 + 1] + log2f(tail->fin_l[h0 + 1]) : INFINITY;
                    // four tiles per TMEM access; columns past the last tile are allocated but never written
                    // and are ignored (key >= n); each key of the unit is owned by exactly one thread
                    for (int it4 = 0; it4 < tiles_total; it4 += 4) {
                        float z[16];
                        tmem_ld16(tmem_warp + 4u * (uint32_t)it4, z);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            float va = fmaxf(z[4 * u] - c0, z[4 * u + 1] - c1), vb = fmaxf(z[4 * u + 2] - c0, z[4 * u + 3] - c1);
                            va = fmaxf(va, __shfl_xor_sync(0xffffffffu, va, 1));
                            vb = fmaxf(vb, __shfl_xor_sync(0xffffffffu, vb, 1));
                            va = fmaxf(va, __shfl_xor_sync(0xffffffffu, va, 2));
                            vb = fmaxf(vb, __shfl_xor_sync(0xffffffffu, vb, 2));
                            const int key = (it4 + u) * kTileKeys + warp * 16 + (lane >> 2) + ((lane & 1) ? 8 : 0);
                            if ((lane & 2) == 0 && key < n_keys_all) s_sum[key] += fast_exp2((lane & 1) ? vb : va);
                        }
                    }
                    tmem_fence_before_sync();
                }
            } else {
                float c[8];
#pragma unroll
                for (int h = 0; h < 8; ++h) c[h] = (h < p.g) ? tail->fin_m[h] + log2f(tail->fin_l[h]) : INFINITY;
                const float* g_log = p.logits + (size_t)unit_local * p.C * 8;
#pragma unroll 4   // independent loads: a few L2 round trips for the unit's logits instead of one per iteration
                for (int t = tid; t < n_keys_all; t += kDecodeThreads) {
                    const float4 x0 = __ldcg(reinterpret_cast<const float4*>(g_log + (size_t)t * 8));
                    const float4 x1 = __ldcg(reinterpret_cast<const float4*>(g_log + (size_t)t * 8 + 4));
                    float v = x0.x - c[0];
                    v = fmaxf(v, x0.y - c[1]); v = fmaxf(v, x0.z - c[2]); v = fmaxf(v, x0.w - c[3]);
                    v = fmaxf(v, x1.x - c[4]); v = fmaxf(v, x1.y - c[5]); v = fmaxf(v, x1.z - c[6]);
                    v = fmaxf(v, x1.w - c[7]);
                    atomicAdd(sacc + t, fast_exp2(v));
                }
            }
        }
    }

    // The last CTA of a (layer, sequence) publishes the new length.
    __syncthreads();
    if (use_tmem && warp == kConsumerWarps) {
        tmem_fence_after_sync();
        tmem_dealloc(*(volatile uint32_t*)&tail->tmem_base, (uint32_t)p.tmem_cols);
    }
    if (ACCUM == 1) {
        float* gsum = p.sacc + (size_t)unit * p.C;
        for (int t = tid; t < n; t += kDecodeThreads) gsum[t] = s_sum[t];
    }
    if (tid == 0) {
        const int per_seq = p.h_kv * p.splits;
        const int prev = atomicAdd(&p.seq_done[lseq_global], 1);
        if (prev == per_seq - 1) {
            p.seq_done[lseq_global] = 0;
            p.len[lseq_global] = n;
        }
    }
}

// ---------------------------------------------------------------------------------------------
static size_t decode_smem_bytes(int C, int accum, int splits, int stages) {
    return 1024 + (size_t)stages * kStageBytes + decode_sum_bytes(C, (accum && splits == 1) ? 1 : 0) + sizeof(DecodeSmemTail);
}

// TMEM columns a window-step CTA allocates for its logits: 4 per 64-key tile, a power of two >= 32.
int decode_tmem_cols(int C) {
    const int need = 4 * ((C + kTileKeys - 1) / kTileKeys);
    int cols = 32;
    while (cols < need) cols <<= 1;
    return cols;   // C <= 4096 -> at most 256
}

// Key split of a launch with few units: about two CTAs per SM, so that all of them run in one wave (measured
// on 4..256 units of 18 tiles: 2 and 3 per SM are equal, 4 and more cost a second wave and 30-50 % more
// time); the tiles are then spread evenly (no CTA without a tile).
int decode_pick_splits(int units_in_launch, int C, int sm_count) {
    const int max_tiles = (C + kTileKeys - 1) / kTileKeys;
    if (units_in_launch >= 2 * sm_count) return 1;
    int s_max = (2 * sm_count) / units_in_launch;
    if (s_max > 32) s_max = 32;
    if (s_max < 1) s_max = 1;
    const int tiles_per_split = (max_tiles + s_max - 1) / s_max;
    return (max_tiles + tiles_per_split - 1) / tiles_per_split;
}

// Resident CTAs per SM matter more than ring depth: with four consumer warps per CTA the per-warp
// dependent chain (ldmatrix -> mma -> shuffles -> exp2 -> mma) needs >= 8-12 warps per SM to hide, so take
// the stage count that allows the most CTAs per SM (up to 3), then the deepest ring that still fits.
int decode_pick_stages(int C, int accum, int splits, size_t* smem_bytes) {
    const size_t cap = 227 * 1024;
    int best = 2, best_score = -1;
    // Window steps hold TMEM: resident CTAs x columns must stay within the SM's 512 columns, so that no
    // CTA ever waits for its allocation.
    const int cta_cap = (accum && splits == 1) ? min(3, 512 / decode_tmem_cols(C)) : 3;
    for (int st = 2; st <= kMaxStages; ++st) {
        const size_t b = decode_smem_bytes(C, accum, splits, st);
        if (b > cap) break;
        int ctas = (int)(cap / (b + 1024));  // 1 KB per-CTA reservation
        if (ctas > cta_cap) ctas = cta_cap;
        const int score = ctas * 100 + st;
        if (score > best_score) {
            best_score = score;
            best = st;
        }
    }
    if (smem_bytes) *smem_bytes = decode_smem_bytes(C, accum, splits, best);
    return best;
}

cudaError_t decode_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(gkv_decode_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gkv_decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gkv_decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_decode(const DecodeLaunch& p_in, const DecodeMaps& maps, cudaStream_t s) {
    DecodeLaunch p = p_in;
    p.tmem_cols = decode_tmem_cols(p.C);
    const size_t smem = decode_smem_bytes(p.C, p.accum, p.splits, p.stages);
    const int grid = p.n_layers * p.batch * p.h_kv * p.splits;
    if (!p.accum) gkv_decode_kernel<0><<<grid, kDecodeThreads, smem, s>>>(p, maps);
    else if (p.splits == 1) gkv_decode_kernel<1><<<grid, kDecodeThreads, smem, s>>>(p, maps);
    else gkv_decode_kernel<2><<<grid, kDecodeThreads, smem, s>>>(p, maps);
    return cudaGetLastError();
}

}  // namespace gkv
