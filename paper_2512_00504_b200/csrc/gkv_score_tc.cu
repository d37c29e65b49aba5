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
// One CTA handles one unit (layer, sequence, KV head) and wk <= 64 window rows of all g heads
// (g * wk <= 256 rows; wider windows take several CTAs that add into the same sums).
// Warp 0 streams K tiles by TMA, warp 1 issues tcgen05.mma into two 256-column TMEM accumulators,
// warps 2-17 (four groups of four, one TMEM lane quarter per warp) read the accumulators back with
// tcgen05.ld and do the softmax arithmetic, so copy, tensor work and exponentials overlap; the
// groups split an accumulator's columns, which keeps four warps per scheduler to hide latencies.
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
constexpr int kTcQBytes = kTcMaxRows * kRowBytes;            // 64 KB: d-low half (32 KB) then d-high half
constexpr int kTcAccCols = 256;                              // TMEM columns of one accumulator
constexpr uint32_t kTcTmemCols = 512;
constexpr int kTcChunkKeys = 8192;                           // keys whose window sums are held in shared memory at a time

struct __align__(8) ScoreTcTail {
    uint64_t q_full;
    uint64_t k_full[kTcMaxStages];
    uint64_t k_empty[kTcMaxStages];
    uint64_t d_full[2];
    uint64_t d_empty[2];
    uint64_t drain;
    uint64_t chunk_bar;   // the softmax warps meet here when the window sums move on to the next chunk of keys
    uint32_t tmem_base;
    int abort_flag;
    int issued;
};

__device__ __forceinline__ void tc_abort(ScoreTcTail* tail, int32_t* status, int where) {
    if (atomicExch(&tail->abort_flag, 1) == 0 && atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kTcSoftmaxThreads) : "memory"); }

// WK = window rows handled by one CTA (16, 32 or 64); the CTA's local query row of (head h, window
// row k0 + kk) is h * WK + kk.
template <int WK>
__global__ void __launch_bounds__(kTcThreads, 1)
gkv_score_tc_kernel(const ScoreLaunch p, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_q, int n_cta, int stages) {
    constexpr int HW = WK / kTcGroups;   // window rows one softmax group handles in pass 2
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int R = p.g * WK;                          // query rows of this CTA, a multiple of 16
    const int MT = (R + 127) >> 7;                   // 128-row tiles of pass 1
    constexpr int q_half = kTcQBytes / 2;            // bytes of one d-half of the Q tile (d-low, then d-high)
    uint8_t* q_smem = smem;
    uint8_t* k_smem = smem + 2 * q_half;
    float* s_c = reinterpret_cast<float*>(k_smem + stages * kTcKStageBytes);      // [256] m + log2 l of every local row
    float* s_pm = s_c + kTcMaxRows;                                               // [groups][128] partial row maxima
    float* s_pl = s_pm + kTcGroups * 128;                                         // [groups][128] partial row sums
    // [2][c_pad] window sums of this CTA's rows: two groups add into each plane, so every sum has two addends and
    // the result does not depend on the order in which the groups arrive. Caches hold at most kTcChunkKeys rows and
    // fit whole; a longer key range (a prompt being compressed) passes through in chunks of kTcChunkKeys keys, each
    // written out when pass 2, which walks the tiles from the last to the first, leaves it.
    float* s_sum = s_pl + kTcGroups * 128;
    const int c_pad = min((p.C + 63) & ~63, kTcChunkKeys);
    ScoreTcTail* tail = reinterpret_cast<ScoreTcTail*>(s_sum + 2 * c_pad);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit_local = blockIdx.x / n_cta;
    const int part = blockIdx.x - unit_local * n_cta;
    const int k0 = part * WK;                       // first window row of this CTA
    const int head = unit_local % p.h_kv;
    const int ls = unit_local / p.h_kv;             // layer_local * batch + seq
    const int lseq_global = p.layer0 * p.batch + ls;
    const long unit = (long)lseq_global * p.h_kv + head;
    const int n = p.len[lseq_global];
    const int T = (n + kTcTileKeys - 1) / kTcTileKeys;
    const int row0 = (int)(unit * p.C);

    if (tid == 0) {
        mbar_init(smem_u32(&tail->q_full), 1);
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->k_full[s]), 1);
            mbar_init(smem_u32(&tail->k_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tail->d_full[b]), 1);
            mbar_init(smem_u32(&tail->d_empty[b]), kTcSoftmaxThreads / 32);   // one arrival per softmax warp
        }
        mbar_init(smem_u32(&tail->drain), 1);
        mbar_init(smem_u32(&tail->chunk_bar), kTcSoftmaxThreads / 32);
        tail->abort_flag = 0;
        tail->issued = 0;
        fence_mbar_init();
    }
    if (warp == 1) {   // whole warp: the CTA takes all of the SM's tensor memory (one CTA per SM by shared memory)
        tmem_alloc(smem_u32(&tail->tmem_base), kTcTmemCols);
        tmem_relinquish_alloc_permit();
        tmem_fence_before_sync();
    }
    for (int t = tid; t < 2 * c_pad; t += kTcThreads) s_sum[t] = 0.f;
    // rows R .. 128 * MT - 1 of the Q tile take part in the pass-1 products: make them zeros
    for (int e = tid; e < (MT * 128 - R) * 8 * 2; e += kTcThreads) {
        const int half = e / ((MT * 128 - R) * 8);
        const int r = e - half * (MT * 128 - R) * 8;
        *reinterpret_cast<uint4*>(q_smem + half * q_half + (size_t)R * 128 + r * 16) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&tail->tmem_base;
    const int total = 2 * T;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_q);
            const uint32_t qbar = smem_u32(&tail->q_full);
            mbar_arrive_expect_tx(qbar, (uint32_t)R * kRowBytes);
            const int qrow0 = (ls * p.h_q + head * p.g) * p.w + k0;
            for (int h = 0; h < p.g; ++h) {
                tma_load_2d(smem_u32(q_smem + (size_t)h * WK * 128), &tm_q, 0, qrow0 + h * p.w, qbar);
                tma_load_2d(smem_u32(q_smem + q_half + (size_t)h * WK * 128), &tm_q, 64, qrow0 + h * p.w, qbar);
            }
            for (int i = 0, s = 0, round = 0; i < total; ++i) {
                if (round > 0 && !tc_wait(smem_u32(&tail->k_empty[s]), (round - 1) & 1, &tail->abort_flag)) {
                    tc_abort(tail, p.status, 21);
                    break;
                }
                const int tile = (i < T) ? i : total - 1 - i;   // pass 2 walks back: the tiles read last are still in L2
                const uint32_t bar = smem_u32(&tail->k_full[s]);
                const uint32_t dst = smem_u32(k_smem + (size_t)s * kTcKStageBytes);
                const int y = row0 + tile * kTcTileKeys;
                mbar_arrive_expect_tx(bar, kTcKStageBytes);
                tma_load_2d(dst, &tm_k, 0, y, bar);
                tma_load_2d(dst + kBoxBytes, &tm_k, 0, y + 64, bar);
                tma_load_2d(dst + 2 * kBoxBytes, &tm_k, 64, y, bar);
                tma_load_2d(dst + 3 * kBoxBytes, &tm_k, 64, y + 64, bar);
                *(volatile int*)&tail->issued = i + 1;
                if (++s == stages) { s = 0; ++round; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = tc_wait(smem_u32(&tail->q_full), 0, &tail->abort_flag);
            if (!ok) tc_abort(tail, p.status, 22);
            const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem)), k_lo = umma_desc_lo(smem_u32(k_smem));
            const uint32_t idesc1 = umma_idesc_bf16_m128(kTcTileKeys), idesc2 = umma_idesc_bf16_m128(R);
            for (int i = 0, s = 0, round = 0; ok && i < total; ++i) {
                const int buf = i & 1;
                if (i >= 2 && !tc_wait(smem_u32(&tail->d_empty[buf]), ((i >> 1) - 1) & 1, &tail->abort_flag)) {
                    tc_abort(tail, p.status, 23);
                    break;
                }
                if (!tc_wait(smem_u32(&tail->k_full[s]), round & 1, &tail->abort_flag)) {
                    tc_abort(tail, p.status, 24);
                    break;
                }
                tmem_fence_after_sync();
                const uint32_t ks_lo = k_lo + (uint32_t)s * (kTcKStageBytes >> 4);
                const uint32_t d = tmem_base + (uint32_t)buf * kTcAccCols;
                if (i < T) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_bf16(d, umma_desc(q_lo + umma_kstep(ks, q_half)), umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)),
                                  idesc1, ks > 0);
                    if (MT == 2) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(d + 128, umma_desc(q_lo + ((128 * 128) >> 4) + umma_kstep(ks, q_half)),
                                      umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)), idesc1, ks > 0);
                    }
                } else {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_bf16(d, umma_desc(ks_lo + umma_kstep(ks, kTcKStageBytes / 2)), umma_desc(q_lo + umma_kstep(ks, q_half)),
                                  idesc2, ks > 0);
                }
                umma_commit(smem_u32(&tail->k_empty[s]));
                umma_commit(smem_u32(&tail->d_full[buf]));
                if (++s == stages) { s = 0; ++round; }
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

        // ---- pass 1: online (max, sum) of the row this thread owns over its share of the tile's keys.
        // Two 128-row tiles: two groups per tile, 64 keys each; one tile: all four groups, 32 keys each.
        const int rl = (MT == 2) ? (wg >> 1) * 128 + L : L;
        const bool valid = rl < R;
        const int col0 = (MT == 2) ? (wg & 1) * 64 : wg * 32;
        const int nch = (MT == 2) ? 2 : 1;
        const uint32_t t_p1 = t_lane + (uint32_t)((MT == 2) ? (wg >> 1) * 128 + col0 : col0);
        const int last_vis = n - p.w + k0 + (rl % WK);    // last key the row's token sees
        float m_raw = -INFINITY, l = 0.f;                 // maximum in unscaled logits, sum relative to it
        for (int i = 0; i < T; ++i) {
            const int buf = i & 1;
            ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[buf]), (i >> 1) & 1, &tail->abort_flag));
            if (!ok) { tc_abort(tail, p.status, 25); break; }
            tmem_fence_after_sync();
            const int key_base = i * kTcTileKeys + col0;
            const bool need_mask = i * kTcTileKeys + kTcTileKeys - 1 > n - p.w + k0;
            for (int ch = 0; ch < nch; ++ch) {
                float z[32];
                tmem_ld<32>(t_p1 + (uint32_t)(buf * kTcAccCols + ch * 32), z);
                if (valid) {
                    if (need_mask) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (key_base + ch * 32 + j > last_vis) z[j] = -INFINITY;
                    }
                    float c0 = fmaxf(z[0], z[1]), c1 = fmaxf(z[2], z[3]), c2 = fmaxf(z[4], z[5]), c3 = fmaxf(z[6], z[7]);
#pragma unroll
                    for (int j = 8; j < 32; j += 8) {
                        c0 = fmaxf(c0, fmaxf(z[j], z[j + 1]));
                        c1 = fmaxf(c1, fmaxf(z[j + 2], z[j + 3]));
                        c2 = fmaxf(c2, fmaxf(z[j + 4], z[j + 5]));
                        c3 = fmaxf(c3, fmaxf(z[j + 6], z[j + 7]));
                    }
                    const float mn = fmaxf(m_raw, fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)));
                    if (mn != -INFINITY) {
                        const float neg = -mn * scale;
                        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            s0 += fast_exp2(fmaf(z[j], scale, neg));
                            s1 += fast_exp2(fmaf(z[j + 1], scale, neg));
                            s2 += fast_exp2(fmaf(z[j + 2], scale, neg));
                            s3 += fast_exp2(fmaf(z[j + 3], scale, neg));
                        }
                        l = l * fast_exp2(fmaf(m_raw, scale, neg)) + ((s0 + s1) + (s2 + s3));
                        m_raw = mn;
                    }
                }
            }
            tmem_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[buf]));
        }
        // combine the partials of a row and publish c = m + log2 l (scaled, log2 domain)
        s_pm[wg * 128 + L] = m_raw * scale;
        s_pl[wg * 128 + L] = l;
        softmax_bar_sync();
        if ((MT == 2) ? (wg & 1) == 0 : wg == 0) {
            const int first = (MT == 2) ? wg : 0, count = (MT == 2) ? 2 : kTcGroups;   // groups that shared this row
            float mm = -INFINITY, ll = 0.f;
            for (int q = first; q < first + count; ++q) mm = fmaxf(mm, s_pm[q * 128 + L]);
            for (int q = first; q < first + count; ++q) {
                const float mq = s_pm[q * 128 + L];
                ll += (mq == -INFINITY) ? 0.f : s_pl[q * 128 + L] * fast_exp2(mq - mm);
            }
            s_c[rl] = mm + log2f(ll);
        }
        softmax_bar_sync();

        // ---- pass 2: this thread owns key `tile * 128 + L`; group wg covers window rows k0 + wg*HW .. + HW - 1
        float* out = p.sacc + (size_t)unit * p.C;
        // window sums of keys [lo, lo + c_pad) leave shared memory (which is zeroed for the next chunk)
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
        uint32_t chunk_phase = 0;
        int chunk_lo = T > 0 ? ((T - 1) * kTcTileKeys / c_pad) * c_pad : 0;
        for (int i = T; i < total; ++i) {
            const int buf = i & 1;
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
            ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[buf]), (i >> 1) & 1, &tail->abort_flag));
            if (!ok) { tc_abort(tail, p.status, 26); break; }
            tmem_fence_after_sync();
            float v[HW];
#pragma unroll
            for (int j = 0; j < HW; ++j) v[j] = -INFINITY;
            for (int h = 0; h < p.g; ++h) {
                float z[HW];
                tmem_ld<HW>(t_lane + (uint32_t)(buf * kTcAccCols + h * WK + wg * HW), z);
                const float4* c4 = reinterpret_cast<const float4*>(s_c + h * WK + wg * HW);
#pragma unroll
                for (int j = 0; j < HW; j += 4) {
                    const float4 c = c4[j >> 2];
                    v[j] = fmaxf(v[j], fmaf(z[j], scale, -c.x));
                    v[j + 1] = fmaxf(v[j + 1], fmaf(z[j + 1], scale, -c.y));
                    v[j + 2] = fmaxf(v[j + 2], fmaf(z[j + 2], scale, -c.z));
                    v[j + 3] = fmaxf(v[j + 3], fmaf(z[j + 3], scale, -c.w));
                }
            }
            tmem_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[buf]));
            const int key = (total - 1 - i) * kTcTileKeys + L;
            if (key < n) {
                const int first_k = key - (n - p.w) - k0 - wg * HW;   // rows j < first_k decoded before this key existed
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int j = 0; j < HW; j += 2) {
                    s0 += (j >= first_k) ? fast_exp2(v[j]) : 0.f;
                    s1 += (j + 1 >= first_k) ? fast_exp2(v[j + 1]) : 0.f;
                }
                atomicAdd(&s_sum[(wg >> 1) * c_pad + key - chunk_lo], s0 + s1);
            }
        }
        softmax_bar_sync();
        if (ok && !*(volatile int*)&tail->abort_flag) {
            flush_chunk(chunk_lo);   // the chunk of the first tile, walked last
            // rows past the chunk that holds the last key were never in shared memory
            if (n_cta == 1)
                for (int t = (T > 0 ? ((T - 1) * kTcTileKeys / c_pad + 1) * c_pad : 0) + stid; t < p.C; t += kTcSoftmaxThreads) out[t] = 0.f;
        }
    }

    __syncthreads();
    if (*(volatile int*)&tail->abort_flag && tid == 0) {
        // give copies still in flight a bounded time to land before the CTA exits
        mbar_wait_bounded(smem_u32(&tail->q_full), 0);
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

static size_t score_tc_smem_bytes(int C, int rows, int stages) {
    (void)rows;
    return 1024 + (size_t)kTcQBytes + (size_t)stages * kTcKStageBytes +
           sizeof(float) * (kTcMaxRows + 2 * kTcGroups * 128 + 2 * min((C + 63) & ~63, kTcChunkKeys)) + sizeof(ScoreTcTail);
}

// Window rows per CTA for this shape, or 0 when the shape is left to the mma.sync kernel.
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
    // the deepest K ring that fits: bytes in flight per SM are what hides the copy latency (one CTA per SM)
    int stages = 2;
    while (stages < kTcMaxStages && score_tc_smem_bytes(p.C, p.g * wk, stages + 1) <= 227 * 1024) ++stages;
    const size_t smem = score_tc_smem_bytes(p.C, p.g * wk, stages);
    if (n_cta > 1) {
        const size_t off = (size_t)p.layer0 * p.batch * p.h_kv * p.C;
        cudaError_t e = cudaMemsetAsync(p.sacc + off, 0, sizeof(float) * (size_t)units * p.C, s);
        if (e != cudaSuccess) return e;
    }
    if (wk == 16) gkv_score_tc_kernel<16><<<units * n_cta, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages);
    else if (wk == 32) gkv_score_tc_kernel<32><<<units * n_cta, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages);
    else gkv_score_tc_kernel<64><<<units * n_cta, kTcThreads, smem, s>>>(p, tm_k, tm_q, n_cta, stages);
    return cudaGetLastError();
}

}  // namespace gkv
