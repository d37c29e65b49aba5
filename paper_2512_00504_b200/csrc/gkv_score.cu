// Local score recomputed from the observation window (Section 3: Eq. 1 window attention, max over
// the query heads of a KV head, Eq. 2 mean over the window). Writes w * S into the window-sum
// buffer, the same quantity the decode kernel accumulates step by step.
//
// The contraction Q_win K^T runs on mma.sync m16n8k16 with the (window row, head) pairs on the M
// side and keys on the N side. Each consumer warp owns up to two 16-row m-tiles with their Q
// fragments resident in registers, and streams every K tile of the unit from shared memory (TMA
// ring shared by the CTA). Softmax needs each row's final normaliser before the max over heads, so
// the keys are streamed twice: pass 1 keeps an online (max, sum) per row, pass 2 recomputes the
// logits, forms log2 p = z - (m + log2 l), takes the max over the heads of the group by lane
// shuffles, exponentiates once, and adds over the window rows. Row ownership makes both passes free
// of CTA-wide barriers. Window token k sees the keys t <= n - w + k.
#include "gkv_common.cuh"
#include "gkv_internal.h"

namespace gkv {

constexpr int kScoreWarps = 8;                       // consumer warps
constexpr int kScoreThreads = (kScoreWarps + 1) * 32;
constexpr int kScoreStages = 4;                      // K-only stages of 16 KB
constexpr int kScoreMT = 2;                          // m-tiles per warp
constexpr int kScoreRowsPerCta = kScoreWarps * kScoreMT * 16;

struct __align__(8) ScoreSmemTail {
    uint64_t full_bar[kScoreStages];
    uint64_t empty_bar[kScoreStages];
    int abort_flag;
    int issued;
};

// GP = heads per window row after padding (4 or 8): an m-tile holds 16 / GP window rows.
template <int GP>
__global__ void __launch_bounds__(kScoreThreads, 1)
gkv_score_kernel(const ScoreLaunch p, const __grid_constant__ CUtensorMap tm_k, int wsplit) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* s_sum = reinterpret_cast<float*>(smem + kScoreStages * kTileBytes);       // [C] window sums
    ScoreSmemTail* tail = reinterpret_cast<ScoreSmemTail*>(smem + kScoreStages * kTileBytes + sizeof(float) * ((p.C + 63) & ~63));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit_local = blockIdx.x / wsplit;
    const int part = blockIdx.x - unit_local * wsplit;     // which slice of the window rows
    const int head = unit_local % p.h_kv;
    const int ls = unit_local / p.h_kv;
    const int lseq_global = p.layer0 * p.batch + ls;
    const long unit = (long)lseq_global * p.h_kv + head;
    const int n = p.len[lseq_global];
    const int tiles = (n + kTileKeys - 1) / kTileKeys;
    const int row0 = (int)(unit * p.C);

    constexpr int WR_PER_TILE = 16 / GP;                    // window rows per m-tile
    const int wr_per_cta = kScoreRowsPerCta / GP;           // window rows one CTA covers
    const int wr_base_cta = part * wr_per_cta;

    if (tid == 0) {
        for (int s = 0; s < kScoreStages; ++s) {
            mbar_init(smem_u32(&tail->full_bar[s]), 1);
            mbar_init(smem_u32(&tail->empty_bar[s]), kScoreWarps);
        }
        tail->abort_flag = 0;
        tail->issued = 0;
        fence_mbar_init();
    }
    for (int t = tid; t < p.C; t += kScoreThreads) s_sum[t] = 0.f;
    __syncthreads();

    const int total_iters = 2 * tiles;
    if (warp == kScoreWarps) {
        if (lane == 0) {
            prefetch_tensormap(&tm_k);
            for (int j = 0; j < total_iters; ++j) {
                const int s = j % kScoreStages;
                if (j >= kScoreStages) {
                    if (!mbar_wait_bounded(smem_u32(&tail->empty_bar[s]), ((j / kScoreStages) - 1) & 1)) {
                        if (atomicCAS(p.status, 0, kStatusTimeout) == 0) { p.status[1] = 11; p.status[2] = blockIdx.x; }
                        tail->abort_flag = 1;
                        break;
                    }
                }
                if (*(volatile int*)&tail->abort_flag) break;
                const int it = (j < tiles) ? j : j - tiles;
                const uint32_t bar = smem_u32(&tail->full_bar[s]);
                const uint32_t dst = smem_u32(smem + (size_t)s * kTileBytes);
                mbar_arrive_expect_tx(bar, kTileBytes);
                tma_load_2d(dst, &tm_k, 0, row0 + it * kTileKeys, bar);
                tma_load_2d(dst + kBoxBytes, &tm_k, 64, row0 + it * kTileKeys, bar);
                *(volatile int*)&tail->issued = j + 1;
            }
        }
    } else {
        // ---- rows of this warp: m-tile mt covers window rows wr0 + mt*WR_PER_TILE ...
        const int wr0 = wr_base_cta + warp * kScoreMT * WR_PER_TILE;
        const int r_lo = lane >> 2;                           // fragment row (and r_lo + 8)
        // A fragments of Q: a0 = (row r_lo, k 2c..), a1 = (row r_lo+8, ..), a2 = (row r_lo, k+8), a3 = (row r_lo+8, k+8)
        uint32_t qa[kScoreMT][8][4];
        int wr_of[kScoreMT][2];                               // window row of fragment rows r_lo, r_lo+8
        bool valid[kScoreMT][2];
        bool any_rows = false;
#pragma unroll
        for (int mt = 0; mt < kScoreMT; ++mt) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int r = r_lo + half * 8;
                const int wr = wr0 + mt * WR_PER_TILE + r / GP;
                const int h = r % GP;
                wr_of[mt][half] = wr;
                valid[mt][half] = (wr < p.w) && (h < p.g);
                any_rows |= (wr0 + mt * WR_PER_TILE) < p.w;
                const __nv_bfloat16* qrow = p.q_win +
                    (((size_t)ls * p.h_q + (size_t)head * p.g + h) * p.w + wr) * kHeadDim + (lane & 3) * 2;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    uint32_t x0 = 0u, x1 = 0u;
                    if (valid[mt][half]) {
                        x0 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16);
                        x1 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8);
                    }
                    qa[mt][ks][half] = x0;
                    qa[mt][ks][2 + half] = x1;
                }
            }
        }
        // online row statistics (per thread: its two columns of every n-tile), log2 domain
        float rm[kScoreMT][2], rl[kScoreMT][2], rc[kScoreMT][2];
#pragma unroll
        for (int mt = 0; mt < kScoreMT; ++mt) {
            rm[mt][0] = rm[mt][1] = -INFINITY;
            rl[mt][0] = rl[mt][1] = 0.f;
            rc[mt][0] = rc[mt][1] = INFINITY;
        }
        // K ldmatrix as the B operand ([n = key][k = d] rows): matrix i of an x4 covers d chunk
        // (2*ksp + (i >> 1)) ... laid out so that regs {0,1} feed k step 2*ksp and {2,3} k step 2*ksp+1
        const int b_row = lane & 7, b_mat = lane >> 3;

        for (int j = 0; j < total_iters; ++j) {
            const int s = j % kScoreStages;
            if (!mbar_wait_bounded(smem_u32(&tail->full_bar[s]), (j / kScoreStages) & 1)) {
                if (atomicCAS(p.status, 0, kStatusTimeout) == 0) { p.status[1] = 12; p.status[2] = blockIdx.x; }
                tail->abort_flag = 1;
                break;
            }
            if (*(volatile int*)&tail->abort_flag) break;
            const bool pass2 = j >= tiles;
            const int it = pass2 ? j - tiles : j;
            if (j == tiles) {
                // end of pass 1: combine the four column-slices of every row, c = m + log2(l)
#pragma unroll
                for (int mt = 0; mt < kScoreMT; ++mt)
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float m = rm[mt][half], l = rl[mt][half];
#pragma unroll
                        for (int o = 1; o < 4; o <<= 1) {
                            const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
                            const float l2 = __shfl_xor_sync(0xffffffffu, l, o);
                            const float mn = fmaxf(m, m2);
                            l = ((m == -INFINITY) ? 0.f : l * fast_exp2(m - mn)) +
                                ((m2 == -INFINITY) ? 0.f : l2 * fast_exp2(m2 - mn));
                            m = mn;
                        }
                        rc[mt][half] = valid[mt][half] ? m + log2f(l) : INFINITY;
                    }
            }
            if (any_rows) {
                const uint32_t kaddr = smem_u32(smem + (size_t)s * kTileBytes);
                const int tile_key0 = it * kTileKeys;
                const bool need_mask = tile_key0 + kTileKeys > n - p.w;   // window keys or the tail
#pragma unroll 1
                for (int nt = 0; nt < 8; ++nt) {
                    const int key0 = tile_key0 + nt * 8;
                    if (key0 >= n) break;
                    uint32_t kb[4][4];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)   // d chunks 4*q4 .. 4*q4+3 of keys key0..key0+7
                        ldmatrix_x4(kaddr + tile_off(nt * 8 + b_row, q4 * 4 + b_mat), kb[q4]);
                    const int ca = key0 + (lane & 3) * 2, cb = ca + 1;   // this thread's two keys
                    float e_sum0 = 0.f, e_sum1 = 0.f;
#pragma unroll
                    for (int mt = 0; mt < kScoreMT; ++mt) {
                        if ((wr0 + mt * WR_PER_TILE) >= p.w) continue;   // warp-uniform
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            mma_bf16_16816(c, qa[mt][ks], kb[ks >> 1][(ks & 1) * 2], kb[ks >> 1][(ks & 1) * 2 + 1]);
                        float z[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) z[i] = c[i] * p.scale_log2;
                        if (need_mask) {
                            // row half 0 -> c[0], c[1]; half 1 -> c[2], c[3]; columns ca, cb
#pragma unroll
                            for (int half = 0; half < 2; ++half) {
                                const int last = n - p.w + wr_of[mt][half];   // last visible key of the row
                                if (ca > last || ca >= n) z[half * 2] = -INFINITY;
                                if (cb > last || cb >= n) z[half * 2 + 1] = -INFINITY;
                            }
                        }
                        if (!pass2) {
#pragma unroll
                            for (int half = 0; half < 2; ++half) {
                                const float za = z[half * 2], zb = z[half * 2 + 1];
                                const float mn = fmaxf(rm[mt][half], fmaxf(za, zb));
                                if (mn != -INFINITY) {
                                    rl[mt][half] = rl[mt][half] * fast_exp2(rm[mt][half] - mn) +
                                                   fast_exp2(za - mn) + fast_exp2(zb - mn);
                                    rm[mt][half] = mn;
                                }
                            }
                        } else {
                            // log2 of the normalised weight, max over the heads of the group
                            float v[4];
#pragma unroll
                            for (int half = 0; half < 2; ++half) {
                                v[half * 2] = z[half * 2] - rc[mt][half];
                                v[half * 2 + 1] = z[half * 2 + 1] - rc[mt][half];
                            }
#pragma unroll
                            for (int o = 4; o < 4 * GP; o <<= 1)
#pragma unroll
                                for (int i = 0; i < 4; ++i) v[i] = fmaxf(v[i], __shfl_xor_sync(0xffffffffu, v[i], o));
                            if (((lane >> 2) & (GP - 1)) == 0) {   // one lane per (window row, column pair)
                                e_sum0 += fast_exp2(v[0]) + fast_exp2(v[2]);
                                e_sum1 += fast_exp2(v[1]) + fast_exp2(v[3]);
                            }
                        }
                    }
                    if (pass2 && ((lane >> 2) & (GP - 1)) == 0) {
                        if (ca < n) atomicAdd(&s_sum[ca], e_sum0);
                        if (cb < n) atomicAdd(&s_sum[cb], e_sum1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->empty_bar[s]));
        }
    }

    __syncthreads();
    if (*(volatile int*)&tail->abort_flag) {
        if (tid == 0) {
            const int issued = *(volatile int*)&tail->issued;
            for (int j = max(0, issued - kScoreStages); j < issued; ++j)
                mbar_wait_bounded(smem_u32(&tail->full_bar[j % kScoreStages]), (j / kScoreStages) & 1);
        }
        return;
    }
    float* out = p.sacc + (size_t)unit * p.C;
    if (wsplit == 1) {
        for (int t = tid; t < p.C; t += kScoreThreads) out[t] = (t < n) ? s_sum[t] : 0.f;
    } else {
        for (int t = tid; t < n; t += kScoreThreads) atomicAdd(&out[t], s_sum[t]);   // buffer zeroed by the host
    }
}

static size_t score_smem_bytes(int C) {
    return 1024 + (size_t)kScoreStages * kTileBytes + sizeof(float) * ((C + 63) & ~63) + sizeof(ScoreSmemTail);
}

cudaError_t score_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(gkv_score_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gkv_score_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024);
}

cudaError_t launch_score(const ScoreLaunch& p, const CUtensorMap& tm_k, cudaStream_t s) {
    const int gp = (p.g <= 4) ? 4 : 8;
    const int rows = p.w * gp;
    const int wsplit = (rows + kScoreRowsPerCta - 1) / kScoreRowsPerCta;
    const int units = p.n_layers * p.batch * p.h_kv;
    const size_t smem = score_smem_bytes(p.C);
    if (wsplit > 1) {
        // several CTAs add into one unit's sums
        const size_t off = (size_t)p.layer0 * p.batch * p.h_kv * p.C;
        cudaError_t e = cudaMemsetAsync(p.sacc + off, 0, sizeof(float) * (size_t)units * p.C, s);
        if (e != cudaSuccess) return e;
    }
    if (gp == 4) gkv_score_kernel<4><<<units * wsplit, kScoreThreads, smem, s>>>(p, tm_k, wsplit);
    else gkv_score_kernel<8><<<units * wsplit, kScoreThreads, smem, s>>>(p, tm_k, wsplit);
    return cudaGetLastError();
}

}  // namespace gkv
