// Redundancy level of every cached key (the paper's appendix on combining the global score with other
// methods): Kbar = K / (|K| + eps), Cm = Kbar Kbar^T, entries below the threshold tau zeroed, the
// columns of the most recent tokens zeroed, cbar[t] = sum over k of the masked column t.
//
// Cm is symmetric and so is the threshold mask, so the column sum of column t equals the sum over
// row t: the thread that owns an accumulator row owns a key and adds up its own row, no
// cross-thread reduction. The Gram matrix is taken of the RAW bf16 keys on tcgen05 (products exact,
// fp32 accumulation) and scaled by the two inverse norms in the epilogue, so normalisation costs no
// precision before the threshold comparison.
//
// Two launches: gkv_keynorm_kernel writes 1 / (|K_t| + eps) per cached row; gkv_redundancy_tc_kernel
// (one CTA per unit and block of 256 keys) keeps its 256 keys resident in shared memory as the A
// operand (two 128-row tiles), streams all keys of the unit as 128-key B tiles by TMA, accumulates
// D[own key][other key] in four 128-column TMEM accumulators (warp 0 copies; the 128 x 128 products
// are issued by two threads, warps 1 and 18, one per turn parity), and 16 epilogue warps in two
// sets, one per turn parity, scale, threshold and add; every wait is bounded and latches a status
// word like the scoring kernel's. The softmax and the max-normalisation
// of the appendix reduce to exp(cbar - max cbar), which the eviction kernel applies.
#include "gkv_common.cuh"
#include "gkv_internal.h"
#include "gkv_tcgen05.cuh"

namespace gkv {

constexpr int kRdGroups = 4;
constexpr int kRdEpiThreads = kRdGroups * 128;
constexpr int kRdIssuerB = 2 + kRdEpiThreads / 32;          // the warp after the epilogue warps: second tcgen05.mma issuer
constexpr int kRdThreads = 64 + kRdEpiThreads + 32;
constexpr int kRdTileKeys = 128;
constexpr int kRdBlockRows = 256;
constexpr int kRdMaxStages = 4;
constexpr int kRdStageBytes = kRdTileKeys * kRowBytes;       // 32 KB: d-low half then d-high half
constexpr int kRdABytes = kRdBlockRows * kRowBytes;          // 64 KB
constexpr int kRdAccCols = 128;                              // TMEM columns of one accumulator (four of them)
constexpr uint32_t kRdTmemCols = 512;

// ---------------------------------------------------------------------------------------------
// inv[unit][t] = 1 / (|K[unit][t]| + eps) for t < len, 0 beyond. 16 lanes per row, 16 rows per pass.
__global__ void __launch_bounds__(256) gkv_keynorm_kernel(const RedundancyLaunch p) {
    const int blocks_per_unit = (p.C + 127) / 128;
    const int unit_local = blockIdx.x / blocks_per_unit;
    const int rb = blockIdx.x - unit_local * blocks_per_unit;
    const int ls = unit_local / p.h_kv;
    const int lseq_global = p.layer0 * p.batch + ls;
    const long unit = (long)lseq_global * p.h_kv + (unit_local - ls * p.h_kv);
    const int n = p.len[lseq_global];
    const int sub = threadIdx.x >> 4, c = threadIdx.x & 15;
    const uint4* k4 = reinterpret_cast<const uint4*>(p.k_cache + (size_t)unit * p.C * kHeadDim);
    float* inv = p.inv_norm + (size_t)unit * p.C;
    for (int it = 0; it < 8; ++it) {                   // warp-uniform trip count: the shuffles below need every lane
        const int r = rb * 128 + it * 16 + sub;
        float ss = 0.f;
        if (r < n) {
            const uint4 x = k4[(size_t)r * 16 + c];
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
                ss = fmaf(lo, lo, ss);
                ss = fmaf(hi, hi, ss);
            }
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (c == 0 && r < p.C) inv[r] = (r < n) ? __frcp_rn(__fsqrt_rn(ss) + p.eps) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------------
struct __align__(8) RedundancyTail {
    uint64_t a_full;
    uint64_t k_full[kRdMaxStages];
    uint64_t k_empty[kRdMaxStages];
    uint64_t d_full[4];
    uint64_t d_empty[4];
    uint64_t drain[2];
    uint32_t tmem_base;
    int abort_flag;
    int issued;
};

__device__ __forceinline__ void rd_abort(RedundancyTail* tail, int32_t* status, int where) {
    if (atomicExch(&tail->abort_flag, 1) == 0 && atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}
// s += t where t >= thr (not for NaN).
__device__ __forceinline__ void add_if_ge(float& s, float t, float thr) {
    asm("{.reg .pred p; setp.ge.f32 p, %1, %2; @p add.f32 %0, %0, %1;}" : "+f"(s) : "f"(t), "f"(thr));
}
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kRdEpiThreads) : "memory"); }

// LONG: the unit's inverse norms do not fit shared memory (prompts of more than 8192 tokens being compressed): they are
// read from the workspace (L2) with plain loads, 32 per chunk of columns, the same addresses for every lane.
template <bool LONG>
__global__ void __launch_bounds__(kRdThreads, 1)
gkv_redundancy_tc_kernel(const RedundancyLaunch p, const __grid_constant__ CUtensorMap tm_k, int blocks_per_unit,
                         int stages) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int a_half = kRdABytes / 2;
    uint8_t* a_smem = smem;
    uint8_t* k_smem = smem + kRdABytes;
    const int c_pad = LONG ? 0 : (p.C + 127) & ~127;
    float* s_inv = reinterpret_cast<float*>(k_smem + stages * kRdStageBytes);   // [c_pad] inverse norms of the unit, 0 beyond n
    float* s_part = s_inv + c_pad;                                              // [groups][128] partial row sums
    RedundancyTail* tail = reinterpret_cast<RedundancyTail*>(s_part + kRdGroups * 128);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit_local = blockIdx.x / blocks_per_unit;
    const int a0 = (blockIdx.x - unit_local * blocks_per_unit) * kRdBlockRows;   // first key of this CTA's block
    const int ls = unit_local / p.h_kv;
    const int lseq_global = p.layer0 * p.batch + ls;
    const long unit = (long)lseq_global * p.h_kv + (unit_local - ls * p.h_kv);
    const int n = p.len[lseq_global];
    if (a0 >= n) return;                              // the whole CTA: no key of the cache in this block
    const int T = (n + kRdTileKeys - 1) / kRdTileKeys;
    const int row0 = (int)(unit * p.C);
    const int MT = (min(kRdBlockRows, n - a0) + 127) >> 7;   // row tiles of this block = turns per key tile
    const int mt_shift = MT - 1;
    const int total = T << mt_shift;                           // turns: one 128 x 128 product each

    if (tid == 0) {
        mbar_init(smem_u32(&tail->a_full), 1);
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&tail->k_full[s]), 1);
            mbar_init(smem_u32(&tail->k_empty[s]), MT);                   // one commit per turn that read the tile
        }
        for (int b = 0; b < 4; ++b) {
            mbar_init(smem_u32(&tail->d_full[b]), 1);
            mbar_init(smem_u32(&tail->d_empty[b]), kRdEpiThreads / 64);   // the eight warps that read this accumulator
        }
        mbar_init(smem_u32(&tail->drain[0]), 1);
        mbar_init(smem_u32(&tail->drain[1]), 1);
        tail->abort_flag = 0;
        tail->issued = 0;
        fence_mbar_init();
    }
    if (warp == 1) {   // whole warp: all of the SM's tensor memory (one CTA per SM by shared memory)
        tmem_alloc(smem_u32(&tail->tmem_base), kRdTmemCols);
        tmem_relinquish_alloc_permit();
        tmem_fence_before_sync();
    }
    const float* ginv = p.inv_norm + (size_t)unit * p.C;
    for (int t = tid; t < c_pad; t += kRdThreads) s_inv[t] = (t < n) ? ginv[t] : 0.f;
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tmem_base = *(volatile uint32_t*)&tail->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_k);
            const uint32_t abar = smem_u32(&tail->a_full);
            mbar_arrive_expect_tx(abar, (uint32_t)MT * 128 * kRowBytes);
            for (int rb = 0; rb < 2 * MT; ++rb) {      // 64-row boxes; rows past the tensor's end arrive as zeros
                tma_load_2d(smem_u32(a_smem + (size_t)rb * kBoxBytes), &tm_k, 0, row0 + a0 + rb * 64, abar);
                tma_load_2d(smem_u32(a_smem + a_half + (size_t)rb * kBoxBytes), &tm_k, 64, row0 + a0 + rb * 64, abar);
            }
            for (int i = 0, s = 0, round = 0; i < T; ++i) {
                if (round > 0 && !tc_wait(smem_u32(&tail->k_empty[s]), (round - 1) & 1, &tail->abort_flag)) {
                    rd_abort(tail, p.status, 31);
                    break;
                }
                const uint32_t bar = smem_u32(&tail->k_full[s]);
                const uint32_t dst = smem_u32(k_smem + (size_t)s * kRdStageBytes);
                const int y = row0 + i * kRdTileKeys;
                mbar_arrive_expect_tx(bar, kRdStageBytes);
                tma_load_2d(dst, &tm_k, 0, y, bar);
                tma_load_2d(dst + kBoxBytes, &tm_k, 0, y + 64, bar);
                tma_load_2d(dst + 2 * kBoxBytes, &tm_k, 64, y, bar);
                tma_load_2d(dst + 3 * kBoxBytes, &tm_k, 64, y + 64, bar);
                *(volatile int*)&tail->issued = i + 1;
                if (++s == stages) { s = 0; ++round; }
            }
        }
    } else if (warp == 1 || warp == kRdIssuerB) {
        // ------------------------------------------------------------------ MMA issuers
        // A turn is one 128 x 128 product (a row tile of the block times a key tile, eight instructions) into one of
        // four 128-column accumulators: turn t uses accumulator t % 4. Turns of parity 0 belong to issuer 0 and epilogue
        // set 0, those of parity 1 to issuer 1 and set 1, so each pair works through its own two accumulators. One thread
        // needs longer to get a product out (two waits, the instructions, two commits) than the tensor core to run it;
        // with two threads one product's instructions are queued while the other's execute, and with two accumulators
        // per pair a pair's next product runs under its epilogue. A commit covers the instructions of the thread that
        // makes it, so a ring slot is released by every turn that read it (its barrier counts them). With two row tiles
        // issuer `rt` always takes row tile `rt`; with one, the issuers take alternate key tiles and the ring depth is
        // even (see the launch), so that a slot always belongs to the same issuer.
        if (lane == 0) {
            const int me = warp == 1 ? 0 : 1;
            bool ok = tc_wait(smem_u32(&tail->a_full), 0, &tail->abort_flag);
            if (!ok) rd_abort(tail, p.status, 32);
            const uint32_t a_lo = umma_desc_lo(smem_u32(a_smem)) + (uint32_t)(MT == 2 ? me * ((128 * 128) >> 4) : 0);
            const uint32_t k_lo = umma_desc_lo(smem_u32(k_smem));
            const uint32_t idesc = umma_idesc_bf16_m128(kRdTileKeys);
            uint64_t a_desc[8];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) a_desc[ks] = umma_desc(a_lo + umma_kstep(ks, a_half));
            const int lstep = 2 >> mt_shift;           // key tiles between two turns of one issuer
            int s = (me >> mt_shift) % stages, round = (me >> mt_shift) / stages;
            for (int t = me; ok && t < total; t += 2) {
                const int acc = t & 3, use = t >> 2;
                if (use > 0 && !tc_wait(smem_u32(&tail->d_empty[acc]), (use - 1) & 1, &tail->abort_flag)) {
                    rd_abort(tail, p.status, 33);
                    break;
                }
                if (!tc_wait(smem_u32(&tail->k_full[s]), round & 1, &tail->abort_flag)) {
                    rd_abort(tail, p.status, 34);
                    break;
                }
                tmem_fence_after_sync();
                const uint64_t k_desc = umma_desc(k_lo + (uint32_t)s * (kRdStageBytes >> 4));
                const uint32_t d = tmem_base + (uint32_t)(acc * kRdAccCols);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_bf16(d, a_desc[ks], k_desc + umma_kstep(ks, kRdStageBytes / 2), idesc, ks > 0);
                umma_commit(smem_u32(&tail->k_empty[s]));
                umma_commit(smem_u32(&tail->d_full[acc]));
                s += lstep;
                while (s >= stages) { s -= stages; ++round; }
            }
            umma_commit(smem_u32(&tail->drain[me]));     // everything this thread issued has completed before TMEM is given back
            mbar_wait_bounded(smem_u32(&tail->drain[me]), 0);
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int wg = (warp - 2) >> 2;
        const int q4 = warp & 3;
        const int L = q4 * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q4 * 32) << 16);
        // Two sets of two groups: set 0 reads the turns of parity 0, set 1 those of parity 1, so one set's TMEM loads
        // run under the other's arithmetic. With two row tiles a set always has row tile `set`; with one, the sets take
        // alternate key tiles. The two groups of a set take 64 of a turn's 128 columns each.
        const int set = wg >> 1, sub = wg & 1;
        const int rl = (MT == 2) ? set * 128 + L : L;
        const int col0 = sub * 64;
        const int row = a0 + rl;                       // the key this thread sums for
        const float inv_r = (row < n) ? (LONG ? ginv[row] : s_inv[row]) : 0.f;
        const float thr = (row < n) ? __fdiv_rn(p.tau, inv_r) : INFINITY;   // Cm >= tau  <=>  G * inv_col >= tau / inv_row
        float sum = 0.f;
        bool ok = true;
        for (int t = set; t < total; t += 2) {
            const int i = t >> mt_shift, buf = t & 3;   // key tile and accumulator of this turn
            ok = __all_sync(0xffffffffu, ok && tc_wait(smem_u32(&tail->d_full[buf]), (t >> 2) & 1, &tail->abort_flag));
            if (!ok) { rd_abort(tail, p.status, 35); break; }
            tmem_fence_after_sync();
            for (int ch = 0; ch < 2; ++ch) {
                float gacc[32];
                tmem_ld<32>(t_lane + (uint32_t)(buf * kRdAccCols + col0 + ch * 32), gacc);
                const int colbase = i * kRdTileKeys + col0 + ch * 32;
                float4 ivl[8];
                const float4* iv = LONG ? ivl : reinterpret_cast<const float4*>(s_inv + colbase);
                if (LONG) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int c = colbase + 4 * j;
                        ivl[j] = make_float4(c < n ? __ldg(ginv + c) : 0.f, c + 1 < n ? __ldg(ginv + c + 1) : 0.f,
                                             c + 2 < n ? __ldg(ginv + c + 2) : 0.f, c + 3 < n ? __ldg(ginv + c + 3) : 0.f);
                    }
                }
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                if (i + 1 < T) {
                    // per element a multiply, a compare into a predicate and an add under it (one instruction on the ALU
                    // pipe, two on the FMA pipe; a compare + select + add would put two on the ALU pipe, which throttles first)
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 c = iv[j >> 2];
                        add_if_ge(s0, gacc[j] * c.x, thr);
                        add_if_ge(s1, gacc[j + 1] * c.y, thr);
                        add_if_ge(s2, gacc[j + 2] * c.z, thr);
                        add_if_ge(s3, gacc[j + 3] * c.w, thr);
                    }
                } else {
                    // last tile: columns past the end of the cache hold whatever the rows beyond it contain (possibly
                    // NaN or Inf bit patterns); their inverse norm is 0 and a select drops them whatever the product is
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 c = iv[j >> 2];
                        const float t0 = gacc[j] * c.x, t1 = gacc[j + 1] * c.y, t2 = gacc[j + 2] * c.z, t3 = gacc[j + 3] * c.w;
                        s0 += (c.x != 0.f && t0 >= thr) ? t0 : 0.f;
                        s1 += (c.y != 0.f && t1 >= thr) ? t1 : 0.f;
                        s2 += (c.z != 0.f && t2 >= thr) ? t2 : 0.f;
                        s3 += (c.w != 0.f && t3 >= thr) ? t3 : 0.f;
                    }
                }
                sum += (s0 + s1) + (s2 + s3);
            }
            tmem_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->d_empty[buf]));
        }
        s_part[wg * 128 + L] = sum;
        epilogue_bar_sync();
        if (!*(volatile int*)&tail->abort_flag && ((MT == 2) ? sub == 0 : wg == 0) && row < n) {
            float tot;   // the partials of the groups that shared this row (two column halves; with one row tile also the two sets), fixed order
            if (MT == 2) tot = s_part[(2 * set) * 128 + L] + s_part[(2 * set + 1) * 128 + L];
            else tot = (s_part[L] + s_part[128 + L]) + (s_part[256 + L] + s_part[384 + L]);
            p.cbar[(size_t)unit * p.C + row] = (row < n - p.recent) ? tot * inv_r : 0.f;   // recent tokens: column zeroed
        }
    }

    __syncthreads();
    if (*(volatile int*)&tail->abort_flag && tid == 0) {
        mbar_wait_bounded(smem_u32(&tail->a_full), 0);
        const int issued = *(volatile int*)&tail->issued;
        for (int i = max(0, issued - stages); i < issued; ++i)
            mbar_wait_bounded(smem_u32(&tail->k_full[i % stages]), (i / stages) & 1);
    }
    __syncthreads();
    if (warp == 1) {
        tmem_fence_after_sync();
        tmem_dealloc(tmem_base, kRdTmemCols);
    }
}

constexpr int kRdMaxShared = 8192;   // keys whose inverse norms are kept in shared memory
static size_t redundancy_smem_bytes(int C, int stages) {
    return 1024 + (size_t)kRdABytes + (size_t)stages * kRdStageBytes +
           sizeof(float) * ((C > kRdMaxShared ? 0 : ((C + 127) & ~127)) + kRdGroups * 128) + sizeof(RedundancyTail);
}

cudaError_t redundancy_kernel_setup() {
    cudaError_t e = cudaFuncSetAttribute(gkv_redundancy_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gkv_redundancy_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_keynorm(const RedundancyLaunch& p, cudaStream_t s) {
    const int units = p.n_layers * p.batch * p.h_kv;
    gkv_keynorm_kernel<<<units * ((p.C + 127) / 128), 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_redundancy(const RedundancyLaunch& p, const CUtensorMap& tm_k, cudaStream_t s) {
    const int units = p.n_layers * p.batch * p.h_kv;
    const int blocks_per_unit = (p.C + kRdBlockRows - 1) / kRdBlockRows;
    int stages = 2;
    while (stages < kRdMaxStages && redundancy_smem_bytes(p.C, stages + 1) <= 227 * 1024) ++stages;
    stages &= ~1;   // a block with one row tile has its issuers take alternate key tiles: a ring slot must stay with one of them
    if (p.C > kRdMaxShared)
        gkv_redundancy_tc_kernel<true><<<units * blocks_per_unit, kRdThreads, redundancy_smem_bytes(p.C, stages), s>>>(
            p, tm_k, blocks_per_unit, stages);
    else
        gkv_redundancy_tc_kernel<false><<<units * blocks_per_unit, kRdThreads, redundancy_smem_bytes(p.C, stages), s>>>(
            p, tm_k, blocks_per_unit, stages);
    return cudaGetLastError();
}

}  // namespace gkv
