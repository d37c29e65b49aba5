// The compression step after scoring: max-normalise the local score, merge it with the decayed
// history into the global score (Section 5, Eq. 3-5), select the top-(b-w) candidates per KV head
// (ties toward the lower position), and compact K, V, F and pos in place.
//
// A unit is one (layer, sequence, KV head). All per-row score state of a unit (at most C <= 4096
// rows) lives in shared memory. The selection is a radix select on the fp32 bit patterns (mapped so
// that they order as unsigned integers) followed by one ordered scan that assigns destinations.
//
// The fused kernel is persistent and warp-specialised: eight "selection" warps take units from a
// device-wide counter and produce each unit's kept list; a ninth "copy" warp moves the rows of the
// unit before, so the selection of one unit (latency-bound: a few dependent passes over a few
// thousand scores) runs while the copy engine streams the rows of another. The copy warp gathers
// the rows of 32 consecutive destination rows into a shared-memory stage with bulk copies
// (cp.async.bulk global -> shared, consecutive source rows merged into one copy) and writes the
// stage to its contiguous destination with one bulk copy per tensor; no row passes through
// registers and no CTA-wide barrier sits in the copy loop. In place is safe because kept[r] >= r
// and kept is ascending: a group's destination ends below the sources of every later group, and
// the rows a group overwrites are sources of that group or of earlier ones, whose loads have
// completed before the group is stored.
#include "gkv_common.cuh"
#include "gkv_internal.h"

namespace gkv {

constexpr int kEvictThreads = 256;
constexpr int kCompactUnroll = 4;

// Barrier among the 256 threads that run the score phases (all threads of the staged and prompt kernels; the
// selection warps of the fused kernel, whose copy warp does not take part).
__device__ __forceinline__ void sel_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

struct EvictShared {
    int hist[256];
    int warp_sums[16];
    float warp_max[8];
    int digit, k_rem, first_evicted, is_last;
    int32_t* status;   // the launch's status word (checked build: where a bad index is reported)
};

// inclusive prefix sum over the 256 threads of the CTA
__device__ __forceinline__ int block_incl_scan(int v, int* warp_sums, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    if (lane == 31) warp_sums[warp] = v;
    sel_sync();
    int base = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) base += (i < warp) ? warp_sums[i] : 0;
    sel_sync();
    return v + base;
}

// the same for two counters at once (full 32-bit range each)
__device__ __forceinline__ int2 block_incl_scan2(int a, int b, int* warp_sums, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int ta = __shfl_up_sync(0xffffffffu, a, o), tb = __shfl_up_sync(0xffffffffu, b, o);
        if (lane >= o) { a += ta; b += tb; }
    }
    if (lane == 31) { warp_sums[warp] = a; warp_sums[8 + warp] = b; }
    sel_sync();
    int base_a = 0, base_b = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        base_a += (i < warp) ? warp_sums[i] : 0;
        base_b += (i < warp) ? warp_sums[8 + i] : 0;
    }
    sel_sync();
    return make_int2(a + base_a, b + base_b);
}

__device__ __forceinline__ float block_max(float v, float* warp_max, int tid) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((tid & 31) == 0) warp_max[tid >> 5] = v;
    sel_sync();
    float r = warp_max[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) r = fmaxf(r, warp_max[i]);
    sel_sync();
    return r;
}

// Section 5: S_hat = S / max S over the n_c candidates; F = merge(alpha * F_prev, S_hat) on the
// n_h rows with history, F = S_hat elsewhere. `s_f` receives F for t < n_c.
// `sums` holds w * S (the 1/w of Eq. 2 cancels in the normalisation).
__device__ void merge_phase(const float* sums, const float* f_prev, float* s_f,
                            int n_c, int n_h, float alpha, int mode, EvictShared* sh, int tid) {
    float mx = 0.f;
    for (int t = tid; t < n_c; t += kEvictThreads) {
        const float s = sums[t];
        s_f[t] = s;
        mx = fmaxf(mx, s);
    }
    mx = block_max(mx, sh->warp_max, tid);
    for (int t = tid; t < n_c; t += kEvictThreads) {
        const float shat = (mx > 0.f) ? __fdiv_rn(s_f[t], mx) : 0.f;
        float f = shat;
        if (t < n_h && mode != GKV_MODE_LOCAL) {
            const float fp = alpha * f_prev[t];
            if (mode == GKV_MODE_MAX) f = fmaxf(fp, shat);
            else if (mode == GKV_MODE_MEAN) f = fp + (1.f - alpha) * shat;
            else f = fp + shat;
        }
        s_f[t] = f;
    }
    sel_sync();
}

// Appendix on combining the global score with other methods, SnapKV: sequence-wise max-pooling of the score
// the selection runs on (odd kernel, window clipped at the ends of the candidate range).
__device__ void pool_phase(const float* s_f, float* s_sel, int n_c, int kernel, int tid) {
    const int half = kernel >> 1;
    for (int t = tid; t < n_c; t += kEvictThreads) {
        float m = s_f[t];
        for (int u = max(t - half, 0); u <= min(t + half, n_c - 1); ++u) m = fmaxf(m, s_f[u]);
        s_sel[t] = m;
    }
    sel_sync();
}

// Same appendix, redundancy term: R = softmax(cbar), R' = R / max R = exp(cbar - max cbar) (maximum over all
// n cached tokens), selection score = lambda P - (1 - lambda) R' with P = s_in (F, or pooled F; s_in may be s_sel).
__device__ void combine_phase(const float* __restrict__ cbar, const float* s_in, float* s_sel, int n, int n_c,
                              float lambda, EvictShared* sh, int tid) {
    float mx = -INFINITY;
    for (int t = tid; t < n; t += kEvictThreads) mx = fmaxf(mx, cbar[t]);
    mx = block_max(mx, sh->warp_max, tid);
    for (int t = tid; t < n_c; t += kEvictThreads)
        s_sel[t] = lambda * s_in[t] - (1.f - lambda) * fast_exp2((cbar[t] - mx) * 1.4426950408889634f);
    sel_sync();
}

// F in s_f -> the scores the selection runs on in s_sel (s_sel == s_f when no optional term is on):
// P = maxpool(F) if pooling is on, then lambda P - (1 - lambda) R' if the redundancy term is on.
__device__ __forceinline__ bool has_selection_terms(const EvictLaunch& p) { return p.cbar != nullptr || p.pool_kernel > 1; }
__device__ void selection_scores(const EvictLaunch& p, long unit, const float* s_f, float* s_sel, int n, int n_c,
                                 EvictShared* sh, int tid) {
    const bool pool = p.pool_kernel > 1;
    if (pool) pool_phase(s_f, s_sel, n_c, p.pool_kernel, tid);
    if (p.cbar) combine_phase(p.cbar + (size_t)unit * p.C, pool ? s_sel : s_f, s_sel, n, n_c, p.lambda, sh, tid);
}

// fp32 bit pattern -> unsigned integer with the same order (negative values included: the combined
// score of the redundancy term is lambda * F - (1 - lambda) * R').
__device__ __forceinline__ uint32_t ordered_bits(uint32_t x) {
    return x ^ (static_cast<uint32_t>(static_cast<int32_t>(x) >> 31) | 0x80000000u);
}

// Top-n_keep of s_f[0..n_c) with ties toward the lower index; kept rows ascending into s_kept,
// followed by the w window rows n_c .. n_c+w-1. Returns (CTA-uniform) the first row that moves.
// s_evict (may be NULL) receives the n_c - n_keep evicted rows in ascending order.
template <typename KT>   // element type of the kept list: int, or uint16_t where rows are known to be < 65536
__device__ int select_phase(const float* s_f, KT* s_kept, int* s_evict, int n_c, int n_keep, int w, EvictShared* sh,
                            int tid) {
    const uint32_t* bits = reinterpret_cast<const uint32_t*>(s_f);
    const int lane = tid & 31;
    uint32_t prefix = 0;
    int k = n_keep;
    sh->hist[tid] = 0;
    sel_sync();
    // Radix select, 8 bits a pass from the top: the histogram of the candidates that match the prefix found so far,
    // a scan from the top digit down, and the digit that holds the k-th largest joins the prefix. Scores crowd into a
    // few top digits (same sign and exponent), so equal digits within a warp are counted once (match) and added with
    // one atomic. A pass whose digit holds exactly the k candidates still wanted ends the search early: all of them
    // are kept, whatever their lower bits.
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        const uint32_t mask = (shift == 24) ? 0u : (0xffffffffu << (shift + 8));
        for (int t0 = 0; t0 < n_c; t0 += kEvictThreads) {
            const int t = t0 + tid;
            const uint32_t x = (t < n_c) ? ordered_bits(bits[t]) : 0u;
            const bool in = t < n_c && (x & mask) == prefix;
            const uint32_t d = in ? ((x >> shift) & 255u) : 256u;
            const uint32_t peers = __match_any_sync(0xffffffffu, d);
            if (in && (peers & ((1u << lane) - 1u)) == 0u) atomicAdd(&sh->hist[d], __popc(peers));
        }
        sel_sync();
        // thread tid looks at digit 255 - tid (and clears it for the next pass); `ge` = matching elements with digit >= mine
        const int mine = sh->hist[255 - tid];
        sh->hist[255 - tid] = 0;
        const int ge = block_incl_scan(mine, sh->warp_sums, tid);
        const int gt = ge - mine;
        if (ge >= k && gt < k) {  // exactly one digit holds the k-th largest
            sh->digit = 255 - tid;
            sh->k_rem = k - gt;
            sh->is_last = (mine == k - gt);
        }
        sel_sync();
        prefix |= static_cast<uint32_t>(sh->digit) << shift;
        k = sh->k_rem;
        if (sh->is_last) {      // (CTA-uniform) every candidate of this digit is kept: threshold = the digit's lowest pattern
            k = n_c;
            break;
        }
    }
    // prefix = ordered bit pattern T of the n_keep-th largest score; take everything above it and the
    // first k rows equal to it
    const uint32_t T = prefix;
    const int per = (n_c + kEvictThreads - 1) / kEvictThreads;
    const int t0 = tid * per, t1 = min(t0 + per, n_c);
    int gt = 0, eq = 0;
    for (int t = t0; t < t1; ++t) {
        const uint32_t x = ordered_bits(bits[t]);
        gt += (x > T);
        eq += (x == T);
    }
    if (tid == 0) sh->first_evicted = n_c;
    const int2 incl = block_incl_scan2(gt, eq, sh->warp_sums, tid);
    int gt_before = incl.x - gt, eq_before = incl.y - eq;
    int first_drop = n_c;
    for (int t = t0; t < t1; ++t) {
        const uint32_t x = ordered_bits(bits[t]);
        const int kept_before = gt_before + min(eq_before, k);   // kept rows below t
        bool dropped = false;
        if (x > T) {
            if (GKV_BOUNDS_OK(kept_before >= 0 && kept_before < n_keep, sh->status, 61)) s_kept[kept_before] = (KT)t;
            ++gt_before;
        } else if (x == T) {
            if (eq_before < k) {
                if (GKV_BOUNDS_OK(kept_before >= 0 && kept_before < n_keep, sh->status, 62)) s_kept[kept_before] = (KT)t;
            } else {
                dropped = true;
            }
            ++eq_before;
        } else {
            dropped = true;
        }
        if (dropped) {
            first_drop = min(first_drop, t);
            if (s_evict && GKV_BOUNDS_OK(t - kept_before >= 0 && t - kept_before < n_c - n_keep, sh->status, 63))
                s_evict[t - kept_before] = t;
        }
    }
    if (first_drop < n_c) atomicMin(&sh->first_evicted, first_drop);
    for (int r = tid; r < w; r += kEvictThreads) s_kept[n_keep + r] = (KT)(n_c + r);
    sel_sync();
    return sh->first_evicted;
}

// Sink-plus-recent policy (StreamingLLM, a baseline of the paper's experimental setup) as a selection without a
// score: rows 0 .. n_sink - 1 stay, rows n_sink .. n_sink + (n - b) - 1 leave, the rest moves up. Writes the same
// outputs as select_phase, clears s_f (no score is recorded) and returns the first row that moves.
template <typename KT>
__device__ int streaming_phase(float* s_f, KT* s_kept, int* s_evict, int n, int n_c, int b, int n_sink, int tid) {
    const int shift = n - b;
    for (int t = tid; t < n_c; t += kEvictThreads) s_f[t] = 0.f;
    for (int r = tid; r < b; r += kEvictThreads) s_kept[r] = (KT)(r < n_sink ? r : r + shift);
    if (s_evict)
        for (int e = tid; e < shift; e += kEvictThreads) s_evict[e] = n_sink + e;
    sel_sync();
    return n_sink;
}

// Move the rows kept[r] -> r for r in [r_first, b) of one unit's K and V, restricted to the
// 16-byte chunks [chunk0, chunk0 + cpr) of every row (cpr divides 16).
// (`n_rows` = rows of the unit that hold tokens and `status` are used by the checked build only.)
__device__ void compact_phase(__nv_bfloat16* kbase, __nv_bfloat16* vbase, const int* kept, int b, int r_first,
                              int chunk0, int cpr, int tid, int n_rows, int32_t* status) {
    (void)n_rows; (void)status;
    const int rows_per_pass = kEvictThreads / cpr;
    const int my_r = tid / cpr;
    const int my_c = chunk0 + (tid - my_r * cpr);
    uint4* k4 = reinterpret_cast<uint4*>(kbase);
    uint4* v4 = reinterpret_cast<uint4*>(vbase);
    for (int r0 = r_first; r0 < b; r0 += kCompactUnroll * rows_per_pass) {
        uint4 kx[kCompactUnroll], vx[kCompactUnroll];
        int src[kCompactUnroll];
#pragma unroll
        for (int u = 0; u < kCompactUnroll; ++u) {
            const int r = r0 + u * rows_per_pass + my_r;
            src[u] = (r < b) ? kept[r] : -1;
            if (src[u] >= 0 && !GKV_BOUNDS_OK(src[u] >= r && src[u] < n_rows, status, 64)) src[u] = -1;
            if (src[u] >= 0) {
                kx[u] = k4[(size_t)src[u] * 16 + my_c];
                vx[u] = v4[(size_t)src[u] * 16 + my_c];
            }
        }
        __syncthreads();  // the whole group is in registers before any of its rows is overwritten
#pragma unroll
        for (int u = 0; u < kCompactUnroll; ++u) {
            const int r = r0 + u * rows_per_pass + my_r;
            if (src[u] >= 0) {
                k4[(size_t)r * 16 + my_c] = kx[u];
                v4[(size_t)r * 16 + my_c] = vx[u];
            }
        }
    }
}

// The same move for whole rows, without register staging: the rows of a group of kCopyRows consecutive
// DESTINATION rows are gathered into a shared-memory stage by 16-byte cp.async (the stage holds them
// in destination order), and once they have landed one bulk copy per tensor writes the stage to the
// group's contiguous destination. kCopyStages - 2 groups of loads are in flight while older groups
// are stored. In place is safe for the same reason as above: a group's destination ends below the
// sources of every later group, and its own rows are all in shared memory before it is stored.
constexpr int kCopyRows = 32;
constexpr int kCopyStages = 5;
constexpr int kCopyStageBytes = kCopyRows * kRowBytes * 2;   // K rows then V rows
constexpr int kCopyRingBytes = kCopyStages * kCopyStageBytes;

// Source and destination may be the same buffers (compaction in place) or different ones (gather of a prompt).
__device__ void compact_phase_async(const __nv_bfloat16* ksrc, const __nv_bfloat16* vsrc, __nv_bfloat16* kbase,
                                    __nv_bfloat16* vbase, const int* kept, int b, int r_first, uint8_t* ring, int tid,
                                    int n_rows, int32_t* status) {
    (void)n_rows; (void)status;
    constexpr int D = kCopyStages - 2;                        // groups of loads in flight
    const int n_groups = (b - r_first + kCopyRows - 1) / kCopyRows;
    const uint32_t ring_addr = smem_u32(ring);
    const uint4* k4 = reinterpret_cast<const uint4*>(ksrc);
    const uint4* v4 = reinterpret_cast<const uint4*>(vsrc);
    for (int j = 0; j < n_groups + D; ++j) {
        // the stage group j loads into was last read by the store issued two iterations ago
        if (tid == 0) bulk_wait_read<1>();
        __syncthreads();
        if (j < n_groups) {
            const uint32_t stage = ring_addr + (uint32_t)(j % kCopyStages) * kCopyStageBytes;
            const int r0 = r_first + j * kCopyRows;
            // 32 rows x 16 chunks x 2 tensors = 1024 copies over 256 threads
#pragma unroll
            for (int u = 0; u < 2 * kCopyRows * 16 / kEvictThreads; ++u) {
                const int e = u * kEvictThreads + tid;
                const int is_v = e >> 9, row = (e >> 4) & (kCopyRows - 1), chunk = e & 15;
                const int r = r0 + row;
                if (r < b && GKV_BOUNDS_OK(kept[r] >= r && kept[r] < n_rows, status, 65)) {
                    const uint4* src = (is_v ? v4 : k4) + (size_t)kept[r] * 16 + chunk;
                    cp_async_16(stage + (uint32_t)(is_v * kCopyRows * kRowBytes + row * kRowBytes + chunk * 16), src);
                }
            }
        }
        cp_async_commit();
        cp_async_wait_group<D>();          // this thread's copies of group j - D have landed
        fence_proxy_async_smem();          // ... and are visible to the bulk copy engine
        __syncthreads();
        const int jd = j - D;
        if (jd >= 0 && tid == 0) {
            const uint32_t stage = ring_addr + (uint32_t)(jd % kCopyStages) * kCopyStageBytes;
            const int r0 = r_first + jd * kCopyRows;
            const uint32_t bytes = (uint32_t)min(kCopyRows, b - r0) * kRowBytes;
            bulk_store(kbase + (size_t)r0 * kHeadDim, stage, bytes);
            bulk_store(vbase + (size_t)r0 * kHeadDim, stage + kCopyRows * kRowBytes, bytes);
            bulk_commit();
        }
    }
    if (tid == 0) bulk_wait<0>();          // all rows written before the state is published
    __syncthreads();
}

struct UnitIndex {
    int unit_local, lseq_global;
    long unit;
};
__device__ __forceinline__ UnitIndex unit_of(const EvictLaunch& p, int unit_local) {
    UnitIndex u;
    u.unit_local = unit_local;
    const int ls = unit_local / p.h_kv;
    const int head = unit_local - ls * p.h_kv;
    u.lseq_global = p.layer0 * p.batch + ls;
    u.unit = (long)u.lseq_global * p.h_kv + head;
    return u;
}

// Record the per-row state after selection: compact F and pos, clear the window sums, export kept.
template <typename KT>
__device__ void write_score_state(const EvictLaunch& p, const UnitIndex& u, const float* s_f, const KT* s_kept,
                                  int* s_pos, const int* s_evict, int n, int tid) {
    const int n_keep = p.b - p.w;
    float* f = p.f + (size_t)u.unit * p.C;
    for (int r = tid; r < p.C; r += kEvictThreads)
        f[r] = (r < n_keep && GKV_BOUNDS_OK((int)s_kept[r] >= r && (int)s_kept[r] < n - p.w, p.status, 66)) ? s_f[s_kept[r]] : 0.f;
    if (p.pos) {
        int32_t* pos = p.pos + (size_t)u.unit * p.C;
        for (int t = tid; t < n; t += kEvictThreads) s_pos[t] = pos[t];
        sel_sync();
        for (int r = tid; r < p.b; r += kEvictThreads) pos[r] = s_pos[s_kept[r]];
    }
    if (p.evict_log) {   // what left the cache: original positions when they are tracked, else pre-compaction rows
        int32_t* log = p.evict_log + (size_t)u.unit * (p.C - p.b);
        const int n_ev = n - p.b;
        for (int e = tid; e < p.C - p.b; e += kEvictThreads)
            log[e] = (e < n_ev) ? (p.pos ? s_pos[s_evict[e]] : s_evict[e]) : -1;
    }
    float* sacc = p.sacc + (size_t)u.unit * p.C;
    for (int t = tid; t < p.C; t += kEvictThreads) sacc[t] = 0.f;
    if (p.kept_out) {
        int32_t* ko = p.kept_out + (size_t)u.unit_local * p.b;
        for (int r = tid; r < p.b; r += kEvictThreads) ko[r] = s_kept[r];
    }
}

// The last CTA of a (layer, sequence) publishes len = b and n_hist = b - w.
__device__ void publish_state(const EvictLaunch& p, const UnitIndex& u, int ctas_per_seq, EvictShared* sh, int tid) {
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(&p.seq_done[u.lseq_global], 1);
        if (prev == ctas_per_seq - 1) {
            p.seq_done[u.lseq_global] = 0;
            p.len[u.lseq_global] = p.b;
            p.len[(size_t)p.L_total * p.batch + u.lseq_global] = p.b - p.w;
        }
    }
}

// s_sel (the scores the selection runs on) is s_f itself unless an optional term is on. `kept_bufs` kept lists
// of b entries follow the scores (two in the fused kernel: one being produced, one being copied from).
__device__ __forceinline__ void carve(uint8_t* smem, const EvictLaunch& p, float** s_f, int** s_kept, int** s_pos,
                                      EvictShared** sh, float** s_sel, int** s_evict, int kept_bufs = 1) {
    *sh = reinterpret_cast<EvictShared*>(smem);
    *s_f = reinterpret_cast<float*>(smem + sizeof(EvictShared));
    *s_kept = reinterpret_cast<int*>(*s_f + p.C);
    *s_pos = *s_kept + kept_bufs * p.b;
    const bool terms = p.cbar != nullptr || p.pool_kernel > 1;
    *s_sel = terms ? reinterpret_cast<float*>(*s_pos + (p.pos ? p.C : 0)) : *s_f;
    *s_evict = p.evict_log ? *s_pos + (p.pos ? p.C : 0) + (terms ? p.C : 0) : nullptr;
}
static size_t evict_state_bytes(const EvictLaunch& p, int kept_bufs = 1) {
    return sizeof(EvictShared) + sizeof(float) * p.C + sizeof(int) * p.b * kept_bufs + (p.pos ? sizeof(int) * p.C : 0) +
           ((p.cbar || p.pool_kernel > 1) ? sizeof(float) * p.C : 0) + (p.evict_log ? sizeof(int) * (p.C - p.b) : 0);
}
static size_t evict_smem_bytes(const EvictLaunch& p) { return evict_state_bytes(p); }

// ---------------------------------------------------------------------------------------------
// Whole step in one launch: merge -> select -> score-state update on the selection warps, K/V compaction on the
// copy warp, one unit behind.
constexpr int kFusedThreads = kEvictThreads + 32;
constexpr int kFusedMaxStages = 8;

struct __align__(16) FusedPipe {
    uint64_t kept_full[2];    // selection -> copy: the kept list in buffer i is complete (tid 0 arrives)
    uint64_t kept_empty[2];   // copy -> selection: every load that reads buffer i has been issued
    uint64_t taken[2];        // copy -> selection: the copy warp has started on the list in buffer i
    uint64_t ring_full[kFusedMaxStages];   // the rows of a stage have landed
    long unit[2];             // the unit whose kept list is in buffer i, or -1: no more
    int r_first[2];           // first destination row that moves
    int n_rows[2];            // rows of that unit that hold tokens (checked build)
    uint32_t dst_row[kFusedMaxStages];     // per stage: first destination row (in rows of the whole K / V tensor), rows held
    int st_rows[kFusedMaxStages];
    int cur_item, abort_flag, is_last, go;
};

// Shared memory of the fused kernel (byte offsets): the selection warps' score arrays, two kept lists of b 16-bit
// rows (one being produced, one being copied from; C <= 4096), the hand-over structure, the copy ring.
struct FusedLayout {
    int f, fp, sel, pos, evict, kept, pipe, ring;
};
__host__ __device__ inline FusedLayout fused_layout(int C, int b, bool terms, bool has_pos, bool has_log) {
    FusedLayout l;
    int off = (int)sizeof(EvictShared);
    l.f = off;      off += 4 * C;                       // F (the sums arrive here first)
    l.fp = off;     off += 4 * C;                       // F_prev
    l.sel = terms ? off : l.f;   off += terms ? 4 * C : 0;
    l.pos = off;    off += has_pos ? 4 * C : 0;
    l.evict = off;  off += has_log ? 4 * (C - b) : 0;
    l.kept = off;   off += 2 * 2 * b;
    l.pipe = (off + 15) & ~15;
    l.ring = (l.pipe + (int)sizeof(FusedPipe) + 127) & ~127;
    return l;
}

__device__ __forceinline__ bool evict_wait(uint32_t bar, uint32_t parity, const int* abort_flag) {
    for (uint32_t i = 0; i < kWaitSpins; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*(volatile const int*)abort_flag) return false;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void evict_abort(FusedPipe* pipe, int32_t* status, int where) {
    if (atomicExch(&pipe->abort_flag, 1) == 0 && atomicCAS(status, 0, kStatusTimeout) == 0) {
        status[1] = where;
        status[2] = blockIdx.x;
    }
}

__global__ void __launch_bounds__(kFusedThreads, 5) gkv_evict_fused_kernel(const EvictLaunch p, int stages) {
    extern __shared__ __align__(128) uint8_t evict_smem[];
    const FusedLayout lay = fused_layout(p.C, p.b, has_selection_terms(p), p.pos != nullptr, p.evict_log != nullptr);
    EvictShared* sh = reinterpret_cast<EvictShared*>(evict_smem);
    float* s_f = reinterpret_cast<float*>(evict_smem + lay.f);
    float* s_fp = reinterpret_cast<float*>(evict_smem + lay.fp);
    float* s_sel = reinterpret_cast<float*>(evict_smem + lay.sel);
    int* s_pos = reinterpret_cast<int*>(evict_smem + lay.pos);
    int* s_evict = p.evict_log ? reinterpret_cast<int*>(evict_smem + lay.evict) : nullptr;
    uint16_t* s_kept = reinterpret_cast<uint16_t*>(evict_smem + lay.kept);
    FusedPipe* pipe = reinterpret_cast<FusedPipe*>(evict_smem + lay.pipe);
    uint8_t* ring = evict_smem + lay.ring;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total = p.n_layers * p.batch * p.h_kv;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&pipe->kept_full[i]), 1);
            mbar_init(smem_u32(&pipe->kept_empty[i]), 1);
            mbar_init(smem_u32(&pipe->taken[i]), 1);
        }
        for (int s = 0; s < stages; ++s) mbar_init(smem_u32(&pipe->ring_full[s]), 1);
        pipe->abort_flag = 0;
        pipe->is_last = 0;
        sh->status = p.status;
        fence_mbar_init();
    }
    __syncthreads();

    if (warp < kEvictThreads / 32) {
        // ------------------------------------------------------------------ selection warps
        int handed = 0;      // units handed to the copy warp so far
        bool ok = true;
        for (int k = 0; ok; ++k) {
            // Units are handed out first come, first served: this CTA's index first, then numbers from a device-wide
            // counter. The barrier also ends the previous unit's use of the score arrays.
            // A CTA asks for its next unit only once its copy warp has started on the unit before: it then holds one
            // unit in the copy and one in the selection, not three, and the units go to the CTAs that get through
            // them fastest.
            if (tid == 0) {
                int item = -1;
                if (handed == 0 || evict_wait(smem_u32(&pipe->taken[(handed - 1) & 1]), ((handed - 1) >> 1) & 1, &pipe->abort_flag))
                    item = (k == 0) ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(p.work, 1);
                else
                    evict_abort(pipe, p.status, 40);
                pipe->cur_item = item < total ? item : -1;
            }
            sel_sync();
            const int item = *(volatile int*)&pipe->cur_item;
            if (item < 0) break;
            const UnitIndex u = unit_of(p, item);
            // The unit's window sums and recorded scores start their way into shared memory at once (all C entries:
            // the length is not known yet), so the length, the sums and the scores cost one memory round trip, not three.
            {
                const float* gs = p.sacc + (size_t)u.unit * p.C;
                const float* gf = p.f + (size_t)u.unit * p.C;
                for (int t = tid; t < p.C; t += kEvictThreads) {
                    cp_async_4(smem_u32(s_f + t), gs + t);
                    cp_async_4(smem_u32(s_fp + t), gf + t);
                }
                cp_async_commit();
            }
            const int n = p.len[u.lseq_global];
            const int n_h = p.len[(size_t)p.L_total * p.batch + u.lseq_global];
            cp_async_wait_all();
            sel_sync();
            if (n <= p.b) {  // nothing to evict: only the window sums restart
                float* sacc = p.sacc + (size_t)u.unit * p.C;
                for (int t = tid; t < p.C; t += kEvictThreads) sacc[t] = 0.f;
                if (p.evict_log)
                    for (int e = tid; e < p.C - p.b; e += kEvictThreads) p.evict_log[(size_t)u.unit * (p.C - p.b) + e] = -1;
                continue;
            }
            const int buf = handed & 1;
            uint16_t* kept = s_kept + buf * p.b;
            const int n_c = n - p.w;
            const bool scored = p.policy != GKV_POLICY_STREAMING;
            if (scored) {
                merge_phase(s_f, s_fp, s_f, n_c, n_h, p.alpha, p.mode, sh, tid);
                selection_scores(p, u.unit, s_f, s_sel, n, n_c, sh, tid);
            }
            // the copy warp has issued every load that reads this buffer's previous list (two units ago)
            if (handed >= 2) {   // one thread waits, the barrier hands its verdict (and the ordering) to the others
                if (tid == 0) pipe->go = evict_wait(smem_u32(&pipe->kept_empty[buf]), ((handed >> 1) - 1) & 1, &pipe->abort_flag);
                sel_sync();
                if (!*(volatile int*)&pipe->go) { evict_abort(pipe, p.status, 41); break; }
            }
            const int r_first = scored ? select_phase(s_sel, kept, s_evict, n_c, p.b - p.w, p.w, sh, tid)
                                       : streaming_phase(s_f, kept, s_evict, n, n_c, p.b, p.n_sink, tid);
            if (tid == 0) {
                pipe->unit[buf] = u.unit;
                pipe->r_first[buf] = r_first;
                pipe->n_rows[buf] = n;
                mbar_arrive(smem_u32(&pipe->kept_full[buf]));
            }
            ++handed;
            write_score_state(p, u, s_f, kept, s_pos, s_evict, n, tid);
        }
        // the end of the list: a buffer that carries -1
        if (tid == 0 && !*(volatile int*)&pipe->abort_flag) {
            const int buf = handed & 1;
            if (handed < 2 || evict_wait(smem_u32(&pipe->kept_empty[buf]), ((handed >> 1) - 1) & 1, &pipe->abort_flag)) {
                pipe->unit[buf] = -1;
                mbar_arrive(smem_u32(&pipe->kept_full[buf]));
            } else {
                evict_abort(pipe, p.status, 42);
            }
        }
    } else {
        // ------------------------------------------------------------------ copy warp
        const int D = stages - 2;                      // groups of loads in flight
        const uint32_t ring_addr = smem_u32(ring);
        uint32_t G = 0, stored = 0;                    // ring groups loaded / stored so far, across units
        bool ok = true;
        // store ring group `stored`: its rows have landed (and with them every row loaded before)
        auto store_next = [&]() {
            const int st = stored % stages;
            if (!evict_wait(smem_u32(&pipe->ring_full[st]), (stored / stages) & 1, &pipe->abort_flag)) {
                evict_abort(pipe, p.status, 44);
                ok = false;
                return;
            }
            if (lane == 0) {
                const uint32_t src = ring_addr + (uint32_t)st * kCopyStageBytes;
                const uint32_t bytes = (uint32_t)pipe->st_rows[st] * kRowBytes;
                const size_t dst = (size_t)pipe->dst_row[st] * kHeadDim;
                bulk_store(p.k_cache + dst, src, bytes);
                bulk_store(p.v_cache + dst, src + kCopyRows * kRowBytes, bytes);
                bulk_commit();
            }
            ++stored;
        };
        for (int k = 0; ok; ++k) {
            const int buf = k & 1;
            // while the next list is not there yet, the groups already loaded go out
            while (ok && stored < G && !mbar_try_wait(smem_u32(&pipe->kept_full[buf]), (k >> 1) & 1)) store_next();
            if (!ok) break;
            if (!evict_wait(smem_u32(&pipe->kept_full[buf]), (k >> 1) & 1, &pipe->abort_flag)) {
                evict_abort(pipe, p.status, 43);
                break;
            }
            const long unit = *(volatile long*)&pipe->unit[buf];
            if (unit < 0) break;
            const int r_first = *(volatile int*)&pipe->r_first[buf];
            if (lane == 0) mbar_arrive(smem_u32(&pipe->taken[buf]));
            const uint16_t* kept = s_kept + buf * p.b;
            const uint4* k4 = reinterpret_cast<const uint4*>(p.k_cache + (size_t)unit * p.C * kHeadDim);
            const uint4* v4 = reinterpret_cast<const uint4*>(p.v_cache + (size_t)unit * p.C * kHeadDim);
            for (int r0 = r_first; r0 < p.b && ok; r0 += kCopyRows, ++G) {
                const int st = G % stages;
                // the stage was last read by the store of ring group G - stages; stores issued so far: groups < `stored`
                if (lane == 0) bulk_wait_read<1>();
                __syncwarp();
                const int rows = min(kCopyRows, p.b - r0);
                const uint32_t bar = smem_u32(&pipe->ring_full[st]);
                if (lane == 0) {
                    pipe->dst_row[st] = (uint32_t)(unit * p.C + r0);
                    pipe->st_rows[st] = rows;
                    mbar_arrive_expect_tx(bar, (uint32_t)rows * 2 * kRowBytes);
                }
                __syncwarp();
                // lane i owns destination row r0 + i; runs of consecutive source rows travel as one copy
                const bool valid = lane < rows;
                const int src = valid ? (int)kept[r0 + lane] : -2;
                const int prev = __shfl_up_sync(0xffffffffu, src, 1);
                const bool start = valid && (lane == 0 || src != prev + 1);
                const uint32_t starts = __ballot_sync(0xffffffffu, start);
                if (start) {
                    const uint32_t rest = (lane == 31) ? 0u : (starts >> (lane + 1));
                    int run = rest ? __ffs(rest) : rows - lane;
                    // (checked build: a run must start at or above its destination and end inside the unit's tokens;
                    // a bad one is not copied, its bytes are taken off the stage's expected count)
                    if (!GKV_BOUNDS_OK(src >= r0 + lane && src + run <= pipe->n_rows[buf] && r0 + lane + run <= p.b, p.status, 67)) {
                        asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"((uint32_t)run * 2 * kRowBytes) : "memory");
                        run = 0;
                    }
                    if (run > 0) {
                    const uint32_t dst = ring_addr + (uint32_t)st * kCopyStageBytes + (uint32_t)lane * kRowBytes;
                    bulk_load(dst, k4 + (size_t)src * 16, (uint32_t)run * kRowBytes, bar);
                    bulk_load(dst + kCopyRows * kRowBytes, v4 + (size_t)src * 16, (uint32_t)run * kRowBytes, bar);
                    }
                }
                if (G >= (uint32_t)D + stored) store_next();   // keeps D groups of loads in flight
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&pipe->kept_empty[buf]));
        }
        while (ok && stored < G) store_next();
        if (!ok || *(volatile int*)&pipe->abort_flag) {
            // loads still in flight get a bounded time to land before the CTA exits
            for (uint32_t g = stored; g < G; ++g) mbar_wait_bounded(smem_u32(&pipe->ring_full[g % stages]), (g / stages) & 1);
        }
        if (lane == 0) bulk_wait<0>();                 // all rows written
    }

    __syncthreads();
    // The last CTA to finish puts the two counters back to zero and publishes the new state of every sequence of the
    // launch that was compressed: len = b, n_hist = b - w. (No CTA may do that for its own sequence earlier: the other
    // KV heads of the sequence read the old length when they start.)
    if (tid == 0) {
        __threadfence();
        pipe->is_last = atomicAdd(p.work + 1, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (pipe->is_last) {
        const int n_seq = p.n_layers * p.batch;
        for (int ls = tid; ls < n_seq; ls += kFusedThreads) {
            const int lseq = p.layer0 * p.batch + ls;
            if (p.len[lseq] > p.b) {
                p.len[lseq] = p.b;
                p.len[(size_t)p.L_total * p.batch + lseq] = p.b - p.w;
            }
        }
        if (tid == 0) {
            p.work[0] = 0;
            p.work[1] = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// First compression of a prompt that is longer than the cache (Section 3: "compressed after every s
// tokens" starts from a prefilled cache; Section 5: the first step uses the normalised local score alone).
// The prompt's K, V live in the caller's prefill buffers [batch][h_kv][P_max][d] with per-sequence lengths;
// `sums` holds w * S of the prompt's last w tokens over all its keys (scoring kernel). Per unit: prompts of
// at most b tokens are copied whole (no history starts); longer ones keep the top-(b-w) candidates by the
// normalised score (after the optional pooling) plus the window, gathered into cache rows 0..b-1 in
// ascending position, with F_state = the normalised score of the kept rows and pos = prompt position.
__global__ void __launch_bounds__(kEvictThreads) gkv_prompt_compress_kernel(const PromptLaunch p, int ring_offset) {
    extern __shared__ __align__(128) uint8_t evict_smem[];
    EvictShared* sh = reinterpret_cast<EvictShared*>(evict_smem);
    const int tid = threadIdx.x;
    if (tid == 0) sh->status = p.status;     // (read after the barriers of the phases below)
    const int unit_local = blockIdx.x;
    // The unit's scores [P_max] (and the pooled ones) live in shared memory, or, for prompts too long for it, in the
    // workspace: the phases below only need a pointer, and a CTA-wide barrier orders global accesses as well.
    const int n_arrays = (p.pool_kernel > 1 || p.cbar) ? 2 : 1;
    float* s_f = p.f_long ? p.f_long + (size_t)unit_local * n_arrays * p.P_max
                          : reinterpret_cast<float*>(evict_smem + sizeof(EvictShared));
    float* s_sel = (n_arrays == 2) ? s_f + p.P_max : s_f;                      // [P_max] the scores the selection runs on
    int* s_kept = p.f_long ? reinterpret_cast<int*>(evict_smem + sizeof(EvictShared))
                           : reinterpret_cast<int*>(s_f + n_arrays * p.P_max);   // [b]
    const int seq = unit_local / p.h_kv;
    const int lseq_global = p.layer * p.batch + seq;
    const long unit = (long)lseq_global * p.h_kv + (unit_local - seq * p.h_kv);
    const int n = min(p.prompt_len[seq], p.P_max);
    const bool compress = n > p.b;
    const int rows = compress ? p.b : n;                   // rows of the cache after this call
    const int n_keep = p.b - p.w;
    if (compress && p.policy == GKV_POLICY_STREAMING) {
        streaming_phase(s_f, s_kept, (int*)nullptr, n, n - p.w, p.b, p.n_sink, tid);
    } else if (compress) {
        const int n_c = n - p.w;
        merge_phase(p.sums + (size_t)unit_local * p.P_max, nullptr, s_f, n_c, 0, 0.f, GKV_MODE_LOCAL, sh, tid);
        if (p.pool_kernel > 1) pool_phase(s_f, s_sel, n_c, p.pool_kernel, tid);
        if (p.cbar)
            combine_phase(p.cbar + (size_t)unit_local * p.P_max, (p.pool_kernel > 1) ? s_sel : s_f, s_sel, n, n_c, p.lambda, sh, tid);
        select_phase(s_sel, s_kept, nullptr, n_c, n_keep, p.w, sh, tid);
    } else {
        for (int r = tid; r < n; r += kEvictThreads) s_kept[r] = r;
        __syncthreads();
    }
    float* f = p.f + (size_t)unit * p.C;
    float* sacc = p.sacc + (size_t)unit * p.C;
    for (int r = tid; r < p.C; r += kEvictThreads) {
        f[r] = (compress && r < n_keep) ? s_f[s_kept[r]] : 0.f;
        sacc[r] = 0.f;
    }
    if (p.pos) {
        int32_t* pos = p.pos + (size_t)unit * p.C;
        for (int r = tid; r < rows; r += kEvictThreads) pos[r] = s_kept[r];
    }
    if (p.kept_out) {
        int32_t* ko = p.kept_out + (size_t)unit_local * p.b;
        for (int r = tid; r < p.b; r += kEvictThreads) ko[r] = (r < rows) ? s_kept[r] : -1;
    }
    compact_phase_async(p.k_src + (size_t)unit_local * p.P_max * kHeadDim, p.v_src + (size_t)unit_local * p.P_max * kHeadDim,
                        p.k_cache + (size_t)unit * p.C * kHeadDim, p.v_cache + (size_t)unit * p.C * kHeadDim, s_kept, rows, 0,
                        evict_smem + ring_offset, tid, n, p.status);
    __syncthreads();
    if (tid == 0) {   // the last CTA of the sequence publishes its length and the rows that carry history
        const int prev = atomicAdd(&p.seq_done[lseq_global], 1);
        if (prev == p.h_kv - 1) {
            p.seq_done[lseq_global] = 0;
            p.len[lseq_global] = rows;
            p.len[(size_t)p.L_total * p.batch + lseq_global] = compress ? n_keep : 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The same step as separate launches (timed one by one); they hand over through the workspace.
__global__ void __launch_bounds__(kEvictThreads) gkv_evict_merge_kernel(const EvictLaunch p) {
    extern __shared__ __align__(128) uint8_t evict_smem[];
    float* s_f; int* s_kept; int* s_pos; EvictShared* sh; float* s_sel; int* s_evict;
    carve(evict_smem, p, &s_f, &s_kept, &s_pos, &sh, &s_sel, &s_evict);
    const int tid = threadIdx.x;
    const UnitIndex u = unit_of(p, blockIdx.x);
    const int n = p.len[u.lseq_global];
    const int n_h = p.len[(size_t)p.L_total * p.batch + u.lseq_global];
    if (n <= p.b || p.policy == GKV_POLICY_STREAMING) return;   // (the policy without a score has nothing to merge)
    const int n_c = n - p.w;
    merge_phase(p.sacc + (size_t)u.unit * p.C, p.f + (size_t)u.unit * p.C, s_f, n_c, n_h, p.alpha, p.mode, sh, tid);
    float* out = p.f_ws + (size_t)u.unit_local * p.C;
    for (int t = tid; t < n_c; t += kEvictThreads) out[t] = s_f[t];
    if (has_selection_terms(p)) {
        selection_scores(p, u.unit, s_f, s_sel, n, n_c, sh, tid);
        float* out2 = p.fsel_ws + (size_t)u.unit_local * p.C;
        for (int t = tid; t < n_c; t += kEvictThreads) out2[t] = s_sel[t];
    }
}

__global__ void __launch_bounds__(kEvictThreads) gkv_evict_select_kernel(const EvictLaunch p) {
    extern __shared__ __align__(128) uint8_t evict_smem[];
    float* s_f; int* s_kept; int* s_pos; EvictShared* sh; float* s_sel; int* s_evict;
    carve(evict_smem, p, &s_f, &s_kept, &s_pos, &sh, &s_sel, &s_evict);
    const int tid = threadIdx.x;
    const UnitIndex u = unit_of(p, blockIdx.x);
    const int n = p.len[u.lseq_global];
    if (n <= p.b) {
        float* sacc = p.sacc + (size_t)u.unit * p.C;
        for (int t = tid; t < p.C; t += kEvictThreads) sacc[t] = 0.f;
        return;
    }
    const int n_c = n - p.w;
    if (tid == 0) sh->status = p.status;
    if (p.policy == GKV_POLICY_STREAMING) {
        streaming_phase(s_f, s_kept, s_evict, n, n_c, p.b, p.n_sink, tid);
    } else {
        const float* in = p.f_ws + (size_t)u.unit_local * p.C;
        for (int t = tid; t < n_c; t += kEvictThreads) s_f[t] = in[t];
        if (has_selection_terms(p)) {
            const float* in2 = p.fsel_ws + (size_t)u.unit_local * p.C;
            for (int t = tid; t < n_c; t += kEvictThreads) s_sel[t] = in2[t];
        }
        __syncthreads();
        select_phase(s_sel, s_kept, s_evict, n_c, p.b - p.w, p.w, sh, tid);
    }
    write_score_state(p, u, s_f, s_kept, s_pos, s_evict, n, tid);
    int32_t* kw = p.kept_ws + (size_t)u.unit_local * p.b;
    for (int r = tid; r < p.b; r += kEvictThreads) kw[r] = s_kept[r];
}

// grid = units x slices: each CTA moves one column slice of every row of its unit.
__global__ void __launch_bounds__(kEvictThreads) gkv_evict_compact_kernel(const EvictLaunch p, int slices) {
    extern __shared__ __align__(128) uint8_t evict_smem[];
    float* s_f; int* s_kept; int* s_pos; EvictShared* sh; float* s_sel; int* s_evict;
    carve(evict_smem, p, &s_f, &s_kept, &s_pos, &sh, &s_sel, &s_evict);
    const int tid = threadIdx.x;
    const int unit_local = blockIdx.x / slices, slice = blockIdx.x - unit_local * slices;
    const UnitIndex u = unit_of(p, unit_local);
    const int n = p.len[u.lseq_global];
    if (n <= p.b) return;
    if (tid == 0) sh->first_evicted = p.b;
    __syncthreads();
    const int32_t* kw = p.kept_ws + (size_t)unit_local * p.b;
    int first = p.b;
    for (int r = tid; r < p.b; r += kEvictThreads) {
        const int s = kw[r];
        s_kept[r] = s;
        if (s != r) first = min(first, r);
    }
    if (first < p.b) atomicMin(&sh->first_evicted, first);
    __syncthreads();
    const int cpr = 16 / slices;
    compact_phase(p.k_cache + (size_t)u.unit * p.C * kHeadDim, p.v_cache + (size_t)u.unit * p.C * kHeadDim, s_kept,
                  p.b, sh->first_evicted, slice * cpr, cpr, tid, n, p.status);
    publish_state(p, u, p.h_kv * slices, sh, tid);
}

// ---------------------------------------------------------------------------------------------
static cudaError_t ensure_smem(const void* fn, size_t bytes) {
    if (bytes <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Launch shape of the fused kernel. Ring depth: the one that keeps the most groups of loads in flight per SM
// (resident CTAs x (stages - 2)); among equals the one with more CTAs, whose selection phases then hide each other.
// Grid: persistent, at most the resident CTAs; with three rounds of units or fewer the rounds are filled equally
// (512 units on 296 slots run as 256 CTAs x 2 units: a unit cannot be split, and a CTA holding two units next to
// CTAs holding one sets the end of the launch).
void evict_plan(const EvictLaunch& p, int* stages, int* grid, size_t* smem, int* ctas_per_sm) {
    const FusedLayout lay = fused_layout(p.C, p.b, p.cbar != nullptr || p.pool_kernel > 1, p.pos != nullptr, p.evict_log != nullptr);
    auto ctas_with = [&](int st) {
        const int by_smem = (int)((227 * 1024) / ((size_t)lay.ring + (size_t)st * kCopyStageBytes + 1024));
        return by_smem > 5 ? 5 : by_smem;
    };
    int st = 3, best = -1;
    for (int c = 3; c <= kFusedMaxStages; ++c) {
        const int score = ctas_with(c) * (c - 2) * 8 + ctas_with(c);
        if (ctas_with(c) >= 1 && score > best) { best = score; st = c; }
    }
    const int sm = p.sm_count > 0 ? p.sm_count : 148;
    const long total = (long)p.n_layers * p.batch * p.h_kv;
    const long resident = (long)max(1, ctas_with(st)) * sm;
    long g = total < resident ? total : resident;
    if (total > resident) {
        const long rounds = (total + resident - 1) / resident;
        if (rounds <= 3) g = (total + rounds - 1) / rounds;
    }
    *stages = st;
    *grid = (int)g;
    *smem = (size_t)lay.ring + (size_t)st * kCopyStageBytes;
    if (ctas_per_sm) *ctas_per_sm = max(1, ctas_with(st));
}

cudaError_t launch_evict_fused(const EvictLaunch& p, cudaStream_t s) {
    int stages, grid;
    size_t smem;
    evict_plan(p, &stages, &grid, &smem, nullptr);
    cudaError_t e = ensure_smem((const void*)gkv_evict_fused_kernel, smem);
    if (e != cudaSuccess) return e;
    gkv_evict_fused_kernel<<<grid, kFusedThreads, smem, s>>>(p, stages);
    return cudaGetLastError();
}
cudaError_t launch_prompt_compress(const PromptLaunch& p, cudaStream_t s) {
    const size_t scores = p.f_long ? 0 : sizeof(float) * p.P_max * ((p.pool_kernel > 1 || p.cbar) ? 2 : 1);
    const size_t state = sizeof(EvictShared) + scores + sizeof(int) * p.b;
    const size_t ring = (state + 127) & ~size_t(127);
    const size_t smem = ring + kCopyRingBytes;
    cudaError_t e = ensure_smem((const void*)gkv_prompt_compress_kernel, smem);
    if (e != cudaSuccess) return e;
    gkv_prompt_compress_kernel<<<p.batch * p.h_kv, kEvictThreads, smem, s>>>(p, (int)ring);
    return cudaGetLastError();
}
cudaError_t launch_evict_merge(const EvictLaunch& p, cudaStream_t s) {
    const size_t smem = evict_smem_bytes(p);
    cudaError_t e = ensure_smem((const void*)gkv_evict_merge_kernel, smem);
    if (e != cudaSuccess) return e;
    gkv_evict_merge_kernel<<<p.n_layers * p.batch * p.h_kv, kEvictThreads, smem, s>>>(p);
    return cudaGetLastError();
}
cudaError_t launch_evict_select(const EvictLaunch& p, cudaStream_t s) {
    const size_t smem = evict_smem_bytes(p);
    cudaError_t e = ensure_smem((const void*)gkv_evict_select_kernel, smem);
    if (e != cudaSuccess) return e;
    gkv_evict_select_kernel<<<p.n_layers * p.batch * p.h_kv, kEvictThreads, smem, s>>>(p);
    return cudaGetLastError();
}
cudaError_t launch_evict_compact(const EvictLaunch& p, int sm_count, cudaStream_t s) {
    const size_t smem = evict_smem_bytes(p);
    cudaError_t e = ensure_smem((const void*)gkv_evict_compact_kernel, smem);
    if (e != cudaSuccess) return e;
    const int units = p.n_layers * p.batch * p.h_kv;
    int slices = 1;
    while (slices < 16 && units * slices < 4 * sm_count) slices <<= 1;  // column slices for small batches
    gkv_evict_compact_kernel<<<units * slices, kEvictThreads, smem, s>>>(p, slices);
    return cudaGetLastError();
}

}  // namespace gkv
