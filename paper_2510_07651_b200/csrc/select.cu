// Pooling + per-head top-budget selection + ordered index emission (Algorithm 2: the num_hh best
// candidates below the cutoff, their indices ascending), and the row gather that builds the compacted cache.
//
//   select_cluster_kernel  one thread-block cluster per (batch item, KV head).  Every CTA pools
//                     its contiguous share of the candidates into order-preserving uint32 keys
//                     held in shared memory; three radix passes (11 + 11 + 10 bits) whose
//                     histograms are summed in the leading CTA's shared memory find the key of
//                     the n_hh-th largest candidate and how many of its ties are kept; the
//                     CTAs exchange their counts and emit the kept indices in ascending order
//   pool_key_kernel + select_kernel   the same selection with one CTA per head and the keys in
//                     global memory: the path for sequences too long for a cluster's shared memory
//   gather_kernel     16-byte vector copy of the kept K/V rows (and optionally their scores)
#include "obc_common.cuh"

#include <cooperative_groups.h>
#include <mutex>
namespace cg = cooperative_groups;

namespace obc {

namespace {

// fp32 -> uint32 whose unsigned order equals the float order; -0.0 is folded onto +0.0
__device__ __forceinline__ uint32_t float_key(float x) {
    uint32_t u = __float_as_uint(x + 0.0f);          // -0.0 + 0.0 = +0.0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ int seq_len(const SelectShape& s, int b) { return s.seq_lens ? s.seq_lens[b] : s.Nmax; }
__device__ __forceinline__ int budget_of(const SelectShape& s, int b) { return s.budgets ? s.budgets[b] : s.budget; }

__global__ void __launch_bounds__(256)
pool_key_kernel(SelectShape s, const float* __restrict__ scores, uint32_t* __restrict__ keys) {
    pdl_wait();
    const int unit = blockIdx.y, b = unit / s.Hkv;
    const int N = seq_len(s, b), lo = s.n_sink, hi = N - s.n_recent;
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= s.Nmax) return;
    const float* sc = scores + (size_t)unit * s.Nmax;
    uint32_t key = 0;
    if (p >= lo && p < hi) {
        float val;
        const int half = s.pool_kernel / 2;
        if (s.pool_mode == OBC_POOL_NONE || s.pool_kernel == 1) {
            val = sc[p];
        } else if (s.pool_mode == OBC_POOL_MAX) {
            val = -INFINITY;
            for (int t = p - half; t <= p + half; ++t)
                if (t >= lo && t < hi) val = fmaxf(val, sc[t]);
        } else {
            val = 0.f;
            for (int t = p - half; t <= p + half; ++t)
                if (t >= lo && t < hi) val = __fadd_rn(val, sc[t]);
            val = __fdiv_rn(val, (float)s.pool_kernel);
        }
        key = float_key(val);
    }
    keys[(size_t)unit * s.Nmax + p] = key;
}

constexpr int SEL_NT = 1024;

__global__ void __launch_bounds__(SEL_NT)
select_kernel(SelectShape s, const uint32_t* __restrict__ keys_all, int32_t* __restrict__ idx_all) {
    pdl_wait();
    __shared__ uint32_t hist[256];
    __shared__ uint32_t sh_prefix, sh_remaining;
    __shared__ uint32_t warp_gt[32], warp_eq[32];

    const int unit = blockIdx.x, b = unit / s.Hkv;
    const int N = seq_len(s, b), budget = budget_of(s, b);
    const int lo = s.n_sink, hi = N - s.n_recent, n = hi - lo;
    const int n_hh = budget - s.n_sink - s.n_recent;
    const uint32_t* keys = keys_all + (size_t)unit * s.Nmax;
    int32_t* idx = idx_all + (size_t)unit * s.idx_stride;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (n_hh < 0 || n_hh > n || budget > s.idx_stride || N > s.Nmax || hi < lo) {   // bad per-sequence budget
        for (int j = tid; j < s.idx_stride; j += SEL_NT) idx[j] = -1;
        return;
    }
    // protected ranges and padding
    for (int j = tid; j < s.n_sink; j += SEL_NT) idx[j] = j;
    for (int j = tid; j < s.n_recent; j += SEL_NT) idx[s.n_sink + n_hh + j] = hi + j;
    for (int j = budget + tid; j < s.idx_stride; j += SEL_NT) idx[j] = -1;
    if (n_hh == 0) return;

    // ---- radix search for the key T of the n_hh-th largest candidate -----------------------
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)n_hh;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int base = 0; base < n; base += SEL_NT) {
            const int i = base + tid;
            const bool in = i < n;
            const uint32_t key = in ? keys[lo + i] : 0u;
            const bool pred = in && ((key & mask) == prefix);
            const unsigned act = __ballot_sync(0xffffffffu, pred);
            if (pred) {
                const uint32_t dgt = (key >> shift) & 255u;
                const unsigned peers = __match_any_sync(act, dgt);
                if (lane == __ffs(peers) - 1) atomicAdd(&hist[dgt], (uint32_t)__popc(peers));
            }
        }
        __syncthreads();
        if (warp == 0) {
            // lane owns bins [8*lane, 8*lane+8); find the highest bin D with
            // count(bins > D) < remaining <= count(bins >= D)
            uint32_t loc[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { loc[j] = hist[lane * 8 + j]; tot += loc[j]; }
            uint32_t above = 0;                                  // sum over lanes > lane
            uint32_t incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t t = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += t;
            }
            above = incl - tot;
            if (above < remaining && remaining <= above + tot) {
                uint32_t run = above;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (run < remaining && remaining <= run + loc[j]) {
                        sh_prefix = prefix | ((uint32_t)(lane * 8 + j) << shift);
                        sh_remaining = remaining - run;
                        run = 0xffffffffu;                       // found: stop matching
                    } else if (run != 0xffffffffu) {
                        run += loc[j];
                    }
                }
            }
        }
        __syncthreads();
        prefix = sh_prefix; remaining = sh_remaining; mask |= 255u << shift;
        __syncthreads();
    }
    const uint32_t T = prefix, k_eq = remaining;      // keep all keys > T and the first k_eq keys == T

    // ---- ordered emission: each warp owns a contiguous segment of the candidates -----------
    const int seg = ((n + 31) / 32 + 31) / 32 * 32;
    const int s0 = warp * seg, s1 = min(s0 + seg, n);
    uint32_t cgt = 0, ceq = 0;
    for (int i = s0 + lane; i < s1; i += 32) {
        const uint32_t key = keys[lo + i];
        cgt += key > T; ceq += key == T;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cgt += __shfl_xor_sync(0xffffffffu, cgt, o);
        ceq += __shfl_xor_sync(0xffffffffu, ceq, o);
    }
    if (lane == 0) { warp_gt[warp] = cgt; warp_eq[warp] = ceq; }
    __syncthreads();
    uint32_t gt_before = 0, eq_before = 0;
    for (int w = 0; w < warp; ++w) { gt_before += warp_gt[w]; eq_before += warp_eq[w]; }
    uint32_t eq_run = eq_before;
    uint32_t out = s.n_sink + gt_before + min(eq_before, k_eq);
    const unsigned lt_mask = (1u << lane) - 1u;
    for (int base = s0; base < s1; base += 32) {
        const int i = base + lane;
        const uint32_t key = i < s1 ? keys[lo + i] : 0u;
        const bool is_eq = i < s1 && key == T;
        const unsigned beq = __ballot_sync(0xffffffffu, is_eq);
        const bool sel = i < s1 && (key > T || (is_eq && eq_run + __popc(beq & lt_mask) < k_eq));
        const unsigned bsel = __ballot_sync(0xffffffffu, sel);
        if (sel) idx[out + __popc(bsel & lt_mask)] = lo + i;
        out += __popc(bsel);
        eq_run += __popc(beq);
    }
}

// ---- cluster path ----------------------------------------------------------------------------
constexpr int CL_NT = 512;                    // threads per CTA
constexpr int CL_BINS = 2048;                 // 11-bit digits
constexpr int CL_MAX_SEG = 20 * 1024;         // candidates per CTA (two 4-byte shared arrays of this size)

constexpr int CL_GATHER = 2 * CL_BINS;        // survivors of the first pass that every CTA can hold (all CTAs' lists together):
                                              // they lie over the histograms of passes 1 and 2, which are used only when the lists do not fit

struct ClusterShared {                        // fixed part of the CTA's shared memory
    uint32_t sum[3][CL_BINS];                 // per radix pass: histogram of the whole head (every CTA adds into every copy)
    uint32_t local[CL_BINS];                  // this CTA's histogram of the current pass
    uint32_t found[2];                        // result of a pass: prefix, remaining
    uint32_t n_list;                          // candidates of this CTA that survive the first pass
    uint32_t rank_gt[16], rank_eq[16];        // kept-candidate counts of every CTA of the cluster
    uint32_t rank_list[16], rank_above[16];   // per CTA: survivors of the first pass, candidates in higher bins
    uint32_t before[2];                       // kept candidates (greater, equal) in the CTAs before this one
    uint32_t warp_gt[CL_NT / 32], warp_eq[CL_NT / 32];
    uint32_t scan[CL_NT / 32];
    // slot r of the gathered lists: the survivors of CTA r (CL_GATHER / C keys each), in the space of sum[1] and sum[2]
    __device__ __forceinline__ uint32_t* gathered() { return &sum[1][0]; }
};

// The highest bin D of hist[0 .. CL_BINS) with count(bins > D) < remaining <= count(bins >= D), found by the
// whole CTA (thread t owns bins [4t, 4t+4)); found[0] = D, found[1] = remaining - count(bins > D).
__device__ __forceinline__ void find_bin(const uint32_t* hist, uint32_t remaining, uint32_t* scan, uint32_t* found) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t loc[4], tot = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) { loc[j] = hist[tid * 4 + j]; tot += loc[j]; }
    uint32_t incl = tot;                           // suffix sum over the lanes >= lane
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += t;
    }
    if (lane == 0) scan[warp] = incl;
    __syncthreads();
    uint32_t wsum = lane < CL_NT / 32 ? scan[lane] : 0u;          // suffix sum over the warps > warp
#pragma unroll
    for (int o = 1; o < CL_NT / 32; o <<= 1) {
        const uint32_t t = __shfl_down_sync(0xffffffffu, wsum, o);
        if (lane + o < CL_NT / 32) wsum += t;
    }
    const uint32_t above_warps = __shfl_sync(0xffffffffu, wsum, min(warp + 1, 31));
    const uint32_t above = incl - tot + (warp + 1 < CL_NT / 32 ? above_warps : 0u);
    if (above < remaining && remaining <= above + tot) {
        uint32_t run = above;
#pragma unroll
        for (int j = 3; j >= 0; --j) {
            if (run != 0xffffffffu) {
                if (remaining <= run + loc[j]) {
                    found[0] = (uint32_t)(tid * 4 + j);
                    found[1] = remaining - run;
                    run = 0xffffffffu;
                } else {
                    run += loc[j];
                }
            }
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(CL_NT)
select_cluster_kernel(SelectShape s, const float* __restrict__ scores, int32_t* __restrict__ idx_all, int seg_cap,
                      const uint32_t* __restrict__ keys_in) {
    extern __shared__ __align__(16) uint8_t sel_smem[];
    ClusterShared& sh = *reinterpret_cast<ClusterShared*>(sel_smem);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sel_smem + ((sizeof(ClusterShared) + 15) & ~(size_t)15));   // 16-byte aligned
    float* stage = reinterpret_cast<float*>(keys + seg_cap);          // seg_cap + pool_kernel - 1 floats

    pdl_wait();
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int unit = blockIdx.x / C, b = unit / s.Hkv;
    const int N = seq_len(s, b), budget = budget_of(s, b);
    const int lo = s.n_sink, hi = N - s.n_recent, n = hi - lo;
    const int n_hh = budget - s.n_sink - s.n_recent;
    int32_t* idx = idx_all + (size_t)unit * s.idx_stride;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gtid = rank * CL_NT + tid, gthreads = C * CL_NT;

    // these tests depend on the unit only, so all CTAs of the cluster leave together
    if (n_hh < 0 || n_hh > n || budget > s.idx_stride || N > s.Nmax || hi < lo) {   // bad per-sequence budget
        for (int j = gtid; j < s.idx_stride; j += gthreads) idx[j] = -1;
        return;
    }
    for (int j = gtid; j < s.n_sink; j += gthreads) idx[j] = j;
    for (int j = gtid; j < s.n_recent; j += gthreads) idx[s.n_sink + n_hh + j] = hi + j;
    for (int j = budget + gtid; j < s.idx_stride; j += gthreads) idx[j] = -1;
    if (n_hh == 0) return;

    // ---- this CTA's share of the candidates: [c0, c1) of [0, n) --------------------------------
    const int seg = ((n + C - 1) / C + 31) / 32 * 32;
    const int c0 = min(rank * seg, n), c1 = min(c0 + seg, n), m = c1 - c0;
    if (tid == 0) sh.n_list = 0;
    if (keys_in) for (int i = tid; i < 4 * CL_BINS; i += CL_NT) (&sh.sum[0][0])[i] = 0;   // sum[3][] and local[]

    if (keys_in) {                                 // the caller has the (pooled) keys already: [units][Nmax]
        const uint32_t* kin = keys_in + (size_t)unit * s.Nmax + lo + c0;
        for (int i = tid; i < m; i += CL_NT) keys[i] = kin[i];
        __syncthreads();
        cluster.barrier_arrive();
    } else {
        // pooled keys: stage the scores with their halo, then pool out of shared memory
        const float* sc = scores + (size_t)unit * s.Nmax;
        const int half = (s.pool_mode == OBC_POOL_NONE) ? 0 : s.pool_kernel / 2;
        const float pad = s.pool_mode == OBC_POOL_MAX ? -INFINITY : 0.f;
        // nine loads in flight per thread: a share of 4096 candidates and its halo travel in one round trip
        constexpr int LD = 9;
        for (int base = 0; base < m + 2 * half; base += LD * CL_NT) {
            float val[LD];
    #pragma unroll
            for (int u = 0; u < LD; ++u) {
                const int i = base + u * CL_NT + tid, p = lo + c0 + i - half;
                val[u] = (i < m + 2 * half && p >= lo && p < hi) ? sc[p] : pad;
            }
            if (base == 0)                             // the histograms are cleared while the loads travel
                for (int i = tid; i < 4 * CL_BINS; i += CL_NT) (&sh.sum[0][0])[i] = 0;   // sum[3][] and local[]
    #pragma unroll
            for (int u = 0; u < LD; ++u) {
                const int i = base + u * CL_NT + tid;
                if (i < m + 2 * half) stage[i] = val[u];
            }
        }
        if (m + 2 * half <= 0)                         // a CTA without candidates issued no loads above
            for (int i = tid; i < 4 * CL_BINS; i += CL_NT) (&sh.sum[0][0])[i] = 0;
        __syncthreads();
        cluster.barrier_arrive();                      // this CTA's histograms are clear: others may add to them after their wait
        for (int i = tid; i < m; i += CL_NT) {
            float val;
            if (half == 0) {
                val = stage[i];
            } else if (half <= 3) {                    // kernels up to 7: all taps read before they are combined
                float tap[7];
    #pragma unroll
                for (int t = 0; t < 7; ++t) tap[t] = t <= 2 * half ? stage[i + t] : pad;
                if (s.pool_mode == OBC_POOL_MAX) {
                    val = -INFINITY;
    #pragma unroll
                    for (int t = 0; t < 7; ++t) val = fmaxf(val, tap[t]);      // padding taps are -inf
                } else {                               // taps in ascending index order; padding adds +0
                    val = 0.f;
    #pragma unroll
                    for (int t = 0; t < 7; ++t) if (t <= 2 * half) val = __fadd_rn(val, tap[t]);
                    val = __fdiv_rn(val, (float)s.pool_kernel);
                }
            } else if (s.pool_mode == OBC_POOL_MAX) {
                val = -INFINITY;
                for (int t = 0; t <= 2 * half; ++t) val = fmaxf(val, stage[i + t]);
            } else {
                val = 0.f;
                for (int t = 0; t <= 2 * half; ++t) val = __fadd_rn(val, stage[i + t]);
                val = __fdiv_rn(val, (float)s.pool_kernel);
            }
            keys[i] = float_key(val);
        }
    }
    // (the first cluster barrier is split: arrival above, once this CTA's histograms were clear; the wait comes just
    // before the first remote additions, behind the pooling and the first local histogram)

    // ---- radix search for the key T of the n_hh-th largest candidate ---------------------------
    // Pass 0 histograms the top 11 bits of all keys of the CTA.  Every CTA adds its non-empty bins into the `sum`
    // copy of every CTA of the cluster, so that after one cluster barrier each CTA finds by itself the bin D that
    // holds the n_hh-th largest key.  The keys of bin D (a few hundred of a 32k-token head) are copied to a list,
    // and every CTA hands its list, and how many of its candidates lie in the bins above D, to all the others:
    // after a second barrier each CTA settles the remaining 21 bits on its own copy of all the lists and knows
    // what the CTAs before it keep, without further exchanges.  Only when the lists do not fit their slots (keys
    // that all but coincide) do passes 1 and 2 run across the cluster as pass 0 did.
    uint32_t* list = reinterpret_cast<uint32_t*>(stage);
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)n_hh;
    const int slot_cap = CL_GATHER / C;
    bool gathered_path = false;
    for (int ps = 0; ps < 3 && !gathered_path; ++ps) {
        const int shift = ps == 0 ? 21 : ps == 1 ? 10 : 0;
        const uint32_t dmask = ps == 2 ? 1023u : 2047u;
        const uint32_t* src = ps == 0 ? keys : list;
        const int cnt = ps == 0 ? m : (int)sh.n_list;
        for (int base = 0; base < cnt; base += CL_NT) {
            const int i = base + tid;
            const bool pred = i < cnt && (ps < 2 || (src[i] & mask) == prefix);   // the list holds pass 0's bin only
            if (pred) atomicAdd(&sh.local[(src[i] >> shift) & dmask], 1u);
        }
        __syncthreads();
        if (ps == 0) cluster.barrier_wait();       // every CTA of the cluster runs and has cleared its histograms
        for (int bin = tid; bin < CL_BINS; bin += CL_NT) {
            const uint32_t c = sh.local[bin];
            if (c) for (int r = 0; r < C; ++r) atomicAdd(cluster.map_shared_rank(&sh.sum[ps][bin], r), c);
        }
        cluster.sync();                            // every copy of sum[ps] holds the whole head
        find_bin(sh.sum[ps], remaining, sh.scan, sh.found);
        const uint32_t digit = sh.found[0];
        remaining = sh.found[1];
        prefix |= digit << shift; mask |= dmask << shift;
        if (ps == 0) {
            // survivors of the first pass -> list (any order); candidates of this CTA in the bins above D
            uint32_t above = 0;
            for (int bin = (int)digit + 1 + tid; bin < CL_BINS; bin += CL_NT) above += sh.local[bin];
            for (int i = tid; i < m; i += CL_NT) {        // survivors are few: one shared-memory atomic each
                const uint32_t key = keys[i];
                if ((key & mask) == prefix) list[atomicAdd(&sh.n_list, 1u)] = key;
            }
            if (tid < 2) sh.before[tid] = 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) above += __shfl_xor_sync(0xffffffffu, above, o);
            if (lane == 0) sh.scan[warp] = above;
            __syncthreads();                       // the list and its length are complete
            const int nl = (int)sh.n_list;
            if (tid < C) {                         // length and higher-bin count into every CTA
                uint32_t ab = 0;
                for (int w = 0; w < CL_NT / 32; ++w) ab += sh.scan[w];
                cluster.map_shared_rank(&sh.rank_list[0], tid)[rank] = (uint32_t)nl;
                cluster.map_shared_rank(&sh.rank_above[0], tid)[rank] = ab;
            }
            if (nl <= slot_cap)                    // the keys themselves, into slot `rank` of every CTA (warp w serves CTA w mod C)
                for (int r = warp % C; r < C; r += CL_NT / 32) {
                    uint32_t* dst = cluster.map_shared_rank(sh.gathered(), r) + rank * slot_cap;
                    const int step = (CL_NT / 32 >= C ? CL_NT / 32 / C : 1) * 32;
                    for (int i = (CL_NT / 32 >= C ? warp / C : 0) * 32 + lane; i < nl; i += step) dst[i] = list[i];
                }
            for (int bin = tid; bin < CL_BINS; bin += CL_NT) sh.local[bin] = 0;
            cluster.sync();                        // lists and counts have arrived everywhere
            bool fits = true;
            for (int r = 0; r < C; ++r) fits = fits && (int)sh.rank_list[r] <= slot_cap;   // the same answer in every CTA
            if (fits) {
                // ---- the remaining 21 bits, on this CTA's copy of all lists (no cluster traffic) ----
                for (int half_pass = 0; half_pass < 2; ++half_pass) {
                    const int sh2 = half_pass == 0 ? 10 : 0;
                    const uint32_t dm2 = half_pass == 0 ? 2047u : 1023u;
                    for (int r = warp % C; r < C; r += CL_NT / 32) {          // warp w reads slot w mod C
                        const int nr = (int)sh.rank_list[r];
                        const uint32_t* g = sh.gathered() + r * slot_cap;
                        const int step = (CL_NT / 32 >= C ? CL_NT / 32 / C : 1) * 32;
                        for (int i = (CL_NT / 32 >= C ? warp / C : 0) * 32 + lane; i < nr; i += step)
                            if ((g[i] & mask) == prefix) atomicAdd(&sh.local[(g[i] >> sh2) & dm2], 1u);
                    }
                    __syncthreads();
                    find_bin(sh.local, remaining, sh.scan, sh.found);
                    prefix |= sh.found[0] << sh2; mask |= dm2 << sh2; remaining = sh.found[1];
                    if (half_pass == 0) {
                        for (int bin = tid; bin < CL_BINS; bin += CL_NT) sh.local[bin] = 0;
                        __syncthreads();
                    }
                }
                // what the CTAs before this one keep: their candidates above bin D, and of their lists the keys > T, == T
                uint32_t bg = 0, be = 0;
                if (tid < rank) bg = sh.rank_above[tid];
                for (int r = warp % C; r < rank; r += CL_NT / 32) {
                    const int nr = (int)sh.rank_list[r];
                    const uint32_t* g = sh.gathered() + r * slot_cap;
                    const int step = (CL_NT / 32 >= C ? CL_NT / 32 / C : 1) * 32;
                    for (int i = (CL_NT / 32 >= C ? warp / C : 0) * 32 + lane; i < nr; i += step) { bg += g[i] > prefix; be += g[i] == prefix; }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    bg += __shfl_xor_sync(0xffffffffu, bg, o);
                    be += __shfl_xor_sync(0xffffffffu, be, o);
                }
                if (lane == 0 && (bg | be)) { atomicAdd(&sh.before[0], bg); atomicAdd(&sh.before[1], be); }
                gathered_path = true;              // leaves the pass loop; the barrier below publishes `before`
            } else {
                // the exchanged passes 1 and 2 add into the histograms that the lists have overwritten: clear them
                // everywhere before any CTA adds to another's copy
                for (int i = tid; i < 2 * CL_BINS; i += CL_NT) sh.gathered()[i] = 0;
                cluster.sync();
            }
        } else {
            for (int bin = tid; bin < CL_BINS; bin += CL_NT) sh.local[bin] = 0;
        }
        __syncthreads();
    }
    const uint32_t T = prefix, k_eq = remaining;   // keep all keys > T and the first k_eq keys == T

    // ---- ordered emission: each warp owns a contiguous run of this CTA's candidates, in blocks of 256 keys of
    // which a lane holds eight consecutive ones (two 16-byte reads) ------------------------------------------------
    const int wseg = ((m + CL_NT / 32 - 1) / (CL_NT / 32) + 255) / 256 * 256;
    const int s0 = min(warp * wseg, m), s1 = min(s0 + wseg, m);
    auto load8 = [&](int i, uint32_t (&k8)[8]) -> unsigned {           // returns the mask of keys that exist
        if (i + 8 <= s1) {
            const uint4 a = *reinterpret_cast<const uint4*>(keys + i), b = *reinterpret_cast<const uint4*>(keys + i + 4);
            k8[0] = a.x; k8[1] = a.y; k8[2] = a.z; k8[3] = a.w; k8[4] = b.x; k8[5] = b.y; k8[6] = b.z; k8[7] = b.w;
            return 0xffu;
        }
        unsigned have = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { const bool in = i + j < s1; k8[j] = in ? keys[i + j] : 0u; have |= (unsigned)in << j; }
        return have;
    };
    uint32_t cgt = 0, ceq = 0;
    for (int base = s0; base < s1; base += 256) {
        uint32_t k8[8];
        const unsigned have = load8(base + lane * 8, k8);
#pragma unroll
        for (int j = 0; j < 8; ++j) { cgt += ((have >> j) & 1u) && k8[j] > T; ceq += ((have >> j) & 1u) && k8[j] == T; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cgt += __shfl_xor_sync(0xffffffffu, cgt, o);
        ceq += __shfl_xor_sync(0xffffffffu, ceq, o);
    }
    if (lane == 0) { sh.warp_gt[warp] = cgt; sh.warp_eq[warp] = ceq; }
    __syncthreads();
    if (!gathered_path) {                          // the CTAs' totals were not derived from the lists: exchange them
        if (tid < C) {                             // this CTA's totals into every CTA of the cluster
            uint32_t tg = 0, te = 0;
            for (int w = 0; w < CL_NT / 32; ++w) { tg += sh.warp_gt[w]; te += sh.warp_eq[w]; }
            cluster.map_shared_rank(&sh.rank_gt[0], tid)[rank] = tg;
            cluster.map_shared_rank(&sh.rank_eq[0], tid)[rank] = te;
        }
        cluster.sync();
        if (tid == 0) {
            uint32_t bg = 0, be = 0;
            for (int r = 0; r < rank; ++r) { bg += sh.rank_gt[r]; be += sh.rank_eq[r]; }
            sh.before[0] = bg; sh.before[1] = be;
        }
        __syncthreads();
    }
    uint32_t gt_run = sh.before[0], eq_run = sh.before[1];             // kept candidates before the block at hand
    for (int w = 0; w < warp; ++w) { gt_run += sh.warp_gt[w]; eq_run += sh.warp_eq[w]; }
    for (int base = s0; base < s1; base += 256) {
        uint32_t k8[8];
        const int i = base + lane * 8;
        const unsigned have = load8(i, k8);
        uint32_t g = 0, e = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { g += ((have >> j) & 1u) && k8[j] > T; e += ((have >> j) & 1u) && k8[j] == T; }
        uint32_t gi = g, ei = e;                   // inclusive scans over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t tg = __shfl_up_sync(0xffffffffu, gi, o), te = __shfl_up_sync(0xffffffffu, ei, o);
            if (lane >= o) { gi += tg; ei += te; }
        }
        uint32_t eq_at = eq_run + ei - e;          // equal keys before this lane's first key: the first k_eq of them are kept
        uint32_t out = s.n_sink + gt_run + (gi - g) + min(eq_at, k_eq);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (!((have >> j) & 1u)) continue;
            if (k8[j] > T) idx[out++] = lo + c0 + i + j;
            else if (k8[j] == T) { if (eq_at < k_eq) idx[out++] = lo + c0 + i + j; ++eq_at; }
        }
        gt_run += __shfl_sync(0xffffffffu, gi, 31);
        eq_run += __shfl_sync(0xffffffffu, ei, 31);
    }
}

// four 16-byte vectors of K and of V per thread, all loads issued before the first store (`vecs`
// vectors per row; a thread's vectors are a quarter of the unit's vectors apart)
__global__ void __launch_bounds__(256)
gather_kernel(int units, int Hkv, int idx_stride, int vecs, int elem_bytes,
              TensorView k, TensorView v, TensorView ko, TensorView vo,
              const int32_t* __restrict__ idx, const float* __restrict__ s_in, float* __restrict__ s_out, int Nmax) {
    pdl_wait();
    const int unit = blockIdx.y, b = unit / Hkv, g = unit % Hkv;
    const int total = idx_stride * vecs, quarter = (total + 3) / 4;
    const int e0 = blockIdx.x * blockDim.x + threadIdx.x;
    if (e0 >= quarter) return;
    const size_t eb = (size_t)elem_bytes;
    const char* kb = (const char*)k.ptr + ((size_t)b * k.sb + (size_t)g * k.sh) * eb;
    const char* vb = (const char*)v.ptr + ((size_t)b * v.sb + (size_t)g * v.sh) * eb;
    char* kob = (char*)ko.ptr + ((size_t)b * ko.sb + (size_t)g * ko.sh) * eb;
    char* vob = (char*)vo.ptr + ((size_t)b * vo.sb + (size_t)g * vo.sh) * eb;
    int src[4], j[4], c[4];
    uint4 kv[4], vv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * quarter;
        j[u] = e / vecs; c[u] = e % vecs;
        src[u] = e < total ? idx[(size_t)unit * idx_stride + j[u]] : -1;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (src[u] >= 0) {
            kv[u] = __ldg(reinterpret_cast<const uint4*>(kb + (size_t)src[u] * k.st * eb) + c[u]);
            vv[u] = __ldg(reinterpret_cast<const uint4*>(vb + (size_t)src[u] * v.st * eb) + c[u]);
        }
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (src[u] >= 0) {
            reinterpret_cast<uint4*>(kob + (size_t)j[u] * ko.st * eb)[c[u]] = kv[u];
            reinterpret_cast<uint4*>(vob + (size_t)j[u] * vo.st * eb)[c[u]] = vv[u];
            if (s_in && c[u] == 0) s_out[(size_t)unit * idx_stride + j[u]] = s_in[(size_t)unit * Nmax + src[u]];
        }
}


// ---- head-adaptive budgets: pieces around the two selection kernels ------------------------------------
// keys of the tokens every head keeps by its own ranking are raised to the largest key, so that the
// ranking across heads takes them first
__global__ void __launch_bounds__(256)
adaptive_boost_kernel(int units, int Nmax, int n_sink, int n_safe, int safe_stride,
                      const int32_t* __restrict__ idx_safe, uint32_t* __restrict__ keys) {
    pdl_wait();
    const int unit = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (unit >= units || j >= n_safe) return;
    const int p = idx_safe[(size_t)unit * safe_stride + n_sink + j];
    if (p >= 0 && p < Nmax) keys[(size_t)unit * Nmax + p] = 0xffffffffu;
}

// vidx [B][total]: the tokens chosen across the heads of a batch item, ascending in h * Nmax + p.  One block
// per (b, h) finds its head's stretch by binary search and writes the head's row of idx: sinks, chosen
// tokens, recent tail, -1 padding; counts[b, h] = tokens kept (or -1, with a row of -1, when the row does
// not fit idx_stride or the budget does not fit the sequence).
// First position of the ascending array a[0, n) whose value is >= v (n if none), found by the whole block: every
// round the threads probe evenly spaced positions of the remaining range at once, so 16384 entries take three
// round trips to memory where a binary search by one thread takes fourteen.  Called by all threads of the block.
template <typename Less>
__device__ __forceinline__ int block_lower_bound(int n, Less value_below) {
    int lo = 0, hi = n;
    while (hi > lo) {
        const int step = (hi - lo + (int)blockDim.x - 1) / (int)blockDim.x;
        const int pos = lo + (int)threadIdx.x * step;
        const int cnt = __syncthreads_count(pos < hi && value_below(pos));   // the probes below v are a prefix
        if (cnt == 0) { hi = lo; }
        else { const int last = lo + (cnt - 1) * step; lo = last + 1; hi = min(last + step, hi); }
    }
    return lo;
}

__global__ void __launch_bounds__(256)
adaptive_split_kernel(SelectShape s, int total, const int32_t* __restrict__ vidx_all,
                      int32_t* __restrict__ idx_all, int32_t* __restrict__ counts) {
    pdl_wait();
    const int unit = blockIdx.x, b = unit / s.Hkv, h = unit % s.Hkv;
    const int N = seq_len(s, b), lo = s.n_sink, hi = N - s.n_recent;
    const int n_hh = s.budget - s.n_sink - s.n_recent;
    const int32_t* vidx = vidx_all + (size_t)b * total;
    int32_t* idx = idx_all + (size_t)unit * s.idx_stride;
    auto lower_bound = [&](int v) {                       // first position whose virtual index is >= v
        return block_lower_bound(total, [&](int i) { return vidx[i] < v; });
    };
    const int seg0 = lower_bound(h * s.Nmax), seg1 = lower_bound((h + 1) * s.Nmax), c = seg1 - seg0;
    const int kept = s.n_sink + c + s.n_recent;
    const bool bad = N > s.Nmax || hi < lo || n_hh < 0 || n_hh > hi - lo || kept > s.idx_stride;
    if (bad) {
        for (int j = threadIdx.x; j < s.idx_stride; j += blockDim.x) idx[j] = -1;
        if (threadIdx.x == 0) counts[unit] = -1;
        return;
    }
    for (int j = threadIdx.x; j < s.n_sink; j += blockDim.x) idx[j] = j;
    for (int j = threadIdx.x; j < c; j += blockDim.x) idx[s.n_sink + j] = vidx[seg0 + j] - h * s.Nmax;
    for (int j = threadIdx.x; j < s.n_recent; j += blockDim.x) idx[s.n_sink + c + j] = hi + j;
    for (int j = kept + threadIdx.x; j < s.idx_stride; j += blockDim.x) idx[j] = -1;
    if (threadIdx.x == 0) counts[unit] = kept;
}

// A token shard's share of the kept indices: row (b, h) of idx is ascending (padding -1 at the end), so the entries
// in [t0, t0 + n) are one stretch, found by binary search; written relative to the shard, padded with -1.
__global__ void __launch_bounds__(256)
shard_indices_kernel(int idx_stride, int t0, int n, const int32_t* __restrict__ idx_all,
                     int32_t* __restrict__ local_all, int32_t* __restrict__ counts) {
    pdl_wait();
    const int unit = blockIdx.x;
    const int32_t* idx = idx_all + (size_t)unit * idx_stride;
    int32_t* local = local_all + (size_t)unit * idx_stride;
    auto lower_bound = [&](int v) {                       // first entry >= v; the -1 padding counts as past every token
        return block_lower_bound(idx_stride, [&](int i) { const int x = idx[i]; return x >= 0 && x < v; });
    };
    const int seg0 = lower_bound(t0), seg1 = lower_bound(t0 + n), c = seg1 - seg0;
    for (int j = threadIdx.x; j < idx_stride; j += blockDim.x) local[j] = j < c ? idx[seg0 + j] - t0 : -1;
    if (threadIdx.x == 0) counts[unit] = c;
}

}  // namespace

obc_status launch_shard_indices(int units, int idx_stride, int t0, int n, const int32_t* idx, int32_t* local, int32_t* counts,
                                cudaStream_t stream) {
    ProfScope ps("shard_indices", stream);
    OBC_CUDA_TRY(launch_pdl(shard_indices_kernel, dim3((unsigned)units), dim3(256), 0, stream, 1, idx_stride, t0, n, idx, local, counts));
    return OBC_OK;
}

size_t select_workspace_bytes(int B, int Hkv, int Nmax) { return align_up((size_t)B * Hkv * Nmax * 4, 256); }

// Cluster size for the one-cluster-per-head path, or 0 when a head does not fit a cluster's shared memory.
static int select_cluster_size(int Nmax, int* seg_cap) {
    int C = 8;
    if ((Nmax + C - 1) / C > 8192) C = 16;
    const int seg = ((Nmax + C - 1) / C + 31) / 32 * 32;
    if (seg > CL_MAX_SEG) return 0;
    *seg_cap = seg;
    return C;
}

// keys_in: when given, [units][Nmax] keys that take the place of pooling `scores` (which may then be null);
// `ws` is then not written
static obc_status launch_select_impl(const SelectShape& s, const float* scores, const uint32_t* keys_in, int32_t* idx,
                                     void* ws, cudaStream_t stream);
obc_status launch_select(const SelectShape& s, const float* scores, int32_t* idx, void* ws, cudaStream_t stream) {
    return launch_select_impl(s, scores, nullptr, idx, ws, stream);
}
static obc_status launch_select_impl(const SelectShape& s, const float* scores, const uint32_t* keys_in, int32_t* idx,
                                     void* ws, cudaStream_t stream) {
    const int units = s.B * s.Hkv;
    int seg_cap = 0;
    const int C = select_cluster_size(s.Nmax, &seg_cap);
    if (C > 0) {
        const size_t smem = sizeof(ClusterShared) + (size_t)seg_cap * 8 + (size_t)s.pool_kernel * 4 + 16;
        OBC_CUDA_TRY(cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (C > 8) OBC_CUDA_TRY(cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)(units * C)); cfg.blockDim = dim3(CL_NT); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        // whether the device can host such a cluster depends on the cluster size and the shared memory alone: asked once
        // per (device, size, bytes) and remembered (the query costs as much host time as the launch)
        thread_local struct { int dev, C; size_t smem; int max_clusters; } seen[4] = {};
        thread_local int seen_next = 0;
        int dev = -1, max_clusters = -1;
        (void)cudaGetDevice(&dev);
        for (const auto& e : seen) if (e.C == C && e.smem == smem && e.dev == dev) max_clusters = e.max_clusters;
        if (max_clusters < 0) {
            if (cudaOccupancyMaxActiveClusters(&max_clusters, select_cluster_kernel, &cfg) != cudaSuccess) { max_clusters = 0; (void)cudaGetLastError(); }
            seen[seen_next] = {dev, C, smem, max_clusters};
            seen_next = (seen_next + 1) % 4;
        }
        if (max_clusters > 0) {
            { ProfScope ps("select_cluster", stream);
              OBC_CUDA_TRY(launch_pdl(select_cluster_kernel, dim3((unsigned)(units * C)), dim3(CL_NT), smem, stream, C, s, scores, idx, seg_cap, keys_in)); }
            return OBC_OK;
        }
        (void)cudaGetLastError();                  // the device cannot host such a cluster: one CTA per head
    }
    if (keys_in) {
        { ProfScope ps("select", stream); OBC_CUDA_TRY(launch_pdl(select_kernel, dim3(units), dim3(SEL_NT), 0, stream, 1, s, keys_in, idx)); }
        return OBC_OK;
    }
    uint32_t* keys = (uint32_t*)ws;
    { ProfScope ps("pool_key", stream); OBC_CUDA_TRY(launch_pdl(pool_key_kernel, dim3((s.Nmax + 255) / 256, units), dim3(256), 0, stream, 1, s, scores, keys)); }
    { ProfScope ps("select", stream); OBC_CUDA_TRY(launch_pdl(select_kernel, dim3(units), dim3(SEL_NT), 0, stream, 1, s, (const uint32_t*)keys, idx)); }
    return OBC_OK;
}

// ---- allocation-free variant: the key scratch is part of the library image -----------------------
// One key per score, shared by every call on the device (see obc_select_noalloc in obcache.h).
static __device__ __align__(256) uint32_t g_select_keys[OBC_SELECT_NOALLOC_MAX_KEYS];

// Device address of g_select_keys on the current device.  In host code the array's name only
// stands for the symbol; the address a kernel can use comes from the runtime, per device.
static obc_status select_static_keys(uint32_t** out) {
    constexpr int kMaxDev = 64;
    static std::mutex mu;
    static uint32_t* ptrs[kMaxDev] = {};
    int dev = 0;
    OBC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return OBC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!ptrs[dev]) {
        uint32_t* ptr = nullptr;
        OBC_CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_select_keys));
        if (!ptr) return OBC_ERR_CUDA;
        ptrs[dev] = ptr;
    }
    *out = ptrs[dev];
    return OBC_OK;
}

obc_status launch_select_static(const SelectShape& s, const float* scores, int32_t* idx, cudaStream_t stream) {
    const int units = s.B * s.Hkv;
    if ((long long)units * s.Nmax > (long long)OBC_SELECT_NOALLOC_MAX_KEYS) return OBC_ERR_CAPACITY;
    uint32_t* keys = nullptr;
    obc_status st = select_static_keys(&keys);
    if (st != OBC_OK) return st;
    // every key a head reads is written by pool_key_kernel of this call: nothing has to be cleared
    { ProfScope ps("pool_key", stream); OBC_CUDA_TRY(launch_pdl(pool_key_kernel, dim3((s.Nmax + 255) / 256, units), dim3(256), 0, stream, 1, s, scores, keys)); }
    { ProfScope ps("select", stream); OBC_CUDA_TRY(launch_pdl(select_kernel, dim3(units), dim3(SEL_NT), 0, stream, 1, s, (const uint32_t*)keys, idx)); }
    return OBC_OK;
}

obc_status launch_gather(int B, int Hkv, int idx_stride, int Nmax, int elem_bytes,
                         TensorView k, TensorView v, TensorView ko, TensorView vo, const int32_t* idx,
                         const float* s_in, float* s_out, cudaStream_t stream) {
    const int vecs = kD * elem_bytes / 16;
    const long long total = ((long long)idx_stride * vecs + 3) / 4;    // four vectors per thread
    {
        ProfScope ps("gather", stream);
        OBC_CUDA_TRY(launch_pdl(gather_kernel, dim3((unsigned)((total + 255) / 256), B * Hkv), dim3(256), 0, stream, 1,
                                B * Hkv, Hkv, idx_stride, vecs, elem_bytes, k, v, ko, vo, idx, s_in, s_out, Nmax));
    }
    return OBC_OK;
}

// ---- head-adaptive budgets -------------------------------------------------------------------------------
// workspace: pooled keys [units][Nmax] | every head's own selection [units][n_sink + n_safe + n_recent] |
// the selection across heads [B][Hkv * n_hh]
struct AdaptivePlan { size_t off_keys, off_safe, off_vidx, bytes; int safe_stride, total; };
static AdaptivePlan make_adaptive_plan(const SelectShape& s, int n_safe) {
    AdaptivePlan p{};
    const size_t units = (size_t)s.B * s.Hkv;
    const int n_hh = s.budget - s.n_sink - s.n_recent;
    p.safe_stride = s.n_sink + n_safe + s.n_recent;
    p.total = s.Hkv * (n_hh > 0 ? n_hh : 0);
    size_t off = 0;
    p.off_keys = off; off = align_up(off + units * s.Nmax * 4, 256);
    p.off_safe = off; off = align_up(off + units * (size_t)(p.safe_stride > 0 ? p.safe_stride : 1) * 4, 256);
    p.off_vidx = off; off = align_up(off + (size_t)s.B * (size_t)(p.total > 0 ? p.total : 1) * 4, 256);
    p.bytes = off;
    return p;
}
size_t select_adaptive_workspace_bytes(const SelectShape& s, int n_safe) { return make_adaptive_plan(s, n_safe).bytes; }

obc_status launch_select_adaptive(const SelectShape& s, int n_safe, const float* scores, int32_t* idx, int32_t* counts,
                                  void* ws, cudaStream_t stream) {
    const AdaptivePlan plan = make_adaptive_plan(s, n_safe);
    const int units = s.B * s.Hkv;
    uint32_t* keys = (uint32_t*)((char*)ws + plan.off_keys);
    int32_t* idx_safe = (int32_t*)((char*)ws + plan.off_safe);
    int32_t* vidx = (int32_t*)((char*)ws + plan.off_vidx);
    { ProfScope ps("pool_key", stream); OBC_CUDA_TRY(launch_pdl(pool_key_kernel, dim3((s.Nmax + 255) / 256, units), dim3(256), 0, stream, 1, s, scores, keys)); }
    if (n_safe > 0) {
        SelectShape own = s;                              // every head's own ranking, n_safe scored tokens each
        own.budget = s.n_sink + n_safe + s.n_recent; own.budgets = nullptr; own.idx_stride = plan.safe_stride;
        obc_status st = launch_select_impl(own, nullptr, keys, idx_safe, nullptr, stream);
        if (st != OBC_OK) return st;
        { ProfScope ps("adaptive_boost", stream);
          OBC_CUDA_TRY(launch_pdl(adaptive_boost_kernel, dim3((n_safe + 255) / 256, units), dim3(256), 0, stream, 1, units, s.Nmax, s.n_sink, n_safe, plan.safe_stride, (const int32_t*)idx_safe, keys)); }
    }
    if (plan.total > 0) {
        // all heads of a batch item as one sequence of Hkv * Nmax keys (the keys of protected and padding
        // positions are 0 and rank below every candidate); equal keys keep the lowest head, then the lowest index
        SelectShape all{s.B, 1, s.Hkv * s.Nmax, nullptr, plan.total, nullptr, plan.total, 0, 0, OBC_POOL_NONE, 1};
        obc_status st = launch_select_impl(all, nullptr, keys, vidx, nullptr, stream);
        if (st != OBC_OK) return st;
    }
    { ProfScope ps("adaptive_split", stream);
      OBC_CUDA_TRY(launch_pdl(adaptive_split_kernel, dim3(units), dim3(256), 0, stream, 1, s, plan.total, (const int32_t*)vidx, idx, counts)); }
    return OBC_OK;
}

}  // namespace obc
