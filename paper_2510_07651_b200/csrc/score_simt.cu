// CUDA-core (fp32 FMA) score kernels: the path for fp32 caches and for row counts too small or
// too irregular for the tensor-core kernels.  Two passes over K/V per (batch item, KV head):
//
//   pass 1  split-KV streaming softmax over the window rows: per split, running max / sum of
//           exp2 and the un-normalised partial output  (Sec. 3: A = softmax(QK^T/sqrt(d)), O = AV)
//   combine merges the splits into log2-sum-exp, O (fp32) and ||o_r||^2 per row
//   pass 2  recomputes the logits tile by tile together with v_p . o_r and folds the score
//           arithmetic of Eq. 4-6 (in the expanded form of Algorithm 1) and the sum over window
//           rows and the GQA group (App. A.5) into registers; one fp32 store per token and plane.
//
// No W x N matrix is written to global memory.
#include "obc_common.cuh"

namespace obc {

namespace {
constexpr int TN = 64;        // tokens per tile
constexpr int RC = 32;        // window rows per chunk (8 warps x 4 rows)
constexpr int KS = kD + 4;    // padded row stride (floats) of the token-major smem tiles
constexpr int NT = 256;

// A length read on the device cannot be checked by the host: it is clamped to [0, max_len] so that no row
// beyond the caller's buffers is ever addressed.
__device__ __forceinline__ int seq_len(const ScoreShape& s, int b) {
    return s.seq_lens ? min(max(s.seq_lens[b], 0), s.Nmax) : s.Nmax;
}
// length the causal mask counts from: the sequence's own length, or (token-sharded caches) the distance from the
// shard's first token to the end of the whole sequence
__device__ __forceinline__ int mask_len(const ScoreShape& s, int b) { return s.mask_lens ? s.mask_lens[b] : seq_len(s, b); }

template <typename T>
__device__ __forceinline__ const T* row_ptr(const TensorView& t, int b, int h, long long tok) {
    return reinterpret_cast<const T*>(t.ptr) + b * t.sb + h * t.sh + tok * t.st;
}

__device__ __forceinline__ float elem_to_float(float x) { return x; }
__device__ __forceinline__ float elem_to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// cooperative load of `rows` x 128 elements into fp32 smem (row stride `stride` floats);
// rows >= valid are zero-filled.  get(row) returns the global row pointer.
template <typename T, typename F>
__device__ __forceinline__ void load_rows(float* dst, int stride, int rows, int valid, F get) {
    for (int idx = threadIdx.x; idx < rows * (kD / 4); idx += NT) {
        int row = idx >> 5, c4 = idx & 31;
        float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < valid) f = load4<T>(get(row) + c4 * 4);
        *reinterpret_cast<float4*>(dst + row * stride + c4 * 4) = f;
    }
}

__device__ __forceinline__ float dot4(float4 a, float4 b, float acc) {
    acc = fmaf(a.x, b.x, acc); acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc); acc = fmaf(a.w, b.w, acc);
    return acc;
}

// acc[i][j] += sum_c A[(warp*4+i)][c] * Bt[(lane+32j)][c]   (A row stride kD, Bt row stride KS)
__device__ __forceinline__ void tile_gemm(const float* __restrict__ sA, const float* __restrict__ sB,
                                          int warp, int lane, float (&acc)[4][2]) {
#pragma unroll 4
    for (int c4 = 0; c4 < kD / 4; ++c4) {
        float4 b0 = *reinterpret_cast<const float4*>(sB + lane * KS + c4 * 4);
        float4 b1 = *reinterpret_cast<const float4*>(sB + (lane + 32) * KS + c4 * 4);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 a = *reinterpret_cast<const float4*>(sA + (warp * 4 + i) * kD + c4 * 4);
            acc[i][0] = dot4(a, b0, acc[i][0]);
            acc[i][1] = dot4(a, b1, acc[i][1]);
        }
    }
}

// ------------------------------------------------------------------------------------------ pass 1
template <typename T>
__global__ void __launch_bounds__(NT, 2)
simt_pass1_kernel(ScoreShape s, SimtPlan plan, TensorView q, TensorView k, TensorView v, float* ws) {
    pdl_wait();
    extern __shared__ __align__(16) float smem[];
    float* sK = smem;                       // [TN][KS]
    float* sV = sK + TN * KS;               // [TN][kD]
    float* sQ = sV + TN * kD;               // [RC][kD]
    float* sP = sQ + RC * kD;               // [RC][TN]

    const int split = blockIdx.x, unit = blockIdx.y, r0 = blockIdx.z * RC;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int N = seq_len(s, b);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float sl2 = s.scale * kLog2e;
    // the status word of the workspace header is only raised by the tensor-core kernels
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0)
        *reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(ws) + plan.off_flag) = 0u;

    load_rows<T>(sQ, kD, RC, min(RC, s.R - r0), [&](int row) {
        int r = r0 + row;
        return row_ptr<T>(q, b, g * s.G + r / s.W, r % s.W);
    });

    float m2[4], l[4], o[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m2[i] = -INFINITY; l[i] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) o[i][c] = 0.f;
    }
    long long last[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = r0 + warp * 4 + i;
        last[i] = (r < s.R) ? (s.causal ? min((long long)mask_len(s, b) - s.W + (r % s.W), (long long)N - 1) : (long long)N - 1) : -1;
    }

    const int tile_lo = split * plan.tiles_per_split;
    const int tile_hi = min(tile_lo + plan.tiles_per_split, (N + TN - 1) / TN);
    if (tile_lo >= (N + TN - 1) / TN) return;      // a split past the end of a shorter sequence: the merge does not read it
    for (int tile = tile_lo; tile < tile_hi; ++tile) {
        const int t0 = tile * TN;
        __syncthreads();
        load_rows<T>(sK, KS, TN, min(TN, N - t0), [&](int row) { return row_ptr<T>(k, b, g, t0 + row); });
        load_rows<T>(sV, kD, TN, min(TN, N - t0), [&](int row) { return row_ptr<T>(v, b, g, t0 + row); });
        __syncthreads();

        float acc[4][2] = {};
        tile_gemm(sQ, sK, warp, lane, acc);

#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s0 = (t0 + lane <= last[i]) ? acc[i][0] * sl2 : -INFINITY;
            float s1 = (t0 + lane + 32 <= last[i]) ? acc[i][1] * sl2 : -INFINITY;
            float mt = warp_max(fmaxf(s0, s1));
            float mn = fmaxf(m2[i], mt);
            float p0 = 0.f, p1 = 0.f, corr = 1.f;
            if (mn != -INFINITY) {
                corr = exp2f(m2[i] - mn);              // m2 = -inf -> 0
                p0 = exp2f(s0 - mn); p1 = exp2f(s1 - mn);
            }
            float ps = warp_sum(p0 + p1);
            l[i] = l[i] * corr + ps;
            m2[i] = mn;
#pragma unroll
            for (int c = 0; c < 4; ++c) o[i][c] *= corr;
            sP[(warp * 4 + i) * TN + lane] = p0;
            sP[(warp * 4 + i) * TN + lane + 32] = p1;
        }
        __syncwarp();
        // O[rows of this warp][lane*4 .. +3] += P[row][p] * V[p][lane*4 .. +3]
#pragma unroll 2
        for (int p4 = 0; p4 < TN / 4; ++p4) {
            float4 pr[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) pr[i] = *reinterpret_cast<const float4*>(sP + (warp * 4 + i) * TN + p4 * 4);
#pragma unroll
            for (int pp = 0; pp < 4; ++pp) {
                float4 vv = *reinterpret_cast<const float4*>(sV + (p4 * 4 + pp) * kD + lane * 4);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float pw = pp == 0 ? pr[i].x : pp == 1 ? pr[i].y : pp == 2 ? pr[i].z : pr[i].w;
                    o[i][0] = fmaf(pw, vv.x, o[i][0]); o[i][1] = fmaf(pw, vv.y, o[i][1]);
                    o[i][2] = fmaf(pw, vv.z, o[i][2]); o[i][3] = fmaf(pw, vv.w, o[i][3]);
                }
            }
        }
        __syncwarp();
    }

    float* part_m = ws + plan.off_part_m / 4;
    float* part_l = ws + plan.off_part_l / 4;
    float* part_o = ws + plan.off_part_o / 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = r0 + warp * 4 + i;
        if (r >= s.R) continue;
        size_t row = ((size_t)unit * plan.n_splits + split) * s.R + r;
        if (lane == 0) { part_m[row] = m2[i]; part_l[row] = l[i]; }
        *reinterpret_cast<float4*>(part_o + row * kD + lane * 4) = make_float4(o[i][0], o[i][1], o[i][2], o[i][3]);
    }
}

// ------------------------------------------------------------------------------------------ combine
// one block of 128 threads per (unit, output row): merge the splits.  Output rows >= R are padding
// for the tensor-core pass: O = 0, ||o||^2 = 0 and log2-sum-exp = +inf, so that they weigh 0.
// Every load of a block is issued before the first one is used: thread t reads the statistics of
// split t, warp w the float4 partial outputs of splits w, w+4, ... (pass 1 writes every partial,
// zeros where a split saw no token), so a block costs one round trip to L2 instead of one per split.
constexpr int CMB_NT = 128;
// splits that hold tokens of a sequence of N tokens: the others ran no tile and wrote nothing
__device__ __forceinline__ int active_splits(const SimtPlan& plan, int N) {
    const int tiles = (N + plan.tile_tokens - 1) / plan.tile_tokens;
    return min(plan.n_splits, (tiles + plan.tiles_per_split - 1) / plan.tiles_per_split);
}
constexpr int CMB_INFLIGHT = 10;                       // float4 loads in flight per thread

__device__ __forceinline__ float block128_reduce(float x, bool take_max, float* red) {
    x = take_max ? warp_max(x) : warp_sum(x);
    __syncthreads();                                   // red may still be read from an earlier call
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    return take_max ? fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3])) : (red[0] + red[1]) + (red[2] + red[3]);
}

__global__ void __launch_bounds__(CMB_NT)
simt_combine_kernel(ScoreShape s, SimtPlan plan, float* ws) {
    pdl_wait();
    const int r = blockIdx.x % plan.rows_out, unit = blockIdx.x / plan.rows_out;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t orow = (size_t)unit * plan.rows_out + r;
    __nv_bfloat16* obf = plan.want_obf ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(ws) + plan.off_obf) : nullptr;
    float* cpair = plan.want_obf ? ws + plan.off_cpair / 4 + (orow >> 1) * 4 + (orow & 1) : nullptr;
    if (r >= s.R) {
        (ws + plan.off_o / 4)[orow * kD + tid] = 0.f;
        if (obf) obf[orow * kD + tid] = __float2bfloat16(0.f);
        if (tid == 0) {
            (ws + plan.off_lse2 / 4)[orow] = INFINITY; (ws + plan.off_onorm / 4)[orow] = 0.f;
            if (cpair) { cpair[0] = -INFINITY; cpair[2] = 0.f; }
        }
        return;
    }
    __shared__ float red[4];
    __shared__ float sW[CMB_NT];
    __shared__ __align__(16) float sAcc[4][kD];
    const float* part_m = ws + plan.off_part_m / 4;
    const float* part_l = ws + plan.off_part_l / 4;
    const float* part_o = ws + plan.off_part_o / 4;
    const size_t row0 = (size_t)unit * plan.n_splits * s.R + r;          // split sp: row0 + sp * R
    const size_t sstride = (size_t)s.R * kD;                             // floats between the outputs of two splits
    float M = -INFINITY, L = 0.f, Mrun = -INFINITY;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int n_act = active_splits(plan, seq_len(s, unit / s.Hkv));
    for (int base = 0; base < n_act; base += CMB_NT) {
        const int sp = base + tid, cnt = min(CMB_NT, n_act - base);
        const float m = sp < n_act ? part_m[row0 + (size_t)sp * s.R] : -INFINITY;
        const float l = sp < n_act ? part_l[row0 + (size_t)sp * s.R] : 0.f;
        const float* po = part_o + (row0 + (size_t)base * s.R) * kD + lane * 4;
        for (int j0 = warp; j0 < cnt || j0 == warp; j0 += 4 * CMB_INFLIGHT) {
            float4 o4[CMB_INFLIGHT];
#pragma unroll
            for (int u = 0; u < CMB_INFLIGHT; ++u) {
                const int j = j0 + 4 * u;
                o4[u] = j < cnt ? *reinterpret_cast<const float4*>(po + (size_t)j * sstride) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (j0 == warp) {                          // first round: weights of this batch of splits
                M = block128_reduce(m, true, red);
                if (M > Mrun) {                        // (only with more than 128 splits) rescale what was summed
                    const float f = Mrun == -INFINITY ? 0.f : exp2f(Mrun - M);
                    L *= f; acc.x *= f; acc.y *= f; acc.z *= f; acc.w *= f;
                    Mrun = M;
                }
                const float w = m == -INFINITY ? 0.f : exp2f(m - Mrun);
                L = fmaf(l, w, L);
                sW[tid] = w;
                __syncthreads();
            }
#pragma unroll
            for (int u = 0; u < CMB_INFLIGHT; ++u) {
                const int j = j0 + 4 * u;
                const float w = j < cnt ? sW[j] : 0.f;
                acc.x = fmaf(o4[u].x, w, acc.x); acc.y = fmaf(o4[u].y, w, acc.y);
                acc.z = fmaf(o4[u].z, w, acc.z); acc.w = fmaf(o4[u].w, w, acc.w);
            }
        }
        __syncthreads();                               // sW is rewritten by the next batch
    }
    *reinterpret_cast<float4*>(&sAcc[warp][lane * 4]) = acc;
    L = block128_reduce(L, false, red);                // its barriers also publish sAcc
    // (L = 0: the row saw no token, which only a shard of a longer sequence can show; it then weighs nothing in the merge)
    const float oc = L > 0.f ? ((sAcc[0][tid] + sAcc[1][tid]) + (sAcc[2][tid] + sAcc[3][tid])) / L : 0.f;
    const float onorm = block128_reduce(oc * oc, false, red);
    (ws + plan.off_o / 4)[orow * kD + tid] = oc;
    if (obf) obf[orow * kD + tid] = __float2bfloat16(-2.f * oc);
    if (tid == 0) {
        const float lse2 = Mrun + log2f(L);
        (ws + plan.off_lse2 / 4)[orow] = lse2;
        (ws + plan.off_onorm / 4)[orow] = onorm;
        if (cpair) { cpair[0] = -lse2; cpair[2] = onorm; }
    }
}

// The same merge with one warp per (unit, output row), for many rows (a window of thousands of queries, a large
// batch): no block-wide barrier, lane t holds head-dim elements 4t..4t+3, the splits are added in order, eight at a time.
constexpr int CMBW_MAX_SPLITS = 8;
// FEW: at most CMBW_MAX_SPLITS splits, one batch of loads and the maximum taken from it (one round trip to L2 in all)
template <bool FEW>
__global__ void __launch_bounds__(CMB_NT)
simt_combine_rows_kernel(ScoreShape s, SimtPlan plan, float* ws) {
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long rows_total = (long long)s.B * s.Hkv * plan.rows_out;
    const long long orow = (long long)blockIdx.x * (CMB_NT / 32) + (threadIdx.x >> 5);
    if (orow >= rows_total) return;
    const int r = (int)(orow % plan.rows_out), unit = (int)(orow / plan.rows_out);
    __nv_bfloat16* obf = plan.want_obf ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(ws) + plan.off_obf) : nullptr;
    float* cpair = plan.want_obf ? ws + plan.off_cpair / 4 + (orow >> 1) * 4 + (orow & 1) : nullptr;
    float4 oc = make_float4(0.f, 0.f, 0.f, 0.f);
    float lse2 = INFINITY, onorm = 0.f;                    // padding rows weigh 0
    if (r < s.R) {
        const float* part_m = ws + plan.off_part_m / 4;
        const float* part_l = ws + plan.off_part_l / 4;
        const float* part_o = ws + plan.off_part_o / 4;
        const size_t row0 = (size_t)unit * plan.n_splits * s.R + r;          // split sp: row0 + sp * R
        const int n_act = active_splits(plan, seq_len(s, unit / s.Hkv));
        float M = -INFINITY, L = 0.f;
        float m[CMBW_MAX_SPLITS], l[CMBW_MAX_SPLITS];
        float4 o4[CMBW_MAX_SPLITS];
        auto load_batch = [&](int base) {                                    // every load of the batch before the first use
#pragma unroll
            for (int u = 0; u < CMBW_MAX_SPLITS; ++u) {
                const int sp = base + u;
                const bool on = sp < n_act;
                m[u] = on ? part_m[row0 + (size_t)sp * s.R] : -INFINITY;
                l[u] = on ? part_l[row0 + (size_t)sp * s.R] : 0.f;
                o4[u] = on ? *reinterpret_cast<const float4*>(part_o + (row0 + (size_t)sp * s.R) * kD + lane * 4)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        };
        load_batch(0);
        // the row's maximum over the splits: from the first batch when that is all of them (one round trip in all),
        // otherwise the lanes read the splits' maxima side by side
        float mrest = -INFINITY;
        if (!FEW)
            for (int sp = CMBW_MAX_SPLITS + lane; sp < n_act; sp += 32) mrest = fmaxf(mrest, part_m[row0 + (size_t)sp * s.R]);
#pragma unroll
        for (int u = 0; u < CMBW_MAX_SPLITS; ++u) M = fmaxf(M, m[u]);
        if (!FEW && n_act > CMBW_MAX_SPLITS) M = fmaxf(M, warp_max(mrest));
        for (int base = 0; base < (FEW ? 1 : n_act); base += CMBW_MAX_SPLITS) {
            if (base > 0) load_batch(base);
#pragma unroll
            for (int u = 0; u < CMBW_MAX_SPLITS; ++u) {
                const float w = m[u] == -INFINITY ? 0.f : exp2f(m[u] - M);
                L = fmaf(l[u], w, L);
                oc.x = fmaf(o4[u].x, w, oc.x); oc.y = fmaf(o4[u].y, w, oc.y);
                oc.z = fmaf(o4[u].z, w, oc.z); oc.w = fmaf(o4[u].w, w, oc.w);
            }
        }
        if (L > 0.f) { oc.x /= L; oc.y /= L; oc.z /= L; oc.w /= L; }       // L = 0: a shard in which the row sees no token
        onorm = warp_sum((oc.x * oc.x + oc.y * oc.y) + (oc.z * oc.z + oc.w * oc.w));
        lse2 = M + log2f(L);
    }
    *reinterpret_cast<float4*>(ws + plan.off_o / 4 + orow * kD + lane * 4) = oc;
    if (obf) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(-2.f * oc.x, -2.f * oc.y), hi = __floats2bfloat162_rn(-2.f * oc.z, -2.f * oc.w);
        *reinterpret_cast<uint2*>(obf + orow * kD + lane * 4) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
    if (lane == 0) {
        (ws + plan.off_lse2 / 4)[orow] = lse2;
        (ws + plan.off_onorm / 4)[orow] = onorm;
        if (cpair) { cpair[0] = -lse2; cpair[2] = onorm; }
    }
}

// One block of 128 threads per (unit, output row), like the combine kernel, but the row comes from the
// caller: o [B,Hq,W,d] and the natural-log LSE [B,Hq,W] of an attention kernel that already ran.
// Row r of KV head g is (query head g*G + r / W, window query r % W).
template <typename T>
__global__ void __launch_bounds__(CMB_NT)
given_prep_kernel(ScoreShape s, SimtPlan plan, TensorView o, const float* lse, float* ws) {
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0)     // no wait of this call can have given up yet
        *reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(ws) + plan.off_flag) = 0u;
    const int r = blockIdx.x % plan.rows_out, unit = blockIdx.x / plan.rows_out;
    const int tid = threadIdx.x;
    const size_t orow = (size_t)unit * plan.rows_out + r;
    __nv_bfloat16* obf = plan.want_obf ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(ws) + plan.off_obf) : nullptr;
    float* cpair = plan.want_obf ? ws + plan.off_cpair / 4 + (orow >> 1) * 4 + (orow & 1) : nullptr;
    __shared__ float red[4];
    float oc = 0.f, lse2 = INFINITY;             // padding rows weigh 0
    if (r < s.R) {
        const int b = unit / s.Hkv, g = unit % s.Hkv, h = g * s.G + r / s.W, i = r % s.W;
        oc = elem_to_float(row_ptr<T>(o, b, h, i)[tid]);
        lse2 = lse[((size_t)b * s.Hq + h) * s.W + i] * kLog2e;
    }
    const float onorm = block128_reduce(oc * oc, false, red);
    (ws + plan.off_o / 4)[orow * kD + tid] = oc;
    if (obf) obf[orow * kD + tid] = __float2bfloat16(-2.f * oc);
    if (tid == 0) {
        (ws + plan.off_lse2 / 4)[orow] = lse2;
        (ws + plan.off_onorm / 4)[orow] = onorm;
        if (cpair) { cpair[0] = -lse2; cpair[2] = onorm; }
    }
}

// ------------------------------------------------------------------------------------------ pass 2
template <typename T>
__global__ void __launch_bounds__(NT, 2)
simt_pass2_kernel(ScoreShape s, SimtPlan plan, TensorView q, TensorView k, TensorView v,
                  const float* ws, float* scores) {
    pdl_wait();
    extern __shared__ __align__(16) float smem[];
    float* sK = smem;                       // [TN][KS]
    float* sV = sK + TN * KS;               // [TN][KS]
    float* sQ = sV + TN * KS;               // [RC][kD]   (reused for the final cross-warp sum)
    float* sO = sQ + RC * kD;               // [RC][kD]
    float* sNv = sO + RC * kD;              // [TN]
    float* sNv1 = sNv + TN;                 // [TN]
    float* sLse = sNv1 + TN;                // [RC]
    float* sNo = sLse + RC;                 // [RC]

    const int unit = blockIdx.y, t0 = blockIdx.x * TN;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int N = seq_len(s, b);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t plane = (size_t)s.B * s.Hkv * s.Nmax;
    float* out = scores + (size_t)unit * s.Nmax;

    if (t0 >= N) {                          // padding beyond the sequence: scores are 0
        for (int i = threadIdx.x; i < TN * s.n_planes; i += NT) {
            int p = t0 + (i % TN);
            if (p < s.Nmax) out[(size_t)(i / TN) * plane + p] = 0.f;
        }
        return;
    }

    load_rows<T>(sK, KS, TN, min(TN, N - t0), [&](int row) { return row_ptr<T>(k, b, g, t0 + row); });
    load_rows<T>(sV, KS, TN, min(TN, N - t0), [&](int row) { return row_ptr<T>(v, b, g, t0 + row); });
    __syncthreads();
    // ||v_p||^2: each warp covers 8 tokens
    for (int tkn = warp * 8; tkn < warp * 8 + 8; ++tkn) {
        float4 f = *reinterpret_cast<const float4*>(sV + tkn * KS + lane * 4);
        float sq = warp_sum(f.x * f.x + f.y * f.y + f.z * f.z + f.w * f.w);
        float ab = warp_sum((fabsf(f.x) + fabsf(f.y)) + (fabsf(f.z) + fabsf(f.w)));
        if (lane == 0) { sNv[tkn] = sq; sNv1[tkn] = ab; }
    }

    const float sl2 = s.scale * kLog2e;
    const float* o_all = ws + plan.off_o / 4 + (size_t)unit * plan.rows_out * kD;
    const float* lse_all = ws + plan.off_lse2 / 4 + (size_t)unit * plan.rows_out;
    const float* no_all = ws + plan.off_onorm / 4 + (size_t)unit * plan.rows_out;

    float sv[2] = {0.f, 0.f}, sk[2] = {0.f, 0.f}, sx[2] = {0.f, 0.f}, sa[2] = {0.f, 0.f};

    for (int r0 = 0; r0 < s.R; r0 += RC) {
        __syncthreads();
        const int valid = min(RC, s.R - r0);
        load_rows<T>(sQ, kD, RC, valid, [&](int row) {
            int r = r0 + row;
            return row_ptr<T>(q, b, g * s.G + r / s.W, r % s.W);
        });
        load_rows<float>(sO, kD, RC, valid, [&](int row) { return o_all + (size_t)(r0 + row) * kD; });
        if (threadIdx.x < RC) {
            bool ok = threadIdx.x < valid;
            sLse[threadIdx.x] = ok ? lse_all[r0 + threadIdx.x] : 0.f;
            sNo[threadIdx.x] = ok ? no_all[r0 + threadIdx.x] : 0.f;
        }
        __syncthreads();

        float az[4][2] = {}, at[4][2] = {};
        tile_gemm(sQ, sK, warp, lane, az);
        tile_gemm(sO, sV, warp, lane, at);

#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + warp * 4 + i;
            if (r >= s.R) continue;
            const long long last = s.causal ? min((long long)mask_len(s, b) - s.W + (r % s.W), (long long)N - 1) : (long long)N - 1;
            const float lse = sLse[warp * 4 + i], no = sNo[warp * 4 + i];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int tl = lane + 32 * j;
                if (t0 + tl > last) continue;              // masked pair: contributes 0
                const float nv = sNv[tl];
                const float a = exp2f(fmaf(az[i][j], sl2, -lse));
                const float Z = az[i][j] * s.scale;
                const float t = at[i][j];
                const float a2 = a * a;
                sa[j] += a;
                sv[j] = fmaf(a2, nv, sv[j]);
                sk[j] = fmaf(a2 * Z * Z, no + nv - 2.f * t, sk[j]);      // Alg. 1: |o|^2+|v|^2-2 v.o
                sx[j] = fmaf(2.f * a2 * Z, nv - t, sx[j]);               // Eq. 6 cross term
            }
        }
    }

    // sum over the 8 warps (each warp held 4 of every 32 rows)
    __syncthreads();
    float* red = sQ;                        // [8][4][TN]
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int tl = lane + 32 * j;
        red[(warp * 4 + 0) * TN + tl] = sv[j];
        red[(warp * 4 + 1) * TN + tl] = sk[j];
        red[(warp * 4 + 2) * TN + tl] = sx[j];
        red[(warp * 4 + 3) * TN + tl] = sa[j];
    }
    __syncthreads();
    if (threadIdx.x < TN) {
        const int tl = threadIdx.x, p = t0 + tl;
        float tv = 0.f, tk = 0.f, tx = 0.f, ta = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            tv += red[(w * 4 + 0) * TN + tl]; tk += red[(w * 4 + 1) * TN + tl];
            tx += red[(w * 4 + 2) * TN + tl]; ta += red[(w * 4 + 3) * TN + tl];
        }
        if (p < s.Nmax) {
            const bool live = p < N;
            int pl = 0;
            if (s.variants & OBC_VAR_V)    out[(size_t)(pl++) * plane + p] = live ? tv : 0.f;
            if (s.variants & OBC_VAR_K)    out[(size_t)(pl++) * plane + p] = live ? tk : 0.f;
            if (s.variants & OBC_VAR_VK)   out[(size_t)(pl++) * plane + p] = live ? tv + tk + tx : 0.f;
            if (s.variants & OBC_VAR_ATTN) out[(size_t)(pl++) * plane + p] = live ? ta : 0.f;
            if (s.variants & OBC_VAR_VATP) out[(size_t)(pl++) * plane + p] = live ? ta * sNv1[tl] : 0.f;
        }
    }
}

constexpr size_t kSmemPass1 = (size_t)(TN * KS + TN * kD + RC * kD + RC * TN) * 4;
constexpr size_t kSmemPass2 = (size_t)(2 * TN * KS + 2 * RC * kD + 2 * TN + 2 * RC) * 4;

template <typename T>
obc_status launch_pass1_typed(const ScoreShape& s, const SimtPlan& plan, TensorView q, TensorView k, TensorView v,
                              float* ws, cudaStream_t stream) {
    const int units = s.B * s.Hkv, chunks = (s.R + RC - 1) / RC;
    OBC_CUDA_TRY(cudaFuncSetAttribute(simt_pass1_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemPass1));
    { ProfScope ps("simt_pass1", stream); OBC_CUDA_TRY(launch_pdl(simt_pass1_kernel<T>, dim3(plan.n_splits, units, chunks), dim3(NT), kSmemPass1, stream, 1, s, plan, q, k, v, ws)); }
    return launch_combine(s, plan, ws, stream);
}

template <typename T>
obc_status launch_pass2_typed(const ScoreShape& s, const SimtPlan& plan, TensorView q, TensorView k, TensorView v,
                              float* scores, float* ws, cudaStream_t stream) {
    const int units = s.B * s.Hkv;
    OBC_CUDA_TRY(cudaFuncSetAttribute(simt_pass2_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemPass2));
    { ProfScope ps("simt_pass2", stream); OBC_CUDA_TRY(launch_pdl(simt_pass2_kernel<T>, dim3((s.Nmax + TN - 1) / TN, units), dim3(NT), kSmemPass2, stream, 1, s, plan, q, k, v, ws, scores)); }
    return OBC_OK;
}
}  // namespace

SimtPlan make_simt_plan(const ScoreShape& s, int rows_out, bool want_obf) {
    SimtPlan p{};
    const int units = s.B * s.Hkv, chunks = (s.R + RC - 1) / RC;
    const int tiles = (s.Nmax + TN - 1) / TN;
    // enough CTAs for ~2 waves of 148 SMs x 2 resident CTAs, at least 8 tiles per split
    int want = (148 * 2 * 2 + units * chunks - 1) / (units * chunks);
    int max_splits = (tiles + 7) / 8;
    int n = want < 1 ? 1 : want;
    if (n > max_splits) n = max_splits;
    if (n < 1) n = 1;
    p.tiles_per_split = (tiles + n - 1) / n;
    p.n_splits = (tiles + p.tiles_per_split - 1) / p.tiles_per_split;
    p.tile_tokens = TN;
    p.rows_out = rows_out;
    p.want_obf = want_obf ? 1 : 0;
    size_t rows = (size_t)units * s.R, prow = rows * p.n_splits, orow = (size_t)units * rows_out, off = 0;
    p.off_flag = off;   off = 256;
    p.off_part_m = off; off = align_up(off + prow * 4, 256);
    p.off_part_l = off; off = align_up(off + prow * 4, 256);
    p.off_part_o = off; off = align_up(off + prow * kD * 4, 256);
    p.off_lse2 = off;   off = align_up(off + orow * 4, 256);
    p.off_onorm = off;  off = align_up(off + orow * 4, 256);
    p.off_o = off;      off = align_up(off + orow * kD * 4, 256);
    p.off_obf = off;    off = align_up(off + (want_obf ? orow * kD * 2 : 0), 1024);
    p.off_cpair = off; p.off_nv = off;             // tensor-core plan only
    p.bytes = off;
    return p;
}

// ---- token-sharded caches: a shard's window attention out of the workspace, and the merge of the shards' ----------
// one warp per window row: o [B,Hq,W,d] fp32 and the natural-log lse [B,Hq,W] from the combined arrays
__global__ void __launch_bounds__(CMB_NT)
export_attention_kernel(ScoreShape s, SimtPlan plan, const float* ws, float* o_out, float* lse_out) {
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (CMB_NT / 32) + (threadIdx.x >> 5);   // (unit, r) = ((b, g), (head of the group, query))
    if (row >= (long long)s.B * s.Hkv * s.R) return;
    const long long unit = row / s.R, r = row % s.R;
    const size_t src = (size_t)unit * plan.rows_out + r;
    // rows of a unit are its G heads' W queries in order, and the units follow (b, g): the same order as [B,Hq,W]
    *reinterpret_cast<float4*>(o_out + (size_t)row * kD + lane * 4) =
        *reinterpret_cast<const float4*>(ws + plan.off_o / 4 + src * kD + lane * 4);
    if (lane == 0) lse_out[row] = (ws + plan.off_lse2 / 4)[src] * 0.6931471805599453f;
}

// one warp per row: lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s over the n_parts shards
__global__ void __launch_bounds__(CMB_NT)
merge_attention_kernel(int n_parts, long long rows, const float* __restrict__ o_parts, const float* __restrict__ lse_parts,
                       float* __restrict__ o_out, float* __restrict__ lse_out) {
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (CMB_NT / 32) + (threadIdx.x >> 5);
    if (row >= rows) return;
    float M = -INFINITY;
    for (int sp = 0; sp < n_parts; ++sp) M = fmaxf(M, lse_parts[(size_t)sp * rows + row]);
    float L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp = 0; sp < n_parts; ++sp) {
        const float ls = lse_parts[(size_t)sp * rows + row];
        const float w = ls == -INFINITY ? 0.f : expf(ls - M);
        const float4 o4 = *reinterpret_cast<const float4*>(o_parts + ((size_t)sp * rows + row) * kD + lane * 4);
        L += w;
        acc.x = fmaf(o4.x, w, acc.x); acc.y = fmaf(o4.y, w, acc.y); acc.z = fmaf(o4.z, w, acc.z); acc.w = fmaf(o4.w, w, acc.w);
    }
    if (L > 0.f) { acc.x /= L; acc.y /= L; acc.z /= L; acc.w /= L; }
    *reinterpret_cast<float4*>(o_out + (size_t)row * kD + lane * 4) = acc;
    if (lane == 0) lse_out[row] = M + logf(L);
}

obc_status launch_export_attention(const ScoreShape& s, const SimtPlan& plan, const void* ws, float* o_out, float* lse_out,
                                   cudaStream_t stream) {
    const long long rows = (long long)s.B * s.Hkv * s.R;
    ProfScope ps("export_attention", stream);
    OBC_CUDA_TRY(launch_pdl(export_attention_kernel, dim3((unsigned)((rows + CMB_NT / 32 - 1) / (CMB_NT / 32))), dim3(CMB_NT), 0, stream, 1,
                            s, plan, (const float*)ws, o_out, lse_out));
    return OBC_OK;
}

obc_status launch_merge_attention(int n_parts, long long rows, const float* o_parts, const float* lse_parts,
                                  float* o_out, float* lse_out, cudaStream_t stream) {
    ProfScope ps("merge_attention", stream);
    OBC_CUDA_TRY(launch_pdl(merge_attention_kernel, dim3((unsigned)((rows + CMB_NT / 32 - 1) / (CMB_NT / 32))), dim3(CMB_NT), 0, stream, 1,
                            n_parts, rows, o_parts, lse_parts, o_out, lse_out));
    return OBC_OK;
}

obc_status launch_combine(const ScoreShape& s, const SimtPlan& plan, void* ws, cudaStream_t stream) {
    const long long rows = (long long)s.B * s.Hkv * plan.rows_out;
    // a warp per row when there are many rows: with 8192 rows of 16 splits (ragged batch of 8) 23 us against 31 us for a
    // block per row; with 1024 rows of 18 splits (one 32k layer) the block per row wins, 8.5 us against 14.5 us
    if ((plan.n_splits <= CMBW_MAX_SPLITS && rows >= 1024) || rows >= 4096) {
        ProfScope ps("combine", stream);
        const dim3 grid((unsigned)((rows + CMB_NT / 32 - 1) / (CMB_NT / 32)));
        if (plan.n_splits <= CMBW_MAX_SPLITS) OBC_CUDA_TRY(launch_pdl(simt_combine_rows_kernel<true>, grid, dim3(CMB_NT), 0, stream, 1, s, plan, (float*)ws));
        else OBC_CUDA_TRY(launch_pdl(simt_combine_rows_kernel<false>, grid, dim3(CMB_NT), 0, stream, 1, s, plan, (float*)ws));
        return OBC_OK;
    }
    { ProfScope ps("combine", stream); OBC_CUDA_TRY(launch_pdl(simt_combine_kernel, dim3(s.B * s.Hkv * plan.rows_out), dim3(CMB_NT), 0, stream, 1, s, plan, (float*)ws)); }
    return OBC_OK;
}

obc_status launch_given_prep(const ScoreShape& s, const SimtPlan& plan, const GivenAttention& given,
                             void* ws, cudaStream_t stream) {
    const dim3 grid(s.B * s.Hkv * plan.rows_out), block(CMB_NT);
    ProfScope ps("given_prep", stream);
    if (given.o_dtype == OBC_F32)
        OBC_CUDA_TRY(launch_pdl(given_prep_kernel<float>, grid, block, 0, stream, 1, s, plan, given.o, given.lse, (float*)ws));
    else
        OBC_CUDA_TRY(launch_pdl(given_prep_kernel<__nv_bfloat16>, grid, block, 0, stream, 1, s, plan, given.o, given.lse, (float*)ws));
    return OBC_OK;
}

obc_status launch_simt_pass1_combine(const ScoreShape& s, const SimtPlan& plan, int dtype,
                                     TensorView q, TensorView k, TensorView v, void* ws, cudaStream_t stream) {
    if (dtype == OBC_F32) return launch_pass1_typed<float>(s, plan, q, k, v, (float*)ws, stream);
    return launch_pass1_typed<__nv_bfloat16>(s, plan, q, k, v, (float*)ws, stream);
}

obc_status launch_simt_pass2(const ScoreShape& s, const SimtPlan& plan, int dtype,
                             TensorView q, TensorView k, TensorView v,
                             float* scores, void* ws, cudaStream_t stream) {
    if (dtype == OBC_F32) return launch_pass2_typed<float>(s, plan, q, k, v, scores, (float*)ws, stream);
    return launch_pass2_typed<__nv_bfloat16>(s, plan, q, k, v, scores, (float*)ws, stream);
}

}  // namespace obc
