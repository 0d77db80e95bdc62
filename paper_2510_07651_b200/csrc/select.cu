// Pooling + per-head top-budget selection + ordered index emission (Algorithm 2's
// "topk(S[..., :cutoff], num_hh) -> sort"), and the row gather that builds the compacted cache.
//
//   pool_key_kernel   pooled score of every candidate token -> order-preserving uint32 key
//   select_kernel     one CTA per (batch item, KV head): 4 x 8-bit radix passes find the key of
//                     the n_hh-th largest candidate and how many of its ties are kept; two
//                     warp-segmented sweeps then emit the kept indices in ascending order
//   gather_kernel     16-byte vector copy of the kept K/V rows (and optionally their scores)
#include "obc_common.cuh"

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

// one 16-byte vector per thread; `vecs` vectors per row
__global__ void __launch_bounds__(256)
gather_kernel(int units, int Hkv, int idx_stride, int vecs, int elem_bytes,
              TensorView k, TensorView v, TensorView ko, TensorView vo,
              const int32_t* __restrict__ idx, const float* __restrict__ s_in, float* __restrict__ s_out, int Nmax) {
    const int unit = blockIdx.y, b = unit / Hkv, g = unit % Hkv;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = e / vecs, c = e % vecs;
    if (j >= idx_stride) return;
    const int src = idx[(size_t)unit * idx_stride + j];
    if (src < 0) return;
    const size_t eb = (size_t)elem_bytes;
    const char* kp = (const char*)k.ptr + ((size_t)b * k.sb + (size_t)g * k.sh + (size_t)src * k.st) * eb;
    const char* vp = (const char*)v.ptr + ((size_t)b * v.sb + (size_t)g * v.sh + (size_t)src * v.st) * eb;
    char* kop = (char*)ko.ptr + ((size_t)b * ko.sb + (size_t)g * ko.sh + (size_t)j * ko.st) * eb;
    char* vop = (char*)vo.ptr + ((size_t)b * vo.sb + (size_t)g * vo.sh + (size_t)j * vo.st) * eb;
    reinterpret_cast<uint4*>(kop)[c] = __ldg(reinterpret_cast<const uint4*>(kp) + c);
    reinterpret_cast<uint4*>(vop)[c] = __ldg(reinterpret_cast<const uint4*>(vp) + c);
    if (s_in && c == 0) s_out[(size_t)unit * idx_stride + j] = s_in[(size_t)unit * Nmax + src];
}

}  // namespace

size_t select_workspace_bytes(int B, int Hkv, int Nmax) { return align_up((size_t)B * Hkv * Nmax * 4, 256); }

obc_status launch_select(const SelectShape& s, const float* scores, int32_t* idx, void* ws, cudaStream_t stream) {
    uint32_t* keys = (uint32_t*)ws;
    const int units = s.B * s.Hkv;
    { ProfScope ps("pool_key", stream); pool_key_kernel<<<dim3((s.Nmax + 255) / 256, units), 256, 0, stream>>>(s, scores, keys); }
    OBC_CUDA_TRY(cudaGetLastError());
    { ProfScope ps("select", stream); select_kernel<<<units, SEL_NT, 0, stream>>>(s, keys, idx); }
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

obc_status launch_gather(int B, int Hkv, int idx_stride, int Nmax, int elem_bytes,
                         TensorView k, TensorView v, TensorView ko, TensorView vo, const int32_t* idx,
                         const float* s_in, float* s_out, cudaStream_t stream) {
    const int vecs = kD * elem_bytes / 16;
    const long long total = (long long)idx_stride * vecs;
    {
        ProfScope ps("gather", stream);
        gather_kernel<<<dim3((unsigned)((total + 255) / 256), B * Hkv), 256, 0, stream>>>(
            B * Hkv, Hkv, idx_stride, vecs, elem_bytes, k, v, ko, vo, idx, s_in, s_out, Nmax);
    }
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

}  // namespace obc
