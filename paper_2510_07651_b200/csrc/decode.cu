// Decode-time rescoring + eviction step (W = 1: only the newest query of each head scores the
// cache).  Sec. 3 "Decoding" / "Cache Eviction"; Sec. 4.2 (scores accumulated over steps);
// App. C.2.2 (sinks + recent window protected, one eviction per step once over budget).
//
// CUDA cores only: with G <= 8 score rows per KV head the contractions are matrix-vector
// products bound by HBM traffic, so one thread owns one cache slot (a 256-byte K or V row read
// as 16-byte vectors) and reductions over slots use warp shuffles.
//
//   decode_pass1   append (k_t, v_t); logits of every live slot (kept in the workspace so K is
//                  read once); per-chunk softmax statistics and partial outputs
//   decode_combine merge the chunks: log2-sum-exp, o_r, ||o_r||^2
//   decode_score   v_p . o_r and ||v_p||^2 per slot, score, s_acc += score, per-chunk argmin of
//                  the evictable slots
//   decode_final   per (b, g): pick the slot to free, update pos / state
#include "obc_common.cuh"

namespace obc {
namespace {

constexpr int CH = 256;                  // slots per chunk = threads per block
constexpr size_t kStageBytes = (size_t)CH * 256;   // one chunk of 256-byte rows in shared memory

struct DecodePlan {
    int chunks;
    size_t off_z, off_pm, off_pl, off_po, off_lse, off_no, off_o, off_min, bytes;
};

DecodePlan make_plan(const DecodeShape& s) {
    DecodePlan p{};
    p.chunks = (s.cap + CH - 1) / CH;
    const size_t units = (size_t)s.B * s.Hkv;
    size_t off = 0;
    p.off_z = off;   off = align_up(off + units * s.G * s.cap * 4, 256);
    p.off_pm = off;  off = align_up(off + units * p.chunks * s.G * 4, 256);
    p.off_pl = off;  off = align_up(off + units * p.chunks * s.G * 4, 256);
    p.off_po = off;  off = align_up(off + units * p.chunks * s.G * kD * 4, 256);
    p.off_lse = off; off = align_up(off + units * s.G * 4, 256);
    p.off_no = off;  off = align_up(off + units * s.G * 4, 256);
    p.off_o = off;   off = align_up(off + units * s.G * kD * 4, 256);
    p.off_min = off; off = align_up(off + units * p.chunks * 16, 256);
    p.bytes = off;
    return p;
}

struct MinCand { float val; int pos; int slot; int pad; };

// four packed pairs (lo, hi) of the eight bf16 of a 16-byte chunk
__device__ __forceinline__ void unpack8x2(uint4 u, float2 (&f)[4]) {
    f[0] = make_float2(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u));
    f[1] = make_float2(__uint_as_float(u.y << 16), __uint_as_float(u.y & 0xffff0000u));
    f[2] = make_float2(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u));
    f[3] = make_float2(__uint_as_float(u.w << 16), __uint_as_float(u.w & 0xffff0000u));
}

__device__ __forceinline__ const __nv_bfloat16* bf_row(const TensorView& t, int b, int h, long long tok) {
    return reinterpret_cast<const __nv_bfloat16*>(t.ptr) + b * t.sb + h * t.sh + tok * t.st;
}

// Cooperative copy of the 256-byte rows [c0, c0 + CH) of one cache into shared memory, in two steps so
// that the caller can put work between them: load_rows issues all 16 loads of a thread before any
// use (a warp reads two whole rows per instruction, coalesced; rows at or beyond `hi` are not
// read), store_rows puts the 16-byte chunk c of row r at chunk c ^ (r & 15), so that the thread
// that owns row r later reads its row without bank conflicts.
__device__ __forceinline__ void load_rows(uint4 (&v)[16], const TensorView& t, int b, int g, int c0, int hi) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const int i = threadIdx.x + k * CH, r = i >> 4, c = i & 15;
        // plain loads: the new token's row was stored by this CTA just before
        v[k] = c0 + r < hi ? reinterpret_cast<const uint4*>(bf_row(t, b, g, c0 + r))[c] : make_uint4(0, 0, 0, 0);
    }
}
__device__ __forceinline__ void store_rows(uint4* dst, const uint4 (&v)[16]) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const int i = threadIdx.x + k * CH, r = i >> 4, c = i & 15;
        dst[r * 16 + (c ^ (r & 15))] = v[k];
    }
}
__device__ __forceinline__ uint4 staged_chunk(const uint4* src, int r, int c) { return src[r * 16 + (c ^ (r & 15))]; }

template <int G>
__global__ void __launch_bounds__(CH)
decode_pass1_kernel(DecodeShape s, DecodePlan plan, TensorView q, TensorView kt, TensorView vt,
                    TensorView kc, TensorView vc, float* s_acc, int32_t* pos, const int32_t* state,
                    int step_pos, char* ws) {
    pdl_wait();
    extern __shared__ __align__(16) uint4 sRows[];                      // [CH][16]: the chunk's K rows
    __shared__ __align__(16) float sQ[G][kD];
    __shared__ float sP[G][CH];
    __shared__ __align__(16) float sO[8][G][kD];
    __shared__ float sRed[8][G];
    __shared__ float sM[G];

    const int unit = blockIdx.y, chunk = blockIdx.x, c0 = chunk * CH;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];
    const bool valid = next >= 0 && next < s.cap;
    const int hi = valid ? max(hi_old, next + 1) : hi_old;

    float* part_m = (float*)(ws + plan.off_pm) + ((size_t)unit * plan.chunks + chunk) * G;
    float* part_l = (float*)(ws + plan.off_pl) + ((size_t)unit * plan.chunks + chunk) * G;
    if (c0 >= hi) {
        if (tid < G) { part_m[tid] = -INFINITY; part_l[tid] = 0.f; }
        return;
    }
    for (int i = tid; i < G * kD; i += CH) {
        const int r = i / kD, c = i % kD;
        sQ[r][c] = __bfloat162float(bf_row(q, b, g * G + r, 0)[c]);
    }
    if (valid && next >= c0 && next < c0 + CH) {       // this chunk owns the slot of the new token
        __nv_bfloat16* kdst = const_cast<__nv_bfloat16*>(bf_row(kc, b, g, next));
        __nv_bfloat16* vdst = const_cast<__nv_bfloat16*>(bf_row(vc, b, g, next));
        if (tid < 16) reinterpret_cast<uint4*>(kdst)[tid] = reinterpret_cast<const uint4*>(bf_row(kt, b, g, 0))[tid];
        else if (tid < 32) reinterpret_cast<uint4*>(vdst)[tid - 16] = reinterpret_cast<const uint4*>(bf_row(vt, b, g, 0))[tid - 16];
        else if (tid == 32) { pos[(size_t)unit * s.cap + next] = step_pos; s_acc[(size_t)unit * s.cap + next] = 0.f; }
    }
    __syncthreads();                                       // the new token's row is in place
    uint4 stage[16];
    load_rows(stage, kc, b, g, c0, hi);
    store_rows(sRows, stage);
    __syncthreads();
    load_rows(stage, vc, b, g, c0, hi);                    // V rows travel while the logits are computed

    const int slot = c0 + tid;
    const bool live = slot < hi && ((valid && slot == next) || pos[(size_t)unit * s.cap + slot] >= 0);
    const float sl2 = s.scale * kLog2e;
    float z2[G];
#pragma unroll
    for (int r = 0; r < G; ++r) z2[r] = 0.f;
    if (live) {
        float2 zz[G];                                      // two partial dot products per row (packed fp32x2)
#pragma unroll
        for (int r = 0; r < G; ++r) zz[r] = make_float2(0.f, 0.f);
#pragma unroll 4
        for (int c = 0; c < 16; ++c) {
            float2 kf[4];
            unpack8x2(staged_chunk(sRows, tid, c), kf);
#pragma unroll
            for (int r = 0; r < G; ++r) {
                const float4 qa = *reinterpret_cast<const float4*>(&sQ[r][c * 8]);
                const float4 qb = *reinterpret_cast<const float4*>(&sQ[r][c * 8 + 4]);
                zz[r] = __ffma2_rn(make_float2(qa.x, qa.y), kf[0], zz[r]); zz[r] = __ffma2_rn(make_float2(qa.z, qa.w), kf[1], zz[r]);
                zz[r] = __ffma2_rn(make_float2(qb.x, qb.y), kf[2], zz[r]); zz[r] = __ffma2_rn(make_float2(qb.z, qb.w), kf[3], zz[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < G; ++r) z2[r] = zz[r].x + zz[r].y;
    }
    float* zbuf = (float*)(ws + plan.off_z) + (size_t)unit * G * s.cap;
#pragma unroll
    for (int r = 0; r < G; ++r) {
        z2[r] = live ? z2[r] * sl2 : -INFINITY;
        if (slot < s.cap) zbuf[(size_t)r * s.cap + slot] = z2[r];
        const float wm = warp_max(z2[r]);
        if (lane == 0) sRed[warp][r] = wm;
    }
    __syncthreads();
    if (tid < G) {
        float m = -INFINITY;
        for (int w = 0; w < 8; ++w) m = fmaxf(m, sRed[w][tid]);
        sM[tid] = m;
    }
    __syncthreads();
    float lsum[G];
#pragma unroll
    for (int r = 0; r < G; ++r) {
        const float p = live ? exp2f(z2[r] - sM[r]) : 0.f;
        sP[r][tid] = p;
        lsum[r] = warp_sum(p);
    }
    __syncthreads();                                       // sRed reads done, sP complete, K rows no longer read
    store_rows(sRows, stage);
#pragma unroll
    for (int r = 0; r < G; ++r) if (lane == 0) sRed[warp][r] = lsum[r];

    // partial outputs: warp w covers slots c0+32w .. +31, lane owns channels 4*lane .. +3
    const unsigned live_mask = __ballot_sync(0xffffffffu, live);
    float o[G][4];
#pragma unroll
    for (int r = 0; r < G; ++r) { o[r][0] = o[r][1] = o[r][2] = o[r][3] = 0.f; }
    __syncthreads();                                       // V rows staged
    for (int t = 0; t < 32; ++t) {
        if (!((live_mask >> t) & 1u)) continue;
        // channels 4*lane .. +3 of slot row: half (lane & 1) of the 16-byte chunk lane / 2
        const int row = warp * 32 + t;
        const uint2 raw = reinterpret_cast<const uint2*>(&sRows[row * 16 + ((lane >> 1) ^ (row & 15))])[lane & 1];
        float4 vv;
        vv.x = __uint_as_float(raw.x << 16); vv.y = __uint_as_float(raw.x & 0xffff0000u);
        vv.z = __uint_as_float(raw.y << 16); vv.w = __uint_as_float(raw.y & 0xffff0000u);
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float p = sP[r][warp * 32 + t];
            o[r][0] = fmaf(p, vv.x, o[r][0]); o[r][1] = fmaf(p, vv.y, o[r][1]);
            o[r][2] = fmaf(p, vv.z, o[r][2]); o[r][3] = fmaf(p, vv.w, o[r][3]);
        }
    }
#pragma unroll
    for (int r = 0; r < G; ++r)
        *reinterpret_cast<float4*>(&sO[warp][r][lane * 4]) = make_float4(o[r][0], o[r][1], o[r][2], o[r][3]);
    __syncthreads();
    float* part_o = (float*)(ws + plan.off_po) + ((size_t)unit * plan.chunks + chunk) * G * kD;
    for (int i = tid; i < G * kD; i += CH) {
        const int r = i / kD, c = i % kD;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) acc += sO[w][r][c];
        part_o[i] = acc;
    }
    if (tid < G) {
        float l = 0.f;
        for (int w = 0; w < 8; ++w) l += sRed[w][tid];
        part_m[tid] = sM[tid]; part_l[tid] = l;
    }
}

// one block of 128 threads per (b, g, row): merge the chunk partials.  The statistics of the chunks
// are read one per thread and the partial outputs eight at a time, so the block costs a couple of
// round trips to L2 however many chunks there are.
__device__ __forceinline__ float decode_block_reduce(float x, bool take_max, float* red) {
    x = take_max ? warp_max(x) : warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
    __syncthreads();
    return take_max ? fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3])) : (red[0] + red[1]) + (red[2] + red[3]);
}

__global__ void __launch_bounds__(kD)
decode_combine_kernel(DecodeShape s, DecodePlan plan, char* ws) {
    pdl_wait();
    const int G = s.G, unit = blockIdx.x / G, r = blockIdx.x % G, c = threadIdx.x;
    __shared__ float red[4];
    __shared__ float sW[kD];
    const float* pm = (const float*)(ws + plan.off_pm) + (size_t)unit * plan.chunks * G + r;
    const float* pl = (const float*)(ws + plan.off_pl) + (size_t)unit * plan.chunks * G + r;
    const float* po = (const float*)(ws + plan.off_po) + ((size_t)unit * plan.chunks * G + r) * kD + c;
    float M = -INFINITY;
    for (int ch = c; ch < plan.chunks; ch += kD) M = fmaxf(M, pm[(size_t)ch * G]);
    M = decode_block_reduce(M, true, red);
    float L = 0.f, oc = 0.f;
    for (int base = 0; base < plan.chunks; base += kD) {
        const int ch = base + c, cnt = min(kD, plan.chunks - base);
        float w = 0.f;
        if (ch < plan.chunks) {
            const float m = pm[(size_t)ch * G];
            if (m != -INFINITY) { w = exp2f(m - M); L = fmaf(pl[(size_t)ch * G], w, L); }
        }
        __syncthreads();
        sW[c] = w;
        __syncthreads();
        for (int j0 = 0; j0 < cnt; j0 += 8) {
            float o8[8], w8[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {                  // chunks without a live slot hold no partial output
                w8[u] = j0 + u < cnt ? sW[j0 + u] : 0.f;
                o8[u] = w8[u] != 0.f ? po[(size_t)(base + j0 + u) * G * kD] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) oc = fmaf(o8[u], w8[u], oc);
        }
    }
    L = decode_block_reduce(L, false, red);
    oc = L > 0.f ? oc / L : 0.f;
    const float sq = decode_block_reduce(oc * oc, false, red);
    ((float*)(ws + plan.off_o))[((size_t)unit * G + r) * kD + c] = oc;
    if (c == 0) {
        ((float*)(ws + plan.off_lse))[(size_t)unit * G + r] = M + log2f(L);
        ((float*)(ws + plan.off_no))[(size_t)unit * G + r] = sq;
    }
}

template <int G>
__global__ void __launch_bounds__(CH)
decode_score_kernel(DecodeShape s, DecodePlan plan, TensorView vc, float* s_acc, const int32_t* pos,
                    const int32_t* state, int step_pos, char* ws) {
    pdl_wait();
    extern __shared__ __align__(16) uint4 sRows[];                      // [CH][16]: the chunk's V rows
    __shared__ __align__(16) float sO[G][kD];
    __shared__ float sLse[G], sNo[G];
    __shared__ MinCand sMin[8];

    const int unit = blockIdx.y, chunk = blockIdx.x, c0 = chunk * CH;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];
    const bool valid = next >= 0 && next < s.cap;
    const int hi = valid ? max(hi_old, next + 1) : hi_old;
    MinCand* part_min = (MinCand*)(ws + plan.off_min) + (size_t)unit * plan.chunks + chunk;
    if (c0 >= hi) {
        if (tid == 0) *part_min = MinCand{INFINITY, -1, -1, 0};
        return;
    }
    for (int i = tid; i < G * kD; i += CH) sO[i / kD][i % kD] = ((const float*)(ws + plan.off_o))[(size_t)unit * G * kD + i];
    if (tid < G) {
        sLse[tid] = ((const float*)(ws + plan.off_lse))[(size_t)unit * G + tid];
        sNo[tid] = ((const float*)(ws + plan.off_no))[(size_t)unit * G + tid];
    }
    {
        uint4 stage[16];
        load_rows(stage, vc, b, g, c0, hi);
        store_rows(sRows, stage);
    }
    __syncthreads();

    const int slot = c0 + tid;
    const int my_pos = slot < hi ? pos[(size_t)unit * s.cap + slot] : -1;
    const bool live = my_pos >= 0;
    MinCand cand{INFINITY, -1, -1, 0};
    if (live) {
        float nv, t[G];
        float2 nn = make_float2(0.f, 0.f), tt[G];          // packed fp32x2 partial sums
#pragma unroll
        for (int r = 0; r < G; ++r) tt[r] = make_float2(0.f, 0.f);
#pragma unroll 4
        for (int c = 0; c < 16; ++c) {
            float2 vf[4];
            unpack8x2(staged_chunk(sRows, tid, c), vf);
#pragma unroll
            for (int j = 0; j < 4; ++j) nn = __ffma2_rn(vf[j], vf[j], nn);
#pragma unroll
            for (int r = 0; r < G; ++r) {
                const float4 oa = *reinterpret_cast<const float4*>(&sO[r][c * 8]);
                const float4 ob = *reinterpret_cast<const float4*>(&sO[r][c * 8 + 4]);
                tt[r] = __ffma2_rn(make_float2(oa.x, oa.y), vf[0], tt[r]); tt[r] = __ffma2_rn(make_float2(oa.z, oa.w), vf[1], tt[r]);
                tt[r] = __ffma2_rn(make_float2(ob.x, ob.y), vf[2], tt[r]); tt[r] = __ffma2_rn(make_float2(ob.z, ob.w), vf[3], tt[r]);
            }
        }
        nv = nn.x + nn.y;
#pragma unroll
        for (int r = 0; r < G; ++r) t[r] = tt[r].x + tt[r].y;
        const float* zbuf = (const float*)(ws + plan.off_z) + (size_t)unit * G * s.cap;
        float sc = 0.f;
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float z2 = zbuf[(size_t)r * s.cap + slot];
            const float a = exp2f(z2 - sLse[r]);
            const float Z = z2 * 0.6931471805599453f;          // back from log2 units: scale * q.k
            const float a2 = a * a;
            if (s.variant == OBC_VAR_V) sc = fmaf(a2, nv, sc);
            else if (s.variant == OBC_VAR_K) sc = fmaf(a2 * Z * Z, sNo[r] + nv - 2.f * t[r], sc);
            else if (s.variant == OBC_VAR_VK)
                sc += a2 * nv + a2 * Z * Z * (sNo[r] + nv - 2.f * t[r]) + 2.f * a2 * Z * (nv - t[r]);
            else sc += a;
        }
        const float acc = s_acc[(size_t)unit * s.cap + slot] + sc;
        s_acc[(size_t)unit * s.cap + slot] = acc;
        if (my_pos >= s.n_sink && my_pos <= step_pos - s.n_recent) cand = MinCand{acc, my_pos, slot, 0};
    }
    // argmin of (value, -pos): smallest accumulator, equal values -> highest position
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MinCand other;
        other.val = __shfl_xor_sync(0xffffffffu, cand.val, o);
        other.pos = __shfl_xor_sync(0xffffffffu, cand.pos, o);
        other.slot = __shfl_xor_sync(0xffffffffu, cand.slot, o);
        if (other.slot >= 0 && (cand.slot < 0 || other.val < cand.val || (other.val == cand.val && other.pos > cand.pos)))
            { cand.val = other.val; cand.pos = other.pos; cand.slot = other.slot; }
    }
    if (lane == 0) sMin[warp] = cand;
    __syncthreads();
    if (tid == 0) {
        MinCand best = sMin[0];
        for (int w = 1; w < 8; ++w) {
            const MinCand o2 = sMin[w];
            if (o2.slot >= 0 && (best.slot < 0 || o2.val < best.val || (o2.val == best.val && o2.pos > best.pos))) best = o2;
        }
        *part_min = best;
    }
}

__global__ void __launch_bounds__(128)
decode_final_kernel(DecodeShape s, DecodePlan plan, int32_t* pos, int32_t* state, const char* ws) {
    pdl_wait();
    const int unit = blockIdx.x * blockDim.x + threadIdx.x;
    if (unit >= s.B * s.Hkv) return;
    int live = state[unit * 4 + 0];
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];
    const bool valid = next >= 0 && next < s.cap;
    if (!valid) { state[unit * 4 + 3] = 1; return; }       // no room: the step was not applied
    const int hi = max(hi_old, next + 1);
    live += 1;
    int new_next = hi;
    if (live > s.budget) {
        const MinCand* pm = (const MinCand*)(ws + plan.off_min) + (size_t)unit * plan.chunks;
        MinCand best{INFINITY, -1, -1, 0};
        for (int ch = 0; ch < plan.chunks; ++ch) {
            const MinCand o2 = pm[ch];
            if (o2.slot >= 0 && (best.slot < 0 || o2.val < best.val || (o2.val == best.val && o2.pos > best.pos))) best = o2;
        }
        if (best.slot >= 0) {
            pos[(size_t)unit * s.cap + best.slot] = -1;
            live -= 1;
            new_next = best.slot;
        }
    }
    state[unit * 4 + 0] = live;
    state[unit * 4 + 1] = new_next;
    state[unit * 4 + 2] = hi;
}

template <int G>
obc_status launch_g(const DecodeShape& s, const DecodePlan& plan, TensorView q, TensorView kt, TensorView vt,
                    TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                    int step_pos, char* ws, cudaStream_t stream) {
    const int units = s.B * s.Hkv;
    { ProfScope ps("decode_pass1", stream); OBC_CUDA_TRY(cudaFuncSetAttribute(decode_pass1_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStageBytes));
      OBC_CUDA_TRY(launch_pdl(decode_pass1_kernel<G>, dim3(plan.chunks, units), dim3(CH), kStageBytes, stream, 1, s, plan, q, kt, vt, kc, vc, s_acc, pos, state, step_pos, ws)); }
    { ProfScope ps("decode_combine", stream); OBC_CUDA_TRY(launch_pdl(decode_combine_kernel, dim3(units * s.G), dim3(kD), 0, stream, 1, s, plan, ws)); }
    { ProfScope ps("decode_score", stream); OBC_CUDA_TRY(cudaFuncSetAttribute(decode_score_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStageBytes));
      OBC_CUDA_TRY(launch_pdl(decode_score_kernel<G>, dim3(plan.chunks, units), dim3(CH), kStageBytes, stream, 1, s, plan, vc, s_acc, pos, state, step_pos, ws)); }
    { ProfScope ps("decode_final", stream); OBC_CUDA_TRY(launch_pdl(decode_final_kernel, dim3((units + 127) / 128), dim3(128), 0, stream, 1, s, plan, pos, state, ws)); }
    return OBC_OK;
}

}  // namespace

size_t decode_workspace_bytes(const DecodeShape& s) { return make_plan(s).bytes; }

obc_status launch_decode(const DecodeShape& s, TensorView q, TensorView kt, TensorView vt,
                         TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                         int step_pos, void* ws, cudaStream_t stream) {
    const DecodePlan plan = make_plan(s);
    char* w = (char*)ws;
#define OBC_DECODE_CASE(Gv) case Gv: return launch_g<Gv>(s, plan, q, kt, vt, kc, vc, s_acc, pos, state, step_pos, w, stream)
    switch (s.G) {
        OBC_DECODE_CASE(1); OBC_DECODE_CASE(2); OBC_DECODE_CASE(3); OBC_DECODE_CASE(4);
        OBC_DECODE_CASE(5); OBC_DECODE_CASE(6); OBC_DECODE_CASE(7); OBC_DECODE_CASE(8);
    }
#undef OBC_DECODE_CASE
    return OBC_ERR_UNSUPPORTED;
}

}  // namespace obc
