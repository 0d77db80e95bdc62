// Decode-time rescoring + eviction step (W = 1: only the newest query of each head scores the
// cache).  Sec. 3 "Decoding" / "Cache Eviction"; Sec. 4.2 (scores accumulated over steps);
// App. C.2.2 (sinks + recent window protected, one eviction per step once over budget).
//
// With G <= 8 score rows per KV head the contractions are thin (slots x heads x 128 channels) and
// the step is bound by HBM traffic.  A CTA takes one chunk of 128 slots of one KV head: the 256-byte
// K and V rows travel into shared memory as one tiled bulk copy per chunk (TMA, two 64-channel halves
// with the 128-byte swizzle) and the contractions run as warp-level m16n8k16 MMAs fed by ldmatrix; one
// thread per slot does the softmax and score arithmetic, and reductions over slots use warp shuffles.
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

constexpr int CH = 128;                  // slots per chunk = threads per block
constexpr int NWARP = CH / 32;
constexpr size_t kStageBytes = (size_t)CH * 256;   // one chunk of 256-byte rows in shared memory

struct DecodePlan {
    int chunks;
    size_t off_z, off_pm, off_pl, off_po, off_lse, off_no, off_o, off_ohi, off_olo, off_min, bytes;
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
    p.off_ohi = off; off = align_up(off + units * s.G * kD * 2, 256);     // o as bf16 high and low halves (o = hi + lo)
    p.off_olo = off; off = align_up(off + units * s.G * kD * 2, 256);
    p.off_min = off; off = align_up(off + units * p.chunks * 16, 256);
    p.bytes = off;
    return p;
}

struct MinCand { float val; int pos; int slot; int pad; };

__device__ __forceinline__ const __nv_bfloat16* bf_row(const TensorView& t, int b, int h, long long tok) {
    return reinterpret_cast<const __nv_bfloat16*>(t.ptr) + b * t.sb + h * t.sh + tok * t.st;
}

// ---- a chunk of cache rows as one tiled bulk copy ------------------------------------------------------
// Layout in shared memory: two halves of [CH rows][128 bytes] (channels 0-63, 64-127); the 16-byte piece c of a
// half's row r lands at piece c ^ (r & 7) (the 128-byte swizzle), so the eight rows of an 8x8 ldmatrix tile fall
// into distinct banks.  Rows past the cache's capacity arrive as zeros; rows past the live extent hold whatever
// the cache holds there and are zeroed by the CTA where they could reach an MMA as values.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void chunk_bar_init(uint64_t* bar) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// hint: 0 = default L2 policy, 1 = evict first (rows that are not read again this step), 2 = evict last
__device__ __forceinline__ void copy_chunk_tma(uint4* dst, const CUtensorMap* map, uint64_t* bar, int b, int g, int c0, int hint = 0) {
    const uint32_t d = smem_addr(dst), mb = smem_addr(bar);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mb), "r"((uint32_t)kStageBytes) : "memory");
    if (hint) {
        uint64_t pol;
        if (hint == 1) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
        else asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
        asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
                     ::"r"(d), "l"(map), "r"(mb), "r"(0), "r"(c0), "r"(g), "r"(b), "l"(pol) : "memory");
        asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
                     ::"r"(d + (uint32_t)(kStageBytes / 2)), "l"(map), "r"(mb), "r"(64), "r"(c0), "r"(g), "r"(b), "l"(pol) : "memory");
        return;
    }
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(d), "l"(map), "r"(mb), "r"(0), "r"(c0), "r"(g), "r"(b) : "memory");
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(d + (uint32_t)(kStageBytes / 2)), "l"(map), "r"(mb), "r"(64), "r"(c0), "r"(g), "r"(b) : "memory");
}
// bounded wait for the copy of the given phase: false after two seconds
__device__ __forceinline__ bool chunk_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t mb = smem_addr(bar);
    unsigned long long t0 = 0;
    for (;;) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(mb), "r"(parity) : "memory");
        if (ok) return true;
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (!t0) t0 = now;
        else if (now - t0 > 2000000000ull) return false;
    }
}
// piece `piece` (0..15) of staged row `row`
__device__ __forceinline__ int staged_piece(int row, int piece) {
    return (piece >> 3) * (CH * 8) + row * 8 + ((piece & 7) ^ (row & 7));
}

// ---- warp-level tensor-core pieces ------------------------------------------------------------------
// The contractions of a chunk are tiny (256 slots x at most 8 heads x 128 channels) and the kernels are
// bound by memory traffic, but on CUDA cores their instruction count (about 3000 per thread and chunk)
// was what limited the blocks in flight.  One m16n8k16 MMA per 16 slots and 16 channels replaces 128
// multiply-adds per lane; the operands come out of the staged rows with ldmatrix (the 16-byte pieces of
// the swizzled rows are exactly its 8x8 tiles).
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void* p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
// d += a (16x16, row-major) * b (16x8, column-major), bf16 operands, fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// address of the 8x8 tile that lane `lane` names for an x4 load covering 16 staged rows from `row0` and the two
// 16-byte pieces `piece0`, `piece0 + 1`.  rows_major: tiles ordered (rows 0-7, p0), (rows 8-15, p0), (rows 0-7, p1),
// (rows 8-15, p1), the A operand of slots x channels; otherwise (rows 0-7, p0), (rows 0-7, p1), (rows 8-15, p0), ...
__device__ __forceinline__ const uint4* tile_addr(const uint4* sRows, int row0, int piece0, int lane, bool rows_major) {
    const int mi = lane >> 3, rr = lane & 7;
    const int row = row0 + (rows_major ? (mi & 1) : (mi >> 1)) * 8 + rr;
    const int piece = piece0 + (rows_major ? (mi >> 1) : (mi & 1));
    return sRows + staged_piece(row, piece);
}
// x = hi + lo with both halves bf16: two MMAs then carry an fp32 operand to about 16 bits
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

// The chunks arrive as tiled bulk copies through the two tensor maps.  A bulk copy that does not complete within its
// time limit is reported in the unit's state word 3 (value 2).
template <int G>
__global__ void __launch_bounds__(CH)
decode_pass1_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    DecodeShape s, DecodePlan plan, TensorView q, TensorView kt, TensorView vt,
                    TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                    int step_pos, char* ws) {
    extern __shared__ __align__(16) uint4 sStageRaw[];                  // [CH][16]: the chunk's K rows, later its V rows
    uint4* sStage = reinterpret_cast<uint4*>(((uintptr_t)sStageRaw + 1023) & ~(uintptr_t)1023);   // the swizzle's 1024-byte frame
    __shared__ uint64_t sBar;
    if (threadIdx.x == 0) chunk_bar_init(&sBar);
    __syncthreads();                                           // the barrier is initialised for every waiter
    // this is the step's first kernel: the kernel before it in the stream may be the caller's and may have written the
    // cache (the compaction that fills it, for one), so nothing is read before the wait
    pdl_wait();
    if (threadIdx.x == 0)
        copy_chunk_tma(sStage, &map_k, &sBar, blockIdx.y / s.Hkv, blockIdx.y % s.Hkv, blockIdx.x * CH, 1);              // K is read once per step
    __shared__ float sP[G][CH];
    __shared__ __align__(16) float sO[NWARP][G][kD];
    __shared__ float sRed[NWARP][G];
    __shared__ float sM[G];

    const int unit = blockIdx.y, chunk = blockIdx.x, c0 = chunk * CH;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];
    const bool valid = next >= 0 && next < s.cap;
    const int hi = valid ? max(hi_old, next + 1) : hi_old;

    float* part_m = (float*)(ws + plan.off_pm) + ((size_t)unit * plan.chunks + chunk) * G;
    float* part_l = (float*)(ws + plan.off_pl) + ((size_t)unit * plan.chunks + chunk) * G;
    bool copy_failed = false;
    if (c0 >= hi) {
        if (tid < G) { part_m[tid] = -INFINITY; part_l[tid] = 0.f; }
        if (tid == 0 && !chunk_wait(&sBar, 0)) atomicMax(&state[unit * 4 + 3], 2);   // no copy may be under way when the CTA leaves
        return;
    }
    // B operand of the logits: lane (n = lane / 4, t = lane % 4) holds q_n[16 ks + 2t .. +1] and [.. + 8 .. +9]
    uint32_t qf[8][2];
    {
        const int n = lane >> 2, t = lane & 3;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(bf_row(q, b, g * G + (n < G ? n : 0), 0));
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qf[ks][0] = n < G ? qrow[ks * 8 + t] : 0u;
            qf[ks][1] = n < G ? qrow[ks * 8 + 4 + t] : 0u;
        }
    }
    if (valid && next >= c0 && next < c0 + CH) {       // this chunk owns the slot of the new token
        __nv_bfloat16* kdst = const_cast<__nv_bfloat16*>(bf_row(kc, b, g, next));
        __nv_bfloat16* vdst = const_cast<__nv_bfloat16*>(bf_row(vc, b, g, next));
        if (tid < 16) reinterpret_cast<uint4*>(kdst)[tid] = reinterpret_cast<const uint4*>(bf_row(kt, b, g, 0))[tid];
        else if (tid < 32) reinterpret_cast<uint4*>(vdst)[tid - 16] = reinterpret_cast<const uint4*>(bf_row(vt, b, g, 0))[tid - 16];
        else if (tid == 32) { pos[(size_t)unit * s.cap + next] = step_pos; s_acc[(size_t)unit * s.cap + next] = 0.f; }
        // a token that enters the cache starts with an empty score history (the slot's former tenant left its own)
        for (int r = tid; r < s.acc_window; r += CH) s.s_hist[((size_t)unit * s.acc_window + r) * s.cap + next] = 0.f;
    }
    __syncthreads();                                       // the new token's row is in place
    // One buffer: the K rows first; the V rows take their place as soon as the logits are out and travel during
    // the softmax arithmetic.  (Half the shared memory per CTA lets more CTAs of the SM overlap their round trips.)
    const uint4* sRows = sStage;
    const uint4* sVrows = sStage;
    const int slot = c0 + tid;
    const bool live = slot < hi && ((valid && slot == next) || pos[(size_t)unit * s.cap + slot] >= 0);
    const bool owns_new = valid && next >= c0 && next < c0 + CH;
    copy_failed = !chunk_wait(&sBar, 0);
    // the bulk copy was asked for before the new token's row was written: put that row in place here
    if (owns_new && tid < 16)
        sStage[staged_piece(next - c0, tid)] = reinterpret_cast<const uint4*>(bf_row(kt, b, g, 0))[tid];
    __syncthreads();
    const float sl2 = s.scale * kLog2e;
    // logits of the warp's 32 slots: two 16-slot tiles, eight 16-channel steps each
#pragma unroll
    for (int tile = 0; tile < 2; ++tile) {
        const int row0 = warp * 32 + tile * 16;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a[4];
            ldsm_x4(a, tile_addr(sRows, row0, 2 * ks, lane, true));
            mma_bf16(acc, a, qf[ks][0], qf[ks][1]);
        }
        // acc[0], acc[1]: slot row0 + lane / 4, heads 2 (lane % 4), + 1; acc[2], acc[3]: slot + 8
        const int sl = row0 + (lane >> 2), h0 = 2 * (lane & 3);
        if (h0 < G) { sP[h0][sl] = acc[0]; sP[h0][sl + 8] = acc[2]; }
        if (h0 + 1 < G) { sP[h0 + 1][sl] = acc[1]; sP[h0 + 1][sl + 8] = acc[3]; }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // this thread's writes to the buffer precede the bulk copy into it
    __syncthreads();                                       // the K rows are no longer read
    if (tid == 0) copy_chunk_tma(sStage, &map_v, &sBar, b, g, c0, 2);   // V is read again by the score kernel
    float z2[G];
#pragma unroll
    for (int r = 0; r < G; ++r) z2[r] = sP[r][tid];        // this thread's slot; sP[.][tid] is rewritten below by this thread only
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
        for (int w = 0; w < NWARP; ++w) m = fmaxf(m, sRed[w][tid]);
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
    copy_failed |= !chunk_wait(&sBar, 1);
    if (owns_new && tid < 16)
        sStage[staged_piece(next - c0, tid)] = reinterpret_cast<const uint4*>(bf_row(vt, b, g, 0))[tid];
    // rows at or beyond the live extent may hold anything, and 0 x NaN would spoil the outputs: zero them
    if (c0 + CH > hi)
        for (int i = tid; i < CH * 16; i += CH) if (c0 + (i >> 4) >= hi) sStage[staged_piece(i >> 4, i & 15)] = make_uint4(0, 0, 0, 0);
    if (copy_failed) atomicMax(&state[unit * 4 + 3], 2);
    __syncthreads();                                       // sRed reads done, sP complete, V rows staged
#pragma unroll
    for (int r = 0; r < G; ++r) if (lane == 0) sRed[warp][r] = lsum[r];

    // partial outputs of the warp's 32 slots, transposed: (16 channels) x (8 heads) tiles of V^T P^T.  The
    // probabilities enter as bf16 high and low halves; slots without a live token carry p = 0.
    {
        uint32_t ph[2][2], pl[2][2];                       // [16-slot step][k half]: p of head lane / 4, slots 2 (lane % 4), + 1 (+ 8)
        const int n = lane >> 2, t = lane & 3;
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int sl = warp * 32 + kk * 16 + hf * 8 + 2 * t;
                const float p0 = n < G ? sP[n][sl] : 0.f, p1 = n < G ? sP[n][sl + 1] : 0.f;
                split_bf16x2(p0, p1, ph[kk][hf], pl[kk][hf]);
            }
#pragma unroll
        for (int j = 0; j < 8; ++j) {                      // channels 16 j .. 16 j + 15
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                uint32_t a[4];
                ldsm_x4_trans(a, tile_addr(sVrows, warp * 32 + kk * 16, 2 * j, lane, false));
                mma_bf16(acc, a, ph[kk][0], ph[kk][1]);
                mma_bf16(acc, a, pl[kk][0], pl[kk][1]);
            }
            // acc[0], acc[1]: channel 16 j + lane / 4, heads 2 (lane % 4), + 1; acc[2], acc[3]: channel + 8
            const int ch = 16 * j + (lane >> 2), h0 = 2 * t;
            if (h0 < G) { sO[warp][h0][ch] = acc[0]; sO[warp][h0][ch + 8] = acc[2]; }
            if (h0 + 1 < G) { sO[warp][h0 + 1][ch] = acc[1]; sO[warp][h0 + 1][ch + 8] = acc[3]; }
        }
    }
    __syncthreads();
    float* part_o = (float*)(ws + plan.off_po) + ((size_t)unit * plan.chunks + chunk) * G * kD;
    for (int i = tid; i < G * kD; i += CH) {
        const int r = i / kD, c = i % kD;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) acc += sO[w][r][c];
        part_o[i] = acc;
    }
    if (tid < G) {
        float l = 0.f;
        for (int w = 0; w < NWARP; ++w) l += sRed[w][tid];
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
    // the statistics of chunk c (and c + 128, ...) are read once; the partial outputs are requested CMB at a
    // time before their weights are known (a chunk without a live slot wrote none: its value is dropped, not
    // multiplied), so the block costs a couple of round trips to L2 however many chunks there are
    constexpr int CMB = 20;
    float M = -INFINITY;
    for (int ch = c; ch < plan.chunks; ch += kD) M = fmaxf(M, pm[(size_t)ch * G]);
    float first[CMB];
#pragma unroll
    for (int u = 0; u < CMB; ++u) first[u] = u < plan.chunks ? po[(size_t)u * G * kD] : 0.f;
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
        for (int j0 = 0; j0 < cnt; j0 += CMB) {
            float o[CMB];
            if (base == 0 && j0 == 0) {
#pragma unroll
                for (int u = 0; u < CMB; ++u) o[u] = first[u];
            } else {
#pragma unroll
                for (int u = 0; u < CMB; ++u) o[u] = j0 + u < cnt ? po[(size_t)(base + j0 + u) * G * kD] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < CMB; ++u) {
                const float wu = j0 + u < cnt ? sW[j0 + u] : 0.f;
                oc = wu != 0.f ? fmaf(o[u], wu, oc) : oc;
            }
        }
    }
    L = decode_block_reduce(L, false, red);
    oc = L > 0.f ? oc / L : 0.f;
    const float sq = decode_block_reduce(oc * oc, false, red);
    ((float*)(ws + plan.off_o))[((size_t)unit * G + r) * kD + c] = oc;
    {   // the score kernel's MMA operand: o to about 16 bits as two bf16 halves
        const __nv_bfloat16 hi = __float2bfloat16_rn(oc);
        // stored in the order the score kernel's MMA lanes take them: the 32-bit word w = 8 ks + 4 hf + t (channels 2w, 2w + 1;
        // k step ks, half hf, lane-in-group t) goes to word 16 t + 2 ks + hf, so that a lane's sixteen words are four 16-byte loads
        const int w = c >> 1, wpos = (w & 3) * 16 + (w >> 3) * 2 + ((w >> 2) & 1);
        const size_t at = ((size_t)unit * G + r) * kD + wpos * 2 + (c & 1);
        ((__nv_bfloat16*)(ws + plan.off_ohi))[at] = hi;
        ((__nv_bfloat16*)(ws + plan.off_olo))[at] = __float2bfloat16_rn(oc - __bfloat162float(hi));
    }
    if (c == 0) {
        ((float*)(ws + plan.off_lse))[(size_t)unit * G + r] = M + log2f(L);
        ((float*)(ws + plan.off_no))[(size_t)unit * G + r] = sq;
    }
}

template <int G>
__global__ void __launch_bounds__(CH)
decode_score_kernel(const __grid_constant__ CUtensorMap map_v, DecodeShape s, DecodePlan plan, TensorView vc, float* s_acc,
                    const int32_t* pos, int32_t* state, int step_pos, char* ws) {
    extern __shared__ __align__(16) uint4 sRowsRaw[];                   // [CH][16]: the chunk's V rows
    uint4* sRows = reinterpret_cast<uint4*>(((uintptr_t)sRowsRaw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t sBar;
    __shared__ float sLse[G], sNo[G];
    __shared__ float sT[G + 1][CH];                                     // v_slot . o_r (r < G) and ||v_slot||^2
    __shared__ MinCand sMin[NWARP];

    // units and chunks are taken last to first: what the first kernel read last is what the L2 still holds (its V
    // copies ask to stay, its K copies and this kernel's V copies to go first): 65 -> 58 us on 256 units of 4097 slots
    const int unit = (int)(gridDim.y - 1 - blockIdx.y), chunk = (int)(gridDim.x - 1 - blockIdx.x), c0 = chunk * CH;
    const int b = unit / s.Hkv, g = unit % s.Hkv;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The V rows are requested before anything else, and before the wait on the preceding kernel: the cache
    // was last written two kernels back (the new token's row), and which rows are live is sorted out below.
    if (tid == 0) { chunk_bar_init(&sBar); copy_chunk_tma(sRows, &map_v, &sBar, b, g, c0, 1); }
    __syncthreads();                                       // the barrier is initialised for every waiter
    // Likewise this slot's position, logits and accumulator, all written two kernels back or earlier: asked for
    // whether or not the slot turns out to be live, so that no later load has to wait for an earlier one.
    const int slot = c0 + tid;
    const bool in_cache = slot < s.cap;
    const int pos_in = in_cache ? pos[(size_t)unit * s.cap + slot] : -1;
    const float* zbuf = (const float*)(ws + plan.off_z) + (size_t)unit * G * s.cap;
    float zin[G];
#pragma unroll
    for (int r = 0; r < G; ++r) zin[r] = in_cache ? zbuf[(size_t)r * s.cap + slot] : 0.f;
    const float acc_in = in_cache ? s_acc[(size_t)unit * s.cap + slot] : 0.f;
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];   // written by the preceding step's last kernel
    pdl_wait();
    const bool valid = next >= 0 && next < s.cap;
    const int hi = valid ? max(hi_old, next + 1) : hi_old;
    MinCand* part_min = (MinCand*)(ws + plan.off_min) + (size_t)unit * plan.chunks + chunk;
    if (c0 >= hi) {
        if (tid == 0) *part_min = MinCand{INFINITY, -1, -1, 0};
        // no copy may be under way when the CTA leaves
        if (tid == 0 && !chunk_wait(&sBar, 0)) atomicMax(&state[unit * 4 + 3], 2);
        return;
    }
    if (tid < G) {
        sLse[tid] = ((const float*)(ws + plan.off_lse))[(size_t)unit * G + tid];
        sNo[tid] = ((const float*)(ws + plan.off_no))[(size_t)unit * G + tid];
    }
    // B operand of v . o: lane (n = lane / 4, t = lane % 4) holds o_n[16 ks + 2t .. +1] and [.. + 8 .. +9],
    // each fp32 value as a bf16 high and low half (split once per step by the combine kernel)
    uint32_t oh[8][2], ol[8][2];
    {
        const int n = lane >> 2, t = lane & 3;
        const size_t row = ((size_t)unit * G + (n < G ? n : 0)) * (kD / 2) + t * 16;   // the lane's sixteen words, in (ks, hf) order
        const uint4* hrow = reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(ws + plan.off_ohi) + row);
        const uint4* lrow = reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(ws + plan.off_olo) + row);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const uint4 h4 = n < G ? hrow[q4] : make_uint4(0, 0, 0, 0), l4 = n < G ? lrow[q4] : make_uint4(0, 0, 0, 0);
            oh[2 * q4][0] = h4.x; oh[2 * q4][1] = h4.y; oh[2 * q4 + 1][0] = h4.z; oh[2 * q4 + 1][1] = h4.w;
            ol[2 * q4][0] = l4.x; ol[2 * q4][1] = l4.y; ol[2 * q4 + 1][0] = l4.z; ol[2 * q4 + 1][1] = l4.w;
        }
    }
    const int my_pos = slot < hi ? pos_in : -1;
    if (!chunk_wait(&sBar, 0)) atomicMax(&state[unit * 4 + 3], 2);
    __syncthreads();
    if (c0 + CH > hi) {                                    // rows beyond the live extent may hold anything: zero them
        for (int i = tid; i < CH * 16; i += CH) if (c0 + (i >> 4) >= hi) sRows[staged_piece(i >> 4, i & 15)] = make_uint4(0, 0, 0, 0);
        __syncthreads();
    }
    const bool live = my_pos >= 0;
    MinCand cand{INFINITY, -1, -1, 0};
    // v . o_r and ||v||^2 of the warp's 32 slots: two 16-slot tiles, eight 16-channel steps each.  The norms are
    // the diagonal of (tile) x (tile)^T, whose B operand is the tile's own A fragment.
#pragma unroll
    for (int tile = 0; tile < 2; ++tile) {
        const int row0 = warp * 32 + tile * 16;
        float acc[4] = {0.f, 0.f, 0.f, 0.f}, n_lo[4] = {0.f, 0.f, 0.f, 0.f}, n_hi[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a[4];
            ldsm_x4(a, tile_addr(sRows, row0, 2 * ks, lane, true));
            mma_bf16(acc, a, oh[ks][0], oh[ks][1]);
            mma_bf16(acc, a, ol[ks][0], ol[ks][1]);
            mma_bf16(n_lo, a, a[0], a[2]);                 // columns = slots row0 .. + 7
            mma_bf16(n_hi, a, a[1], a[3]);                 // columns = slots row0 + 8 .. + 15
        }
        // acc[0], acc[1]: slot row0 + lane / 4, heads 2 (lane % 4), + 1; acc[2], acc[3]: slot + 8
        const int gq = lane >> 2, tq = lane & 3, sl = row0 + gq, h0 = 2 * tq;
        if (h0 < G) { sT[h0][sl] = acc[0]; sT[h0][sl + 8] = acc[2]; }
        if (h0 + 1 < G) { sT[h0 + 1][sl] = acc[1]; sT[h0 + 1][sl + 8] = acc[3]; }
        // the lane whose column pair 2 tq, 2 tq + 1 contains its own row holds the diagonal entries
        if (tq == (gq >> 1)) {
            sT[G][sl] = (gq & 1) ? n_lo[1] : n_lo[0];
            sT[G][sl + 8] = (gq & 1) ? n_hi[3] : n_hi[2];
        }
    }
    __syncthreads();
    if (live) {
        float nv = sT[G][tid], t[G];
#pragma unroll
        for (int r = 0; r < G; ++r) t[r] = sT[r][tid];
        float sc = 0.f;
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const float z2 = zin[r];
            const float a = exp2f(z2 - sLse[r]);
            const float Z = z2 * 0.6931471805599453f;          // back from log2 units: scale * q.k
            const float a2 = a * a;
            if (s.variant == OBC_VAR_V) sc = fmaf(a2, nv, sc);
            else if (s.variant == OBC_VAR_K) sc = fmaf(a2 * Z * Z, sNo[r] + nv - 2.f * t[r], sc);
            else if (s.variant == OBC_VAR_VK)
                sc += a2 * nv + a2 * Z * Z * (sNo[r] + nv - 2.f * t[r]) + 2.f * a2 * Z * (nv - t[r]);
            else sc += a;
        }
        float acc = acc_in + sc;
        if (s.acc_window > 0) {                                // the last acc_window steps only, summed afresh in ring order
            float* hcol = s.s_hist + (size_t)unit * s.acc_window * s.cap + slot;
            const int now = step_pos % s.acc_window;
            acc = 0.f;
            for (int r0 = 0; r0 < s.acc_window; r0 += 8) {      // eight loads in flight
                float hv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) hv[u] = (r0 + u < s.acc_window && r0 + u != now) ? hcol[(size_t)(r0 + u) * s.cap] : 0.f;
#pragma unroll
                for (int u = 0; u < 8; ++u) acc += (r0 + u == now) ? sc : hv[u];
            }
            hcol[(size_t)now * s.cap] = sc;
        }
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
        for (int w = 1; w < NWARP; ++w) {
            const MinCand o2 = sMin[w];
            if (o2.slot >= 0 && (best.slot < 0 || o2.val < best.val || (o2.val == best.val && o2.pos > best.pos))) best = o2;
        }
        *part_min = best;
    }
}

// one warp per (b, g): the lanes read the chunks' candidates side by side and reduce them with shuffles
__global__ void __launch_bounds__(128)
decode_final_kernel(DecodeShape s, DecodePlan plan, int32_t* pos, int32_t* state, const char* ws) {
    pdl_wait();
    const int unit = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (unit >= s.B * s.Hkv) return;
    int live = state[unit * 4 + 0];
    const int next = state[unit * 4 + 1], hi_old = state[unit * 4 + 2];
    const bool valid = next >= 0 && next < s.cap;
    if (!valid) { if (lane == 0) state[unit * 4 + 3] = 1; return; }       // no room: the step was not applied
    const int hi = max(hi_old, next + 1);
    live += 1;
    int new_next = hi;
    if (live > s.budget) {                                   // uniform over the warp
        const MinCand* pm = (const MinCand*)(ws + plan.off_min) + (size_t)unit * plan.chunks;
        MinCand best{INFINITY, -1, -1, 0};
        for (int ch = lane; ch < plan.chunks; ch += 32) {
            const MinCand o2 = pm[ch];
            if (o2.slot >= 0 && (best.slot < 0 || o2.val < best.val || (o2.val == best.val && o2.pos > best.pos))) best = o2;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            MinCand other;
            other.val = __shfl_xor_sync(0xffffffffu, best.val, o);
            other.pos = __shfl_xor_sync(0xffffffffu, best.pos, o);
            other.slot = __shfl_xor_sync(0xffffffffu, best.slot, o);
            if (other.slot >= 0 && (best.slot < 0 || other.val < best.val || (other.val == best.val && other.pos > best.pos)))
                { best.val = other.val; best.pos = other.pos; best.slot = other.slot; }
        }
        if (best.slot >= 0) {
            if (lane == 0) pos[(size_t)unit * s.cap + best.slot] = -1;
            live -= 1;
            new_next = best.slot;
        }
    }
    if (lane == 0) {
        state[unit * 4 + 0] = live;
        state[unit * 4 + 1] = new_next;
        state[unit * 4 + 2] = hi;
    }
}

// a tensor map over a cache [B, Hkv, cap, d]: its base 16-byte aligned and its strides whole 16-byte units
bool cache_map(CUtensorMap* map, const TensorView& t, const DecodeShape& s) {
    if (((uintptr_t)t.ptr & 15) || (t.st & 7) || (t.sh & 7) || (t.sb & 7) || t.st < kD) return false;
    const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)s.cap, (uint64_t)s.Hkv, (uint64_t)s.B};
    const uint64_t strides[3] = {(uint64_t)t.st * 2, (uint64_t)(s.Hkv > 1 ? t.sh : t.st * s.cap) * 2,
                                 (uint64_t)(s.B > 1 ? t.sb : (s.Hkv > 1 ? t.sh * s.Hkv : t.st * s.cap)) * 2};
    return make_map(map, t.ptr, 4, dims, strides, CH);
}

template <int G>
obc_status launch_g(const DecodeShape& s, const DecodePlan& plan, const CUtensorMap& mk, const CUtensorMap& mv,
                    TensorView q, TensorView kt, TensorView vt,
                    TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                    int step_pos, char* ws, cudaStream_t stream) {
    const int units = s.B * s.Hkv;
    const size_t stage = kStageBytes + 1024;                            // + room to align the swizzled tile
    { ProfScope ps("decode_pass1", stream); OBC_CUDA_TRY(cudaFuncSetAttribute(decode_pass1_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage));
      OBC_CUDA_TRY(launch_pdl(decode_pass1_kernel<G>, dim3(plan.chunks, units), dim3(CH), stage, stream, 1, mk, mv, s, plan, q, kt, vt, kc, vc, s_acc, pos, state, step_pos, ws)); }
    { ProfScope ps("decode_combine", stream); OBC_CUDA_TRY(launch_pdl(decode_combine_kernel, dim3(units * s.G), dim3(kD), 0, stream, 1, s, plan, ws)); }
    { ProfScope ps("decode_score", stream); OBC_CUDA_TRY(cudaFuncSetAttribute(decode_score_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage));
      OBC_CUDA_TRY(launch_pdl(decode_score_kernel<G>, dim3(plan.chunks, units), dim3(CH), stage, stream, 1, mv, s, plan, vc, s_acc, pos, state, step_pos, ws)); }
    { ProfScope ps("decode_final", stream); OBC_CUDA_TRY(launch_pdl(decode_final_kernel, dim3((units + 3) / 4), dim3(128), 0, stream, 1, s, plan, pos, state, ws)); }
    return OBC_OK;
}

}  // namespace

size_t decode_workspace_bytes(const DecodeShape& s) { return make_plan(s).bytes; }

obc_status launch_decode(const DecodeShape& s, TensorView q, TensorView kt, TensorView vt,
                         TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                         int step_pos, void* ws, cudaStream_t stream) {
    const DecodePlan plan = make_plan(s);
    char* w = (char*)ws;
    // (the entry point has checked what a tensor map asks of the caches: 16-byte aligned base, strides whole 16-byte units)
    CUtensorMap mk, mv;
    if (!cache_map(&mk, kc, s) || !cache_map(&mv, vc, s)) { set_last_cuda_error((int)cudaErrorInvalidValue); return OBC_ERR_CUDA; }
#define OBC_DECODE_CASE(Gv) case Gv: return launch_g<Gv>(s, plan, mk, mv, q, kt, vt, kc, vc, s_acc, pos, state, step_pos, w, stream)
    switch (s.G) {
        OBC_DECODE_CASE(1); OBC_DECODE_CASE(2); OBC_DECODE_CASE(3); OBC_DECODE_CASE(4);
        OBC_DECODE_CASE(5); OBC_DECODE_CASE(6); OBC_DECODE_CASE(7); OBC_DECODE_CASE(8);
    }
#undef OBC_DECODE_CASE
    return OBC_ERR_UNSUPPORTED;
}

}  // namespace obc
