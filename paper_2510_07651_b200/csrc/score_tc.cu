// Tensor-core score path for bf16 caches (sm_100a: TMA + tcgen05 MMA with TMEM accumulators).
//
// Pass 2, the fused score kernel, runs here.  For one tile of 128 cached tokens and one chunk of
// up to 128 window rows it issues two contractions with the TOKENS on the MMA M dimension,
//     Z^T = K_tile . Q_chunk^T          (logits,           Sec. 3)
//     T'^T = V_tile . (-2 O_chunk)^T    (-2 v_p . o_r,     Algorithm 1's "VO" term)
// so that a TMEM lane holds one token and an epilogue thread sums that token's score terms
// (Eq. 4-6 in the expanded form of Algorithm 1) over all rows of the chunk serially in registers:
// the sum over window queries and the GQA group (App. A.5) needs no cross-thread reduction and no
// W x N matrix ever leaves the SM.
//
// Warp roles of the 640-thread CTA (persistent, one CTA per SM):
//   warp 0      TMA producer: K/V tiles into a 2-stage ring, Q / -2O when the unit changes
//   warp 1      MMA issuer (one elected lane), double-buffered TMEM accumulators (2 x 256 columns)
//   warps 2-3   idle when pass 1 ran (its two spare warps computed ||v_p||^2 with the V tile at hand);
//               otherwise (attention outputs supplied by the caller, or the l1 variant) the value norms of every tile
//   warps 4-11  epilogue of the even tiles, warps 12-19 epilogue of the odd tiles.  Each tile has two
//               warpgroups: both hold one token per thread (a warp reads the TMEM lanes 32 (warp mod 4) ..),
//               the first sums the first half of the window rows, the second the other half and hands
//               its sums over through shared memory; the first adds them and stores the token's scores.
//               (One warpgroup per tile spent most of its time waiting on its own dependent instructions:
//               an SM sub-partition then runs two epilogue warps; with four it hides them.)
//
// Every mbarrier wait is bounded: on a timeout the kernel raises the status word in the workspace
// header, stops issuing work, waits (bounded) for its own copies in flight, frees TMEM and returns.
#include "obc_common.cuh"

#include <cuda.h>
#include <cudaTypedefs.h>

namespace obc {
namespace {

constexpr int TILE = 128;                       // tokens per tile = MMA M
constexpr unsigned kAllVariants = OBC_VAR_V | OBC_VAR_K | OBC_VAR_VK | OBC_VAR_ATTN | OBC_VAR_VATP;
constexpr int NSTAGE = 2;
constexpr uint32_t kHalfBytes = 128 * 128;      // [128 rows][64 bf16] = 16 KB, one swizzle-128B block
constexpr uint32_t kOperandBytes = 2 * kHalfBytes;
constexpr int kThreads = 640;                   // single-chunk pass 2: 4 service warps + 4 epilogue warpgroups
constexpr int kThreadsBase = 384;               // the multi-chunk pass 2 keeps two epilogue warpgroups
constexpr unsigned long long kWaitNs = 2000000000ull;   // 2 s per wait

// ---- shared memory map (offsets from a 1024-byte aligned base) ------------------------------
constexpr uint32_t OFF_Q = 0;
constexpr uint32_t OFF_O = OFF_Q + kOperandBytes;
constexpr uint32_t OFF_K = OFF_O + kOperandBytes;                 // NSTAGE x 32 KB
constexpr uint32_t OFF_V = OFF_K + NSTAGE * kOperandBytes;        // NSTAGE x 32 KB
constexpr uint32_t OFF_CONST = OFF_V + NSTAGE * kOperandBytes;    // 16 epilogue warps x 32 float4 (row-pair constants of the warp's half)
constexpr int NSLOT = 4;                                          // ring depth of the per-tile value norms
constexpr uint32_t OFF_NV = OFF_CONST + 16 * 32 * 16;             // NSLOT x 128 x (||v||^2, ||v||_1), own-norm kernels only
constexpr int kNumSums = 7;                                       // running sums a token carries (RowSums)
constexpr uint32_t OFF_XCH = OFF_NV + NSLOT * TILE * 8;           // [tile parity][2][kNumSums][128] floats: the second half's sums
constexpr uint32_t OFF_BAR = OFF_XCH + 2 * 2 * kNumSums * TILE * 4;
constexpr uint32_t kNumBars = 2 * NSTAGE + 2 + 4 + 2 + 2 * NSLOT + 4;
constexpr uint32_t OFF_TMEM = OFF_BAR + kNumBars * 8;
constexpr uint32_t kSmemBytes = OFF_TMEM + 16 + 1024;             // + alignment slack

enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_QO_FULL = 2 * NSTAGE, BAR_QO_EMPTY = 2 * NSTAGE + 1,
       BAR_TM_FULL = 2 * NSTAGE + 2,      // [epilogue group][TMEM buffer]
       BAR_TM_EMPTY = 2 * NSTAGE + 6,     // [TMEM buffer]
       BAR_NV = 2 * NSTAGE + 8,           // [epilogue group][slot], own-norm kernels only
       BAR_XCH = 2 * NSTAGE + 8 + 2 * NSLOT };   // [tile parity][2]: the second row half's sums are in shared memory

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Device-side extent of a kernel: every CTA folds its first and last clock reading into two words of
// the workspace header (both by atomicMax, the start as its complement, so that zeros mean "no
// reading").  obc_score_kernel_spans() reads and zeroes them.
// (Taken by a thread that has nothing urgent to do at either end: thread 0 issues the first copies.)
__device__ __forceinline__ void span_begin(unsigned long long* span) {
    if (threadIdx.x == 96) atomicMax(span, ~global_ns());
}
__device__ __forceinline__ void span_end(unsigned long long* span) {
    if (threadIdx.x == 96) atomicMax(span + 1, global_ns());
}
// bounded wait: false after kWaitNs without completion
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try(bar, parity)) return true;
        if (global_ns() - t0 > kWaitNs) return false;
    }
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// the same copy with an L2 eviction-priority hint (a policy made by l2_policy_*)
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int c0, int c1, int c2, int c3, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptors: K-major operand with 128-byte swizzle = rows of 64 bf16 (128 B),
// 8-row groups 1024 B apart (the image a swizzle-128B TMA box of 64 elements x rows leaves).
// The MMA thread builds two descriptors per instruction, so they are kept cheap: the high word of a
// descriptor is a constant and the low word is (address >> 4) plus constant fields; shared memory
// addresses are below 256 KB, so adding a byte offset / 16 to the low word cannot carry out of the
// 14-bit address field.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);       // SBO 1024 B, version 1, 128-byte swizzle
__device__ __forceinline__ uint32_t desc_lo_k(uint32_t addr) { return (addr >> 4) | (1u << 16); }                     // K-major
__device__ __forceinline__ uint32_t desc_lo_mn(uint32_t addr) { return (addr >> 4) | ((kHalfBytes >> 4) << 16); }     // MN-major, LBO 16 KB
__device__ __forceinline__ uint64_t desc_make(uint32_t lo) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(kDescHi));
    return d;
}
__device__ __forceinline__ constexpr uint32_t desc_kstep(int ks, uint32_t half_bytes) {   // K step ks of a [rows][2 x 64] operand
    return (uint32_t)(ks >> 2) * (half_bytes >> 4) + (uint32_t)(ks & 3) * 2u;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128
__host__ __device__ constexpr uint32_t idesc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TILE >> 4) << 24);
}

struct TcParams {
    int B, Hkv, G, W, R, Nmax;
    const int32_t* seq_lens;
    const int32_t* mask_lens;                 // or nullptr: length the causal mask counts from (token-sharded caches)
    float scale;
    int causal;
    unsigned variants;
    int n_chunks, chunk_rows, rows_out;       // rows_out = n_chunks * chunk_rows
    const float* lse2;                        // [units][rows_out]
    const float4* cpair;                      // [units][rows_out / 2]: (-lse2_0, -lse2_1, |o_0|^2, |o_1|^2) per row pair
    const float* nv;                          // [units][Nmax]: ||v_p||^2 from pass 1
    const float* onorm;                       // [units][rows_out]
    float* scores;                            // [planes][units][Nmax]
    unsigned int* status;                     // device status word (workspace header)
    unsigned long long* span;                 // [2]: ~(earliest CTA start), latest CTA end, in globaltimer ns
    int l2_stream;                            // K/V copies carry the "evict first" L2 hint (their last use)
    int csplit;                               // multi-chunk kernel: CTAs that share the row chunks of one tile pair
    float* partial;                           // csplit > 1: [csplit][planes][units][Nmax] partial scores
};

// (a device-side length is clamped to [0, max_len]: the host cannot check it)
__device__ __forceinline__ int tc_seq_len_raw(const int32_t* lens, int b, int nmax) { return lens ? min(max(lens[b], 0), nmax) : nmax; }
__device__ __forceinline__ int tc_seq_len(const TcParams& p, int b) { return tc_seq_len_raw(p.seq_lens, b, p.Nmax); }
__device__ __forceinline__ int tc_mask_len(const TcParams& p, int b) { return p.mask_lens ? p.mask_lens[b] : tc_seq_len(p, b); }

// Last token that any of the window rows [r0, r1] of a unit sees (row r is query position N - W + r mod W
// of its head): tiles that begin after it contribute nothing to these rows and are not visited.  With a
// short window every chunk of rows reaches the end of the cache; with the whole sequence as the window
// (W = N) about half of the (row chunk, token tile) pairs drop out.
__device__ __forceinline__ int rows_last_token(int r0, int r1, int W, int N, int causal) {
    return (causal && r0 / W == r1 / W) ? N - W + (r1 % W) : N - 1;
}

// Multi-chunk pass 2 with the row chunks of a tile pair shared by `csplit` CTAs: position t of a unit with
// P pairs stands for pair zigzag(t mod P) and the chunks c = t / P, t / P + csplit, ...  The zigzag (first,
// last, second, second to last, ...) puts a pair that many rows see next to one that few rows see, so that
// the contiguous runs of positions that the CTAs take weigh about the same under a causal window.
__device__ __forceinline__ void split_position(int t, int positions_in_unit, int csplit, int& pair, int& cs) {
    if (csplit == 1) { pair = t; cs = 0; return; }
    const int P = positions_in_unit / csplit, q = t % P;
    cs = t / P;
    pair = (q & 1) ? P - 1 - (q >> 1) : (q >> 1);
}

// Walks the CTA's share of the token tiles.  All non-empty 128-token tiles of all (batch item,
// KV head) units, in (unit, tile) order, are cut into gridDim.x contiguous, equally long runs, so
// that a CTA stays inside one unit for as long as possible (its Q / O operands stay in shared
// memory) and ragged batches are balanced.  Every role of the CTA runs its own copy.
struct TileWalk {
    int unit, tile, tiles_in_unit;            // current position
    long long left;                           // positions still to visit, including the current one
    const TcParams* p;
    int span;                                 // consecutive tiles of a unit that one position stands for
    int reps;                                 // positions per such group of tiles (CTAs that share its row chunks)
    __device__ __forceinline__ int tiles_of(int b) const {
        return ((tc_seq_len(*p, b) + TILE - 1) / TILE + span - 1) / span * reps;
    }
    __device__ void init(const TcParams& prm, int tiles_per_position = 1, int positions_per_group = 1) {
        p = &prm; span = tiles_per_position; reps = positions_per_group;
        long long total = 0;
        if (p->seq_lens) { for (int b = 0; b < p->B; ++b) total += (long long)p->Hkv * tiles_of(b); }
        else total = (long long)p->B * p->Hkv * tiles_of(0);
        const long long lo = total * blockIdx.x / gridDim.x, hi = total * (blockIdx.x + 1) / gridDim.x;
        left = hi - lo;
        unit = 0; tile = 0; tiles_in_unit = 0;
        if (left <= 0) return;
        long long skip = lo;
        int b = 0;
        for (; b < p->B; ++b) {
            const long long blk = (long long)p->Hkv * tiles_of(b);
            if (skip < blk) break;
            skip -= blk;
        }
        tiles_in_unit = tiles_of(b);
        unit = b * p->Hkv + (int)(skip / tiles_in_unit);
        tile = (int)(skip % tiles_in_unit);
    }
    __device__ __forceinline__ bool done() const { return left <= 0; }
    __device__ __forceinline__ void next() {
        --left;
        if (++tile < tiles_in_unit || left <= 0) return;
        tile = 0;
        do { ++unit; tiles_in_unit = tiles_of(unit / p->Hkv); } while (tiles_in_unit == 0);
    }
};

__device__ __forceinline__ float2 bf16x2_to_f32x2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// waits for the TMEM loads of this thread; the registers are operands so that no use is moved above it
__device__ __forceinline__ void tc_wait_ld16x2(uint32_t (&a)[16], uint32_t (&b)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                   "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                   "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                   "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
                 :: "memory");
}

// ||v||^2 (and, with L1, ||v||_1) of row `tok` of a [128 tokens][128 bf16] tile stored as two
// swizzle-128B halves.  Any order of the row's 16-byte pieces gives the same sums; this one is free
// of bank conflicts when consecutive threads take consecutive rows.
template <bool L1>
__device__ __forceinline__ void value_norms(const uint8_t* vt, int tok, float& l2, float& l1) {
    float2 acc0 = make_float2(0.f, 0.f), acc1 = acc0, acc2 = acc0, acc3 = acc0, ab0 = acc0, ab1 = acc0;
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
            const uint4 u = *reinterpret_cast<const uint4*>(vt + h * kHalfBytes + tok * 128 + ((ch ^ (tok & 7)) << 4));
            const float2 f0 = bf16x2_to_f32x2(u.x), f1 = bf16x2_to_f32x2(u.y);
            const float2 f2 = bf16x2_to_f32x2(u.z), f3 = bf16x2_to_f32x2(u.w);
            acc0 = __ffma2_rn(f0, f0, acc0); acc1 = __ffma2_rn(f1, f1, acc1);
            acc2 = __ffma2_rn(f2, f2, acc2); acc3 = __ffma2_rn(f3, f3, acc3);
            if (L1) {
                ab0 = __fadd2_rn(ab0, __fadd2_rn(make_float2(fabsf(f0.x), fabsf(f0.y)), make_float2(fabsf(f1.x), fabsf(f1.y))));
                ab1 = __fadd2_rn(ab1, __fadd2_rn(make_float2(fabsf(f2.x), fabsf(f2.y)), make_float2(fabsf(f3.x), fabsf(f3.y))));
            }
        }
    const float2 sum = __fadd2_rn(__fadd2_rn(acc0, acc1), __fadd2_rn(acc2, acc3));
    l2 = sum.x + sum.y;
    const float2 sab = __fadd2_rn(ab0, ab1);
    l1 = sab.x + sab.y;
}

// Running sums of one token over the window rows, two rows per packed fp32x2 lane.  With
// a = A_rp, u = a z (z the unscaled logit), b = a + scale u = a (1 + Z):
//   Eq. 6   sum_r a^2 ||(1+Z) v - Z o_r||^2 = |v|^2 S1 + scale S2 + scale^2 S3
//   Eq. 5   sum_r a^2 Z^2 ||v - o_r||^2     = scale^2 (|v|^2 S5 + S3 + S4)
//   Eq. 4   |v|^2 S6;   attention-only: S7
// with S1 = sum b^2, S2 = sum u b t', S3 = sum u^2 |o_r|^2, S4 = sum u^2 t', S5 = sum u^2,
// S6 = sum a^2, S7 = sum a and t' = -2 v.o_r (the expanded norms of Algorithm 1).
struct RowSums { float2 s1, s2, s3, s4, s5, s6, s7; };

// 16 rows of one token: zr = logits, tr = -2 v.o_r, cst = per row pair (-lse2_0, -lse2_1, |o_0|^2, |o_1|^2);
// when only the joint score is computed (VARS == OBC_VAR_VK) the |o|^2 entries arrive multiplied by scale
template <unsigned VARS, bool MASKED>
__device__ __forceinline__ void score_rows16(const uint32_t (&zr)[16], const uint32_t (&tr)[16], const float4* cst,
                                             float2 sl2, float2 sc, RowSums& S, int ptok, int mask_base, int W, int& wi) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 cp = cst[i];
        const float2 z = make_float2(__uint_as_float(zr[2 * i]), __uint_as_float(zr[2 * i + 1]));
        const float2 t2 = make_float2(__uint_as_float(tr[2 * i]), __uint_as_float(tr[2 * i + 1]));
        float2 e = __ffma2_rn(z, sl2, make_float2(cp.x, cp.y));
        if (MASKED) {                                   // row r sees tokens p <= N - W + (r mod W)
            if (ptok > mask_base + wi) e.x = -INFINITY;
            wi = wi + 1 == W ? 0 : wi + 1;
            if (ptok > mask_base + wi) e.y = -INFINITY;
            wi = wi + 1 == W ? 0 : wi + 1;
        }
        const float2 a = make_float2(fast_exp2(e.x), fast_exp2(e.y));
        const float2 u = __fmul2_rn(a, z);
        if (VARS == OBC_VAR_VK) {
            // joint score alone: the constants hold scale |o_r|^2, and s2 collects u (b t' + u scale |o_r|^2),
            // i.e. S2 + scale S3 of the general form below, with one packed instruction less
            const float2 b = __ffma2_rn(u, sc, a);
            S.s1 = __ffma2_rn(b, b, S.s1);
            S.s2 = __ffma2_rn(u, __ffma2_rn(u, make_float2(cp.z, cp.w), __fmul2_rn(b, t2)), S.s2);
        } else if (VARS & OBC_VAR_VK) {
            const float2 b = __ffma2_rn(u, sc, a);
            S.s1 = __ffma2_rn(b, b, S.s1);
            S.s2 = __ffma2_rn(__fmul2_rn(u, b), t2, S.s2);
        }
        if ((VARS & (OBC_VAR_VK | OBC_VAR_K)) && VARS != OBC_VAR_VK) {
            const float2 uu = __fmul2_rn(u, u);
            S.s3 = __ffma2_rn(uu, make_float2(cp.z, cp.w), S.s3);
            if (VARS & OBC_VAR_K) { S.s4 = __ffma2_rn(uu, t2, S.s4); S.s5 = __fadd2_rn(uu, S.s5); }
        }
        if (VARS & OBC_VAR_V) S.s6 = __ffma2_rn(a, a, S.s6);
        if (VARS & (OBC_VAR_ATTN | OBC_VAR_VATP)) S.s7 = __fadd2_rn(a, S.s7);
    }
}

// One (tile, chunk) item of one token: all rows of the chunk, one batch of 16 rows in registers at a time.  (Loading
// the next batch ahead of the math, which doubles the registers, was slower in both kernels: the other epilogue
// warps of the SM sub-partition cover the wait for a batch.)
template <unsigned VARS, bool MASKED>
__device__ __forceinline__ void score_chunk(uint32_t zt, uint32_t tt, int chunk_rows, const float4* cst,
                                                 float2 sl2, float2 sc, RowSums& S, int ptok, int mask_base, int W, int wi) {
    uint32_t z0[16], t0[16];
#pragma unroll 1
    for (int c0 = 0; c0 < chunk_rows; c0 += 16) {
        tc_ld16(zt + c0, z0);
        tc_ld16(tt + c0, t0);
        tc_wait_ld16x2(z0, t0);
        score_rows16<VARS, MASKED>(z0, t0, cst + (c0 >> 1), sl2, sc, S, ptok, mask_base, W, wi);
    }
}

// VARS: variants this instantiation computes (a superset of p.variants).  OWN_NV: no pass 1 ran (the
// caller supplied the attention outputs), so warps 2-3 compute the value norms from the V tiles here.
template <unsigned VARS, bool OWN_NV>
__global__ void __launch_bounds__(kThreads, 1)
tc_pass2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o,
                const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                const __grid_constant__ TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + OFF_BAR;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_TMEM);
    float4* sConst = reinterpret_cast<float4*>(smem + OFF_CONST);   // [16 epilogue warps][32 row pairs]
    float2* sNv = reinterpret_cast<float2*>(smem + OFF_NV);         // [NSLOT][128] (||v||^2, ||v||_1)
    float* sXch = reinterpret_cast<float*>(smem + OFF_XCH);         // [tile parity][2][kNumSums][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    span_begin(p.span);
    const int units = p.B * p.Hkv;

    if (threadIdx.x == 0) {
        prefetch_tmap(&map_k); prefetch_tmap(&map_v); prefetch_tmap(&map_q); prefetch_tmap(&map_o);
        // a K/V stage is released by the MMA commit and, when the norms are computed here, by warps 2-3
        for (int i = 0; i < NSTAGE; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), OWN_NV ? 3 : 1); }
        if (OWN_NV) for (int i = 0; i < 2 * NSLOT; ++i) mbar_init(bar(BAR_NV + i), 2);
        mbar_init(bar(BAR_QO_FULL), 1); mbar_init(bar(BAR_QO_EMPTY), 1);
        for (int i = 0; i < 4; ++i) mbar_init(bar(BAR_TM_FULL + i), 1);
        for (int i = 0; i < 2; ++i) mbar_init(bar(BAR_TM_EMPTY + i), 8);
        for (int i = 0; i < 4; ++i) mbar_init(bar(BAR_XCH + i), 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + OFF_TMEM), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    bool failed = false;
    int fail_site = 0;                             // source line of the wait that gave up (status word)
    const uint32_t qo_bytes = (uint32_t)p.chunk_rows * 128u * 2u * 2u;   // Q and O chunks, two halves each

    // Every role walks the same tiles (TileWalk); all window rows of a unit (at most 128) are one chunk.
    // Tiles go to the two epilogue groups alternately.  What an epilogue group waits for (accumulators
    // ready) is signalled on barriers of its own, so that each waiter sees every phase of the barriers
    // it uses; a parity wait must never fall two phases behind.  ||v_p||^2 comes from pass 1 (or, with
    // OWN_NV, from warps 2-3 through a ring of NSLOT slots) and the per-row constants from the combine kernel.
    // `item` counts the (tile, chunk) pairs processed so far and indexes the smem stage, TMEM
    // buffer and constant-slot rings.
    TileWalk tw;
    tw.init(p);
    if (!(warp == 0 && lane == 0)) pdl_wait();       // the producer thread waits after its first K/V copies
    if (warp == 0) {
        // ===================================== TMA producer =====================================
        if (lane == 0) {
            uint32_t item = 0, qo_loads = 0;
            int qo_unit = -1;
            const uint64_t pol_stream = l2_policy_evict_first();
            for (; !tw.done() && !failed; tw.next()) {
                const int unit = tw.unit, b = unit / p.Hkv, g = unit % p.Hkv, t0 = tw.tile * TILE;
                const uint32_t st = item % NSTAGE, use = item / NSTAGE;
                if (!mbar_wait(bar(BAR_EMPTY + st), (use & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                mbar_expect_tx(bar(BAR_FULL + st), 2 * kOperandBytes);
                const uint32_t dk = sbase + OFF_K + st * kOperandBytes, dv = sbase + OFF_V + st * kOperandBytes;
                if (p.l2_stream) {                             // last use of the tile: it may leave the cache first
                    tma_load_4d_hint(dk, &map_k, bar(BAR_FULL + st), 0, t0, g, b, pol_stream);
                    tma_load_4d_hint(dk + kHalfBytes, &map_k, bar(BAR_FULL + st), 64, t0, g, b, pol_stream);
                    tma_load_4d_hint(dv, &map_v, bar(BAR_FULL + st), 0, t0, g, b, pol_stream);
                    tma_load_4d_hint(dv + kHalfBytes, &map_v, bar(BAR_FULL + st), 64, t0, g, b, pol_stream);
                } else {
                    tma_load_4d(dk, &map_k, bar(BAR_FULL + st), 0, t0, g, b);
                    tma_load_4d(dk + kHalfBytes, &map_k, bar(BAR_FULL + st), 64, t0, g, b);
                    tma_load_4d(dv, &map_v, bar(BAR_FULL + st), 0, t0, g, b);
                    tma_load_4d(dv + kHalfBytes, &map_v, bar(BAR_FULL + st), 64, t0, g, b);
                }
                // K, V and the sequence lengths were read by pass 1 of this call, so the first tile
                // may be fetched while the preceding kernel drains; -2 O is that kernel's output
                if (item == 0) pdl_wait();
                if (unit != qo_unit) {
                    if (!mbar_wait(bar(BAR_QO_EMPTY), (qo_loads & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                    mbar_expect_tx(bar(BAR_QO_FULL), qo_bytes);
                    const int qrow = (b * p.Hkv * p.G + g * p.G) * p.W;
                    const int orow = unit * p.rows_out;
                    tma_load_2d(sbase + OFF_Q, &map_q, bar(BAR_QO_FULL), 0, qrow);
                    tma_load_2d(sbase + OFF_Q + kHalfBytes, &map_q, bar(BAR_QO_FULL), 64, qrow);
                    tma_load_2d(sbase + OFF_O, &map_o, bar(BAR_QO_FULL), 0, orow);
                    tma_load_2d(sbase + OFF_O + kHalfBytes, &map_o, bar(BAR_QO_FULL), 64, orow);
                    qo_unit = unit; ++qo_loads;
                }
                ++item;
            }
            // drain: every copy this thread issued must have landed before the CTA may exit
            for (uint32_t back = 0; back < NSTAGE && back < item; ++back) {
                const uint32_t it = item - 1 - back;
                (void)mbar_wait(bar(BAR_FULL + it % NSTAGE), (it / NSTAGE) & 1);
            }
            if (qo_loads) (void)mbar_wait(bar(BAR_QO_FULL), (qo_loads - 1) & 1);
        }
    } else if (warp == 1) {
        // ===================================== MMA issuer =======================================
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(p.chunk_rows);
            uint32_t item = 0, qo_loads = 0, tile_seq = 0;
            int qo_unit = -1;
            for (; !tw.done() && !failed; tw.next(), ++tile_seq) {
                const int unit = tw.unit;
                const uint32_t owner = tile_seq & 1;               // epilogue group of this tile
                const bool new_qo = unit != qo_unit;
                if (new_qo) {
                    if (!mbar_wait(bar(BAR_QO_FULL), qo_loads & 1)) { failed = true; fail_site = __LINE__; break; }
                    qo_unit = unit; ++qo_loads;
                }
                const uint32_t st = item % NSTAGE, buf = item & 1;
                if (!mbar_wait(bar(BAR_FULL + st), (item / NSTAGE) & 1)) { failed = true; fail_site = __LINE__; break; }
                if (!mbar_wait(bar(BAR_TM_EMPTY + buf), ((item >> 1) & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                tc_fence_after();
                const uint32_t zt = tmem_base + buf * 256u, tt = zt + 128u;
                const uint32_t ak = desc_lo_k(sbase + OFF_K + st * kOperandBytes), av = desc_lo_k(sbase + OFF_V + st * kOperandBytes);
                const uint32_t bq = desc_lo_k(sbase + OFF_Q), bo = desc_lo_k(sbase + OFF_O);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)                 // d = 128 = 8 steps of K = 16
                    tc_mma(zt, desc_make(ak + desc_kstep(ks, kHalfBytes)), desc_make(bq + desc_kstep(ks, kHalfBytes)), idesc, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc_mma(tt, desc_make(av + desc_kstep(ks, kHalfBytes)), desc_make(bo + desc_kstep(ks, kHalfBytes)), idesc, ks > 0);
                tc_commit(bar(BAR_TM_FULL + owner * 2 + buf)); // accumulators ready for the tile's epilogue group
                tc_commit(bar(BAR_EMPTY + st));                // K/V stage no longer read by the MMA
                // Q / O may be overwritten once these MMAs are done, if the next item needs others
                const bool last_of_unit = tw.left > 1 && tw.tile + 1 == tw.tiles_in_unit;
                if (last_of_unit) tc_commit(bar(BAR_QO_EMPTY));
                ++item;
            }
        }
    } else if (warp < 4) {
        // ================= value norms of every tile (only when no pass 1 supplied them) ===========
        if (OWN_NV) {
            const int t64 = threadIdx.x - 64;                      // 0..63
            uint32_t item = 0;
            for (; !tw.done() && !failed; tw.next(), ++item) {
                const uint32_t st = item % NSTAGE, slot = item % NSLOT, owner = item & 1;
                if (!mbar_wait(bar(BAR_FULL + st), (item / NSTAGE) & 1)) { failed = true; fail_site = __LINE__; break; }
                const uint8_t* vt = smem + OFF_V + st * kOperandBytes;
                // slot `slot` was last read for the tile four back, whose owner took it into registers before
                // releasing the accumulators that the MMA of the tile two back (whose commit freed this stage) needed
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int tok = t64 + 64 * j;
                    float l2, l1;
                    value_norms<(VARS & OBC_VAR_VATP) != 0>(vt, tok, l2, l1);
                    sNv[slot * TILE + tok] = make_float2(l2, l1);
                }
                __syncwarp();
                if (lane == 0) { mbar_arrive(bar(BAR_NV + owner * NSLOT + slot)); mbar_arrive(bar(BAR_EMPTY + st)); }
            }
        }
    } else {
        // ======================================= epilogue =======================================
        const int wg = (warp - 4) >> 3;                            // 0: even tiles, 1: odd tiles
        const int half = ((warp - 4) >> 2) & 1;                    // 0: first half of the window rows (and the stores), 1: the rest
        const int lane_grp = warp & 3;                             // TMEM lanes 32*lane_grp .. +31
        const int tok = lane_grp * 32 + lane;                      // token within the tile
        // the chunk's rows in two runs of whole 16-row batches
        const int rows0 = min(p.chunk_rows, (p.chunk_rows / 2 + 15) / 16 * 16);
        const int r_begin = half ? rows0 : 0, r_count = half ? p.chunk_rows - rows0 : rows0;
        const float2 sl2 = make_float2(p.scale * kLog2e, p.scale * kLog2e), sc = make_float2(p.scale, p.scale);
        const size_t plane = (size_t)units * p.Nmax;
        uint32_t item = 0, tile_seq = 0, mine_seq = 0;
        uint32_t full_par = 0, nv_par = 0;                         // phase parity of this group's barriers, one bit each
        float4* my_const = sConst + (warp - 4) * 32;               // this warp's copy of its rows' constants
        int const_unit = -1;
        for (; !tw.done() && !failed; tw.next()) {
            const bool mine = (tile_seq & 1) == (uint32_t)wg;
            ++tile_seq;
            if (!mine) { ++item; continue; }
            const int unit = tw.unit, b = unit / p.Hkv;
            const int N = tc_seq_len(p, b), t0 = tw.tile * TILE;
            float* out = p.scores + (size_t)unit * p.Nmax;
            const int ptok = t0 + tok;
            // rows of the window that do not see this tile's last token need the causal mask
            const int Nm = tc_mask_len(p, b);
            const bool masked_tile = p.causal && (t0 + TILE - 1 > Nm - p.W);
            RowSums S;
            S.s1 = S.s2 = S.s3 = S.s4 = S.s5 = S.s6 = S.s7 = make_float2(0.f, 0.f);
            const uint32_t buf = item & 1;
            float nv = 0.f, nv1 = 0.f;                             // used after the row loop
            if (!OWN_NV && half == 0 && ptok < N) nv = p.nv[(size_t)unit * p.Nmax + ptok];
            if (unit != const_unit) {                              // at most once per unit: (-lse2, |o|^2) of the warp's row pairs
                __syncwarp();
                {
                    const int rp = (r_begin >> 1) + lane;          // row pair of the chunk
                    float4 c4 = lane * 2 < r_count ? p.cpair[(((size_t)unit * p.rows_out) >> 1) + rp] : make_float4(-INFINITY, -INFINITY, 0.f, 0.f);
                    if (VARS == OBC_VAR_VK) { c4.z *= p.scale; c4.w *= p.scale; }
                    my_const[lane] = c4;
                }
                __syncwarp();
                const_unit = unit;
            }
            if (!mbar_wait(bar(BAR_TM_FULL + wg * 2 + buf), (full_par >> buf) & 1)) { failed = true; fail_site = __LINE__; break; }
            full_par ^= 1u << buf;
            tc_fence_after();
            if (OWN_NV && half == 0) {                             // the norms of this tile (ready long before the accumulators)
                const uint32_t slot = item % NSLOT;
                if (!mbar_wait(bar(BAR_NV + wg * NSLOT + slot), (nv_par >> slot) & 1)) { failed = true; fail_site = __LINE__; break; }
                nv_par ^= 1u << slot;
                const float2 n21 = sNv[slot * TILE + tok];
                nv = n21.x; nv1 = n21.y;
            }
            const float4* cst = my_const;
            const uint32_t zt = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + buf * 256u + (uint32_t)r_begin, tt = zt + 128u;
            if (r_count > 0) {
                if (masked_tile)
                    score_chunk<VARS, true>(zt, tt, r_count, cst, sl2, sc, S, ptok, Nm - p.W, p.W, r_begin % p.W);
                else
                    score_chunk<VARS, false>(zt, tt, r_count, cst, sl2, sc, S, ptok, 0, 0, 0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_TM_EMPTY + buf));
            ++item;
            // the two row halves of the token meet: sums 1..7 of RowSums, packed lanes folded
            float sum[kNumSums] = {S.s1.x + S.s1.y, S.s2.x + S.s2.y, S.s3.x + S.s3.y, S.s4.x + S.s4.y,
                                   S.s5.x + S.s5.y, S.s6.x + S.s6.y, S.s7.x + S.s7.y};
            // slot xs was last used two of this group's tiles ago; the first half read it before it released the
            // accumulators of the tile after that one, without which the tile at hand could not have been computed
            const uint32_t xs = mine_seq & 1;
            float* xch = sXch + ((wg * 2 + xs) * kNumSums) * TILE + tok;
            if (half == 1) {
#pragma unroll
                for (int j = 0; j < kNumSums; ++j) {
                    const bool used = VARS == OBC_VAR_VK ? j < 2 : true;
                    if (used) xch[j * TILE] = sum[j];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_XCH + wg * 2 + xs));
                ++mine_seq;
                continue;
            }
            if (!mbar_wait(bar(BAR_XCH + wg * 2 + xs), (mine_seq >> 1) & 1)) { failed = true; fail_site = __LINE__; break; }
            ++mine_seq;
#pragma unroll
            for (int j = 0; j < kNumSums; ++j) {
                const bool used = VARS == OBC_VAR_VK ? j < 2 : true;
                if (used) sum[j] += xch[j * TILE];
            }
            if (ptok < p.Nmax) {
                const bool live = ptok < N;
                const float s2 = p.scale * p.scale;
                int pl = 0;
                if (p.variants & OBC_VAR_V)    out[(size_t)(pl++) * plane + ptok] = live ? nv * sum[5] : 0.f;
                if (p.variants & OBC_VAR_K)    out[(size_t)(pl++) * plane + ptok] =
                    live ? s2 * (fmaf(nv, sum[4], sum[2]) + sum[3]) : 0.f;
                if (p.variants & OBC_VAR_VK)   out[(size_t)(pl++) * plane + ptok] =
                    live ? fmaf(nv, sum[0], fmaf(p.scale, sum[1], s2 * sum[2])) : 0.f;
                if (p.variants & OBC_VAR_ATTN) out[(size_t)(pl++) * plane + ptok] = live ? sum[6] : 0.f;
                if (p.variants & OBC_VAR_VATP) out[(size_t)(pl++) * plane + ptok] = live ? nv1 * sum[6] : 0.f;
            }
        }
        // padding beyond the last tile of a shorter sequence: zeros
        if (p.seq_lens) {
            const int et = threadIdx.x - 128;                      // 0..511
            const int n_planes = __popc(p.variants);
            for (int unit = blockIdx.x; unit < units; unit += gridDim.x) {
                const int first = (tc_seq_len(p, unit / p.Hkv) + TILE - 1) / TILE * TILE;
                for (int pl = 0; pl < n_planes; ++pl)
                    for (int i = first + et; i < p.Nmax; i += 512) p.scores[(size_t)pl * plane + (size_t)unit * p.Nmax + i] = 0.f;
            }
        }
    }

    if (failed) atomicCAS(p.status, 0u, (unsigned)(fail_site > 0 ? fail_site : 1));   // the first failure is kept
    tc_fence_before();
    __syncthreads();
    span_end(p.span);
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// =================================================================================================
// Pass 2 for more than 128 window rows per KV head (e.g. GQA 7 x W 64 = 448).  The rows are cut
// into chunks of 64.  A CTA holds TWO consecutive token tiles of a unit in its two K/V stages and
// sweeps the row chunks over both: every Q / -2 O chunk (two buffers) is fetched once per tile pair
// and used by two MMA pairs with N = 64 (four TMEM buffers of Z 64 + T' 64 columns), so the fetch
// of the next chunk hides behind twice the tensor work.  Epilogue warpgroup j owns tile j of the
// pair: it sums all chunks of its 128 tokens in registers and stores their scores itself.
// =================================================================================================
constexpr int MC_ROWS = 64;                                       // window rows per chunk
constexpr uint32_t kHalfB64 = 64 * 128;                           // B operand block: [64 rows][64 bf16]
constexpr uint32_t kQoBuf = 4 * kHalfB64;                         // Q chunk (2 x 8 KB) + -2 O chunk (2 x 8 KB)
constexpr uint32_t MC_OFF_QO = 0;                                 // 2 buffers x 32 KB
constexpr uint32_t MC_OFF_K = MC_OFF_QO + 2 * kQoBuf;             // 2 tiles x 32 KB
constexpr uint32_t MC_OFF_V = MC_OFF_K + 2 * kOperandBytes;
constexpr uint32_t MC_OFF_NV = MC_OFF_V + 2 * kOperandBytes;      // [pair parity][tile of the pair][128] x (||v||^2, ||v||_1)
constexpr uint32_t MC_OFF_CONST = MC_OFF_NV + 4 * TILE * 8;       // 4 slots x 32 float4 (per chunk)
constexpr uint32_t MC_OFF_BAR = MC_OFF_CONST + 4 * 32 * 16;
enum { MC_FULL = 0, MC_EMPTY = 2, MC_QO_FULL = 4, MC_QO_EMPTY = 6, MC_TM_FULL = 8, MC_TM_EMPTY = 12,
       MC_NV = 16, MC_CONST = 18, MC_NBARS = 22 };
constexpr uint32_t MC_OFF_TMEM = MC_OFF_BAR + MC_NBARS * 8;
constexpr int kThreadsMulti = kThreadsBase + 32;                      // + warp 12: the second MMA-issuing thread
constexpr uint32_t kSmemMulti = MC_OFF_TMEM + 16 + 1024;

// SPLIT: the general walk (row chunks of a pair shared by several CTAs, hidden tile pairs skipped); without
// it every CTA takes whole pairs and every chunk, which is all a short window over a long cache needs.
template <unsigned VARS, bool SPLIT>
__global__ void __launch_bounds__(kThreadsMulti, 1)
tc_pass2_multi_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o,
                      const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const __grid_constant__ TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + MC_OFF_BAR;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + MC_OFF_TMEM);
    float2* sNv = reinterpret_cast<float2*>(smem + MC_OFF_NV);
    float* sConst = reinterpret_cast<float*>(smem + MC_OFF_CONST);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    span_begin(p.span);
    const int units = p.B * p.Hkv;
    const int nc = p.n_chunks;                                   // chunks of MC_ROWS rows

    if (threadIdx.x == 0) {
        prefetch_tmap(&map_k); prefetch_tmap(&map_v); prefetch_tmap(&map_q); prefetch_tmap(&map_o);
        // two threads issue the MMAs (see below), so what an MMA commit signals takes two arrivals
        for (int i = 0; i < 2; ++i) { mbar_init(bar(MC_FULL + i), 1); mbar_init(bar(MC_EMPTY + i), 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(MC_QO_FULL + i), 1); mbar_init(bar(MC_QO_EMPTY + i), 2); }
        for (int i = 0; i < 4; ++i) { mbar_init(bar(MC_TM_FULL + i), 2); mbar_init(bar(MC_TM_EMPTY + i), 4); }
        for (int i = 0; i < 2; ++i) mbar_init(bar(MC_NV + i), 2);
        for (int i = 0; i < 4; ++i) mbar_init(bar(MC_CONST + i), 2);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + MC_OFF_TMEM), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    bool failed = false;
    int fail_site = 0;                             // source line of the wait that gave up (status word)
    const uint32_t qo_bytes = MC_ROWS * 128u * 2u * 2u;

    // A position of the walk is a pair of tiles (2 * tw.tile + j, j = 0, 1; the second one may lie past
    // the end of a unit with an odd tile count: it is computed all the same and stores only zeros).
    // `pitem` counts positions, `citem` row chunks over all positions; the chunk's two MMA pairs are
    // items 2 * citem + j.  Rings: K/V stage j; Q/O buffer citem & 1; constant slot citem & 3; TMEM
    // buffer item & 3, so that epilogue group j always sees buffers j and j + 2.
    TileWalk tw;
    tw.init(p, 2, SPLIT ? p.csplit : 1);
    const int cstep = SPLIT ? p.csplit : 1;
    // a chunk of 64 rows can lose sight of a tile pair only if the window is longer than the chunk (with up to
    // 64 window rows per head every chunk holds some head's last query, which sees the whole cache)
    const bool may_skip = SPLIT && p.causal && p.W > MC_ROWS;
    if (!(warp == 0 && lane == 0)) pdl_wait();       // the producer thread waits after its first K/V copies
    if (warp == 0) {
        // ===================================== TMA producer =====================================
        if (lane == 0) {
            uint32_t pitem = 0, citem = 0;
            for (; !tw.done() && !failed; tw.next(), ++pitem) {
                const int unit = tw.unit, b = unit / p.Hkv, g = unit % p.Hkv;
                int pair, cs;
                if (SPLIT) split_position(tw.tile, tw.tiles_in_unit, cstep, pair, cs); else { pair = tw.tile; cs = 0; }
                for (int j = 0; j < 2 && !failed; ++j) {
                    if (!mbar_wait(bar(MC_EMPTY + j), (pitem & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                    const int t0 = (pair * 2 + j) * TILE;
                    mbar_expect_tx(bar(MC_FULL + j), 2 * kOperandBytes);
                    const uint32_t dk = sbase + MC_OFF_K + j * kOperandBytes, dv = sbase + MC_OFF_V + j * kOperandBytes;
                    tma_load_4d(dk, &map_k, bar(MC_FULL + j), 0, t0, g, b);
                    tma_load_4d(dk + kHalfBytes, &map_k, bar(MC_FULL + j), 64, t0, g, b);
                    tma_load_4d(dv, &map_v, bar(MC_FULL + j), 0, t0, g, b);
                    tma_load_4d(dv + kHalfBytes, &map_v, bar(MC_FULL + j), 64, t0, g, b);
                }
                if (pitem == 0) pdl_wait();                        // K and V were read by pass 1; -2 O is the preceding kernel's output
                const int pair_first = pair * 2 * TILE, Nu = tc_mask_len(p, b);
                for (int c = cs; c < nc && !failed; c += cstep) {
                    if (may_skip && rows_last_token(c * MC_ROWS, min(c * MC_ROWS + MC_ROWS, p.R) - 1, p.W, Nu, 1) < pair_first) continue;
                    const uint32_t qb = citem & 1;
                    if (!mbar_wait(bar(MC_QO_EMPTY + qb), ((citem >> 1) & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                    mbar_expect_tx(bar(MC_QO_FULL + qb), qo_bytes);
                    const int qrow = (b * p.Hkv * p.G + g * p.G) * p.W + c * MC_ROWS;
                    const int orow = unit * p.rows_out + c * MC_ROWS;
                    const uint32_t dq = sbase + MC_OFF_QO + qb * kQoBuf, dob = dq + 2 * kHalfB64;
                    tma_load_2d(dq, &map_q, bar(MC_QO_FULL + qb), 0, qrow);
                    tma_load_2d(dq + kHalfB64, &map_q, bar(MC_QO_FULL + qb), 64, qrow);
                    tma_load_2d(dob, &map_o, bar(MC_QO_FULL + qb), 0, orow);
                    tma_load_2d(dob + kHalfB64, &map_o, bar(MC_QO_FULL + qb), 64, orow);
                    ++citem;
                }
            }
            // drain: every copy this thread issued must have landed before the CTA may exit
            if (pitem > 0) {
                (void)mbar_wait(bar(MC_FULL + 0), (pitem - 1) & 1);
                (void)mbar_wait(bar(MC_FULL + 1), (pitem - 1) & 1);
            }
            for (uint32_t back = 0; back < 2 && back < citem; ++back) {
                const uint32_t it = citem - 1 - back;
                (void)mbar_wait(bar(MC_QO_FULL + (it & 1)), (it >> 1) & 1);
            }
        }
    } else if (warp == 1 || warp == 12) {
        // ===================================== MMA issuers ======================================
        // One thread gets a tcgen05.mma out about every 88 cycles here (it shares its scheduler with two epilogue
        // warps), and a 128x64x16 MMA keeps the tensor pipe busy for 32: so two threads issue, warp 1 the logits
        // Z = K Q^T and warp 12 the cross terms T' = V (-2 O)^T.  Each commits what it issued; the barriers that
        // an MMA commit signals count two arrivals.
        const bool z_side = warp == 1;
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(MC_ROWS);
            uint32_t pitem = 0, citem = 0;
            for (; !tw.done() && !failed; tw.next(), ++pitem) {
                if (!mbar_wait(bar(MC_FULL + 0), pitem & 1) || !mbar_wait(bar(MC_FULL + 1), pitem & 1)) { failed = true; fail_site = __LINE__; break; }
                int pair, cs;
                if (SPLIT) split_position(tw.tile, tw.tiles_in_unit, cstep, pair, cs); else { pair = tw.tile; cs = 0; }
                const int pair_first = pair * 2 * TILE, Nu = tc_mask_len(p, tw.unit / p.Hkv);
                for (int c = cs; c < nc && !failed; c += cstep) {
                    if (may_skip && rows_last_token(c * MC_ROWS, min(c * MC_ROWS + MC_ROWS, p.R) - 1, p.W, Nu, 1) < pair_first) continue;
                    const uint32_t qb = citem & 1;
                    if (!mbar_wait(bar(MC_QO_FULL + qb), (citem >> 1) & 1)) { failed = true; fail_site = __LINE__; break; }
                    const uint32_t bq = desc_lo_k(sbase + MC_OFF_QO + qb * kQoBuf), bo = bq + ((2 * kHalfB64) >> 4);
                    for (int j = 0; j < 2; ++j) {
                        const uint32_t item = 2 * citem + j, buf = item & 3;
                        if (!mbar_wait(bar(MC_TM_EMPTY + buf), ((item >> 2) & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                        tc_fence_after();
                        const uint32_t zt = tmem_base + buf * 128u, tt = zt + 64u;
                        const uint32_t ak = desc_lo_k(sbase + MC_OFF_K + j * kOperandBytes), av = desc_lo_k(sbase + MC_OFF_V + j * kOperandBytes);
                        if (z_side) {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)         // d = 128 = 8 steps of K = 16
                                tc_mma(zt, desc_make(ak + desc_kstep(ks, kHalfBytes)), desc_make(bq + desc_kstep(ks, kHalfB64)), idesc, ks > 0);
                        } else {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)
                                tc_mma(tt, desc_make(av + desc_kstep(ks, kHalfBytes)), desc_make(bo + desc_kstep(ks, kHalfB64)), idesc, ks > 0);
                        }
                        tc_commit(bar(MC_TM_FULL + buf));          // this thread's accumulator of the item is ready
                    }
                    if (failed) break;
                    tc_commit(bar(MC_QO_EMPTY + qb));              // this Q / O buffer may be refilled
                    ++citem;
                }
                if (!failed) { tc_commit(bar(MC_EMPTY + 0)); tc_commit(bar(MC_EMPTY + 1)); }   // both tiles no longer read
            }
        }
    } else if (warp < 4) {
        // ==================== ||v_p||^2 per tile, per-row constants per chunk ===================
        // At a new position the constants of the first chunk go out before the norms are computed: the epilogue needs
        // them as soon as the first accumulators are ready, the norms only when the position's last chunk is summed.
        const int t64 = threadIdx.x - 64;                          // 0..63
        uint32_t pitem = 0, citem = 0;
        for (; !tw.done() && !failed; tw.next(), ++pitem) {
            const int unit = tw.unit;
            auto norms = [&]() -> bool {
                for (int j = 0; j < 2; ++j) {
                    if (!mbar_wait(bar(MC_FULL + j), pitem & 1)) { fail_site = __LINE__; return false; }
                    const uint8_t* vt = smem + MC_OFF_V + j * kOperandBytes;
                    float2* nvdst = sNv + ((pitem & 1) * 2 + j) * TILE;
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int tok = t64 + 64 * jj;
                        float l2, l1;
                        value_norms<(VARS & OBC_VAR_VATP) != 0>(vt, tok, l2, l1);
                        nvdst[tok] = make_float2(l2, l1);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(MC_EMPTY + j));
                }
                if (lane == 0) mbar_arrive(bar(MC_NV + (pitem & 1)));
                return true;
            };
            bool norms_done = false;
            int pair, cs;
            if (SPLIT) split_position(tw.tile, tw.tiles_in_unit, cstep, pair, cs); else { pair = tw.tile; cs = 0; }
            const int pair_first = pair * 2 * TILE, Nu = tc_mask_len(p, unit / p.Hkv);
            for (int c = cs; c < nc && !failed; c += cstep) {
                if (may_skip && rows_last_token(c * MC_ROWS, min(c * MC_ROWS + MC_ROWS, p.R) - 1, p.W, Nu, 1) < pair_first) continue;
                const uint32_t cs = citem & 3;
                const size_t crow = (size_t)unit * p.rows_out + (size_t)c * MC_ROWS + t64;
                const float2 cst = make_float2(-p.lse2[crow], p.onorm[crow] * (VARS == OBC_VAR_VK ? p.scale : 1.f));
                // slot cs was last read by the chunk four back; the chunk two back has been summed once
                // the TMEM buffers this chunk is going to use are free again
                const uint32_t i0 = 2 * citem, i1 = i0 + 1;
                if (!mbar_wait(bar(MC_TM_EMPTY + (i0 & 3)), ((i0 >> 2) & 1) ^ 1) ||
                    !mbar_wait(bar(MC_TM_EMPTY + (i1 & 3)), ((i1 >> 2) & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                float* cdst = sConst + cs * 128 + (t64 >> 1) * 4 + (t64 & 1);      // row pair: (-lse2_0, -lse2_1, |o_0|^2, |o_1|^2)
                cdst[0] = cst.x; cdst[2] = cst.y;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(MC_CONST + cs));
                ++citem;
                if (!norms_done) { norms_done = true; if (!norms()) { failed = true; break; } }
            }
            if (!failed && !norms_done && !norms()) failed = true;
        }
    } else if (warp < 12) {
        // ======================================= epilogue =======================================
        const int wg = (warp - 4) >> 2;                            // owns tile wg of every pair
        const int lane_grp = warp & 3;                             // TMEM lanes 32*lane_grp .. +31
        const int tok = lane_grp * 32 + lane;                      // token within the tile
        const float2 sl2 = make_float2(p.scale * kLog2e, p.scale * kLog2e), sc = make_float2(p.scale, p.scale);
        const size_t plane = (size_t)units * p.Nmax;
        uint32_t pitem = 0, citem = 0;
        for (; !tw.done() && !failed; tw.next(), ++pitem) {
            const int unit = tw.unit, b = unit / p.Hkv;
            int pair, cs;
            if (SPLIT) split_position(tw.tile, tw.tiles_in_unit, cstep, pair, cs); else { pair = tw.tile; cs = 0; }
            const int N = tc_seq_len(p, b), Nm = tc_mask_len(p, b), t0 = (pair * 2 + wg) * TILE;
            const int ptok = t0 + tok;
            const bool masked_tile = p.causal && (t0 + TILE - 1 > Nm - p.W);
            RowSums S;
            S.s1 = S.s2 = S.s3 = S.s4 = S.s5 = S.s6 = S.s7 = make_float2(0.f, 0.f);
            const int pair_first = pair * 2 * TILE;
            for (int c = cs; c < nc; c += cstep) {
                if (may_skip && rows_last_token(c * MC_ROWS, min(c * MC_ROWS + MC_ROWS, p.R) - 1, p.W, Nm, 1) < pair_first) continue;
                const uint32_t item = 2 * citem + wg, buf = item & 3, cs = citem & 3;
                if (!mbar_wait(bar(MC_CONST + cs), (citem >> 2) & 1)) { failed = true; fail_site = __LINE__; break; }
                if (!mbar_wait(bar(MC_TM_FULL + buf), (item >> 2) & 1)) { failed = true; fail_site = __LINE__; break; }
                tc_fence_after();
                const float4* cst = reinterpret_cast<const float4*>(sConst + cs * 128);
                const uint32_t zt = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + buf * 128u, tt = zt + 64u;
                // a chunk whose rows lie in one head sees the whole tile as soon as its first row does (with the whole
                // sequence as the window that is every item off the diagonal)
                bool use_mask = masked_tile;
                if (use_mask) {
                    const int wfirst = (c * MC_ROWS) % p.W;
                    if (wfirst + MC_ROWS <= p.W && t0 + TILE - 1 <= Nm - p.W + wfirst) use_mask = false;
                }
                if (use_mask)
                    score_chunk<VARS, true>(zt, tt, MC_ROWS, cst, sl2, sc, S, ptok, Nm - p.W, p.W, (c * MC_ROWS) % p.W);
                else
                    score_chunk<VARS, false>(zt, tt, MC_ROWS, cst, sl2, sc, S, ptok, 0, 0, 0);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(MC_TM_EMPTY + buf));
                ++citem;
            }
            if (failed) break;
            if (!mbar_wait(bar(MC_NV + (pitem & 1)), (pitem >> 1) & 1)) { failed = true; fail_site = __LINE__; break; }
            const float2 nv21 = sNv[((pitem & 1) * 2 + wg) * TILE + tok];
            const float nv = nv21.x, nv1 = nv21.y;
            if (ptok < p.Nmax) {
                // with the chunks of the pair shared by several CTAs each writes its part of the sums (the scores are
                // linear in them) into its own copy of the planes; tc_partial_sum_kernel adds the copies in order
                float* out = (cstep > 1 ? p.partial + (size_t)cs * __popc(p.variants) * plane : p.scores) + (size_t)unit * p.Nmax;
                const bool live = ptok < N;
                const float s2 = p.scale * p.scale;
                int pl = 0;
                if (p.variants & OBC_VAR_V)    out[(size_t)(pl++) * plane + ptok] = live ? nv * (S.s6.x + S.s6.y) : 0.f;
                if (p.variants & OBC_VAR_K)    out[(size_t)(pl++) * plane + ptok] =
                    live ? s2 * (fmaf(nv, S.s5.x + S.s5.y, S.s3.x + S.s3.y) + (S.s4.x + S.s4.y)) : 0.f;
                if (p.variants & OBC_VAR_VK)   out[(size_t)(pl++) * plane + ptok] =
                    live ? fmaf(nv, S.s1.x + S.s1.y, fmaf(p.scale, S.s2.x + S.s2.y, s2 * (S.s3.x + S.s3.y))) : 0.f;
                if (p.variants & OBC_VAR_ATTN) out[(size_t)(pl++) * plane + ptok] = live ? S.s7.x + S.s7.y : 0.f;
                if (p.variants & OBC_VAR_VATP) out[(size_t)(pl++) * plane + ptok] = live ? nv1 * (S.s7.x + S.s7.y) : 0.f;
            }
        }
        // padding beyond the last tile of a shorter sequence: zeros
        if (p.seq_lens) {
            const int et = threadIdx.x - 128;                      // 0..255
            const int n_planes = __popc(p.variants);
            for (int unit = blockIdx.x; unit < units; unit += gridDim.x) {
                const int first = (tc_seq_len(p, unit / p.Hkv) + TILE - 1) / TILE * TILE;
                for (int pl = 0; pl < n_planes; ++pl)
                    for (int i = first + et; i < p.Nmax; i += 256) p.scores[(size_t)pl * plane + (size_t)unit * p.Nmax + i] = 0.f;
            }
        }
    }

    if (failed) atomicCAS(p.status, 0u, (unsigned)(fail_site > 0 ? fail_site : 1));   // the first failure is kept
    tc_fence_before();
    __syncthreads();
    span_end(p.span);
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// scores = sum over the csplit partial copies, in order, for the tokens that pass 2 visited (whole tile
// pairs up to the unit's length; the zero padding beyond is written by pass 2 itself)
__global__ void __launch_bounds__(256)
tc_partial_sum_kernel(TcParams p, int n_planes) {
    pdl_wait();
    const int unit = blockIdx.y, b = unit / p.Hkv;
    const int N = tc_seq_len(p, b);
    const int end = min((N + 2 * TILE - 1) / (2 * TILE) * (2 * TILE), p.Nmax);
    const size_t plane = (size_t)p.B * p.Hkv * p.Nmax;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < end; i += gridDim.x * blockDim.x)
        for (int pl = 0; pl < n_planes; ++pl) {
            const size_t at = (size_t)pl * plane + (size_t)unit * p.Nmax + i;
            float sum = 0.f;
            for (int cs = 0; cs < p.csplit; ++cs) sum += p.partial[(size_t)cs * n_planes * plane + at];
            p.scores[at] = sum;
        }
}

// =================================================================================================
// Pass 1 on tensor cores: streaming softmax statistics and window outputs (Sec. 3: A = softmax(Z),
// O = A V over the perturbation window, Eq. 9), split over the cached tokens.
//
// Rows of the window (one chunk of up to 128) sit on the MMA M dimension, so a TMEM lane holds one
// row and the softmax thread that owns it reduces along the tile without cross-thread traffic.
// Two softmax warpgroups take alternate token tiles; each keeps its own running statistics and its
// own output accumulator; at the end the CTA merges the two and writes one partial result per
// token split, which the combine kernel merges across splits.  For tile t and warpgroup w = t mod 2:
//     S_w  = Q_chunk . K_tile^T                    (tcgen05, accumulator in TMEM)
//     P_w  = exp2(S_w * scale*log2e - m_used)      (registers -> bf16 -> TMEM, over S_w's columns)
//     O_w += P_w . V_tile                          (tcgen05: A operand from TMEM, V as MN-major B)
// m_used is the exponent reference of the row; it is only moved up (and O_w, l rescaled) when the
// tile maximum exceeds it by more than 8 (a factor 256), which keeps P within bf16/fp32 range.
// MMAs issued by one thread execute in order, so S_w of tile t+2 cannot overwrite P_w before
// P_w . V of tile t has read it, and a commit after S_w(t) also covers P_w . V of tile t-2.
//
//   warp 0      TMA producer (Q chunk once, K/V tiles into a 3-stage ring)
//   warp 1      MMA issuer
//   warps 4-7   softmax warpgroup 0 (even tiles), warps 8-11 softmax warpgroup 1 (odd tiles)
// TMEM columns: S_0 [0,128)  S_1 [128,256)  O_0 [256,384)  O_1 [384,512)
// =================================================================================================
constexpr int kThreadsP1 = 384;
constexpr int P1_NSTAGE = 3;
constexpr uint32_t P1_OFF_Q = 0;
constexpr uint32_t P1_OFF_K = P1_OFF_Q + kOperandBytes;
constexpr uint32_t P1_OFF_V = P1_OFF_K + P1_NSTAGE * kOperandBytes;
constexpr uint32_t P1_OFF_BAR = P1_OFF_V + P1_NSTAGE * kOperandBytes;
enum { P1_FULL = 0, P1_EMPTY = P1_NSTAGE, P1_QFULL = 2 * P1_NSTAGE, P1_SFULL = 2 * P1_NSTAGE + 1,
       P1_PFULL = 2 * P1_NSTAGE + 3, P1_ODONE = 2 * P1_NSTAGE + 5, P1_NBARS = 2 * P1_NSTAGE + 6 };
constexpr uint32_t P1_OFF_TMEM = P1_OFF_BAR + P1_NBARS * 8;
constexpr uint32_t kSmemP1 = P1_OFF_TMEM + 16 + 1024;
constexpr float kRescaleThreshold = 8.f;                   // log2 units

struct P1Params {
    int B, Hq, Hkv, G, W, R, Nmax;
    const int32_t* seq_lens;
    const int32_t* mask_lens;                              // or nullptr: length the causal mask counts from
    float scale;
    int causal;
    int n_chunks, chunk_rows;
    int n_splits, tiles_per_split;                         // CTAs per (unit, chunk); each writes one partial
    int l2_stream;                                         // K/V copies carry the "evict first" L2 hint
    float* part_m; float* part_l; float* part_o;           // [units][n_splits][R] (x d for part_o)
    float* nv;                                             // [units][Nmax]: ||v_p||^2, written by the CTAs of the last row chunk; null: not wanted
    unsigned int* status;
    unsigned long long* span;                              // [2]: ~(earliest CTA start), latest CTA end, in globaltimer ns
    // One CTA per (unit, row chunk) and no padding rows: the CTA writes the merged results itself (what the combine
    // kernel would make of its single partial) and no combine kernel runs.  Null out_o: partial results as above.
    float* out_o; __nv_bfloat16* out_obf;                  // [units][R][d]: O and -2 O
    float* out_lse2; float* out_onorm; float* out_cpair;   // [units][R]; row-pair constants as float4 per pair
};

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
// waits for this thread's TMEM loads; the registers are operands so that no use is moved above it
__device__ __forceinline__ void tc_wait_ld32(uint32_t* r) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]: the A operand (rows on lanes, K packed two bf16 per column) is read from TMEM
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// (V as the MN-major B operand of P.V: 64 contiguous head-dim elements per 128-byte row, 8 tokens per
// 1024-byte group = stride byte offset, the next 64 head-dim elements one 16 KB block further = leading
// byte offset: the image of a [tokens][head_dim] tile loaded as two 64-wide boxes; see desc_lo_mn.)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Row chunk of a block.  Under a causal window a chunk of rows visits the tiles up to its last row's position;
// with more CTAs than SMs the chunks that visit most tiles are handed out first.  When the chunks do not
// straddle heads (cph chunks per head), blocks are ordered by the chunk's place within its head, last place
// first; otherwise by chunk, last first.
__device__ __forceinline__ void p1_chunk_of_block(const P1Params& p, int vu, int& unit, int& c) {
    const int cph = p.W / p.chunk_rows;
    if (p.causal && p.n_chunks > 1 && p.W % p.chunk_rows == 0 && p.G * cph == p.n_chunks) {
        const int per_place = p.B * p.Hkv * p.G;
        const int place = cph - 1 - vu / per_place, rest = vu % per_place;
        unit = rest / p.G;
        c = (rest % p.G) * cph + place;
        return;
    }
    unit = vu / p.n_chunks;
    c = p.n_chunks - 1 - vu % p.n_chunks;
}

__global__ void __launch_bounds__(kThreadsP1, 1)
tc_pass1_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ P1Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + P1_OFF_BAR;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + P1_OFF_TMEM);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    span_begin(p.span);

    const int split = blockIdx.x;
    int unit, c;
    p1_chunk_of_block(p, blockIdx.y, unit, c);
    const int b = unit / p.Hkv, g = unit % p.Hkv;
    const bool nv_job = p.nv != nullptr && c == p.n_chunks - 1;     // this CTA also writes ||v_p||^2 of the tiles it visits
    if (threadIdx.x == 0) {
        prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
        // a K/V stage is released by the MMA commit and, where they are at work, by the two ||v||^2 warps
        for (int i = 0; i < P1_NSTAGE; ++i) { mbar_init(bar(P1_FULL + i), 1); mbar_init(bar(P1_EMPTY + i), nv_job ? 3 : 1); }
        mbar_init(bar(P1_QFULL), 1); mbar_init(bar(P1_ODONE), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar(P1_SFULL + i), 1); mbar_init(bar(P1_PFULL + i), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + P1_OFF_TMEM), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    int fail_site = 0;                             // source line of the wait that gave up (status word)
    pdl_wait();                                    // above, only the span words of the workspace header were touched (atomically)
    // the status word starts at 0: no wait of this call can have given up yet (each lasts seconds)
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *p.status = 0u;
    const int N = tc_seq_len_raw(p.seq_lens, b, p.Nmax);
    // a split past the end of a shorter sequence has nothing to do and the merge does not read its partial result
    // (the lengths may be the preceding kernel's output, so they are read after the wait)
    const bool idle_split = split > 0 && split * p.tiles_per_split * TILE >= N;
    const int tile_lo = split * p.tiles_per_split;
    // tiles past the last token that any row of this chunk sees are not visited
    const int Nm = p.mask_lens ? p.mask_lens[b] : N;       // a shard of a longer sequence: its distance to that sequence's end
    const int chunk_last = rows_last_token(c * p.chunk_rows, min((c + 1) * p.chunk_rows, p.R) - 1, p.W, Nm, p.causal);
    const int tile_hi = min(min(tile_lo + p.tiles_per_split, (N + TILE - 1) / TILE), chunk_last / TILE + 1);
    const int n_tiles = max(tile_hi - tile_lo, 0);

    if (idle_split) {
        // nothing to compute and nothing to store
    } else if (warp == 0) {
        // ===================================== TMA producer =====================================
        if (lane == 0 && n_tiles > 0) {
            mbar_expect_tx(bar(P1_QFULL), (uint32_t)p.chunk_rows * 256u);
            const int qrow = (b * p.Hq + g * p.G) * p.W + c * p.chunk_rows;
            tma_load_2d(sbase + P1_OFF_Q, &map_q, bar(P1_QFULL), 0, qrow);
            tma_load_2d(sbase + P1_OFF_Q + kHalfBytes, &map_q, bar(P1_QFULL), 64, qrow);
            int issued = 0;
            const uint64_t pol_stream = l2_policy_evict_first();
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t st = i % P1_NSTAGE;
                if (!mbar_wait(bar(P1_EMPTY + st), ((i / P1_NSTAGE) & 1) ^ 1)) { failed = true; fail_site = __LINE__; break; }
                mbar_expect_tx(bar(P1_FULL + st), 2 * kOperandBytes);
                const uint32_t dk = sbase + P1_OFF_K + st * kOperandBytes, dv = sbase + P1_OFF_V + st * kOperandBytes;
                const int t0 = (tile_lo + i) * TILE;
                if (p.l2_stream) {                             // the cache cannot hold K and V until pass 2 anyway
                    tma_load_4d_hint(dk, &map_k, bar(P1_FULL + st), 0, t0, g, b, pol_stream);
                    tma_load_4d_hint(dk + kHalfBytes, &map_k, bar(P1_FULL + st), 64, t0, g, b, pol_stream);
                    tma_load_4d_hint(dv, &map_v, bar(P1_FULL + st), 0, t0, g, b, pol_stream);
                    tma_load_4d_hint(dv + kHalfBytes, &map_v, bar(P1_FULL + st), 64, t0, g, b, pol_stream);
                } else {
                    tma_load_4d(dk, &map_k, bar(P1_FULL + st), 0, t0, g, b);
                    tma_load_4d(dk + kHalfBytes, &map_k, bar(P1_FULL + st), 64, t0, g, b);
                    tma_load_4d(dv, &map_v, bar(P1_FULL + st), 0, t0, g, b);
                    tma_load_4d(dv + kHalfBytes, &map_v, bar(P1_FULL + st), 64, t0, g, b);
                }
                ++issued;
            }
            for (int back = 0; back < P1_NSTAGE && back < issued; ++back) {   // drain own copies
                const int it = issued - 1 - back;
                (void)mbar_wait(bar(P1_FULL + it % P1_NSTAGE), (it / P1_NSTAGE) & 1);
            }
            (void)mbar_wait(bar(P1_QFULL), 0);
        }
    } else if (warp == 1) {
        // ===================================== MMA issuer =======================================
        if (lane == 0 && n_tiles > 0) {
            const uint32_t idesc_s = idesc_bf16(TILE);
            const uint32_t idesc_pv = idesc_bf16(kD) | (1u << 16);           // B operand (V) is MN-major
            auto issue_s = [&](int j) -> bool {                              // S_w = Q . K_j^T
                const uint32_t st = j % P1_NSTAGE;
                if (!mbar_wait(bar(P1_FULL + st), (j / P1_NSTAGE) & 1)) return false;
                tc_fence_after();
                const uint32_t ak = desc_lo_k(sbase + P1_OFF_K + st * kOperandBytes), aq = desc_lo_k(sbase + P1_OFF_Q);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc_mma(tmem_base + (j & 1) * 128u, desc_make(aq + desc_kstep(ks, kHalfBytes)), desc_make(ak + desc_kstep(ks, kHalfBytes)), idesc_s, ks > 0);
                tc_commit(bar(P1_SFULL + (j & 1)));
                return true;
            };
            failed = !mbar_wait(bar(P1_QFULL), 0);
            if (!failed) failed = !issue_s(0);
            if (!failed && n_tiles > 1) failed = !issue_s(1);
            if (failed) fail_site = __LINE__;
            for (int i = 0; i < n_tiles && !failed; ++i) {
                const uint32_t w = i & 1;
                if (!mbar_wait(bar(P1_PFULL + w), (i >> 1) & 1)) { failed = true; fail_site = __LINE__; break; }
                tc_fence_after();
                const uint32_t av = desc_lo_mn(sbase + P1_OFF_V + (i % P1_NSTAGE) * kOperandBytes);
                const uint32_t first = i > 1;                                // the warpgroup's first tile initialises O_w
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)                               // 128 tokens = 8 steps of K = 16 (2048 bytes of V each)
                    tc_mma_ts(tmem_base + 256u + w * 128u, tmem_base + w * 128u + ks * 8, desc_make(av + ks * (2048 >> 4)),
                              idesc_pv, ks > 0 ? 1u : first);
                tc_commit(bar(P1_EMPTY + (i % P1_NSTAGE)));                  // S(i) and P.V(i) have read the stage
                if (i + 2 < n_tiles && !issue_s(i + 2)) { failed = true; fail_site = __LINE__; break; }
            }
            if (!failed) tc_commit(bar(P1_ODONE));
        }
    } else if (warp < 4) {
        // ============ ||v_p||^2 of every cached token (CTAs of the last row chunk) ===============
        // Pass 2 needs it per token; the V tile is in shared memory here anyway, and these two warps
        // have nothing else to do, whereas in pass 2 every issue slot next to the epilogue counts.
        // (The last chunk holds the last window row, which sees every token, so its CTAs visit every tile.  The
        // pass-2 kernel for more than 128 window rows computes the norms itself: p.nv is null then.)
        if (nv_job) {
            const int t64 = threadIdx.x - 64;                                // 0..63
            for (int i = 0; i < n_tiles && !failed; ++i) {
                const uint32_t st = i % P1_NSTAGE;
                if (!mbar_wait(bar(P1_FULL + st), (i / P1_NSTAGE) & 1)) { failed = true; fail_site = __LINE__; break; }
                const uint8_t* vt = smem + P1_OFF_V + st * kOperandBytes;
                const int t0 = (tile_lo + i) * TILE;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int tok = t64 + 64 * j;
                    float2 acc0 = make_float2(0.f, 0.f), acc1 = acc0, acc2 = acc0, acc3 = acc0;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            const uint4 u = *reinterpret_cast<const uint4*>(vt + h * kHalfBytes + tok * 128 + ((ch ^ (tok & 7)) << 4));
                            const float2 f0 = bf16x2_to_f32x2(u.x), f1 = bf16x2_to_f32x2(u.y);
                            const float2 f2 = bf16x2_to_f32x2(u.z), f3 = bf16x2_to_f32x2(u.w);
                            acc0 = __ffma2_rn(f0, f0, acc0); acc1 = __ffma2_rn(f1, f1, acc1);
                            acc2 = __ffma2_rn(f2, f2, acc2); acc3 = __ffma2_rn(f3, f3, acc3);
                        }
                    const float2 sum = __fadd2_rn(__fadd2_rn(acc0, acc1), __fadd2_rn(acc2, acc3));
                    if (t0 + tok < p.Nmax) p.nv[(size_t)unit * p.Nmax + t0 + tok] = sum.x + sum.y;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(P1_EMPTY + st));
            }
        }
    } else {
        // ======================================= softmax ========================================
        const int w = (warp - 4) >> 2;                                       // warpgroup: tiles w, w+2, ...
        const int lane_grp = warp & 3;
        const int row = lane_grp * 32 + lane;                                // row within the chunk
        const int rows_valid = min(p.chunk_rows, p.R - c * p.chunk_rows);
        const int r = c * p.chunk_rows + row;
        const bool valid = row < rows_valid;
        const int last = valid ? (p.causal ? min(Nm - p.W + (r % p.W), N - 1) : N - 1) : -1;   // last visible token
        const int first_masked = min(p.causal ? Nm - p.W + 1 : N, N);        // tiles reaching it need the mask
        const float sl2 = p.scale * kLog2e;
        const uint32_t lane_addr = (uint32_t)(lane_grp * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + w * 128u, tO = tmem_base + lane_addr + 256u + w * 128u;
        float m_used = -INFINITY, l = 0.f;
        int my_tiles = 0;

        for (int i = w; i < n_tiles && !failed; i += 2, ++my_tiles) {
            const int t0 = (tile_lo + i) * TILE;
            if (!mbar_wait(bar(P1_SFULL + w), my_tiles & 1)) { failed = true; fail_site = __LINE__; break; }
            tc_fence_after();
            const int nvis = last - t0 + 1;                                  // columns j < nvis are visible
            // (a warp whose rows all see the whole tile skips the mask: under a whole-sequence window that is every tile off the diagonal)
            const bool masked = t0 + TILE > first_masked && __any_sync(0xffffffffu, nvis < TILE);

            // sweep 1: tile maximum of the row (raw logits; the scale is positive)
            float mt = -INFINITY;
            {
                uint32_t sa[32], sb[32];
                tc_ld32(tS, sa);
#pragma unroll
                for (int pc = 0; pc < 4; pc += 2) {
                    tc_wait_ld32(sa);
                    tc_ld32(tS + (pc + 1) * 32, sb);
                    if (masked) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (pc * 32 + j >= nvis) sa[j] = 0xff800000u;
                    }
#pragma unroll
                    for (int j = 0; j < 32; j += 2) mt = fmax3(mt, __uint_as_float(sa[j]), __uint_as_float(sa[j + 1]));
                    tc_wait_ld32(sb);
                    if (pc + 2 < 4) tc_ld32(tS + (pc + 2) * 32, sa);
                    if (masked) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) if ((pc + 1) * 32 + j >= nvis) sb[j] = 0xff800000u;
                    }
#pragma unroll
                    for (int j = 0; j < 32; j += 2) mt = fmax3(mt, __uint_as_float(sb[j]), __uint_as_float(sb[j + 1]));
                }
            }
            mt *= sl2;
            const bool need = mt > m_used + kRescaleThreshold;               // also true for the first visible tile
            const float factor = need ? fast_exp2(m_used - mt) : 1.f;        // m_used = -inf -> 0
            if (my_tiles > 0 && __any_sync(0xffffffffu, valid && need && m_used != -INFINITY)) {
                // P.V of this warpgroup's previous tile is complete (the commit that signalled S covers it)
#pragma unroll 1
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t ov[32];
                    tc_ld32(tO + q4 * 32, ov);
                    tc_wait_ld32(ov);
#pragma unroll
                    for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * factor);
                    tc_st32(tO + q4 * 32, ov);
                }
            }
            l *= factor;
            if (need) m_used = mt;
            const float m_eff = m_used == -INFINITY ? 0.f : m_used;
            const float2 sl2v = make_float2(sl2, sl2), negm = make_float2(-m_eff, -m_eff);

            // sweep 2: P = exp2(S * scale*log2e - m_used) as bf16 over the first 64 columns of S_w
            float2 lsum = make_float2(0.f, 0.f);
            {
                uint32_t sa[32], sb[32];
                auto piece = [&](uint32_t* sv, int pc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float2 x = make_float2(__uint_as_float(sv[j]), __uint_as_float(sv[j + 1]));
                        x = __ffma2_rn(x, sl2v, negm);
                        if (masked) {
                            if (pc * 32 + j >= nvis) x.x = -INFINITY;
                            if (pc * 32 + j + 1 >= nvis) x.y = -INFINITY;
                        }
                        const float2 e = make_float2(fast_exp2(x.x), fast_exp2(x.y));
                        lsum = __fadd2_rn(lsum, e);
                        pk[j >> 1] = pack_bf16x2(e.x, e.y);
                    }
                    tc_st16(tS + pc * 16, pk);
                };
                tc_ld32(tS, sa);
#pragma unroll
                for (int pc = 0; pc < 4; pc += 2) {
                    tc_wait_ld32(sa);
                    tc_ld32(tS + (pc + 1) * 32, sb);
                    piece(sa, pc);
                    tc_wait_ld32(sb);
                    if (pc + 2 < 4) tc_ld32(tS + (pc + 2) * 32, sa);
                    piece(sb, pc + 1);
                }
            }
            l += lsum.x + lsum.y;
            tc_wait_st();
            if (t0 + TILE > N && t0 + row >= N) {                            // tail: V rows past the sequence must not reach the MMA
                uint8_t* vrow = smem + P1_OFF_V + (i % P1_NSTAGE) * kOperandBytes + row * 128;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    *reinterpret_cast<uint4*>(vrow + (ch << 4)) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(vrow + kHalfBytes + (ch << 4)) = make_uint4(0, 0, 0, 0);
                }
                fence_async_smem();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P1_PFULL + w));
        }

        // ---- the CTA's partial result: merge the two warpgroups, then store whole 512-byte rows ----
        // A warp may read its 32 TMEM lanes in any column, so the thread of row r in either
        // warpgroup can read both accumulators of that row.  The warpgroups exchange (m, l) through
        // shared memory (the Q region, which the MMAs no longer read), then warpgroup w merges
        // head-dim columns [64 w, 64 w + 64) into a [128 rows][32 x 16 B] tile in the first K/V stage
        // (16-byte chunks XOR-swizzled by the row), and all eight warps store 512-byte rows.
        float* xm = reinterpret_cast<float*>(smem + P1_OFF_Q);               // [2][128]
        float* xl = xm + 256;                                                // [2][128]
        uint8_t* xo = smem + P1_OFF_K;
        bool have = my_tiles > 0 && !failed;
        if (n_tiles > 0) {                                                   // all MMAs done: accumulators final, smem free
            if (!mbar_wait(bar(P1_ODONE), 0)) { failed = true; fail_site = __LINE__; have = false; }
            tc_fence_after();
        }
        xm[w * 128 + row] = have ? m_used : -INFINITY;
        xl[w * 128 + row] = l;
        asm volatile("bar.sync 1, 256;" ::: "memory");                       // both softmax warpgroups
        {
            const float m0 = xm[row], m1 = xm[128 + row];
            const float M = fmaxf(m0, m1);
            const float f0 = m0 == -INFINITY ? 0.f : fast_exp2(m0 - M), f1 = m1 == -INFINITY ? 0.f : fast_exp2(m1 - M);
            const uint32_t tO0 = tmem_base + lane_addr + 256u + w * 64u, tO1 = tO0 + 128u;   // this half of O_0 and O_1
            const size_t prow0 = ((size_t)unit * p.n_splits + split) * p.R + (size_t)c * p.chunk_rows;   // row 0 of the chunk
            const bool fin = p.out_o != nullptr;
            const float Lrow = fmaf(xl[row], f0, xl[128 + row] * f1);
            // (L = 0: the row saw no token, which only a shard of a longer sequence can show)
            const float o_scale = fin ? (Lrow > 0.f ? 1.f / Lrow : 0.f) : 1.f;
            const float g0 = f0 * o_scale, g1 = f1 * o_scale;
            float sq = 0.f;                                                  // squared norm of this thread's 64 output columns
            if (w == 0 && valid && !fin) { p.part_m[prow0 + row] = M; p.part_l[prow0 + row] = Lrow; }
#pragma unroll 1
            for (int q = 0; q < 2; ++q) {
                // CTA-uniform: warpgroup 0 owns tiles iff the split has any, warpgroup 1 iff it has two or more
                // (an accumulator that no MMA wrote is never read; one whose row saw no token holds zeros)
                uint32_t oa[32], ob[32];
                if (n_tiles > 0) { tc_ld32(tO0 + q * 32, oa); tc_wait_ld32(oa); }
                if (n_tiles > 1) { tc_ld32(tO1 + q * 32, ob); tc_wait_ld32(ob); }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (n_tiles > 0)
                        o = make_float4(__uint_as_float(oa[4 * j]) * g0, __uint_as_float(oa[4 * j + 1]) * g0,
                                        __uint_as_float(oa[4 * j + 2]) * g0, __uint_as_float(oa[4 * j + 3]) * g0);
                    if (n_tiles > 1) {
                        o.x = fmaf(__uint_as_float(ob[4 * j]), g1, o.x);     o.y = fmaf(__uint_as_float(ob[4 * j + 1]), g1, o.y);
                        o.z = fmaf(__uint_as_float(ob[4 * j + 2]), g1, o.z); o.w = fmaf(__uint_as_float(ob[4 * j + 3]), g1, o.w);
                    }
                    sq = fmaf(o.x, o.x, fmaf(o.y, o.y, fmaf(o.z, o.z, fmaf(o.w, o.w, sq))));
                    const int chunk = w * 16 + q * 8 + j;
                    *reinterpret_cast<uint4*>(xo + row * 512 + ((chunk ^ (row & 31)) << 4)) =
                        make_uint4(__float_as_uint(o.x), __float_as_uint(o.y), __float_as_uint(o.z), __float_as_uint(o.w));
                }
            }
            float* xs = xl + 256;                                            // [2][128]: the two halves of ||o||^2; then [128] log2-sum-exp
            if (fin) {
                xs[w * 128 + row] = sq;
                if (w == 0) xs[256 + row] = M + log2f(Lrow);
            }
            asm volatile("bar.sync 2, 256;" ::: "memory");                   // the merged tile is complete
            const int row_lo = (warp - 4) * 16;                              // 8 warps x 16 rows
            uint4 rowv[16];
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) {
                const int orow = row_lo + rr;
                rowv[rr] = *reinterpret_cast<const uint4*>(xo + orow * 512 + ((lane ^ (orow & 31)) << 4));
            }
            if (fin) {
                // rows of the unit are rows of the outputs (one split, no padding rows): O, -2 O in bf16, and per row
                // the log2-sum-exp, ||o||^2 and the row's half of its pair's constants
#pragma unroll
                for (int rr = 0; rr < 16; ++rr) {
                    const int orow = row_lo + rr;
                    if (orow < rows_valid) {
                        *reinterpret_cast<uint4*>(p.out_o + (prow0 + orow) * kD + lane * 4) = rowv[rr];
                        const uint32_t b0 = pack_bf16x2(-2.f * __uint_as_float(rowv[rr].x), -2.f * __uint_as_float(rowv[rr].y));
                        const uint32_t b1 = pack_bf16x2(-2.f * __uint_as_float(rowv[rr].z), -2.f * __uint_as_float(rowv[rr].w));
                        *reinterpret_cast<uint2*>(p.out_obf + (prow0 + orow) * kD + lane * 4) = make_uint2(b0, b1);
                    }
                }
                if (lane < 16 && row_lo + lane < rows_valid) {
                    const int orow = row_lo + lane;
                    const size_t gr = prow0 + orow;
                    const float lse2 = xs[256 + orow], on = xs[orow] + xs[128 + orow];
                    p.out_lse2[gr] = lse2; p.out_onorm[gr] = on;
                    float* cp = p.out_cpair + (gr >> 1) * 4 + (gr & 1);
                    cp[0] = -lse2; cp[2] = on;
                }
            } else {
#pragma unroll
                for (int rr = 0; rr < 16; ++rr) {                            // one coalesced 512-byte row per instruction
                    const int orow = row_lo + rr;
                    if (orow < rows_valid) *reinterpret_cast<uint4*>(p.part_o + (prow0 + orow) * kD + lane * 4) = rowv[rr];
                }
            }
        }
        tc_fence_before();
    }

    if (failed) atomicCAS(p.status, 0u, (unsigned)(fail_site > 0 ? fail_site : 1));   // the first failure is kept
    tc_fence_before();
    __syncthreads();
    span_end(p.span);
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------------------------
// Row chunks.  Pass 1 cuts the R window rows into n_chunks pieces of chunk_rows <= 128 (its MMA M
// dimension).  Pass 2 takes the rows whole when R <= 128 and in pieces of 64 otherwise; rows_out is
// the padded row count of the combined arrays it reads.
struct TcChunks { int n_chunks, chunk_rows, rows_out; };
TcChunks tc_chunks(int R) {
    TcChunks c;
    c.n_chunks = (R + 127) / 128;
    c.chunk_rows = ((R + c.n_chunks - 1) / c.n_chunks + 15) / 16 * 16;
    c.rows_out = c.n_chunks > 1 ? (R + MC_ROWS - 1) / MC_ROWS * MC_ROWS : c.chunk_rows;
    return c;
}

size_t l2_bytes() {
    static size_t n = 0;
    if (!n) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev) != cudaSuccess || v <= 0) v = 126 << 20;
        n = (size_t)v;
    }
    return n;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 148;
    }
    return n;
}

}  // namespace

bool tc_shape_supported(const ScoreShape& s) { return s.R >= 64; }

bool tc_supported(const ScoreShape& s, int dtype, const TensorView& q) {
    if (dtype != OBC_BF16 || !tc_shape_supported(s)) return false;
    // the window rows of a KV head's group must be one uniformly strided run of rows
    return q.sh == (long long)s.W * q.st && q.sb == (long long)s.Hq * q.sh;
}

// Multi-chunk pass 2: with fewer tile pairs than about two per SM (a short cache scored over a long window)
// the row chunks of every pair are shared by several CTAs.
static int tc_chunk_split(const ScoreShape& s, const TcChunks& ch) {
    if (ch.n_chunks <= 1) return 1;
    const long long pairs = (long long)s.B * s.Hkv * (((s.Nmax + TILE - 1) / TILE + 1) / 2);
    const int nc = ch.rows_out / MC_ROWS, sms = sm_count();
    if (pairs >= 2LL * sms) return 1;
    // about seven positions per SM: on the 4k whole-sequence window 8 CTAs per pair took 272 us, 4 took 305, 3 took 326,
    // 12 took 270 and 16 took 282 (every position loads its tile pair again and adds a copy of the score planes)
    int c = (int)((7LL * sms + pairs - 1) / pairs);
    if (c > 8) c = 8;
    if (c > nc) c = nc;
    return c < 1 ? 1 : c;
}

// Workspace plan of the tensor-core path: the SIMT plan's layout with splits counted in 128-token tiles.
static SimtPlan make_tc_plan(const ScoreShape& s) {
    const TcChunks ch = tc_chunks(s.R);
    const int units = s.B * s.Hkv, vus = units * ch.n_chunks;
    const int tiles = (s.Nmax + TILE - 1) / TILE;
    int n = sm_count() / vus;                          // one wave of CTAs when the sequences are equal
    // (48 tiles per CTA: with 32 the ragged batch of 8 spent 6 % more in pass 1 on prologues and tails, with 64 the last wave ran half empty)
    if (s.seq_lens) { const int cap = (tiles + 47) / 48; if (cap > n) n = cap; }   // ragged: bound the work per CTA
    if (n < 1) n = 1;
    if (n > tiles) n = tiles;
    SimtPlan p{};
    p.tiles_per_split = (tiles + n - 1) / n;                                   // per pass-1 CTA
    p.n_splits = (tiles + p.tiles_per_split - 1) / p.tiles_per_split;          // CTAs, and partial results, per unit
    p.tile_tokens = TILE;
    p.rows_out = ch.rows_out;
    p.want_obf = 1;
    const size_t rows = (size_t)units * s.R, prow = rows * p.n_splits, orow = (size_t)units * ch.rows_out;
    size_t off = 0;
    p.off_flag = off;   off = 256;
    p.off_part_m = off; off = align_up(off + prow * 4, 256);
    p.off_part_l = off; off = align_up(off + prow * 4, 256);
    p.off_part_o = off; off = align_up(off + prow * kD * 4, 256);
    p.off_lse2 = off;   off = align_up(off + orow * 4, 256);
    p.off_onorm = off;  off = align_up(off + orow * 4, 256);
    p.off_o = off;      off = align_up(off + orow * kD * 4, 256);
    p.off_obf = off;    off = align_up(off + orow * kD * 2, 1024);
    p.off_cpair = off;  off = align_up(off + orow * 8, 256);
    p.off_nv = off;     off = align_up(off + (size_t)units * s.Nmax * 4, 256);
    p.bytes = off;
    return p;
}

// the partial score planes of a shared multi-chunk pass 2 follow the plan's arrays
static size_t tc_partial_bytes(const ScoreShape& s) {
    const int cs = tc_chunk_split(s, tc_chunks(s.R));
    return cs > 1 ? (size_t)cs * s.n_planes * s.B * s.Hkv * s.Nmax * 4 : 0;
}

size_t tc_workspace_bytes(const ScoreShape& s) { return make_tc_plan(s).bytes + tc_partial_bytes(s); }

obc_status launch_attention_tc(const ScoreShape& s, TensorView q, TensorView k, TensorView v, void* ws, cudaStream_t stream,
                               SimtPlan* plan_out) {
    return launch_score_tc(s, q, k, v, nullptr, ws, stream, nullptr, plan_out);
}

obc_status launch_score_tc(const ScoreShape& s, TensorView q, TensorView k, TensorView v,
                           float* scores, void* ws, cudaStream_t stream, const GivenAttention* given,
                           SimtPlan* attention_only) {
    const TcChunks ch = tc_chunks(s.R);
    const SimtPlan plan = make_tc_plan(s);
    char* wsb = (char*)ws;
    const int units = s.B * s.Hkv;
    CUtensorMap mq, mo, mk, mv;
    {
        const uint64_t qd[2] = {(uint64_t)kD, (uint64_t)s.B * s.Hq * s.W};
        const uint64_t qs[1] = {(uint64_t)q.st * 2};
        const uint64_t od[2] = {(uint64_t)kD, (uint64_t)units * ch.rows_out};
        const uint64_t os[1] = {(uint64_t)kD * 2};
        const uint64_t kd[4] = {(uint64_t)kD, (uint64_t)s.Nmax, (uint64_t)s.Hkv, (uint64_t)s.B};
        const uint64_t ks[3] = {(uint64_t)k.st * 2, (uint64_t)(s.Hkv > 1 ? k.sh : k.st * s.Nmax) * 2,
                                (uint64_t)(s.B > 1 ? k.sb : (s.Hkv > 1 ? k.sh * s.Hkv : k.st * s.Nmax)) * 2};
        const uint64_t vs[3] = {(uint64_t)v.st * 2, (uint64_t)(s.Hkv > 1 ? v.sh : v.st * s.Nmax) * 2,
                                (uint64_t)(s.B > 1 ? v.sb : (s.Hkv > 1 ? v.sh * s.Hkv : v.st * s.Nmax)) * 2};
        if (!make_map(&mq, q.ptr, 2, qd, qs, (uint32_t)ch.chunk_rows) ||
            !make_map(&mo, wsb + plan.off_obf, 2, od, os, (uint32_t)ch.chunk_rows) ||
            !make_map(&mk, k.ptr, 4, kd, ks, TILE) || !make_map(&mv, v.ptr, 4, kd, vs, TILE)) {
            set_last_cuda_error((int)cudaErrorInvalidValue);
            return OBC_ERR_CUDA;
        }
    }
    // A cache that cannot hold K and V from pass 1 to pass 2 is better streamed through: with the "evict
    // first" hint on the K/V copies pass 1 ran 2 us faster on the 32k Llama layer (134 MB against 126 MB of L2).
    // Smaller caches keep the default policy, so that pass 2 finds in L2 what pass 1 read.
    const bool l2_stream = ch.n_chunks == 1 && !given &&
        (double)units * s.Nmax * kD * 2 * 2 > 0.75 * (double)l2_bytes();
    if (given) {   // the caller's O and LSE take the place of pass 1 + combine; pass 2 computes the value norms itself
        obc_status st = launch_given_prep(s, plan, *given, ws, stream);
        if (st != OBC_OK) return st;
    } else {       // pass 1 + combine
        P1Params p1{};
        p1.B = s.B; p1.Hq = s.Hq; p1.Hkv = s.Hkv; p1.G = s.G; p1.W = s.W; p1.R = s.R; p1.Nmax = s.Nmax;
        p1.seq_lens = s.seq_lens; p1.mask_lens = s.mask_lens; p1.scale = s.scale; p1.causal = s.causal;
        p1.n_chunks = ch.n_chunks; p1.chunk_rows = ch.chunk_rows;
        p1.n_splits = plan.n_splits; p1.tiles_per_split = plan.tiles_per_split;
        p1.l2_stream = l2_stream ? 1 : 0;
        p1.part_m = (float*)(wsb + plan.off_part_m); p1.part_l = (float*)(wsb + plan.off_part_l);
        p1.part_o = (float*)(wsb + plan.off_part_o);
        // only the single-chunk pass 2 without the l1 plane reads the norms that pass 1 leaves
        const bool want_nv = ch.n_chunks == 1 && !attention_only && !(s.variants & OBC_VAR_VATP);
        p1.nv = want_nv ? (float*)(wsb + plan.off_nv) : nullptr;
        p1.status = (unsigned int*)(wsb + plan.off_flag);
        p1.span = (unsigned long long*)(wsb + plan.off_flag + kSpanOffset);
        // with one CTA per (unit, row chunk) and no padding rows there is nothing to merge: pass 1 writes the results itself
        const bool direct = plan.n_splits == 1 && ch.rows_out == s.R;
        if (direct) {
            p1.out_o = (float*)(wsb + plan.off_o); p1.out_obf = (__nv_bfloat16*)(wsb + plan.off_obf);
            p1.out_lse2 = (float*)(wsb + plan.off_lse2); p1.out_onorm = (float*)(wsb + plan.off_onorm);
            p1.out_cpair = (float*)(wsb + plan.off_cpair);
        }
        OBC_CUDA_TRY(cudaFuncSetAttribute(tc_pass1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemP1));
        { ProfScope ps("tc_pass1", stream);
          OBC_CUDA_TRY(launch_pdl(tc_pass1_kernel, dim3(plan.n_splits, units * ch.n_chunks), dim3(kThreadsP1), kSmemP1, stream, 1, mq, mk, mv, p1)); }
        if (!direct) {
            obc_status st = launch_combine(s, plan, ws, stream);
            if (st != OBC_OK) return st;
        }
    }
    if (attention_only) { *attention_only = plan; return OBC_OK; }      // the workspace holds the window attention
    TcParams p{};
    p.B = s.B; p.Hkv = s.Hkv; p.G = s.G; p.W = s.W; p.R = s.R; p.Nmax = s.Nmax; p.seq_lens = s.seq_lens; p.mask_lens = s.mask_lens;
    p.scale = s.scale; p.causal = s.causal; p.variants = s.variants;
    p.n_chunks = ch.n_chunks; p.chunk_rows = ch.chunk_rows; p.rows_out = ch.rows_out;
    p.lse2 = (const float*)(wsb + plan.off_lse2);
    p.onorm = (const float*)(wsb + plan.off_onorm);
    p.scores = scores;
    p.status = (unsigned int*)(wsb + plan.off_flag);
    p.span = (unsigned long long*)(wsb + plan.off_flag + kSpanOffset) + 2;
    p.cpair = (const float4*)(wsb + plan.off_cpair);
    p.nv = (const float*)(wsb + plan.off_nv);
    p.l2_stream = l2_stream ? 1 : 0;
    p.csplit = 1; p.partial = nullptr;
    const long long n_tiles = (long long)units * ((s.Nmax + TILE - 1) / TILE);
    const int grid = (int)(n_tiles < sm_count() ? n_tiles : sm_count());

    if (ch.n_chunks > 1) {                               // more than 128 window rows: chunks of 64, K/V tile kept
        CUtensorMap mq64, mo64;
        const uint64_t qd[2] = {(uint64_t)kD, (uint64_t)s.B * s.Hq * s.W};
        const uint64_t qs[1] = {(uint64_t)q.st * 2};
        const uint64_t od[2] = {(uint64_t)kD, (uint64_t)units * ch.rows_out};
        const uint64_t os[1] = {(uint64_t)kD * 2};
        if (!make_map(&mq64, q.ptr, 2, qd, qs, MC_ROWS) || !make_map(&mo64, wsb + plan.off_obf, 2, od, os, MC_ROWS)) {
            set_last_cuda_error((int)cudaErrorInvalidValue);
            return OBC_ERR_CUDA;
        }
        p.n_chunks = ch.rows_out / MC_ROWS; p.chunk_rows = MC_ROWS;
        p.csplit = tc_chunk_split(s, ch);
        p.partial = (float*)(wsb + plan.bytes);
        const long long positions = (long long)units * (((s.Nmax + TILE - 1) / TILE + 1) / 2) * p.csplit;
        const int mgrid = (int)(positions < sm_count() ? positions : sm_count());
        auto launch_multi = [&](auto kernel) -> obc_status {
            OBC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMulti));
            { ProfScope ps("tc_pass2", stream); OBC_CUDA_TRY(launch_pdl(kernel, dim3(mgrid), dim3(kThreadsMulti), kSmemMulti, stream, 1, mq64, mo64, mk, mv, p)); }
            if (p.csplit > 1) {
                ProfScope ps("partial_sum", stream);
                OBC_CUDA_TRY(launch_pdl(tc_partial_sum_kernel, dim3((s.Nmax + 255) / 256, units), dim3(256), 0, stream, 1, p, s.n_planes));
            }
            return OBC_OK;
        };
        if (p.csplit > 1 || (s.causal && s.W > MC_ROWS)) {
            if (s.variants == OBC_VAR_VK) return launch_multi(tc_pass2_multi_kernel<OBC_VAR_VK, true>);
            if (s.variants == (OBC_VAR_K | OBC_VAR_VK)) return launch_multi(tc_pass2_multi_kernel<OBC_VAR_K | OBC_VAR_VK, true>);
            return launch_multi(tc_pass2_multi_kernel<kAllVariants, true>);
        }
        if (s.variants == OBC_VAR_VK) return launch_multi(tc_pass2_multi_kernel<OBC_VAR_VK, false>);
        if (s.variants == (OBC_VAR_K | OBC_VAR_VK)) return launch_multi(tc_pass2_multi_kernel<OBC_VAR_K | OBC_VAR_VK, false>);
        return launch_multi(tc_pass2_multi_kernel<kAllVariants, false>);
    }

    auto launch = [&](auto kernel) -> obc_status {
        OBC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        { ProfScope ps("tc_pass2", stream); OBC_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(kThreads), kSmemBytes, stream, 1, mq, mo, mk, mv, p)); }
        return OBC_OK;
    };
    if (given) {
        if (s.variants == OBC_VAR_VK) return launch(tc_pass2_kernel<OBC_VAR_VK, true>);
        if (s.variants == (OBC_VAR_K | OBC_VAR_VK)) return launch(tc_pass2_kernel<OBC_VAR_K | OBC_VAR_VK, true>);
        return launch(tc_pass2_kernel<kAllVariants, true>);
    }
    if (s.variants == OBC_VAR_VK) return launch(tc_pass2_kernel<OBC_VAR_VK, false>);
    if (s.variants == (OBC_VAR_K | OBC_VAR_VK)) return launch(tc_pass2_kernel<OBC_VAR_K | OBC_VAR_VK, false>);
    // pass 1 leaves only ||v||^2; the l1 variant takes both norms from the V tiles in pass 2
    if (s.variants & OBC_VAR_VATP) return launch(tc_pass2_kernel<kAllVariants, true>);
    return launch(tc_pass2_kernel<kAllVariants & ~OBC_VAR_VATP, false>);
}

}  // namespace obc
