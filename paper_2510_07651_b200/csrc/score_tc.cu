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
// Warp roles of the 384-thread CTA (persistent, one CTA per SM):
//   warp 0      TMA producer: K/V tiles into a 2-stage ring, Q / -2O chunks when they change
//   warp 1      MMA issuer (one elected lane), double-buffered TMEM accumulators (2 x 256 columns)
//   warps 2-3   ||v_p||^2 of the tile from shared memory, per-row constants into shared memory
//   warps 4-7   epilogue group 0 (even tiles), warps 8-11 epilogue group 1 (odd tiles)
//
// Every mbarrier wait is bounded: on a timeout the kernel raises the status word in the workspace
// header, stops issuing work, waits (bounded) for its own copies in flight, frees TMEM and returns.
#include "obc_common.cuh"

#include <cuda.h>
#include <cudaTypedefs.h>

namespace obc {
namespace {

constexpr int TILE = 128;                       // tokens per tile = MMA M
constexpr int NSTAGE = 2;
constexpr int NSLOT = 4;                        // ring depth of the per-tile constants / norms
constexpr uint32_t kHalfBytes = 128 * 128;      // [128 rows][64 bf16] = 16 KB, one swizzle-128B block
constexpr uint32_t kOperandBytes = 2 * kHalfBytes;
constexpr int kThreads = 384;
constexpr unsigned long long kWaitNs = 2000000000ull;   // 2 s per wait

// ---- shared memory map (offsets from a 1024-byte aligned base) ------------------------------
constexpr uint32_t OFF_Q = 0;
constexpr uint32_t OFF_O = OFF_Q + kOperandBytes;
constexpr uint32_t OFF_K = OFF_O + kOperandBytes;                 // NSTAGE x 32 KB
constexpr uint32_t OFF_V = OFF_K + NSTAGE * kOperandBytes;        // NSTAGE x 32 KB
constexpr uint32_t OFF_NV = OFF_V + NSTAGE * kOperandBytes;       // NSLOT x 128 floats
constexpr uint32_t OFF_CONST = OFF_NV + NSLOT * TILE * 4;         // NSLOT x 128 float2 (lse2, ||o||^2)
constexpr uint32_t OFF_BAR = OFF_CONST + NSLOT * 128 * 8;
constexpr uint32_t kNumBars = 2 * NSTAGE + 2 + 4 + NSLOT;
constexpr uint32_t OFF_TMEM = OFF_BAR + kNumBars * 8;
constexpr uint32_t kSmemBytes = OFF_TMEM + 16 + 1024;             // + alignment slack

enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_QO_FULL = 2 * NSTAGE, BAR_QO_EMPTY = 2 * NSTAGE + 1,
       BAR_TM_FULL = 2 * NSTAGE + 2, BAR_TM_EMPTY = 2 * NSTAGE + 4, BAR_NV = 2 * NSTAGE + 6 };

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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
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
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 64 bf16 (128 B),
// 8-row groups 1024 B apart (the image a swizzle-128B TMA box of 64 elements x rows leaves)
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);           // start address >> 4
    d |= (uint64_t)1 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: 8 rows x 128 B
    d |= (uint64_t)1 << 46;                          // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                          // layout: 128-byte swizzle
    return d;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128
__host__ __device__ constexpr uint32_t idesc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TILE >> 4) << 24);
}

struct TcParams {
    int B, Hkv, G, W, R, Nmax;
    const int32_t* seq_lens;
    float scale;
    int causal;
    unsigned variants;
    int n_chunks, chunk_rows, rows_out;       // rows_out = n_chunks * chunk_rows
    int tiles_per_unit;
    const float* lse2;                        // [units][rows_out]
    const float* onorm;                       // [units][rows_out]
    float* scores;                            // [planes][units][Nmax]
    unsigned int* status;                     // device status word (workspace header)
};

__device__ __forceinline__ int tc_seq_len_raw(const int32_t* lens, int b, int nmax) { return lens ? lens[b] : nmax; }
__device__ __forceinline__ int tc_seq_len(const TcParams& p, int b) { return tc_seq_len_raw(p.seq_lens, b, p.Nmax); }

// VARS: variants this instantiation computes (a superset of p.variants)
template <unsigned VARS>
__global__ void __launch_bounds__(kThreads, 1)
tc_pass2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o,
                const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + OFF_BAR;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_TMEM);
    float* sNv = reinterpret_cast<float*>(smem + OFF_NV);
    float2* sConst = reinterpret_cast<float2*>(smem + OFF_CONST);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = p.B * p.Hkv;
    const long long n_tiles = (long long)units * p.tiles_per_unit;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NSTAGE; ++i) { mbar_init(bar(BAR_FULL + i), 1); mbar_init(bar(BAR_EMPTY + i), 3); }
        mbar_init(bar(BAR_QO_FULL), 1); mbar_init(bar(BAR_QO_EMPTY), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_TM_FULL + i), 1); mbar_init(bar(BAR_TM_EMPTY + i), 4); }
        for (int i = 0; i < NSLOT; ++i) mbar_init(bar(BAR_NV + i), 2);
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
    const bool reload_qo_every_item = p.n_chunks > 1;
    const uint32_t qo_bytes = (uint32_t)p.chunk_rows * 128u * 2u * 2u;   // Q and O chunks, two halves each

    // Every role walks the same list: tiles L = blockIdx.x + i * gridDim.x, L -> (unit, tile);
    // for each non-empty tile, chunks c = 0 .. n_chunks-1.  `item` counts (tile, chunk) pairs that
    // are actually processed and indexes the smem stage / TMEM buffer / constant slot rings.
    if (warp == 0) {
        // ===================================== TMA producer =====================================
        if (lane == 0) {
            uint32_t item = 0, qo_loads = 0;
            int qo_unit = -1;
            for (long long L = blockIdx.x; L < n_tiles && !failed; L += gridDim.x) {
                const int unit = (int)(L / p.tiles_per_unit), tile = (int)(L % p.tiles_per_unit);
                const int b = unit / p.Hkv, g = unit % p.Hkv;
                const int t0 = tile * TILE;
                if (t0 >= tc_seq_len(p, b)) continue;
                for (int c = 0; c < p.n_chunks; ++c, ++item) {
                    if (reload_qo_every_item || unit != qo_unit) {
                        if (!mbar_wait(bar(BAR_QO_EMPTY), (qo_loads & 1) ^ 1)) { failed = true; break; }
                        mbar_expect_tx(bar(BAR_QO_FULL), qo_bytes);
                        const int qrow = (b * p.Hkv * p.G + g * p.G) * p.W + c * p.chunk_rows;
                        const int orow = unit * p.rows_out + c * p.chunk_rows;
                        tma_load_2d(sbase + OFF_Q, &map_q, bar(BAR_QO_FULL), 0, qrow);
                        tma_load_2d(sbase + OFF_Q + kHalfBytes, &map_q, bar(BAR_QO_FULL), 64, qrow);
                        tma_load_2d(sbase + OFF_O, &map_o, bar(BAR_QO_FULL), 0, orow);
                        tma_load_2d(sbase + OFF_O + kHalfBytes, &map_o, bar(BAR_QO_FULL), 64, orow);
                        qo_unit = unit; ++qo_loads;
                    }
                    const uint32_t st = item % NSTAGE, use = item / NSTAGE;
                    if (!mbar_wait(bar(BAR_EMPTY + st), (use & 1) ^ 1)) { failed = true; break; }
                    mbar_expect_tx(bar(BAR_FULL + st), 2 * kOperandBytes);
                    const uint32_t dk = sbase + OFF_K + st * kOperandBytes, dv = sbase + OFF_V + st * kOperandBytes;
                    tma_load_4d(dk, &map_k, bar(BAR_FULL + st), 0, t0, g, b);
                    tma_load_4d(dk + kHalfBytes, &map_k, bar(BAR_FULL + st), 64, t0, g, b);
                    tma_load_4d(dv, &map_v, bar(BAR_FULL + st), 0, t0, g, b);
                    tma_load_4d(dv + kHalfBytes, &map_v, bar(BAR_FULL + st), 64, t0, g, b);
                }
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
            uint32_t item = 0, qo_loads = 0;
            int qo_unit = -1;
            for (long long L = blockIdx.x; L < n_tiles && !failed; L += gridDim.x) {
                const int unit = (int)(L / p.tiles_per_unit), tile = (int)(L % p.tiles_per_unit);
                const int b = unit / p.Hkv;
                if (tile * TILE >= tc_seq_len(p, b)) continue;
                for (int c = 0; c < p.n_chunks; ++c, ++item) {
                    const bool new_qo = reload_qo_every_item || unit != qo_unit;
                    if (new_qo) {
                        if (!mbar_wait(bar(BAR_QO_FULL), qo_loads & 1)) { failed = true; break; }
                        qo_unit = unit; ++qo_loads;
                    }
                    const uint32_t st = item % NSTAGE, buf = item & 1;
                    if (!mbar_wait(bar(BAR_FULL + st), (item / NSTAGE) & 1)) { failed = true; break; }
                    if (!mbar_wait(bar(BAR_TM_EMPTY + buf), ((item >> 1) & 1) ^ 1)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t zt = tmem_base + buf * 256u, tt = zt + 128u;
                    const uint32_t ak = sbase + OFF_K + st * kOperandBytes, av = sbase + OFF_V + st * kOperandBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {               // d = 128 = 8 steps of K = 16
                        const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                        tc_mma(zt, smem_desc_k_sw128(ak + off), smem_desc_k_sw128(sbase + OFF_Q + off), idesc, ks > 0);
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                        tc_mma(tt, smem_desc_k_sw128(av + off), smem_desc_k_sw128(sbase + OFF_O + off), idesc, ks > 0);
                    }
                    tc_commit(bar(BAR_TM_FULL + buf));             // accumulators ready for the epilogue
                    tc_commit(bar(BAR_EMPTY + st));                // K/V stage no longer read by the MMA
                    // Q / O may be overwritten once these MMAs are done, if the next item needs others
                    bool next_needs_qo = reload_qo_every_item;
                    if (!next_needs_qo) {
                        long long Ln = L + gridDim.x;
                        while (Ln < n_tiles) {
                            const int un = (int)(Ln / p.tiles_per_unit), tn = (int)(Ln % p.tiles_per_unit);
                            if (tn * TILE < tc_seq_len(p, un / p.Hkv)) { next_needs_qo = un != unit; break; }
                            Ln += gridDim.x;
                        }
                    }
                    if (next_needs_qo) tc_commit(bar(BAR_QO_EMPTY));
                }
            }
        }
    } else if (warp < 4) {
        // ============================ ||v_p||^2 and per-row constants ===========================
        const int t64 = threadIdx.x - 64;                          // 0..63
        uint32_t item = 0;
        for (long long L = blockIdx.x; L < n_tiles && !failed; L += gridDim.x) {
            const int unit = (int)(L / p.tiles_per_unit), tile = (int)(L % p.tiles_per_unit);
            const int b = unit / p.Hkv;
            if (tile * TILE >= tc_seq_len(p, b)) continue;
            for (int c = 0; c < p.n_chunks; ++c, ++item) {
                const uint32_t st = item % NSTAGE, slot = item % NSLOT;
                // constants first (global loads overlap the wait for the tile)
                const size_t crow = (size_t)unit * p.rows_out + (size_t)c * p.chunk_rows;
                float2 cst[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int r = t64 + 64 * j;
                    cst[j] = r < p.chunk_rows ? make_float2(p.lse2[crow + r], p.onorm[crow + r]) : make_float2(INFINITY, 0.f);
                }
                if (!mbar_wait(bar(BAR_FULL + st), (item / NSTAGE) & 1)) { failed = true; break; }
                const uint8_t* vt = smem + OFF_V + st * kOperandBytes;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int tok = t64 + 64 * j;
                    float acc = 0.f;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            // any order of the row's 16-byte chunks gives the same sum; this one is bank-conflict free
                            const uint4 u = *reinterpret_cast<const uint4*>(vt + h * kHalfBytes + tok * 128 + ((ch ^ (tok & 7)) << 4));
                            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
                                acc = fmaf(lo, lo, acc); acc = fmaf(hi, hi, acc);
                            }
                        }
                    sNv[slot * TILE + tok] = acc;
                    sConst[slot * 128 + tok] = cst[j];
                }
                __syncwarp();
                if (lane == 0) { mbar_arrive(bar(BAR_NV + slot)); mbar_arrive(bar(BAR_EMPTY + st)); }
            }
        }
    } else {
        // ======================================= epilogue =======================================
        const int wg = (warp - 4) >> 2;                            // 0: even tiles, 1: odd tiles
        const int lane_grp = warp & 3;                             // TMEM lanes 32*lane_grp .. +31
        const int tok = lane_grp * 32 + lane;                      // token within the tile
        const float sl2 = p.scale * kLog2e;
        const size_t plane = (size_t)units * p.Nmax;
        uint32_t item = 0, tile_seq = 0;
        for (long long L = blockIdx.x; L < n_tiles && !failed; L += gridDim.x) {
            const int unit = (int)(L / p.tiles_per_unit), tile = (int)(L % p.tiles_per_unit);
            const int b = unit / p.Hkv;
            const int N = tc_seq_len(p, b), t0 = tile * TILE;
            float* out = p.scores + (size_t)unit * p.Nmax;
            const int ptok = t0 + tok;
            if (t0 >= N) {                                         // padding beyond the sequence: zeros
                if (wg == 0 && ptok < p.Nmax) {
                    int pl = 0;
                    for (unsigned v = 1; v <= 8; v <<= 1) if (p.variants & v) out[(size_t)(pl++) * plane + ptok] = 0.f;
                }
                continue;
            }
            const bool mine = (tile_seq & 1) == (uint32_t)wg;
            ++tile_seq;
            if (!mine) { item += p.n_chunks; continue; }
            // rows of the window that do not see this tile's last token need the causal mask
            const bool masked_tile = p.causal && (t0 + TILE - 1 > N - p.W);
            float s_a = 0.f, s_a2 = 0.f, s_k = 0.f, s_j = 0.f;
            float nv = 0.f;
            for (int c = 0; c < p.n_chunks && !failed; ++c, ++item) {
                const uint32_t buf = item & 1, slot = item % NSLOT;
                if (!mbar_wait(bar(BAR_NV + slot), (item / NSLOT) & 1)) { failed = true; break; }
                if (!mbar_wait(bar(BAR_TM_FULL + buf), (item >> 1) & 1)) { failed = true; break; }
                tc_fence_after();
                nv = sNv[slot * TILE + tok];
                const float nv2 = nv + nv;
                const float2* cst = sConst + slot * 128;
                const uint32_t zt = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + buf * 256u, tt = zt + 128u;
                const int rbase = c * p.chunk_rows;
                for (int c0 = 0; c0 < p.chunk_rows; c0 += 16) {
                    uint32_t zr[16], tr[16];
                    tc_ld16(zt + c0, zr);
                    tc_ld16(tt + c0, tr);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float2 cj = cst[c0 + j];                     // (log2-sum-exp, ||o_r||^2)
                        const float z = __uint_as_float(zr[j]), t2 = __uint_as_float(tr[j]);   // t2 = -2 v.o
                        float a = fast_exp2(fmaf(z, sl2, -cj.x));
                        if (masked_tile) {
                            const int r = rbase + c0 + j;
                            if (ptok > N - p.W + (r % p.W)) a = 0.f;
                        }
                        const float Z = z * p.scale, a2 = a * a;
                        if (VARS & OBC_VAR_ATTN) s_a += a;
                        if (VARS & OBC_VAR_V) s_a2 += a2;
                        const float vmo = (nv + cj.y) + t2;                // ||v - o||^2 = |v|^2 + |o|^2 - 2 v.o
                        if (VARS & OBC_VAR_K) s_k = fmaf(a2 * Z * Z, vmo, s_k);
                        if (VARS & OBC_VAR_VK) {
                            // |v|^2 + 2 Z (|v|^2 - v.o) + Z^2 ||v - o||^2, Horner in Z
                            const float h = fmaf(Z, vmo, nv2 + t2);
                            s_j = fmaf(a2, fmaf(Z, h, nv), s_j);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_TM_EMPTY + buf));
            }
            if (!failed && ptok < p.Nmax) {
                const bool live = ptok < N;
                int pl = 0;
                if (p.variants & OBC_VAR_V)    out[(size_t)(pl++) * plane + ptok] = live ? s_a2 * nv : 0.f;
                if (p.variants & OBC_VAR_K)    out[(size_t)(pl++) * plane + ptok] = live ? s_k : 0.f;
                if (p.variants & OBC_VAR_VK)   out[(size_t)(pl++) * plane + ptok] = live ? s_j : 0.f;
                if (p.variants & OBC_VAR_ATTN) out[(size_t)(pl++) * plane + ptok] = live ? s_a : 0.f;
            }
        }
    }

    if (failed) atomicExch(p.status, 1u);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// =================================================================================================
// Pass 1 on tensor cores: streaming softmax statistics and window outputs (Sec. 3: A = softmax(Z),
// O = A V over the perturbation window, Eq. 9), split over the cached tokens.
//
// Rows of the window (one chunk of up to 128) sit on the MMA M dimension, so a TMEM lane holds one
// row and the softmax thread that owns it reduces along the tile without cross-thread traffic:
//     S   = Q_chunk . K_tile^T                     (tcgen05, accumulators double-buffered in TMEM)
//     P   = exp2(S * scale*log2e - m_used)         (registers -> bf16 -> swizzled shared memory)
//     O  += P . V_tile                             (tcgen05, V read as an MN-major B operand)
// m_used is the exponent reference of the row; it is only moved up (and O, l rescaled) when the
// running maximum exceeds it by more than 8 (a factor 256), which keeps P within bf16/fp32 range.
// Each CTA writes (m_used, l, O) of its token split; the combine kernel merges the splits.
//
//   warp 0      TMA producer (Q chunk once, K/V tiles into a 2-stage ring)
//   warp 1      MMA issuer
//   warps 4-7   softmax (thread = row)
// =================================================================================================
constexpr int kThreadsP1 = 256;
constexpr uint32_t P1_OFF_Q = 0;
constexpr uint32_t P1_OFF_P = P1_OFF_Q + kOperandBytes;
constexpr uint32_t P1_OFF_K = P1_OFF_P + kOperandBytes;
constexpr uint32_t P1_OFF_V = P1_OFF_K + NSTAGE * kOperandBytes;
constexpr uint32_t P1_OFF_BAR = P1_OFF_V + NSTAGE * kOperandBytes;
enum { P1_FULL = 0, P1_EMPTY = 2, P1_QFULL = 4, P1_SFULL = 5, P1_SEMPTY = 7, P1_PFULL = 9, P1_PVDONE = 10, P1_NBARS = 11 };
constexpr uint32_t P1_OFF_TMEM = P1_OFF_BAR + P1_NBARS * 8;
constexpr uint32_t kSmemP1 = P1_OFF_TMEM + 16 + 1024;
constexpr float kRescaleThreshold = 8.f;                   // log2 units

struct P1Params {
    int B, Hq, Hkv, G, W, R, Nmax;
    const int32_t* seq_lens;
    float scale;
    int causal;
    int n_chunks, chunk_rows;
    int n_splits, tiles_per_split;
    float* part_m; float* part_l; float* part_o;           // [units][n_splits][R] (x d for part_o)
    unsigned int* status;
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
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// MN-major B operand with 128-byte swizzle: 64 contiguous elements of N per 128-byte row, 8 rows of
// K per 1024-byte group (stride byte offset), the next 64 elements of N one 16 KB block further
// (leading byte offset).  This is the image of a [tokens][head_dim] tile loaded as two 64-wide boxes.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(kHalfBytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(kThreadsP1, 1)
tc_pass1_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, P1Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + P1_OFF_BAR;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + P1_OFF_TMEM);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int split = blockIdx.x, vu = blockIdx.y;
    const int unit = vu / p.n_chunks, c = vu % p.n_chunks;
    const int b = unit / p.Hkv, g = unit % p.Hkv;
    const int N = tc_seq_len_raw(p.seq_lens, b, p.Nmax);
    const int tile_lo = split * p.tiles_per_split;
    const int tile_hi = min(tile_lo + p.tiles_per_split, (N + TILE - 1) / TILE);
    const int n_tiles = max(tile_hi - tile_lo, 0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < NSTAGE; ++i) { mbar_init(bar(P1_FULL + i), 1); mbar_init(bar(P1_EMPTY + i), 1); }
        mbar_init(bar(P1_QFULL), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar(P1_SFULL + i), 1); mbar_init(bar(P1_SEMPTY + i), 4); }
        mbar_init(bar(P1_PFULL), 4); mbar_init(bar(P1_PVDONE), 1);
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
    const uint32_t tmem_o = tmem_base + 256u;
    bool failed = false;

    if (warp == 0) {
        if (lane == 0 && n_tiles > 0) {
            mbar_expect_tx(bar(P1_QFULL), (uint32_t)p.chunk_rows * 256u);
            const int qrow = (b * p.Hq + g * p.G) * p.W + c * p.chunk_rows;
            tma_load_2d(sbase + P1_OFF_Q, &map_q, bar(P1_QFULL), 0, qrow);
            tma_load_2d(sbase + P1_OFF_Q + kHalfBytes, &map_q, bar(P1_QFULL), 64, qrow);
            int issued = 0;
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t st = i % NSTAGE;
                if (!mbar_wait(bar(P1_EMPTY + st), ((i / NSTAGE) & 1) ^ 1)) { failed = true; break; }
                mbar_expect_tx(bar(P1_FULL + st), 2 * kOperandBytes);
                const uint32_t dk = sbase + P1_OFF_K + st * kOperandBytes, dv = sbase + P1_OFF_V + st * kOperandBytes;
                const int t0 = (tile_lo + i) * TILE;
                tma_load_4d(dk, &map_k, bar(P1_FULL + st), 0, t0, g, b);
                tma_load_4d(dk + kHalfBytes, &map_k, bar(P1_FULL + st), 64, t0, g, b);
                tma_load_4d(dv, &map_v, bar(P1_FULL + st), 0, t0, g, b);
                tma_load_4d(dv + kHalfBytes, &map_v, bar(P1_FULL + st), 64, t0, g, b);
                ++issued;
            }
            for (int back = 0; back < NSTAGE && back < issued; ++back) {      // drain own copies
                const int it = issued - 1 - back;
                (void)mbar_wait(bar(P1_FULL + it % NSTAGE), (it / NSTAGE) & 1);
            }
            (void)mbar_wait(bar(P1_QFULL), 0);
        }
    } else if (warp == 1) {
        if (lane == 0 && n_tiles > 0) {
            const uint32_t idesc_s = idesc_bf16(TILE);
            const uint32_t idesc_pv = idesc_bf16(kD) | (1u << 16);           // B operand (V) is MN-major
            auto issue_s = [&](int j) -> bool {
                const uint32_t st = j % NSTAGE;
                if (!mbar_wait(bar(P1_FULL + st), (j / NSTAGE) & 1)) return false;
                if (!mbar_wait(bar(P1_SEMPTY + (j & 1)), ((j >> 1) & 1) ^ 1)) return false;
                tc_fence_after();
                const uint32_t ak = sbase + P1_OFF_K + st * kOperandBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    tc_mma(tmem_base + (j & 1) * 128u, smem_desc_k_sw128(sbase + P1_OFF_Q + off), smem_desc_k_sw128(ak + off), idesc_s, ks > 0);
                }
                tc_commit(bar(P1_SFULL + (j & 1)));
                return true;
            };
            failed = !mbar_wait(bar(P1_QFULL), 0);
            if (!failed) failed = !issue_s(0);
            for (int i = 0; i < n_tiles && !failed; ++i) {
                if (i + 1 < n_tiles && !issue_s(i + 1)) { failed = true; break; }
                if (!mbar_wait(bar(P1_PFULL), i & 1)) { failed = true; break; }
                tc_fence_after();
                const uint32_t av = sbase + P1_OFF_V + (i % NSTAGE) * kOperandBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {                             // 128 tokens = 8 steps of K = 16
                    const uint32_t offp = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    tc_mma(tmem_o, smem_desc_k_sw128(sbase + P1_OFF_P + offp), smem_desc_mn_sw128(av + ks * 2048), idesc_pv, (i > 0) || (ks > 0));
                }
                tc_commit(bar(P1_PVDONE));
                tc_commit(bar(P1_EMPTY + (i % NSTAGE)));
            }
        }
    } else if (warp >= 4) {
        const int lane_grp = warp & 3;
        const int row = lane_grp * 32 + lane;                                // row within the chunk
        const int rows_valid = min(p.chunk_rows, p.R - c * p.chunk_rows);
        const int r = c * p.chunk_rows + row;
        const bool valid = row < rows_valid;
        const int last = valid ? (p.causal ? N - p.W + (r % p.W) : N - 1) : -1;
        const float sl2 = p.scale * kLog2e;
        const uint32_t lane_addr = (uint32_t)(lane_grp * 32) << 16;
        float m_used = -INFINITY, l = 0.f;
        uint8_t* prow = smem + P1_OFF_P + row * 128;

        for (int i = 0; i < n_tiles && !failed; ++i) {
            const uint32_t buf = i & 1;
            const int t0 = (tile_lo + i) * TILE;
            if (!mbar_wait(bar(P1_SFULL + buf), (i >> 1) & 1)) { failed = true; break; }
            tc_fence_after();
            float sv[128];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tc_ld32(tmem_base + lane_addr + buf * 128u + q4 * 32, reinterpret_cast<uint32_t*>(sv) + q4 * 32);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P1_SEMPTY + buf));

            float mt = -INFINITY;
            const int nvis = last - t0 + 1;                                  // columns j < nvis are visible
#pragma unroll
            for (int j = 0; j < 128; ++j) {
                sv[j] = j < nvis ? sv[j] * sl2 : -INFINITY;
                mt = fmaxf(mt, sv[j]);
            }
            const bool need = mt > m_used + kRescaleThreshold;               // also true for the first visible tile
            const float factor = need ? fast_exp2(m_used - mt) : 1.f;        // m_used = -inf -> 0
            if (i > 0) {
                const bool any = __any_sync(0xffffffffu, need && m_used != -INFINITY);
                if (!mbar_wait(bar(P1_PVDONE), (i - 1) & 1)) { failed = true; break; }   // P buffer free, O stable
                if (any) {
                    tc_fence_after();
#pragma unroll 1
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t ov[32];
                        tc_ld32(tmem_o + lane_addr + q4 * 32, ov);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * factor);
                        tc_st32(tmem_o + lane_addr + q4 * 32, ov);
                    }
                    tc_wait_st();
                    tc_fence_before();
                }
            }
            l *= factor;
            if (need) m_used = mt;
            const float m_eff = m_used == -INFINITY ? 0.f : m_used;
            float lsum = 0.f;
#pragma unroll
            for (int ch = 0; ch < 16; ++ch) {                                // 16 chunks of 8 tokens = 16 bytes of bf16
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float p0 = fast_exp2(sv[ch * 8 + 2 * e] - m_eff), p1 = fast_exp2(sv[ch * 8 + 2 * e + 1] - m_eff);
                    lsum += p0 + p1;
                    w[e] = pack_bf16x2(p0, p1);
                }
                *reinterpret_cast<uint4*>(prow + (ch >> 3) * kHalfBytes + (((ch & 7) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            l += lsum;
            if (t0 + TILE > N && t0 + row >= N) {                            // tail: V rows past the sequence must not reach the MMA
                uint8_t* vrow = smem + P1_OFF_V + (i % NSTAGE) * kOperandBytes + row * 128;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    *reinterpret_cast<uint4*>(vrow + (ch << 4)) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(vrow + kHalfBytes + (ch << 4)) = make_uint4(0, 0, 0, 0);
                }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P1_PFULL));
        }

        // partial results of this split
        const size_t prow_idx = ((size_t)unit * p.n_splits + split) * p.R + r;
        if (n_tiles > 0 && !failed) {
            if (!mbar_wait(bar(P1_PVDONE), (n_tiles - 1) & 1)) failed = true;
            tc_fence_after();
#pragma unroll 1
            for (int q4 = 0; q4 < 4 && !failed; ++q4) {
                uint32_t ov[32];
                tc_ld32(tmem_o + lane_addr + q4 * 32, ov);
                tc_wait_ld();
                if (valid) {
                    float4* dst = reinterpret_cast<float4*>(p.part_o + prow_idx * kD + q4 * 32);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        dst[j] = make_float4(__uint_as_float(ov[4 * j]), __uint_as_float(ov[4 * j + 1]),
                                             __uint_as_float(ov[4 * j + 2]), __uint_as_float(ov[4 * j + 3]));
                }
            }
            tc_fence_before();
        } else if (valid) {
            float4* dst = reinterpret_cast<float4*>(p.part_o + prow_idx * kD);
            for (int j = 0; j < 32; ++j) dst[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (valid) { p.part_m[prow_idx] = m_used; p.part_l[prow_idx] = l; }
    }

    if (failed) atomicExch(p.status, 1u);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---- host side ----------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled get_encode() {
    static PFN_cuTensorMapEncodeTiled fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (PFN_cuTensorMapEncodeTiled)ptr;
    }
    return fn;
}

// bf16 tensor map, rank 2 or 4, innermost dimension = head_dim (128), box {64, box_rows, 1, 1}
bool make_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              uint32_t box_rows) {
    PFN_cuTensorMapEncodeTiled enc = get_encode();
    if (!enc) return false;
    cuuint64_t gdim[4]; cuuint64_t gstr[3]; cuuint32_t box[4] = {64, box_rows, 1, 1}; cuuint32_t estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < rank; ++i) gdim[i] = dims[i];
    for (int i = 0; i < rank - 1; ++i) gstr[i] = strides_bytes[i];
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcChunks { int n_chunks, chunk_rows, rows_out; };
TcChunks tc_chunks(int R) {
    TcChunks c;
    c.n_chunks = (R + 127) / 128;
    c.chunk_rows = ((R + c.n_chunks - 1) / c.n_chunks + 15) / 16 * 16;
    c.rows_out = c.n_chunks * c.chunk_rows;
    return c;
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

// Workspace plan of the tensor-core path: the SIMT plan's layout with splits counted in 128-token tiles.
static SimtPlan make_tc_plan(const ScoreShape& s) {
    const TcChunks ch = tc_chunks(s.R);
    const int units = s.B * s.Hkv, vus = units * ch.n_chunks;
    const int tiles = (s.Nmax + TILE - 1) / TILE;
    int n = sm_count() / vus;                          // one wave of CTAs when the sequences are equal
    if (s.seq_lens) { const int cap = (tiles + 31) / 32; if (cap > n) n = cap; }   // ragged: bound the work per CTA
    if (n < 1) n = 1;
    if (n > tiles) n = tiles;
    SimtPlan p{};
    p.tiles_per_split = (tiles + n - 1) / n;
    p.n_splits = (tiles + p.tiles_per_split - 1) / p.tiles_per_split;
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
    p.bytes = off;
    return p;
}

size_t tc_workspace_bytes(const ScoreShape& s) { return make_tc_plan(s).bytes; }

obc_status launch_score_tc(const ScoreShape& s, TensorView q, TensorView k, TensorView v,
                           float* scores, void* ws, cudaStream_t stream) {
    const TcChunks ch = tc_chunks(s.R);
    const SimtPlan plan = make_tc_plan(s);
    char* wsb = (char*)ws;
    OBC_CUDA_TRY(cudaMemsetAsync(wsb + plan.off_flag, 0, 256, stream));
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
    {   // pass 1 + combine
        P1Params p1{};
        p1.B = s.B; p1.Hq = s.Hq; p1.Hkv = s.Hkv; p1.G = s.G; p1.W = s.W; p1.R = s.R; p1.Nmax = s.Nmax;
        p1.seq_lens = s.seq_lens; p1.scale = s.scale; p1.causal = s.causal;
        p1.n_chunks = ch.n_chunks; p1.chunk_rows = ch.chunk_rows;
        p1.n_splits = plan.n_splits; p1.tiles_per_split = plan.tiles_per_split;
        p1.part_m = (float*)(wsb + plan.off_part_m); p1.part_l = (float*)(wsb + plan.off_part_l);
        p1.part_o = (float*)(wsb + plan.off_part_o);
        p1.status = (unsigned int*)(wsb + plan.off_flag);
        OBC_CUDA_TRY(cudaFuncSetAttribute(tc_pass1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemP1));
        { ProfScope ps("tc_pass1", stream);
          tc_pass1_kernel<<<dim3(plan.n_splits, units * ch.n_chunks), kThreadsP1, kSmemP1, stream>>>(mq, mk, mv, p1); }
        OBC_CUDA_TRY(cudaGetLastError());
        obc_status st = launch_combine(s, plan, ws, stream);
        if (st != OBC_OK) return st;
    }
    TcParams p{};
    p.B = s.B; p.Hkv = s.Hkv; p.G = s.G; p.W = s.W; p.R = s.R; p.Nmax = s.Nmax; p.seq_lens = s.seq_lens;
    p.scale = s.scale; p.causal = s.causal; p.variants = s.variants;
    p.n_chunks = ch.n_chunks; p.chunk_rows = ch.chunk_rows; p.rows_out = ch.rows_out;
    p.tiles_per_unit = (s.Nmax + TILE - 1) / TILE;
    p.lse2 = (const float*)(wsb + plan.off_lse2);
    p.onorm = (const float*)(wsb + plan.off_onorm);
    p.scores = scores;
    p.status = (unsigned int*)(wsb + plan.off_flag);
    const long long n_tiles = (long long)units * p.tiles_per_unit;
    const int grid = (int)(n_tiles < sm_count() ? n_tiles : sm_count());

    auto launch = [&](auto kernel) -> obc_status {
        OBC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        { ProfScope ps("tc_pass2", stream); kernel<<<grid, kThreads, kSmemBytes, stream>>>(mq, mo, mk, mv, p); }
        OBC_CUDA_TRY(cudaGetLastError());
        return OBC_OK;
    };
    if (s.variants == OBC_VAR_VK) return launch(tc_pass2_kernel<OBC_VAR_VK>);
    if (s.variants == (OBC_VAR_K | OBC_VAR_VK)) return launch(tc_pass2_kernel<OBC_VAR_K | OBC_VAR_VK>);
    return launch(tc_pass2_kernel<OBC_VAR_V | OBC_VAR_K | OBC_VAR_VK | OBC_VAR_ATTN>);
}

}  // namespace obc
