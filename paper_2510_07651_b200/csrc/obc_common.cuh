// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <utility>
#include "obcache.h"

namespace obc {

constexpr int kD = 128;                  // head_dim the kernels are written for
constexpr float kLog2e = 1.4426950408889634f;

// ---- thread-local record of the last failing CUDA call -------------------------------------
void set_last_cuda_error(int e);
#define OBC_CUDA_TRY(expr)                                              \
    do {                                                                \
        cudaError_t _e = (expr);                                        \
        if (_e != cudaSuccess) { obc::set_last_cuda_error((int)_e); return OBC_ERR_CUDA; } \
    } while (0)

// Brackets one kernel launch with CUDA events while profiling is on (see obc_profile_begin).
struct ProfScope {
    ProfScope(const char* name, cudaStream_t stream);
    ~ProfScope();
    int slot; cudaStream_t stream;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- internal launch descriptions (plain structs, passed by value to kernels) ---------------
struct TensorView {                      // element strides; d contiguous
    const void* ptr;
    long long sb, sh, st;
};

struct ScoreShape {
    int B, Hq, Hkv, G, W, R, Nmax;
    const int32_t* seq_lens;             // device or nullptr
    const int32_t* mask_lens;            // device or nullptr: length the causal mask counts from (token-sharded caches)
    float scale;                         // 1/sqrt(d) resolved
    int causal;
    unsigned variants;
    int n_planes;
};

constexpr size_t kSpanOffset = 64;   // byte offset, in the workspace header, of the four kernel-span words

// SIMT (CUDA-core) score path: workspace layout, computed identically by the size query and the launch
struct SimtPlan {
    int n_splits;                        // KV splits of pass 1
    int tiles_per_split;
    int tile_tokens;                     // tokens per tile of the pass-1 kernel the plan is for
    int rows_out;                        // rows per unit in the combined arrays (R, or R padded)
    int want_obf;                        // also write the bf16 copy of -2*O (tensor-core pass 2)
    size_t off_flag;                             // 256-byte header: device status word, kernel spans at kSpanOffset
    size_t off_part_m, off_part_l, off_part_o;   // partial softmax stats / outputs per split
    size_t off_lse2, off_onorm, off_o;           // combined: log2-sum-exp, ||o||^2, O (fp32)
    size_t off_obf;                              // bf16 [units][rows_out][d] = -2 * O
    size_t off_cpair;                            // float4 per row pair: (-lse2_0, -lse2_1, |o_0|^2, |o_1|^2)
    size_t off_nv;                               // fp32 [units][Nmax]: ||v_p||^2 (written by tensor-core pass 1)
    size_t bytes;
};
SimtPlan make_simt_plan(const ScoreShape& s, int rows_out, bool want_obf);

// Attention outputs supplied by the caller instead of a recompute: o [B,Hq,W,d] (any dtype, strided),
// lse fp32 [B,Hq,W] contiguous, natural log of the row's sum of exp(scaled logit).
struct GivenAttention {
    TensorView o;
    int o_dtype;
    const float* lse;
};
// writes what the combine kernel would have written (log2-sum-exp, ||o||^2, O, -2 O in bf16, row-pair
// constants) from the caller's arrays, and clears the status word
obc_status launch_given_prep(const ScoreShape& s, const SimtPlan& plan, const GivenAttention& given,
                             void* ws, cudaStream_t stream);

// pass 1 + combine (window softmax statistics and outputs), then pass 2 (scores)
obc_status launch_simt_pass1_combine(const ScoreShape& s, const SimtPlan& plan, int dtype,
                                     TensorView q, TensorView k, TensorView v, void* ws, cudaStream_t stream);
obc_status launch_combine(const ScoreShape& s, const SimtPlan& plan, void* ws, cudaStream_t stream);
// the combined window attention of the workspace as o [B,Hq,W,d] and natural-log lse [B,Hq,W]
obc_status launch_export_attention(const ScoreShape& s, const SimtPlan& plan, const void* ws, float* o_out, float* lse_out,
                                   cudaStream_t stream);
obc_status launch_merge_attention(int n_parts, long long rows, const float* o_parts, const float* lse_parts,
                                  float* o_out, float* lse_out, cudaStream_t stream);
// pass 1 + combine of the tensor-core path alone (the workspace then holds the shard's window attention)
obc_status launch_attention_tc(const ScoreShape& s, TensorView q, TensorView k, TensorView v, void* ws, cudaStream_t stream,
                               SimtPlan* plan_out);
obc_status launch_simt_pass2(const ScoreShape& s, const SimtPlan& plan, int dtype,
                             TensorView q, TensorView k, TensorView v,
                             float* scores, void* ws, cudaStream_t stream);

// ---- select / compact -------------------------------------------------------------------------
struct SelectShape {
    int B, Hkv, Nmax;
    const int32_t* seq_lens;
    int budget;
    const int32_t* budgets;
    int idx_stride, n_sink, n_recent, pool_mode, pool_kernel;
};
size_t select_workspace_bytes(int B, int Hkv, int Nmax);
obc_status launch_select(const SelectShape& s, const float* scores, int32_t* idx, void* ws, cudaStream_t stream);
size_t select_adaptive_workspace_bytes(const SelectShape& s, int n_safe);
obc_status launch_select_adaptive(const SelectShape& s, int n_safe, const float* scores, int32_t* idx, int32_t* counts,
                                  void* ws, cudaStream_t stream);
obc_status launch_select_static(const SelectShape& s, const float* scores, int32_t* idx, cudaStream_t stream);
obc_status launch_shard_indices(int units, int idx_stride, int t0, int n, const int32_t* idx, int32_t* local, int32_t* counts,
                                cudaStream_t stream);
obc_status launch_gather(int B, int Hkv, int idx_stride, int Nmax, int elem_bytes,
                         TensorView k, TensorView v, TensorView ko, TensorView vo, const int32_t* idx,
                         const float* s_in, float* s_out, cudaStream_t stream);

// ---- decode step --------------------------------------------------------------------------------
struct DecodeShape {
    int B, Hq, Hkv, G, cap, budget, n_sink, n_recent;
    unsigned variant;
    float scale;
    int acc_window;                      // 0, or the number of steps whose scores make up the accumulator
    float* s_hist;                       // [B,Hkv,acc_window,cap] ring of per-step scores
};
size_t decode_workspace_bytes(const DecodeShape& s);
obc_status launch_decode(const DecodeShape& s, TensorView q, TensorView kt, TensorView vt,
                         TensorView kc, TensorView vc, float* s_acc, int32_t* pos, int32_t* state,
                         int step_pos, void* ws, cudaStream_t stream);

// ---- tensor-core (tcgen05) score path -----------------------------------------------------------
bool tc_shape_supported(const ScoreShape& s);                       // R large enough for the MMA tiles
bool tc_supported(const ScoreShape& s, int dtype, const TensorView& q);   // + bf16, uniformly strided Q rows
size_t tc_workspace_bytes(const ScoreShape& s);
obc_status launch_score_tc(const ScoreShape& s, TensorView q, TensorView k, TensorView v,
                           float* scores, void* ws, cudaStream_t stream, const GivenAttention* given = nullptr,
                           SimtPlan* attention_only = nullptr);   // non-null: stop after pass 1 + combine, return the plan

// ---- tensor maps ----------------------------------------------------------------------------------
// bf16 tensor map of rank 2 or 4 with 128-byte swizzle, innermost dimension = head_dim (128), box
// {64, box_rows, 1, 1}; strides in bytes for dimensions 1..rank-1.  Maps are cached per host thread.
bool make_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              uint32_t box_rows);

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialization: its CTAs may
// become resident while the preceding kernel of the stream is still draining.  A kernel executes
// pdl_wait() before its first access to memory that an earlier kernel may have written (or may
// still read, for its own writes); what precedes the wait is set-up that touches no such memory.
// (Releasing the next kernel earlier, with griddepcontrol.launch_dependents after the wait, was measured
// and is not done: CTAs of the next kernel that sit waiting on an SM slowed the kernel at work.)
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              int cluster_x, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (cluster_x > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// ---- device helpers --------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// 4 consecutive elements of a row -> float4 (fp32 or bf16 storage)
template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) {
    return *reinterpret_cast<const float4*>(p);
}
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
    uint2 u = *reinterpret_cast<const uint2*>(p);
    float4 f;
    f.x = __uint_as_float(u.x << 16); f.y = __uint_as_float(u.x & 0xffff0000u);
    f.z = __uint_as_float(u.y << 16); f.w = __uint_as_float(u.y & 0xffff0000u);
    return f;
}

}  // namespace obc
