// Internal declarations shared by the .cu files of libwide (not part of the public ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "wide.h"

struct wide_prof_rec {
    const char* name;
    cudaEvent_t begin, end;
};

struct wide_ctx {
    int device;
    int sm_count;
    int* d_status;          // [0] device status word (WIDE_OK or WIDE_ERR_TIMEOUT), [1] reorder ticket,
                            // [4..5] grid-barrier counters of the decode kernels, [6] channel pool of the GEMV decode kernel, [8..9] tile queue of the
                            // 256-row down projection, [10..12] work list of the attention prefill kernel (next item, CTAs done, next block of rows to zero;
                            // zero between launches) (16 ints in all)
    float* decode_acc;      // fp32 accumulators of the decode path; zero between calls
    size_t decode_acc_floats;
    unsigned* d_tickets;    // 2048 completion counters, zero between calls: [0, 1024) and [1024, 1152) the decode FFN /
                            // O-projection kernel, [2040, 2048) the token tiles of the one-launch router
    float* attn_part;       // partial (m, l, O) of the key slices of the decode attention
    size_t attn_part_bytes;
    unsigned long long wait_ns;  // bound of every device-side wait
    void* encode_tiled;     // cuTensorMapEncodeTiled, resolved through the runtime
    unsigned long long launches;  // kernels launched by the library so far
    // optional per-launch timing: a pool of event pairs created by wide_profile_begin
    wide_prof_rec* prof;
    int prof_cap, prof_used;
};

// Launch with the programmatic-serialization attribute: the kernel may start its set-up while the kernel before
// it in the stream finishes; it calls grid_dep_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t wide_launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                         Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Counts one kernel launch and, when profiling is on, brackets it with a pair of CUDA events on
// the launching stream.  Usage: { WideLaunch l(ctx, s, "name"); kernel<<<..., s>>>(...); }
struct WideLaunch {
    wide_ctx* ctx;
    cudaStream_t s;
    int idx;
    WideLaunch(wide_ctx* c, cudaStream_t st, const char* name) : ctx(c), s(st), idx(-1) {
        ++ctx->launches;
        if (ctx->prof && ctx->prof_used < ctx->prof_cap) {
            idx = ctx->prof_used++;
            ctx->prof[idx].name = name;
            cudaEventRecord(ctx->prof[idx].begin, s);
        }
    }
    ~WideLaunch() {
        if (idx >= 0) cudaEventRecord(ctx->prof[idx].end, s);
    }
};

#define WIDE_CUDA_CHECK(expr)                         \
    do {                                              \
        cudaError_t err__ = (expr);                   \
        if (err__ != cudaSuccess) return WIDE_ERR_CUDA; \
    } while (0)

static inline bool wide_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t wide_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int wide_elem_bytes(int dtype) { return dtype == WIDE_BF16 ? 2 : 4; }

// ---- element conversion used by the CUDA-core kernels
__device__ __forceinline__ float wide_to_float(float v) { return v; }
__device__ __forceinline__ float wide_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float wide_to_float(double v) { return static_cast<float>(v); }
__device__ __forceinline__ double wide_to_double(float v) { return static_cast<double>(v); }
__device__ __forceinline__ double wide_to_double(__nv_bfloat16 v) { return static_cast<double>(__bfloat162float(v)); }
__device__ __forceinline__ double wide_to_double(double v) { return v; }
__device__ __forceinline__ void wide_store(float* p, float v) { *p = v; }
__device__ __forceinline__ void wide_store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ bool wide_mask_bit(const uint32_t* mask_bits, int words, int t, int g) {
    return (mask_bits[static_cast<size_t>(t) * words + (g >> 5)] >> (g & 31)) & 1u;
}

// Which K-axis kernel serves a prefill call is decided on the device, without a host read-back:
// the per-group kernel (Algorithm 3: only active (tile, group) blocks, scatter-reduce into the
// output) is chosen when the padded active fraction  sum_g ceil(counts[g]/128)*128 / (T*NG)  is at
// most thr_q / 1024, the owner-computes kernel otherwise.  Every kernel of the pair evaluates this
// same integer predicate when it starts; the one that is not chosen returns at once.
// thr_q < 0: never the per-group kernel; thr_q >= 4096: always.  Warp-collective (all 32 lanes).
#define WIDE_KAXIS_NEVER (-1)
#define WIDE_KAXIS_ALWAYS 4096
#ifdef __CUDACC__
__device__ __forceinline__ bool wide_kaxis_group_chosen(const int32_t* __restrict__ counts, int NG, int T, int thr_q) {
    if (counts == nullptr || thr_q < 0) return false;
    if (thr_q >= WIDE_KAXIS_ALWAYS) return true;
    long long tiles = 0;
    for (int g = threadIdx.x & 31; g < NG; g += 32) tiles += (counts[g] + 127) >> 7;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
    return tiles * 128 * 1024 <= static_cast<long long>(thr_q) * T * NG;
}
#endif

// ---- launchers (each returns WIDE_OK or WIDE_ERR_CUDA; arguments already validated)
int wide_launch_route(wide_ctx* ctx, cudaStream_t s, const void* x, int dtype, int T, int D,
                      const void* w_router, const void* w2, int rank, int NG, int mode, int k,
                      const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* ws, unsigned flags);
size_t wide_route_workspace(int T, int NG, int rank);
// Eq. 4 on the RMSNorm of the hidden state, weight-only work prepared once (csrc/route.cu)
size_t wide_route_pair_prepared_size(int D, int rank, int NG);
size_t wide_route_pair_norm_workspace(int T, int rank);
bool wide_route_pair_norm_supported(int D, int rank, int NG);
int wide_launch_route_pair_prepare(wide_ctx* ctx, cudaStream_t s, const void* w1, const void* w2, const void* gamma, int D,
                                   int rank, int NG, void* prepared);
int wide_launch_route_pair_norm(wide_ctx* ctx, cudaStream_t s, const void* x, int T, int D, const void* w1, const void* w2,
                                int rank, int NG, const void* gamma, float eps, void* prepared, uint32_t* mask_bits,
                                float* scores, void* ws);

int wide_launch_reorder(wide_ctx* ctx, cudaStream_t s, const uint32_t* mask_bits, int T, int NG,
                        int tile_m, int32_t* perm, int32_t* counts, uint8_t* tile_map,
                        int32_t* work_list, int32_t* n_work, int32_t* union_list, int32_t* n_union,
                        int32_t* offsets, int32_t* token_order, int32_t* token_rank);

int wide_launch_mask_slice(wide_ctx* ctx, cudaStream_t s, const uint32_t* mask_bits, int T, int NG, int g_begin, int g_end,
                           uint32_t* out);

int wide_launch_unpermute(wide_ctx* ctx, cudaStream_t s, const void* src, const int32_t* perm, const int32_t* counts,
                          const int32_t* offsets, int T, int NG, int G, int elem_bytes, void* dst);

// CUDA-core FFN / O-proj (any shape, fp32 or bf16).  `h` is scratch [T, Dff] in `dtype`.
int wide_launch_ffn_simt(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu, const void* wd,
                         int dtype, int T, int D, int Dff, int G, const uint32_t* mask_bits, void* y,
                         int out_dtype, void* h);
int wide_launch_oproj_simt(wide_ctx* ctx, cudaStream_t s, const void* a, const void* wo, int dtype, int T, int D,
                           int K, int G, const uint32_t* mask_bits, void* y, int out_dtype);

// tcgen05 prefill path (bf16).  `h` is scratch [T, Dff] bf16, `acc` scratch [T, D] fp32 (used when
// the per-group K-axis kernel reduces in fp32 towards a bf16 output).
int wide_launch_ffn_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg,
                               const void* wu, const void* wd, int T, int D, int Dff, int G,
                               const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts,
                               const int32_t* token_order, const int32_t* token_rank, void* y,
                               int out_dtype, void* h, void* acc, unsigned flags);
int wide_launch_ffn_prefill_tp(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu,
                               const void* wd, int T, int D, int Dff, int G, const uint32_t* mask_bits,
                               const int32_t* perm, const int32_t* counts, const int32_t* token_order,
                               const int32_t* token_rank, float* const* shards, int world, int rows_per_rank, void* h);
int wide_launch_scores_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* w_router, int T, int NG,
                          int ld, int D, float* scores, float* wnorm, int max_split, int* ksplit_out, int* chain_out);
// `a_masked` is scratch [T, K] bf16, `acc` scratch [T, D] fp32.
int wide_launch_oproj_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* a, const void* wo, int T,
                                 int D, int K, int G, const uint32_t* mask_bits, const int32_t* perm,
                                 const int32_t* counts, const int32_t* token_order,
                                 const int32_t* token_rank, void* y, int out_dtype, void* a_masked, void* acc,
                                 unsigned flags);

// Per-group GEMM-K (Algorithm 3) and its helpers, csrc/gemmk_group.cu.
int wide_launch_kaxis_prep(wide_ctx* ctx, cudaStream_t s, const int32_t* counts, int NG, int T, int thr_q, void* zero_ptr,
                           size_t zero_bytes, const void* a, const uint32_t* mask_bits, const int32_t* token_rank, int K,
                           int G, void* a_masked);
int wide_launch_gemmk_group_tc(wide_ctx* ctx, cudaStream_t s, const void* A, int lda, const void* B, int T, int N, int K,
                               int G, const int32_t* perm, const int32_t* counts, const int32_t* a_row_of_token, void* Y,
                               bool bf16_red, int thr_q, const char* name);
int wide_launch_kaxis_convert(wide_ctx* ctx, cudaStream_t s, const int32_t* counts, int NG, int T, int thr_q,
                              const float* acc, void* y_bf16, size_t n_elems);

// tcgen05 decode path (bf16, T <= WIDE_DECODE_MAX_TOKENS).
size_t wide_decode_workspace(int T, int D, int inner);
int wide_launch_ffn_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg,
                              const void* wu, const void* wd, int T, int D, int Dff, int G,
                              const uint32_t* mask_bits, void* y, int out_dtype, void* ws);
int wide_launch_oproj_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* a, const void* wo, int T,
                                int D, int K, int G, const uint32_t* mask_bits, void* y,
                                int out_dtype, void* ws);

// CUDA-core decode path for at most WIDE_DECODE_GEMV_MAX_TOKENS tokens (csrc/decode_gemv.cu).  `act` is x
// (FFN) or the attention output (O-projection, wg = wu = nullptr); `ws` as for the tensor-core kernel.
bool wide_decode_gemv_fits(bool is_ffn, int T, int D, int inner, int G);
int wide_launch_decode_gemv(wide_ctx* ctx, cudaStream_t s, bool is_ffn, const void* act, const void* wg, const void* wu,
                            const void* wd, int T, int D, int inner, int G, const uint32_t* mask_bits, void* y,
                            int out_dtype, void* ws);

// 2-D bf16 row-major [rows, cols] tensor map, box = [box_rows, 64 columns], 128-byte swizzle.
bool wide_make_tmap_bf16(const wide_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows);

// tcgen05 masked attention prefill (bf16, head_dim 64 or 128).
int wide_launch_attn_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v, int Tq,
                                int Tk, int Hq, int Hkv, int head_dim, int hpg, const int32_t* perm,
                                const int32_t* counts, int causal, float scale, void* o);

// tcgen05 routed linear layer (GEMM-MN, bf16): y [T, Nout] bf16, zeros for inactive (token, group) pairs.
int wide_launch_linear_mn_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* w, int T, int D, int Nout,
                             int G, const int32_t* perm, const int32_t* counts, void* y);

// Decode form of the masked attention (CUDA cores, split over the keys); needs
// tokens_q * (n_q_heads / n_kv_heads) <= 8 (wide_attn_decode_fits).
bool wide_attn_decode_fits(int Tq, int Hq, int Hkv);
int wide_launch_attn_decode(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                            const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int head_dim, int hpg,
                            int causal, float scale, void* o, unsigned flags);
