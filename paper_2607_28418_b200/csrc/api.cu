// C ABI of libwide: argument validation, workspace sizing and dispatch.  See include/wide.h.
#include <cstdio>
#include <new>

#include <math.h>

#include "internal.h"

namespace {

bool valid_dtype(int d) { return d == WIDE_BF16 || d == WIDE_F32; }
bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// Which implementation serves this FFN / O-proj call.
enum Path { PATH_SIMT, PATH_PREFILL_TC, PATH_DECODE_TC, PATH_NONE };

Path choose_path(int dtype, int tokens, int hidden, int inner, int group, unsigned flags) {
    if (flags & WIDE_FLAG_SIMT) return PATH_SIMT;
    const bool tc_ok = dtype == WIDE_BF16 && hidden % 64 == 0 && inner % 64 == 0 &&
                       (group == 64 || group == 128 || group == 256 || group == 512);
    if (!tc_ok) return PATH_NONE;
    if (flags & WIDE_FLAG_FORCE_DECODE) return tokens <= WIDE_DECODE_MAX_TOKENS ? PATH_DECODE_TC : PATH_NONE;
    if (flags & WIDE_FLAG_FORCE_PREFILL) return PATH_PREFILL_TC;
    return tokens <= WIDE_DECODE_MAX_TOKENS ? PATH_DECODE_TC : PATH_PREFILL_TC;
}

size_t inner_scratch(int dtype, int tokens, int hidden, int inner) {
    // hidden activation / masked attention output [tokens, inner] in dtype, or the decode scratch
    size_t a = wide_align_up(static_cast<size_t>(tokens) * inner * wide_elem_bytes(dtype), 256);
    size_t b = tokens <= WIDE_DECODE_MAX_TOKENS ? wide_decode_workspace(tokens, hidden, inner) : 0;
    return a > b ? a : b;
}

// fp32 sums [tokens, hidden] of the per-group K-axis kernel, behind the inner scratch
size_t acc_scratch(int tokens, int hidden) {
    return wide_align_up(static_cast<size_t>(tokens) * hidden * sizeof(float), 256);
}

}  // namespace

extern "C" {

int wide_version(void) { return WIDE_VERSION; }

const char* wide_strerror(int code) {
    switch (code) {
        case WIDE_OK: return "ok";
        case WIDE_ERR_INVALID_ARG: return "invalid argument";
        case WIDE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape for the requested path";
        case WIDE_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case WIDE_ERR_WORKSPACE: return "workspace missing or too small";
        case WIDE_ERR_CUDA: return "CUDA runtime or driver error";
        case WIDE_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown error code";
    }
}

int wide_create(wide_ctx** out, int device) {
    if (!out) return WIDE_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return WIDE_ERR_CUDA;
    WIDE_CUDA_CHECK(cudaSetDevice(device));
    cudaDeviceProp prop;
    WIDE_CUDA_CHECK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return WIDE_ERR_CUDA;  // built for sm_100a only
    wide_ctx* ctx = new (std::nothrow) wide_ctx();
    if (!ctx) return WIDE_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->wait_ns = 2000000000ull;
    ctx->encode_tiled = nullptr;
    ctx->launches = 0;
    ctx->prof = nullptr;
    ctx->prof_cap = ctx->prof_used = 0;
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        ctx->encode_tiled = fn;
    // decode accumulators: 64 tokens x (2 * inner + hidden) floats for inner <= 32768, hidden <= 16384
    ctx->decode_acc = nullptr;
    ctx->decode_acc_floats = static_cast<size_t>(WIDE_DECODE_MAX_TOKENS) * (2 * 32768 + 16384);
    if (cudaMalloc(&ctx->d_status, 16 * sizeof(int)) != cudaSuccess) {
        delete ctx;
        return WIDE_ERR_CUDA;
    }
    ctx->d_tickets = nullptr;
    ctx->attn_part = nullptr;
    ctx->attn_part_bytes = 4u << 20;
    if (cudaMalloc(&ctx->attn_part, ctx->attn_part_bytes) != cudaSuccess ||
        cudaMalloc(&ctx->decode_acc, ctx->decode_acc_floats * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ctx->d_tickets, 2048 * sizeof(unsigned)) != cudaSuccess ||
        cudaMemset(ctx->d_tickets, 0, 2048 * sizeof(unsigned)) != cudaSuccess ||
        cudaMemset(ctx->d_status, 0, 16 * sizeof(int)) != cudaSuccess ||
        cudaMemset(ctx->decode_acc, 0, ctx->decode_acc_floats * sizeof(float)) != cudaSuccess) {
        cudaFree(ctx->attn_part);
        cudaFree(ctx->decode_acc);
        cudaFree(ctx->d_tickets);
        cudaFree(ctx->d_status);
        delete ctx;
        return WIDE_ERR_CUDA;
    }
    *out = ctx;
    return WIDE_OK;
}

static void free_profile(wide_ctx* ctx) {
    if (!ctx->prof) return;
    for (int i = 0; i < ctx->prof_cap; ++i) {
        cudaEventDestroy(ctx->prof[i].begin);
        cudaEventDestroy(ctx->prof[i].end);
    }
    delete[] ctx->prof;
    ctx->prof = nullptr;
    ctx->prof_cap = ctx->prof_used = 0;
}

int wide_profile_begin(wide_ctx* ctx, int max_records) {
    if (!ctx || max_records <= 0 || max_records > (1 << 20)) return WIDE_ERR_INVALID_ARG;
    free_profile(ctx);
    ctx->prof = new (std::nothrow) wide_prof_rec[max_records];
    if (!ctx->prof) return WIDE_ERR_CUDA;
    for (int i = 0; i < max_records; ++i) {
        if (cudaEventCreate(&ctx->prof[i].begin) != cudaSuccess || cudaEventCreate(&ctx->prof[i].end) != cudaSuccess)
            return WIDE_ERR_CUDA;
        ctx->prof_cap = i + 1;
    }
    ctx->prof_used = 0;
    return WIDE_OK;
}

int wide_profile_end(wide_ctx* ctx, void* stream, char* buf, size_t buf_bytes) {
    if (!ctx || !buf || buf_bytes == 0) return WIDE_ERR_INVALID_ARG;
    buf[0] = 0;
    if (!ctx->prof) return WIDE_ERR_INVALID_ARG;
    WIDE_CUDA_CHECK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    // aggregate by kernel name (names are string literals: compare by pointer, then by text)
    struct Agg { const char* name; int launches; double ms; };
    Agg agg[64];
    int n_agg = 0;
    for (int i = 0; i < ctx->prof_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, ctx->prof[i].begin, ctx->prof[i].end) != cudaSuccess) continue;
        int j = 0;
        for (; j < n_agg; ++j)
            if (agg[j].name == ctx->prof[i].name) break;
        if (j == n_agg) {
            if (n_agg == 64) continue;
            agg[n_agg++] = Agg{ctx->prof[i].name, 0, 0.0};
        }
        agg[j].launches += 1;
        agg[j].ms += ms;
    }
    size_t off = 0;
    for (int j = 0; j < n_agg; ++j) {
        int w = snprintf(buf + off, buf_bytes - off, "%s,%d,%.6f\n", agg[j].name, agg[j].launches, agg[j].ms);
        if (w < 0 || static_cast<size_t>(w) >= buf_bytes - off) break;
        off += static_cast<size_t>(w);
    }
    free_profile(ctx);
    return WIDE_OK;
}

int wide_launch_count(wide_ctx* ctx, unsigned long long* count) {
    if (!ctx || !count) return WIDE_ERR_INVALID_ARG;
    *count = ctx->launches;
    return WIDE_OK;
}

int wide_destroy(wide_ctx* ctx) {
    if (!ctx) return WIDE_ERR_INVALID_ARG;
    free_profile(ctx);
    cudaFree(ctx->attn_part);
    cudaFree(ctx->d_tickets);
    cudaFree(ctx->decode_acc);
    cudaFree(ctx->d_status);
    delete ctx;
    return WIDE_OK;
}

int wide_status(wide_ctx* ctx, void* stream, int* status) {
    if (!ctx || !status) return WIDE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int v = 0;
    WIDE_CUDA_CHECK(cudaMemcpyAsync(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s));
    WIDE_CUDA_CHECK(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), s));
    WIDE_CUDA_CHECK(cudaStreamSynchronize(s));
    if (v != WIDE_OK) {
        // a kernel gave up half-way: restore the invariants later calls rely on
        WIDE_CUDA_CHECK(cudaMemsetAsync(ctx->d_status, 0, 16 * sizeof(int), s));
        WIDE_CUDA_CHECK(cudaMemsetAsync(ctx->decode_acc, 0, ctx->decode_acc_floats * sizeof(float), s));
        WIDE_CUDA_CHECK(cudaMemsetAsync(ctx->d_tickets, 0, 2048 * sizeof(unsigned), s));
        WIDE_CUDA_CHECK(cudaStreamSynchronize(s));
    }
    *status = v;
    return WIDE_OK;
}

int wide_set_wait_limit_ns(wide_ctx* ctx, uint64_t ns) {
    if (!ctx || ns == 0) return WIDE_ERR_INVALID_ARG;
    ctx->wait_ns = ns;
    return WIDE_OK;
}

size_t wide_workspace_bytes(int op, int dtype, int tokens, int hidden, int inner, int group, int n_groups) {
    (void)group;
    if (tokens < 0 || hidden < 0 || inner < 0 || n_groups < 0 || !valid_dtype(dtype)) return 0;
    switch (op) {
        case WIDE_OP_ROUTE: return wide_route_workspace(tokens, n_groups, 64);
        case WIDE_OP_FFN:
        case WIDE_OP_OPROJ: return inner_scratch(dtype, tokens, hidden, inner) + acc_scratch(tokens, hidden);
        default: return 0;
    }
}

int wide_route(wide_ctx* ctx, void* stream, const void* x, int dtype, int tokens, int hidden,
               const void* w_router, const void* w2, int rank, int n_groups, int mode, int k,
               const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* workspace,
               size_t workspace_bytes, unsigned flags) {
    if (!ctx || !x || !w_router || !mask_bits || !valid_dtype(dtype)) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || n_groups <= 0) return WIDE_ERR_INVALID_ARG;
    if (mode == WIDE_ROUTE_TOPK) {
        if (w2 || rank != 0) return WIDE_ERR_INVALID_ARG;
        if (!k_per_token && (k < 0 || k > n_groups)) return WIDE_ERR_INVALID_ARG;
    } else if (mode == WIDE_ROUTE_PAIR_ARGMAX) {
        if (!w2 || rank <= 0 || rank > 64) return WIDE_ERR_INVALID_ARG;
    } else {
        return WIDE_ERR_INVALID_ARG;
    }
    if (n_groups > WIDE_MAX_GROUPS || hidden % 8 != 0) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(x) || !wide_aligned16(w_router) || (w2 && !wide_aligned16(w2)) || !wide_aligned16(workspace))
        return WIDE_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < wide_route_workspace(tokens, n_groups, rank)) return WIDE_ERR_WORKSPACE;
    return wide_launch_route(ctx, static_cast<cudaStream_t>(stream), x, dtype, tokens, hidden, w_router, w2, rank,
                             n_groups, mode, k, k_per_token, mask_bits, scores, workspace, flags);
}

size_t wide_route_pair_prepared_bytes(int hidden, int rank, int n_groups) {
    if (hidden <= 0 || rank <= 0 || n_groups <= 0) return 0;
    return wide_route_pair_prepared_size(hidden, rank, n_groups);
}

size_t wide_route_pair_norm_workspace_bytes(int tokens, int rank) {
    if (tokens < 0 || rank <= 0) return 0;
    return wide_route_pair_norm_workspace(tokens, rank);
}

int wide_route_pair_prepare(wide_ctx* ctx, void* stream, const void* w1, const void* w2, const void* norm_weight, int hidden,
                            int rank, int n_groups, void* prepared, size_t prepared_bytes) {
    if (!ctx || !w1 || !w2 || !prepared || hidden <= 0 || rank <= 0 || n_groups <= 0) return WIDE_ERR_INVALID_ARG;
    if (!wide_route_pair_norm_supported(hidden, rank, n_groups) || !ctx->encode_tiled) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(w1) || !wide_aligned16(w2) || !wide_aligned16(prepared) || (norm_weight && !wide_aligned16(norm_weight)))
        return WIDE_ERR_ALIGNMENT;
    if (prepared_bytes < wide_route_pair_prepared_size(hidden, rank, n_groups)) return WIDE_ERR_WORKSPACE;
    return wide_launch_route_pair_prepare(ctx, static_cast<cudaStream_t>(stream), w1, w2, norm_weight, hidden, rank, n_groups,
                                          prepared);
}

int wide_route_pair_norm(wide_ctx* ctx, void* stream, const void* x, int tokens, int hidden, const void* w1, const void* w2,
                         int rank, int n_groups, const void* norm_weight, float eps, const void* prepared,
                         uint32_t* mask_bits, float* scores, void* workspace, size_t workspace_bytes) {
    if (!ctx || !x || !w1 || !w2 || !prepared || !mask_bits) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || rank <= 0 || n_groups <= 0 || !(eps >= 0.f)) return WIDE_ERR_INVALID_ARG;
    if (!wide_route_pair_norm_supported(hidden, rank, n_groups) || !ctx->encode_tiled) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(x) || !wide_aligned16(w1) || !wide_aligned16(w2) || !wide_aligned16(prepared) ||
        !wide_aligned16(workspace) || (norm_weight && !wide_aligned16(norm_weight)))
        return WIDE_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < wide_route_pair_norm_workspace(tokens, rank)) return WIDE_ERR_WORKSPACE;
    return wide_launch_route_pair_norm(ctx, static_cast<cudaStream_t>(stream), x, tokens, hidden, w1, w2, rank, n_groups,
                                       norm_weight, eps, const_cast<void*>(prepared), mask_bits, scores, workspace);
}

int wide_reorder(wide_ctx* ctx, void* stream, const uint32_t* mask_bits, int tokens, int n_groups,
                 int tile_m, int32_t* perm, int32_t* counts, uint8_t* tile_map, int32_t* work_list,
                 int32_t* n_work, int32_t* union_list, int32_t* n_union, int32_t* offsets, int32_t* token_order,
                 int32_t* token_rank) {
    if (!ctx || !mask_bits || !perm || !counts || !tile_map || !work_list || !n_work || !union_list || !n_union ||
        !offsets)
        return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || n_groups <= 0 || !is_pow2(tile_m) || tile_m < 16) return WIDE_ERR_INVALID_ARG;
    if ((token_order == nullptr) != (token_rank == nullptr)) return WIDE_ERR_INVALID_ARG;
    if (n_groups > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    return wide_launch_reorder(ctx, static_cast<cudaStream_t>(stream), mask_bits, tokens, n_groups, tile_m, perm,
                               counts, tile_map, work_list, n_work, union_list, n_union, offsets, token_order,
                               token_rank);
}

int wide_mask_slice(wide_ctx* ctx, void* stream, const uint32_t* mask_bits, int tokens, int n_groups, int group_begin,
                    int group_end, uint32_t* out_bits) {
    if (!ctx || !mask_bits || !out_bits) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || n_groups <= 0 || group_begin < 0 || group_end < group_begin || group_end > n_groups)
        return WIDE_ERR_INVALID_ARG;
    if (n_groups > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    return wide_launch_mask_slice(ctx, static_cast<cudaStream_t>(stream), mask_bits, tokens, n_groups, group_begin,
                                  group_end, out_bits);
}

int wide_ffn(wide_ctx* ctx, void* stream, const void* x, const void* w_gate, const void* w_up,
             const void* w_down, int dtype, int tokens, int hidden, int d_ff, int group,
             const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts,
             const int32_t* token_order, const int32_t* token_rank, void* y, int out_dtype,
             void* workspace, size_t workspace_bytes, unsigned flags) {
    if (!ctx || !x || !w_gate || !w_up || !w_down || !mask_bits || !y) return WIDE_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || !valid_dtype(out_dtype)) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || d_ff <= 0 || group <= 0 || d_ff % group != 0) return WIDE_ERR_INVALID_ARG;
    if (d_ff / group > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    const Path path = choose_path(dtype, tokens, hidden, d_ff, group, flags);
    if (path == PATH_NONE) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (path == PATH_SIMT && (hidden % 4 != 0 || group % 4 != 0)) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (path == PATH_PREFILL_TC && (!perm || !counts)) return WIDE_ERR_INVALID_ARG;
    if ((token_order == nullptr) != (token_rank == nullptr)) return WIDE_ERR_INVALID_ARG;
    if (!wide_aligned16(x) || !wide_aligned16(w_gate) || !wide_aligned16(w_up) || !wide_aligned16(w_down) ||
        !wide_aligned16(y) || !wide_aligned16(workspace))
        return WIDE_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < inner_scratch(dtype, tokens, hidden, d_ff) + acc_scratch(tokens, hidden))
        return WIDE_ERR_WORKSPACE;
    if ((flags & WIDE_FLAG_KAXIS_GROUP) && (flags & WIDE_FLAG_KAXIS_OWNER)) return WIDE_ERR_INVALID_ARG;
    void* acc = static_cast<uint8_t*>(workspace) + inner_scratch(dtype, tokens, hidden, d_ff);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (path) {
        case PATH_SIMT:
            return wide_launch_ffn_simt(ctx, s, x, w_gate, w_up, w_down, dtype, tokens, hidden, d_ff, group, mask_bits, y,
                                        out_dtype, workspace);
        case PATH_PREFILL_TC:
            return wide_launch_ffn_prefill_tc(ctx, s, x, w_gate, w_up, w_down, tokens, hidden, d_ff, group, mask_bits,
                                              perm, counts, token_order, token_rank, y, out_dtype, workspace, acc, flags);
        default:
            if (!(flags & WIDE_FLAG_DECODE_TC) && wide_decode_gemv_fits(true, tokens, hidden, d_ff, group))
                return wide_launch_decode_gemv(ctx, s, true, x, w_gate, w_up, w_down, tokens, hidden, d_ff, group,
                                               mask_bits, y, out_dtype, workspace);
            return wide_launch_ffn_decode_tc(ctx, s, x, w_gate, w_up, w_down, tokens, hidden, d_ff, group, mask_bits,
                                             y, out_dtype, workspace);
    }
}

int wide_ffn_tp(wide_ctx* ctx, void* stream, const void* x, const void* w_gate, const void* w_up, const void* w_down,
                int dtype, int tokens, int hidden, int d_ff_local, int group, const uint32_t* mask_bits_local,
                const int32_t* perm, const int32_t* counts, const int32_t* token_order, const int32_t* token_rank,
                float* const* y_shards, int world, int rows_per_rank, void* workspace, size_t workspace_bytes) {
    if (!ctx || !x || !w_gate || !w_up || !w_down || !mask_bits_local || !perm || !counts || !y_shards)
        return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || d_ff_local <= 0 || group <= 0 || d_ff_local % group != 0) return WIDE_ERR_INVALID_ARG;
    if (world < 1 || world > 8 || rows_per_rank <= 0 || static_cast<long long>(world) * rows_per_rank < tokens)
        return WIDE_ERR_INVALID_ARG;
    if ((token_order == nullptr) != (token_rank == nullptr)) return WIDE_ERR_INVALID_ARG;
    for (int r = 0; r < world; ++r)
        if (!y_shards[r] || !wide_aligned16(y_shards[r])) return WIDE_ERR_INVALID_ARG;
    if (d_ff_local / group > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (dtype != WIDE_BF16 || hidden % 64 != 0 || (group != 64 && group != 128 && group != 256 && group != 512) ||
        !ctx->encode_tiled)
        return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(x) || !wide_aligned16(w_gate) || !wide_aligned16(w_up) || !wide_aligned16(w_down) ||
        !wide_aligned16(workspace))
        return WIDE_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < inner_scratch(dtype, tokens, hidden, d_ff_local)) return WIDE_ERR_WORKSPACE;
    return wide_launch_ffn_prefill_tp(ctx, static_cast<cudaStream_t>(stream), x, w_gate, w_up, w_down, tokens, hidden,
                                      d_ff_local, group, mask_bits_local, perm, counts, token_order, token_rank, y_shards,
                                      world, rows_per_rank, workspace);
}

int wide_oproj(wide_ctx* ctx, void* stream, const void* attn_out, const void* w_o, int dtype,
               int tokens, int hidden, int attn_dim, int group, const uint32_t* mask_bits,
               const int32_t* perm, const int32_t* counts, const int32_t* token_order,
               const int32_t* token_rank, void* y, int out_dtype, void* workspace,
               size_t workspace_bytes, unsigned flags) {
    if ((token_order == nullptr) != (token_rank == nullptr)) return WIDE_ERR_INVALID_ARG;
    if ((perm == nullptr) != (counts == nullptr)) return WIDE_ERR_INVALID_ARG;
    if ((flags & WIDE_FLAG_KAXIS_GROUP) && ((flags & WIDE_FLAG_KAXIS_OWNER) || !perm)) return WIDE_ERR_INVALID_ARG;
    if (!ctx || !attn_out || !w_o || !mask_bits || !y) return WIDE_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || !valid_dtype(out_dtype)) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || attn_dim <= 0 || group <= 0 || attn_dim % group != 0) return WIDE_ERR_INVALID_ARG;
    if (attn_dim / group > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    const Path path = choose_path(dtype, tokens, hidden, attn_dim, group, flags);
    if (path == PATH_NONE) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (path == PATH_SIMT && (hidden % 4 != 0 || group % 4 != 0)) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(attn_out) || !wide_aligned16(w_o) || !wide_aligned16(y) || !wide_aligned16(workspace))
        return WIDE_ERR_ALIGNMENT;
    if (path != PATH_SIMT &&
        (!workspace || workspace_bytes < inner_scratch(dtype, tokens, hidden, attn_dim) + acc_scratch(tokens, hidden)))
        return WIDE_ERR_WORKSPACE;
    void* acc = workspace ? static_cast<uint8_t*>(workspace) + inner_scratch(dtype, tokens, hidden, attn_dim) : nullptr;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (path) {
        case PATH_SIMT:
            return wide_launch_oproj_simt(ctx, s, attn_out, w_o, dtype, tokens, hidden, attn_dim, group, mask_bits, y,
                                          out_dtype);
        case PATH_PREFILL_TC:
            return wide_launch_oproj_prefill_tc(ctx, s, attn_out, w_o, tokens, hidden, attn_dim, group, mask_bits, perm,
                                                counts, token_order, token_rank, y, out_dtype, workspace, acc, flags);
        default:
            if (!(flags & WIDE_FLAG_DECODE_TC) && wide_decode_gemv_fits(false, tokens, hidden, attn_dim, group))
                return wide_launch_decode_gemv(ctx, s, false, attn_out, nullptr, nullptr, w_o, tokens, hidden, attn_dim,
                                               group, mask_bits, y, out_dtype, workspace);
            return wide_launch_oproj_decode_tc(ctx, s, attn_out, w_o, tokens, hidden, attn_dim, group, mask_bits, y,
                                               out_dtype, workspace);
    }
}

int wide_attn(wide_ctx* ctx, void* stream, const void* q, const void* k, const void* v, int dtype, int tokens_q,
              int tokens_k, int n_q_heads, int n_kv_heads, int head_dim, int heads_per_group,
              const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts, int causal, float scale, void* o,
              unsigned flags) {
    if (!ctx || !q || !k || !v || !o) return WIDE_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return WIDE_ERR_INVALID_ARG;
    if (tokens_q < 0 || tokens_k <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || heads_per_group <= 0)
        return WIDE_ERR_INVALID_ARG;
    if (n_q_heads % n_kv_heads != 0 || n_q_heads % heads_per_group != 0) return WIDE_ERR_INVALID_ARG;
    if (dtype != WIDE_BF16 || (head_dim != 64 && head_dim != 128)) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (n_q_heads / heads_per_group > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(q) || !wide_aligned16(k) || !wide_aligned16(v) || !wide_aligned16(o)) return WIDE_ERR_ALIGNMENT;
    if (tokens_q == 0) return WIDE_OK;
    if (!(scale > 0.f)) scale = 1.0f / sqrtf(static_cast<float>(head_dim));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a handful of query rows per KV head: the split-key decode form, straight from the mask
    const bool decode = mask_bits && !(flags & WIDE_FLAG_FORCE_PREFILL) &&
                        wide_attn_decode_fits(tokens_q, n_q_heads, n_kv_heads);
    if (decode || (flags & WIDE_FLAG_FORCE_DECODE)) {
        if (!mask_bits) return WIDE_ERR_INVALID_ARG;
        if (!wide_attn_decode_fits(tokens_q, n_q_heads, n_kv_heads)) return WIDE_ERR_UNSUPPORTED_SHAPE;
        return wide_launch_attn_decode(ctx, s, q, k, v, mask_bits, tokens_q, tokens_k, n_q_heads, n_kv_heads, head_dim,
                                       heads_per_group, causal ? 1 : 0, scale, o, flags);
    }
    if (!perm || !counts) return WIDE_ERR_INVALID_ARG;
    if (!ctx->encode_tiled) return WIDE_ERR_UNSUPPORTED_SHAPE;
    return wide_launch_attn_prefill_tc(ctx, s, q, k, v, tokens_q, tokens_k, n_q_heads, n_kv_heads, head_dim,
                                       heads_per_group, perm, counts, causal ? 1 : 0, scale, o);
}

int wide_qproj(wide_ctx* ctx, void* stream, const void* x, const void* w, int dtype, int tokens, int hidden,
               int n_out, int group, const int32_t* perm, const int32_t* counts, void* y, unsigned flags) {
    (void)flags;
    if (!ctx || !x || !w || !perm || !counts || !y) return WIDE_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || n_out <= 0 || group <= 0 || n_out % group != 0) return WIDE_ERR_INVALID_ARG;
    if (dtype != WIDE_BF16 || hidden % 64 != 0 || (group != 128 && group != 256 && group != 512) || !ctx->encode_tiled)
        return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (n_out / group > WIDE_MAX_GROUPS) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(x) || !wide_aligned16(w) || !wide_aligned16(y)) return WIDE_ERR_ALIGNMENT;
    return wide_launch_linear_mn_tc(ctx, static_cast<cudaStream_t>(stream), x, w, tokens, hidden, n_out, group, perm,
                                    counts, y);
}

int wide_unpermute(wide_ctx* ctx, void* stream, const void* src_packed, const int32_t* perm,
                   const int32_t* counts, const int32_t* offsets, int tokens, int n_groups,
                   int group, int elem_bytes, void* dst) {
    if (!ctx || !src_packed || !perm || !counts || !offsets || !dst) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || n_groups <= 0 || group <= 0 || (elem_bytes != 2 && elem_bytes != 4)) return WIDE_ERR_INVALID_ARG;
    if ((group * elem_bytes) % 16 != 0) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(src_packed) || !wide_aligned16(dst)) return WIDE_ERR_ALIGNMENT;
    return wide_launch_unpermute(ctx, static_cast<cudaStream_t>(stream), src_packed, perm, counts, offsets, tokens,
                                 n_groups, group, elem_bytes, dst);
}

}  // extern "C"
