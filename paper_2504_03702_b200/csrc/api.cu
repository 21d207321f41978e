// C-ABI layer: argument checks, context life cycle, status word.  No arithmetic of the
// method lives here; every step of the path runs in the kernels of the other files.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "pre_common.cuh"

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int fail_cuda(pre_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int)e;
    return PRE_ECUDA;
}

void release(pre_ctx* c) {
    if (!c) return;
    cudaFree(c->d_status);
    cudaFree(c->d_chunk_off);
    cudaFree(c->d_excess);
    cudaFree(c->d_bin_count);
    cudaFree(c->d_bin_base);
    cudaFree(c->d_bin_cursor);
    cudaFree(c->d_records);
    cudaFree(c->d_slots);
    cudaFree(c->d_enter);
    cudaFree(c->d_active);
    cudaFree(c->d_scaler_partial);
    cudaFree(c->d_scaler_done);
    cudaFree(c->d_ring_done);
    cudaFree(c->d_queue_entry);
    for (int k = 0; k < 2; ++k) { cudaFree(c->d_fused_totals[k]); cudaFree(c->d_fused_hint[k]); }
    cudaFree(c->d_fused_base);
    cudaFree(c->d_fused_sync);
    cudaFree(c->d_rs_summary);
    cudaFree(c->d_rs_jtop);
    cudaFree(c->d_rs_over);
    cudaFree(c->d_rs_guard);
    cudaFree(c->d_rs_handled);
    delete c;
}

template <typename T>
cudaError_t alloc_zero(T** p, size_t count) {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
    if (e != cudaSuccess) { *p = nullptr; return e; }
    return cudaMemset(*p, 0, count * sizeof(T));
}

}  // namespace

extern "C" {

int pre_create(const pre_config* cfg, pre_ctx** out) {
    if (!cfg || !out) return PRE_EINVAL;
    if (cfg->n_instances < 1 || cfg->horizon < 1 || cfg->horizon > PRE_MAX_HORIZON) return PRE_EINVAL;
    if (cfg->capacity_tokens < 1 || cfg->max_requests < 1 || cfg->max_requests >= (1LL << 31)) return PRE_EINVAL;
    if (!std::isfinite(cfg->t_mem) || !std::isfinite(cfg->beta) || cfg->t_mem < 0.0 || cfg->beta < 0.0)
        return PRE_EINVAL;
    if ((long long)cfg->n_instances * cfg->horizon >= (1LL << 40)) return PRE_EINVAL;

    pre_ctx* c = new (std::nothrow) pre_ctx();
    if (!c) return PRE_ENOMEM;
    std::memset(c, 0, sizeof(*c));
    c->cfg = *cfg;
    c->theta = cfg->t_mem * (double)cfg->capacity_tokens;

    cudaError_t e = cudaGetDevice(&c->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, c->device);
    if (e != cudaSuccess) { delete c; return PRE_ECUDA; }
    c->n_sm = prop.multiProcessorCount;

    const int I = cfg->n_instances, H = cfg->horizon;
    const int t = pre_tile_rows_for(I, H, c->n_sm);
    c->tile_rows = t;
    c->n_tiles = (I + t - 1) / t;
    if (pre_tile_smem_bytes(t, H) > (size_t)prop.sharedMemPerBlockOptin) { delete c; return PRE_EINVAL; }

    e = alloc_zero(&c->d_status, 8);     // status | give-up flag, agreed exchange, blocks met | . | exchange counter
    c->d_abort = c->d_status ? c->d_status + 1 : nullptr;
    c->d_epoch = c->d_status ? reinterpret_cast<unsigned int*>(c->d_status + 5) : nullptr;
    if (e == cudaSuccess) {   // the slots start as zeros: the first tags must not be zero
        const unsigned int first = 2;
        e = cudaMemcpy(c->d_epoch, &first, sizeof(first), cudaMemcpyHostToDevice);
    }
    c->max_chunks = pre_sort_max_chunks(cfg->max_requests, c->n_sm);
    if (e == cudaSuccess && pre_chunk_table_words(c->n_tiles, c->max_chunks))
        e = alloc_zero(&c->d_chunk_off, pre_chunk_table_words(c->n_tiles, c->max_chunks));
    if (e == cudaSuccess) e = alloc_zero(&c->d_excess, (size_t)I);
    if (e == cudaSuccess) e = alloc_zero(&c->d_bin_count, (size_t)c->n_tiles);
    if (e == cudaSuccess) e = alloc_zero(&c->d_bin_base, (size_t)c->n_tiles + 1);
    if (e == cudaSuccess) e = alloc_zero(&c->d_bin_cursor, (size_t)c->n_tiles);
    // records: read in windows of four; the fused build pads every tile's list to 16 bytes
    // (the fused build keeps an eighth and 32 records of spare room per list)
    const size_t record_slots = (size_t)cfg->max_requests + (size_t)cfg->max_requests / 4 + 40 * (size_t)c->n_tiles + 64;
    if (e == cudaSuccess) e = alloc_zero(&c->d_records, record_slots);
    c->fused_record_words = (unsigned int)(2 * record_slots < 0xfffffff0ull ? 2 * record_slots : 0xfffffff0ull);
    for (int k = 0; k < 2; ++k) {
        if (e == cudaSuccess) e = alloc_zero(&c->d_fused_totals[k], (size_t)c->n_tiles);
        if (e == cudaSuccess) e = alloc_zero(&c->d_fused_hint[k], (size_t)c->n_tiles + 1);
    }
    if (e == cudaSuccess) e = alloc_zero(&c->d_fused_base, (size_t)c->n_tiles + 1);
    if (e == cudaSuccess) e = alloc_zero(&c->d_fused_sync, 8);
    if (e == cudaSuccess) e = alloc_zero(&c->d_enter, (size_t)I);
    if (e == cudaSuccess) e = alloc_zero(&c->d_active, (size_t)I);
    if (e == cudaSuccess) e = alloc_zero(&c->d_scaler_partial, (size_t)16 * c->n_sm * 3);
    if (e == cudaSuccess) e = alloc_zero(&c->d_scaler_done, 1);
    if (e == cudaSuccess) e = alloc_zero(&c->d_ring_done, 1);
    if (e == cudaSuccess) e = alloc_zero(&c->d_queue_entry, 2);
    c->spin_limit = PRE_DEFAULT_SPIN_LIMIT;
    if (e == cudaSuccess) e = pre_anticipate_configure(c);
    if (e == cudaSuccess) e = pre_fused_configure(c);
    if (e == cudaSuccess) e = pre_route_configure(c);
    if (e == cudaSuccess) e = alloc_zero(&c->d_slots, (size_t)32 * c->route_blocks);
    if (e == cudaSuccess) e = pre_route_summary_configure(c);
    if (e == cudaSuccess) e = alloc_zero(&c->d_rs_guard, 8);
    if (e == cudaSuccess) e = alloc_zero(&c->d_rs_handled, 1);
    if (e == cudaSuccess && c->route_summary_smem) {
        e = alloc_zero(&c->d_rs_summary, (size_t)2 * I);
        if (e == cudaSuccess) e = alloc_zero(&c->d_rs_jtop, (size_t)I);
        if (e == cudaSuccess) e = alloc_zero(&c->d_rs_over, (size_t)I);
    }
    if (e != cudaSuccess) {
        const bool oom = (e == cudaErrorMemoryAllocation);
        cudaGetLastError();
        release(c);
        return oom ? PRE_ENOMEM : (e == cudaErrorInvalidConfiguration || e == cudaErrorInvalidValue ? PRE_EINVAL
                                                                                                     : PRE_ECUDA);
    }
    *out = c;
    return PRE_OK;
}

int pre_destroy(pre_ctx* ctx) {
    if (!ctx) return PRE_EINVAL;
    release(ctx);
    return PRE_OK;
}

int pre_anticipate(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated,
                   const int32_t* d_predicted, const int32_t* d_instance, int64_t n_requests,
                   int64_t* d_curves, int64_t* d_current_d, void* stream) {
    if (!ctx || !d_curves || !d_current_d) return PRE_EINVAL;
    if (n_requests < 0 || n_requests > ctx->cfg.max_requests) return PRE_EINVAL;
    if (n_requests > 0 && (!d_prompt || !d_generated || !d_predicted || !d_instance)) return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_current_d, 8)) return PRE_EINVAL;
    if (!aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_anticipate(ctx, d_prompt, d_generated, d_predicted, d_instance, n_requests,
                                          d_curves, d_current_d, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_route_batch(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted,
                    int64_t n_arrivals, int64_t* d_curves, int64_t* d_queued_p, int64_t* d_current_d,
                    int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                    int64_t* d_n_requests, int32_t* d_choice, double* d_score, void* stream) {
    if (!ctx || n_arrivals < 0 || n_arrivals >= (1LL << 31)) return PRE_EINVAL;
    if (!d_curves || !d_queued_p || !d_current_d || !d_prompt || !d_generated || !d_predicted || !d_instance ||
        !d_n_requests)
        return PRE_EINVAL;
    if (n_arrivals > 0 && (!d_arr_prompt || !d_arr_predicted || !d_choice)) return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_queued_p, 8) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) ||
        !aligned(d_score, 8) || !aligned(d_choice, 4) || !aligned(d_arr_prompt, 4) || !aligned(d_arr_predicted, 4) ||
        !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_route(ctx, d_arr_prompt, d_arr_predicted, n_arrivals, d_curves, d_queued_p,
                                     d_current_d, d_prompt, d_generated, d_predicted, d_instance, d_n_requests,
                                     d_choice, d_score, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_route_admit(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted, int64_t n_arrivals,
                    double overload_level, double overload_share, int32_t* d_queue_prompt,
                    int32_t* d_queue_predicted, int64_t* d_queue_state, int64_t queue_capacity,
                    int32_t* d_queue_choice, int64_t* d_curves, int64_t* d_queued_p, int64_t* d_current_d,
                    int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                    int64_t* d_n_requests, int32_t* d_choice, double* d_score, void* stream) {
    if (!ctx || n_arrivals < 0 || n_arrivals >= (1LL << 30)) return PRE_EINVAL;
    if (queue_capacity < 0 || queue_capacity >= (1LL << 30) || !d_queue_state) return PRE_EINVAL;
    if (queue_capacity > 0 && (!d_queue_prompt || !d_queue_predicted || !d_queue_choice)) return PRE_EINVAL;
    if (!std::isfinite(overload_level) || !std::isfinite(overload_share)) return PRE_EINVAL;
    if (!d_curves || !d_queued_p || !d_current_d || !d_prompt || !d_generated || !d_predicted || !d_instance ||
        !d_n_requests)
        return PRE_EINVAL;
    if (n_arrivals > 0 && (!d_arr_prompt || !d_arr_predicted || !d_choice)) return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_queued_p, 8) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) ||
        !aligned(d_score, 8) || !aligned(d_choice, 4) || !aligned(d_arr_prompt, 4) || !aligned(d_arr_predicted, 4) ||
        !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4) ||
        !aligned(d_queue_prompt, 4) || !aligned(d_queue_predicted, 4) || !aligned(d_queue_choice, 4) ||
        !aligned(d_queue_state, 8))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_route_admit(ctx, d_arr_prompt, d_arr_predicted, n_arrivals, overload_level,
                                           overload_share, d_queue_prompt, d_queue_predicted, d_queue_state,
                                           queue_capacity, d_queue_choice, d_curves, d_queued_p, d_current_d, d_prompt,
                                           d_generated, d_predicted, d_instance, d_n_requests, d_choice, d_score,
                                           static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_step(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
             const int64_t* d_n_requests, int64_t* d_curves, int64_t* d_queued_p, int64_t* d_current_d,
             void* stream) {
    if (!ctx || !d_prompt || !d_generated || !d_predicted || !d_instance || !d_n_requests || !d_curves ||
        !d_queued_p || !d_current_d)
        return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_queued_p, 8) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) ||
        !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_step(ctx, d_prompt, d_generated, d_predicted, d_instance, d_n_requests, d_curves,
                                    d_queued_p, d_current_d, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_tick(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
             const int32_t* d_actual, const int64_t* d_n_requests, int64_t* d_curves, int64_t* d_queued_p,
             int64_t* d_current_d, double overload_level, double overload_share, double idle_level,
             int32_t* d_over_count, int64_t* d_row_max, int64_t* d_summary, int64_t* d_counts, void* stream) {
    if (!ctx || !d_prompt || !d_generated || !d_predicted || !d_instance || !d_n_requests || !d_curves ||
        !d_queued_p || !d_current_d)
        return PRE_EINVAL;
    const int given = (d_over_count != nullptr) + (d_row_max != nullptr) + (d_summary != nullptr);
    if (given != 0 && given != 3) return PRE_EINVAL;
    if (given == 3 && (!std::isfinite(overload_level) || !std::isfinite(overload_share) || !std::isfinite(idle_level)))
        return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_queued_p, 8) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) ||
        !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4) ||
        !aligned(d_actual, 4) || !aligned(d_over_count, 4) || !aligned(d_row_max, 8) || !aligned(d_summary, 8) ||
        !aligned(d_counts, 8))
        return PRE_EINVAL;
    if (given == 0) { overload_level = 0.0; overload_share = 0.0; idle_level = 0.0; }
    cudaError_t e = pre_launch_tick(ctx, d_prompt, d_generated, d_predicted, d_instance, d_actual, d_n_requests, d_curves,
                                    d_queued_p, d_current_d, overload_level, overload_share, idle_level, d_over_count,
                                    d_row_max, d_summary, d_counts, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_refine(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated, int32_t* d_predicted,
               const int32_t* d_instance, const int32_t* d_actual, const int64_t* d_n_requests, int64_t* d_curves,
               int64_t* d_current_d, int64_t* d_counts, void* stream) {
    if (!ctx || !d_prompt || !d_generated || !d_predicted || !d_instance || !d_actual || !d_n_requests ||
        !d_curves || !d_current_d)
        return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) || !aligned(d_counts, 8) ||
        !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) || !aligned(d_instance, 4) ||
        !aligned(d_actual, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_refine(ctx, d_prompt, d_generated, d_predicted, d_instance, d_actual, d_n_requests,
                                      d_curves, ctx->cfg.horizon, nullptr, d_current_d, d_counts,
                                      static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_ring_refine(pre_ctx* ctx, const int32_t* d_prompt, const int32_t* d_generated, int32_t* d_predicted,
                    const int32_t* d_instance, const int32_t* d_actual, const int64_t* d_n_requests, int64_t* d_ring,
                    int32_t width, const int64_t* d_head, int64_t* d_current_d, int64_t* d_counts, void* stream) {
    if (!ctx || !d_prompt || !d_generated || !d_predicted || !d_instance || !d_actual || !d_n_requests || !d_ring ||
        !d_head || !d_current_d)
        return PRE_EINVAL;
    if (width < ctx->cfg.horizon || (long long)ctx->cfg.n_instances * width >= (1LL << 40)) return PRE_EINVAL;
    if (!aligned(d_ring, 8) || !aligned(d_head, 8) || !aligned(d_current_d, 8) || !aligned(d_n_requests, 8) ||
        !aligned(d_counts, 8) || !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) ||
        !aligned(d_instance, 4) || !aligned(d_actual, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_refine(ctx, d_prompt, d_generated, d_predicted, d_instance, d_actual, d_n_requests,
                                      d_ring, width, d_head, d_current_d, d_counts, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_scaler_signals(pre_ctx* ctx, const int64_t* d_curves, double overload_level, double overload_share,
                       double idle_level, int32_t* d_over_count, int64_t* d_row_max, int64_t* d_summary,
                       void* stream) {
    if (!ctx || !d_curves || !d_over_count || !d_row_max || !d_summary) return PRE_EINVAL;
    if (!aligned(d_curves, 16) || !aligned(d_over_count, 4) || !aligned(d_row_max, 8) || !aligned(d_summary, 8))
        return PRE_EINVAL;
    if (!std::isfinite(overload_level) || !std::isfinite(overload_share) || !std::isfinite(idle_level))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_scaler(ctx, d_curves, overload_level, overload_share, idle_level, d_over_count,
                                      d_row_max, d_summary, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_ring_window(pre_ctx* ctx, const int64_t* d_ring, int32_t width, const int64_t* d_head, int64_t* d_window,
                    void* stream) {
    if (!ctx || !d_ring || !d_head || !d_window) return PRE_EINVAL;
    if (width < ctx->cfg.horizon || (long long)ctx->cfg.n_instances * width >= (1LL << 40)) return PRE_EINVAL;
    if (!aligned(d_ring, 8) || !aligned(d_head, 8) || !aligned(d_window, 16)) return PRE_EINVAL;
    cudaError_t e = pre_launch_ring_window(ctx, d_ring, width, d_head, d_window, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_ring_fold(pre_ctx* ctx, const int32_t* d_arr_prompt, const int32_t* d_arr_predicted, const int32_t* d_choice,
                  int64_t n_arrivals, int64_t* d_ring, int32_t width, const int64_t* d_head, void* stream) {
    if (!ctx || !d_ring || !d_head || n_arrivals < 0 || n_arrivals >= (1LL << 31)) return PRE_EINVAL;
    if (width < ctx->cfg.horizon || (long long)ctx->cfg.n_instances * width >= (1LL << 40)) return PRE_EINVAL;
    if (n_arrivals > 0 && (!d_arr_prompt || !d_arr_predicted || !d_choice)) return PRE_EINVAL;
    if (!aligned(d_ring, 8) || !aligned(d_head, 8) || !aligned(d_arr_prompt, 4) || !aligned(d_arr_predicted, 4) ||
        !aligned(d_choice, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_ring_fold(ctx, d_arr_prompt, d_arr_predicted, d_choice, n_arrivals, d_ring, width,
                                         d_head, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_ring_step(pre_ctx* ctx, int32_t* d_prompt, int32_t* d_generated, int32_t* d_predicted, int32_t* d_instance,
                  const int64_t* d_n_requests, int64_t* d_ring, int32_t width, int64_t* d_head, int64_t* d_queued_p,
                  int64_t* d_current_d, void* stream) {
    if (!ctx || !d_prompt || !d_generated || !d_predicted || !d_instance || !d_n_requests || !d_ring || !d_head ||
        !d_queued_p || !d_current_d)
        return PRE_EINVAL;
    if (width < ctx->cfg.horizon || (long long)ctx->cfg.n_instances * width >= (1LL << 40)) return PRE_EINVAL;
    if (!aligned(d_ring, 8) || !aligned(d_head, 8) || !aligned(d_queued_p, 8) || !aligned(d_current_d, 8) ||
        !aligned(d_n_requests, 8) || !aligned(d_prompt, 4) || !aligned(d_generated, 4) || !aligned(d_predicted, 4) ||
        !aligned(d_instance, 4))
        return PRE_EINVAL;
    cudaError_t e = pre_launch_ring_step(ctx, d_prompt, d_generated, d_predicted, d_instance, d_n_requests, d_ring,
                                         width, d_head, d_queued_p, d_current_d, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? PRE_OK : fail_cuda(ctx, e);
}

int pre_status(pre_ctx* ctx, void* stream) {
    if (!ctx) return PRE_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(int), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    if (word & PRE_ST_TIMEOUT) {
        // a build that gave up leaves its counters half-way: start them afresh
        e = pre_fused_reset(ctx, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        return PRE_ETIMEOUT;
    }
    if (word & PRE_ST_CAPACITY) return PRE_ECAPACITY;
    if (word & PRE_ST_BADREQ) return PRE_EBADREQ;
    return PRE_OK;
}

int pre_last_cuda_error(const pre_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int pre_query_layout(const pre_ctx* ctx, int64_t out[4]) {
    if (!ctx || !out) return PRE_EINVAL;
    out[0] = (int64_t)ctx->route_resident_bytes;
    out[1] = ctx->route_threads;
    out[2] = ctx->fused_grid;
    out[3] = pre_fused_max_rows(ctx);
    return PRE_OK;
}

int pre_route_select(pre_ctx* ctx, int32_t path) {
    if (!ctx || path < PRE_ROUTE_AUTO || path > PRE_ROUTE_SUMMARY) return PRE_EINVAL;
    if (path == PRE_ROUTE_SUMMARY && !pre_route_summary_fits(ctx)) return PRE_ESIZE;
    ctx->route_path = path;
    return PRE_OK;
}

int pre_test_set_spin_limit(pre_ctx* ctx, uint32_t polls) {
    if (!ctx) return PRE_EINVAL;
    ctx->spin_limit = polls;
    return PRE_OK;
}

const char* pre_strerror(int code) {
    switch (code) {
        case PRE_OK: return "ok";
        case PRE_EINVAL: return "invalid argument (null or misaligned pointer, size out of range)";
        case PRE_ECAPACITY: return "request table full: some arrivals were not routed";
        case PRE_EBADREQ: return "malformed request or arrival skipped";
        case PRE_ETIMEOUT: return "a bounded device-side wait ran out; the call stopped early";
        case PRE_ECUDA: return "CUDA runtime error";
        case PRE_ENOMEM: return "out of memory";
        case PRE_ESIZE: return "problem larger than the built-in scratch of pre_anticipate_static";
        default: return "unknown error code";
    }
}

int pre_query(const pre_ctx* ctx, int32_t* route_blocks, int32_t* tile_rows) {
    if (!ctx) return PRE_EINVAL;
    if (route_blocks) *route_blocks = ctx->route_blocks;
    if (tile_rows) *tile_rows = ctx->tile_rows;
    return PRE_OK;
}

}  // extern "C"
