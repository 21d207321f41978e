// Internal declarations shared by the kernels and the C-ABI layer.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "preserve_b200.h"

// Bits of the device status word (OR-ed by kernels, read by pre_status).
enum : int { PRE_ST_BADREQ = 1, PRE_ST_CAPACITY = 2, PRE_ST_TIMEOUT = 4 };

// Field limits that let one binned request fit in 64 bits:
//   [ row within tile : 8 | B = P + g : 28 | remaining = D - g : 28 ]
constexpr int PRE_FIELD_BITS = 28;
constexpr int32_t PRE_FIELD_MAX = (1 << PRE_FIELD_BITS) - 1;
constexpr int PRE_MAX_TILE_ROWS = 256;
constexpr int PRE_MAX_HORIZON = 8192;
// Largest number of build tiles (and, in the step kernel, instances) a block counts in shared memory.
constexpr int PRE_SMEM_BINS = 8192;

struct pre_ctx {
    pre_config cfg;
    int device;
    int n_sm;
    int tile_rows;       // T: instance rows per build tile
    int n_tiles;         // ceil(I / T)
    int max_chunks;      // width of the offset table: chunks the sorting pass may cut the table into
    int tile_grid;       // blocks of the persistent tile kernel
    int route_blocks;    // G: blocks of the persistent routing kernel
    int route_threads;
    size_t route_smem;
    size_t route_resident_bytes;  // shared memory per routing block left for resident rows
    size_t route_smem_admit;            // the same two for the kernel with the admission queue
    size_t route_resident_bytes_admit;
    double theta;        // t_mem * M in binary64
    int last_cuda_error;
    // device scratch
    int* d_status;            // status word
    int* d_abort;             // routing kernel gives up when set
    unsigned int* d_epoch;    // running exchange counter of the routing kernel (tags of the exchange slots)
    int64_t* d_queue_entry;   // {head, length} of the admission queue as they were when the call was made
    unsigned int* d_chunk_off;   // [max_chunks x n_tiles] {start : 16 | length : 16} of each tile inside each
                                 // sorted chunk, then [max_chunks] the largest B of each chunk
    unsigned long long* d_excess;   // [I] remaining tokens beyond the window, per instance (zero between calls)
    unsigned int* d_bin_count;   // slow path [n_tiles]   zero between calls
    unsigned int* d_bin_base;    // slow path [n_tiles+1]
    unsigned int* d_bin_cursor;  // slow path [n_tiles]   zero between calls
    unsigned long long* d_records;  // [max_requests]
    unsigned long long* d_slots;    // [2][G][16] routing exchange, one 128-byte line per block and parity
    unsigned long long* d_enter;    // [I] tokens entering the window at step H-1 (zero between calls)
    unsigned int* d_active;         // [I] live requests per instance (zero between calls)
    long long* d_scaler_partial;    // [16 * n_sm][3] block totals of the kernels that sum the scaler's signals
    unsigned int* d_scaler_done;    // blocks of that kernel that have finished (zero between calls)
    unsigned int* d_ring_done;      // the same for the kernel that advances a ring of maps
    // fused (single-launch) build: 0 blocks when this shape does not use it
    int fused_grid;
    size_t fused_smem;
    unsigned int fused_bar_base;    // value of the grid-barrier counter before the next launch
    unsigned int fused_launch_id;
    unsigned int spin_limit;        // polls before a bounded device-side wait gives up
    int fused_flip;                 // which of the two totals / hint arrays the next launch uses
    unsigned int fused_record_words;   // room in d_records, in 4-byte words
    unsigned int* d_fused_totals[2];   // [n_tiles] records per tile: one in use, the other zero for the next call
    unsigned int* d_fused_hint[2];     // [n_tiles + 1] where the lengths of one build put the next build's lists
    unsigned int* d_fused_base;     // [n_tiles + 1] where each tile's list starts when laid out exactly
    unsigned int* d_fused_sync;     // [8] barrier counter, largest B, id of an abandoned launch
    // routing on per-row summaries: 0 bytes of shared memory when this shape does not use it
    int route_path;                 // PRE_ROUTE_AUTO / _SCAN / _SUMMARY
    size_t route_summary_smem;
    size_t route_summary_smem_admit;    // the same for the kernel with the admission queue
    unsigned long long* d_rs_summary;   // [I] {token count, largest cell, largest cell + step, cell 0} per row (16 bytes)
    uint32_t* d_rs_jtop;            // [I] the first step of a row's largest cell + step
    int32_t* d_rs_over;             // [I] steps of a row above the overload level (admission queue)
    unsigned long long* d_rs_guard; // [8] what the summarising kernel found (largest cell, totals of the batch, ...)
    int* d_rs_handled;              // 1 when the summary kernel routed the last batch, 0 when it left it to the scanning kernel
};

// Launchers (defined next to their kernels).  Each returns a cudaError_t.
cudaError_t pre_launch_anticipate(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                  const int32_t* predicted, const int32_t* instance, int64_t n,
                                  int64_t* curves, int64_t* current_d, cudaStream_t s);
cudaError_t pre_launch_route(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                             int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                             int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                             int64_t* n_requests, int32_t* choice, double* score, cudaStream_t s);
cudaError_t pre_launch_route_admit(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                   int64_t n_arrivals, double overload_level, double overload_share,
                                   int32_t* queue_prompt, int32_t* queue_predicted, int64_t* queue_state,
                                   int64_t queue_capacity, int32_t* queue_choice, int64_t* curves,
                                   int64_t* queued_p, int64_t* current_d, int32_t* prompt, int32_t* generated,
                                   int32_t* predicted, int32_t* instance, int64_t* n_requests, int32_t* choice,
                                   double* score, cudaStream_t s);
cudaError_t pre_launch_step(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                            int32_t* instance, const int64_t* n_requests, int64_t* curves,
                            int64_t* queued_p, int64_t* current_d, cudaStream_t s);
cudaError_t pre_launch_refine(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated, int32_t* predicted,
                              const int32_t* instance, const int32_t* actual, const int64_t* n_requests,
                              int64_t* curves, int width, const int64_t* head, int64_t* current_d, int64_t* counts,
                              cudaStream_t s);
cudaError_t pre_launch_scaler(pre_ctx* ctx, const int64_t* curves, double overload_level, double overload_share,
                              double idle_level, int32_t* over_count, int64_t* row_max, int64_t* summary,
                              cudaStream_t s);
cudaError_t pre_launch_tick(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                            const int32_t* actual, const int64_t* n_requests, int64_t* curves, int64_t* queued_p,
                            int64_t* current_d, double overload_level, double overload_share, double idle_level,
                            int32_t* over_count, int64_t* row_max, int64_t* summary, int64_t* counts, cudaStream_t s);
cudaError_t pre_launch_step_requests(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                     int32_t* instance, const int64_t* n_requests, int width, cudaStream_t s);
cudaError_t pre_launch_ring_window(pre_ctx* ctx, const int64_t* ring, int width, const int64_t* head,
                                   int64_t* window, cudaStream_t s);
cudaError_t pre_launch_ring_fold(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                 const int32_t* choice, int64_t n_arrivals, int64_t* ring, int width,
                                 const int64_t* head, cudaStream_t s);
cudaError_t pre_launch_ring_step(pre_ctx* ctx, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                 int32_t* instance, const int64_t* n_requests, int64_t* ring, int width,
                                 int64_t* head, int64_t* queued_p, int64_t* current_d, cudaStream_t s);
cudaError_t pre_route_configure(pre_ctx* ctx);  // picks G and the shared-memory size
cudaError_t pre_route_summary_configure(pre_ctx* ctx);   // sets ctx->route_summary_smem (0: this shape keeps the scanning kernel)
bool pre_route_summary_fits(const pre_ctx* ctx);
bool pre_route_summary_admit_fits(const pre_ctx* ctx);
cudaError_t pre_launch_route_summary_admit(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                           int64_t n_arrivals, long long hot, double many, int32_t* queue_prompt,
                                           int32_t* queue_predicted, int64_t* queue_state, int64_t queue_capacity,
                                           int32_t* queue_choice, int64_t* curves, int64_t* queued_p,
                                           int64_t* current_d, int32_t* prompt, int32_t* generated, int32_t* predicted,
                                           int32_t* instance, int64_t* n_requests, int32_t* choice, double* score,
                                           cudaStream_t s);
cudaError_t pre_launch_route_summary(pre_ctx* ctx, const int32_t* arr_prompt, const int32_t* arr_predicted,
                                     int64_t n_arrivals, int64_t* curves, int64_t* queued_p, int64_t* current_d,
                                     int32_t* prompt, int32_t* generated, int32_t* predicted, int32_t* instance,
                                     int64_t* n_requests, int32_t* choice, double* score, cudaStream_t s);
size_t pre_tile_smem_bytes(int tile_rows, int horizon);
int pre_tile_rows_for(int n_instances, int horizon, int n_sm);
int pre_tile_threads(int tile_rows, int horizon);
int pre_sort_max_chunks(int64_t max_requests, int n_sm);
size_t pre_chunk_table_words(int n_tiles, int max_chunks);
cudaError_t pre_anticipate_configure(pre_ctx* ctx);
cudaError_t pre_fused_configure(pre_ctx* ctx);   // sets ctx->fused_grid (0: this shape keeps the two-kernel build)
bool pre_fused_fits(const pre_ctx* ctx, int64_t n);
int64_t pre_fused_max_rows(const pre_ctx* ctx);
cudaError_t pre_launch_anticipate_fused(pre_ctx* ctx, const int32_t* prompt, const int32_t* generated,
                                        const int32_t* predicted, const int32_t* instance, int64_t n,
                                        int64_t* curves, int64_t* current_d, cudaStream_t s);
cudaError_t pre_fused_reset(pre_ctx* ctx, cudaStream_t s);   // after a wait ran out
constexpr unsigned int PRE_DEFAULT_SPIN_LIMIT = 1u << 22;

__device__ __forceinline__ bool pre_request_ok(int32_t P, int32_t g, int32_t D, int32_t inst, int32_t I) {
    return P >= 0 && g >= 0 && D >= 1 && inst >= 0 && inst < I;
}
