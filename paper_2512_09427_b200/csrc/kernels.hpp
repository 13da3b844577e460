// Device side of libodma: kernel parameter blocks and host launchers (kernels.cu).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace odma {

// Status word bits written by kernels.
constexpr uint32_t kStatusTimeout = 1u;

struct DecodeParams {
    // per-step tables (device)
    const int32_t* base;
    const int32_t* cap;
    const int32_t* len;
    const int4* cta;            // three int4 per CTA: {item_begin, item_end, 0, 0}, first item
    const int4* items;          // two int4 per item
    const int4* combine;        // one int4 per split stream: {request, head, first slot, pieces}
    uint32_t* counters;         // per split stream: pieces delivered so far (zero between launches);
                                // nullptr = the caller merges with launch_combine instead
    // tensors
    const void* q;              // [n, q_heads, head_dim]
    void* out;                  // [n, q_heads, head_dim]
    float* lse;                 // [n, q_heads] or nullptr
    float* part_o;              // [slots, group, head_dim] unnormalised partial outputs
    float* part_ml;             // [slots, group, 2] running max (log2 domain) and sum
    const void* pool;           // base of the slab pool (or of the paged copy)
    const void* k_new;          // append fused into the decode kernel: the step's new rows,
    const void* v_new;          // [n, kv_heads, head_dim], one token per request; nullptr = not fused
    int64_t rows_per_array;     // T * kv_heads   (paged: n_pages * kv_heads * 16)
    int32_t layer;
    int32_t q_heads, kv_heads, group, head_dim;
    float scale_log2;           // log2(e) / sqrt(head_dim)
    uint32_t* status;
    // page-16 ablation
    const int32_t* page_table;  // [n, max_pages]
    int32_t max_pages;
    int64_t wait_limit_ns;
    int32_t early_ok;           // the previous kernel of the stream that wrote this pool was a decode kernel (it
                                // appends one row per stream): rows up to two before a stream's end may be
                                // requested before the dependency wait; 0: nothing is read before it
    int32_t chained;            // tcgen05 kernel: the previous kernel of the stream is a decode launch of this
                                // pool on another layer (other K/V arrays, other outputs, the other
                                // scratch set): nothing of this launch waits for it
    int32_t kv_fp8;             // the pool holds E4M3 codes (one byte per element); q, the new rows and out are bf16
    float k_scale, v_scale;     // 8-bit pool: a stored code stands for value * scale (this layer's scales)
    float k_inv, v_inv;         // fp32 reciprocals: what an appended element is multiplied by before rounding
    // tcgen05 kernel: one launch for several layers of a step.  The CTA walks its items once per layer
    // (same plan, the pipeline never drains); layer li of the launch uses K/V arrays of layer + li and
    // the buffers below advanced by li strides.
    int32_t n_layers;           // 1 = the usual launch; more: see SpanParams
    int32_t stages;             // pipeline depth of the tensor-core kernel (2..8)
    int32_t q_slots;            // depth of its query / item-descriptor ring (4..8)
};

// What a launch over several layers needs beyond DecodeParams; a parameter of its own that a
// one-layer launch never reads (the parameter block is fetched line by line, on first use, by every
// CTA: what the usual launch touches stays small).
constexpr int kMaxSpanScales = 32;   // layers of one launch over an 8-bit pool
struct SpanParams {
    int64_t q_stride, new_stride, out_stride;      // bytes between consecutive layers of q / k_new, v_new / out
    int64_t lse_stride;                            // floats between consecutive layers of lse
    int64_t part_o_stride, part_ml_stride;         // floats between consecutive layers' partial results
    int32_t counter_stride;                        // counters between consecutive layers
    int32_t pad;
    float4 scales[kMaxSpanScales];                 // 8-bit pools: {k_scale, v_scale, k_inv, v_inv} of layer + li
};

// Lengths handed to the tensor-core kernel with its arguments instead of through the table in
// device memory (a step that reuses the previous step's plan then needs no copy at all).
constexpr int kInlineLens = 256;
struct InlineLens {
    int32_t n;                  // 0: take the lengths the plan was made with (items' n_tokens)
    int32_t len[kInlineLens];   // length after this step's append, per request of the batch
};

struct TensorMaps {
    CUtensorMap box[4];   // boxes of 16, 32, 48 and 64 rows x 128 bytes (box[k]: 16 (k+1) rows)
};

enum DecodeMode { kModeSlab = 0, kModePaged = 1, kModeProbe = 2 };

// Returns false when (head_dim, group) has no tensor-core instantiation.
bool tc_supported(int32_t head_dim, int32_t group);
// Pipeline stages and query-ring slots that fit into one SM's shared memory (one CTA per SM;
// both 0 when nothing fits).
void tc_shape(int32_t head_dim, int32_t group, int32_t* stages, int32_t* q_slots);
cudaError_t launch_decode_tc(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                             cudaStream_t stream, const InlineLens* lens = nullptr);
// The same decode step on the tcgen05 tensor cores (decode_umma.cu): slab and paged modes;
// `stages` and `q_slots` of the parameter block are ignored (the kernel sizes its own rings).
// An 8-bit (E4M3) pool: head_dim 128, group <= 8, slab mode.  `defer` (16-bit slabs, slab mode)
// picks the variant that reads an item's result out under the softmax of the lane's next item.
bool umma_supported(int32_t head_dim, int32_t group, bool kv_fp8);
cudaError_t launch_decode_umma(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                               cudaStream_t stream, const InlineLens* lens = nullptr, const SpanParams* span = nullptr,
                               bool defer = false);
cudaError_t launch_decode_generic(const DecodeParams& p, int dtype, int n_ctas, cudaStream_t stream);
bool generic_supported(int32_t head_dim);

cudaError_t launch_combine(const int4* combine, int n_combine, const float* part_o,
                           const float* part_ml, void* out, float* lse, int group, int head_dim,
                           int q_heads, int dtype, cudaStream_t stream);

struct AppendParams {
    const int32_t* base;
    const int32_t* cap;
    const int32_t* len;
    const int32_t* cu_new;
    void* pool;
    const void* k_new;
    const void* v_new;
    int64_t rows_per_array;
    int32_t layer, n, kv_heads, n_new_total;
    int32_t row_vecs;           // 16-byte vectors per row
    int32_t one_new_each;       // every request appends exactly one token: token index = request
    int32_t quantize;           // the pool holds E4M3 codes: the bf16 rows are multiplied by k_inv / v_inv in
    float k_inv, v_inv;         // fp32 and rounded to the nearest code (row_vecs counts the stored row)
};
cudaError_t launch_append(const AppendParams& p, cudaStream_t stream);

struct MigrateParams {
    void* pool;
    int64_t rows_per_array;
    int64_t src_base, src_cap, dst_base, dst_cap, len;
    int32_t arrays;             // layers * 2
    int32_t kv_heads, row_vecs;
};
cudaError_t launch_migrate(const MigrateParams& p, cudaStream_t stream);

struct ScatterPagesParams {
    const int32_t* base;
    const int32_t* cap;
    const int32_t* len;
    const int32_t* page_table;
    const void* pool;
    void* pages;
    int64_t rows_per_array;      // slab pool
    int64_t n_pages;
    int32_t n, max_pages, arrays, kv_heads, row_vecs;
};
cudaError_t launch_scatter_pages(const ScatterPagesParams& p, int64_t max_len, cudaStream_t stream);

// Limits of launch_decode_static: pieces (items) per batch, query heads per KV head, head_dim.
constexpr int kStaticSlots = 512;
constexpr int kStaticGroup = 8;
constexpr int kStaticHeadDim = 128;
// The generic decode kernel and the combine kernel with the split partials kept in a
// file-scope device array (no allocation).  The first call on a device looks the array's
// address up; calls that overlap on one GPU share the array and race.
cudaError_t launch_decode_static(DecodeParams p, int dtype, int n_ctas, const int4* combine,
                                 int n_combine, cudaStream_t stream);

// A one-thread kernel that waits on a barrier nobody signals, for at most limit_ns, then
// sets the timeout bit: exercises the bounded-wait path without hanging anything.
cudaError_t launch_wait_selftest(uint32_t* status, int64_t limit_ns, cudaStream_t stream);

}  // namespace odma
