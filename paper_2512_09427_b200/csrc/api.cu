// C ABI of libodma (include/odma.h): argument checks, host bookkeeping, kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "allocator.hpp"
#include "kernels.hpp"
#include "odma.h"
#include "planner.hpp"

using namespace odma;

namespace odma {
int32_t simulate(Allocator& alloc, const odma_sim_params& prm, const odma_sim_request* reqs, int32_t n,
                 odma_sim_result* out);      // simulator.cpp
}

namespace {

constexpr int kStagingSlots = 4;
constexpr int kPlanReuseTokens = 32;   // a plan is reused until the batch grew this much per request
constexpr int64_t kDefaultWaitLimitNs = 2000000000ll;   // 2 s: far above any kernel here

struct ProfRecord {
    int kernel;
    cudaEvent_t start, stop;
};

struct Staging {
    int32_t* host = nullptr;     // pinned
    cudaEvent_t done = nullptr;  // recorded after the copy that read `host`
    bool in_flight = false;
};

}  // namespace

struct odma_pool {
    Allocator alloc;
    void* dev_base = nullptr;
    uint64_t bytes = 0;
    int32_t layers = 0, kv_heads = 0, head_dim = 0, dtype = 0;
    int32_t elem_bytes = 0;     // of a stored K/V element
    int32_t io_bytes = 0;       // of an element of q, out and the rows given to an append
    int32_t io_dtype = 0;       // ODMA_DTYPE_F32 or ODMA_DTYPE_BF16
    std::vector<float> k_scale, v_scale;   // 8-bit pools: dequantisation scale per layer
    int64_t rows_per_array = 0;
    int32_t plan_ctas = 148;
    // The decode kernels start reading slab rows before their dependency wait, on the
    // assumption that the kernel ahead of them in the stream is a decode kernel (which writes
    // only the last row of each stream).  True after a decode launch, false after any other
    // launch of the library that writes the pool (append, migration copy).
    bool decode_was_last = false;
    // what the last decode launch was, for chaining the next one to it (decode_attention_impl)
    bool last_fused_tensor = false;
    void* last_stream = nullptr;
    uint32_t scratch_parity = 0;
    uint32_t* d_counters = nullptr;   // per split stream: pieces delivered (fused combine)
    // a second scratch set: consecutive layers of one step alternate between the two, so that a
    // layer's kernel need not wait for the previous layer's
    // the second scratch set: the upper halves of the allocations behind part_o, part_ml, d_counters
    // (one launch over several layers uses both halves as one region, a layer after the other)
    float* part_o2 = nullptr;
    float* part_ml2 = nullptr;
    uint32_t* d_counters2 = nullptr;
    size_t part_o_floats = 0, part_ml_floats = 0;      // of ONE set
    int32_t last_lo = -1, last_hi = -1;                // layers the last decode launch covered
    int64_t slots_max = 0;
    int64_t table_words_max = 0;
    bool has_maps = false;
    TensorMaps maps{};
    float* part_o = nullptr;
    float* part_ml = nullptr;
    uint32_t* d_status = nullptr;
    Staging staging[kStagingSlots];
    int staging_next = 0;
    // device staging of odma_decode_step_host
    void* d_q = nullptr;
    void* d_k_new = nullptr;
    void* d_v_new = nullptr;
    void* d_out = nullptr;
    int32_t* d_step_table = nullptr;
    // profiling
    bool profiling = false;
    std::vector<ProfRecord> prof;
    // reusable host vectors
    std::vector<int32_t> v_base, v_cap, v_len;
    // The last full plan of a decode step (one new token per request).  While the same
    // requests sit in the same slabs and have only grown a little, the next step reuses its
    // dealing of streams to CTAs and only rewrites the lengths: a stream's last piece takes the
    // growth.  A full plan is made again once the batch has grown by kPlanReuseTokens tokens per
    // request on average, and whenever the batch or a slab changes.
    struct PlanCache {
        bool valid = false;
        std::vector<uint64_t> reqs;
        std::vector<int32_t> base, cap, len0, table;
        std::vector<int32_t> end_word;   // table words holding n_tokens of pieces that end a stream ...
        std::vector<int32_t> end_req;    // ... their request (index in the batch) ...
        std::vector<int32_t> end_tok0;   // ... and first token
        odma_tables desc{};
        uint64_t gen = 0;                // counts full plans
    } plan_cache;
    uint64_t step_table_gen = 0;         // the full plan whose table sits in d_step_table (0: none)
};

struct odma_paged {
    odma_pool* pool = nullptr;
    void* d_pages = nullptr;
    int64_t n_pages = 0;
    TensorMaps maps{};
    bool has_maps = false;
    int32_t* pinned = nullptr;
    int64_t pinned_words = 0;
};

namespace {

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Four views of a [rows x head_dim] row array of 2-byte (bf16) or 1-byte (E4M3) elements: boxes of
// 16, 32, 48 and 64 rows by 128 bytes (the widest inner extent the 128-byte swizzle allows).
int32_t make_tensor_maps(void* base, int64_t rows, int32_t head_dim, int32_t elem_bytes, TensorMaps* out) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
        return ODMA_ERR_CUDA;
    auto encode = reinterpret_cast<EncodeTiledFn>(fn);
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(rows)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(head_dim) * elem_bytes};
    const cuuint32_t estride[2] = {1, 1};
    const CUtensorMapDataType type = elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    for (int k = 0; k < 4; ++k) {
        const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), static_cast<cuuint32_t>(16 * (k + 1))};
        if (encode(&out->box[k], type, 2, base, gdim, gstride, box, estride,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return ODMA_ERR_CUDA;
    }
    return ODMA_OK;
}

struct ProfScope {
    odma_pool* pool;
    cudaStream_t stream;
    cudaEvent_t stop = nullptr;
    ProfScope(odma_pool* p, int kernel, cudaStream_t s) : pool(p), stream(s) {
        if (!p->profiling) return;
        ProfRecord r{kernel, nullptr, nullptr};
        if (cudaEventCreate(&r.start) != cudaSuccess || cudaEventCreate(&r.stop) != cudaSuccess) return;
        cudaEventRecord(r.start, s);
        stop = r.stop;
        p->prof.push_back(r);
    }
    ~ProfScope() {
        if (stop) cudaEventRecord(stop, stream);
    }
};

void clear_profile(odma_pool* p) {
    for (auto& r : p->prof) {
        cudaEventDestroy(r.start);
        cudaEventDestroy(r.stop);
    }
    p->prof.clear();
}

void free_device_side(odma_pool* p) {
    clear_profile(p);
    cudaFree(p->part_o);
    cudaFree(p->part_ml);
    cudaFree(p->d_status);
    cudaFree(p->d_counters);
    cudaFree(p->d_q);
    cudaFree(p->d_k_new);
    cudaFree(p->d_v_new);
    cudaFree(p->d_out);
    cudaFree(p->d_step_table);
    for (auto& s : p->staging) {
        if (s.host) cudaFreeHost(s.host);
        if (s.done) cudaEventDestroy(s.done);
        s = Staging{};
    }
}

// Gather slab, capacity and post-append length of every request of the batch.
int32_t gather_batch(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n) {
    pool->v_base.resize(n);
    pool->v_cap.resize(n);
    pool->v_len.resize(n);
    for (int32_t i = 0; i < n; ++i) {
        const Request* r = pool->alloc.find(reqs[i]);
        if (!r) return ODMA_ERR_UNKNOWN_REQ;
        const int64_t add = n_new ? n_new[i] : 1;
        if (add < 0) return ODMA_ERR_INVALID;
        if (r->len + add > r->cap) return ODMA_ERR_OVERFLOW;
        if (r->len + add < 1) return ODMA_ERR_INVALID;
        pool->v_base[i] = static_cast<int32_t>(r->base);
        pool->v_cap[i] = static_cast<int32_t>(r->cap);
        pool->v_len[i] = static_cast<int32_t>(r->len + add);
    }
    return ODMA_OK;
}

// After gather_batch: may the cached plan of an earlier decode step serve this batch?  Same
// requests in the same slabs, grown only, and by no more than kPlanReuseTokens per request.
bool plan_reusable(const odma_pool* pool, const uint64_t* reqs, int32_t n, int64_t* kv_tokens) {
    const odma_pool::PlanCache& pc = pool->plan_cache;
    if (!pc.valid || static_cast<int32_t>(pc.reqs.size()) != n || !std::equal(reqs, reqs + n, pc.reqs.begin()) ||
        pool->v_base != pc.base || pool->v_cap != pc.cap)
        return false;
    int64_t growth = 0, total = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (pool->v_len[i] < pc.len0[i]) return false;
        growth += pool->v_len[i] - pc.len0[i];
        total += pool->v_len[i];
    }
    *kv_tokens = total;
    return growth <= static_cast<int64_t>(kPlanReuseTokens) * n;
}

int32_t plan_into(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                  int32_t* host_table, uint64_t table_bytes, odma_tables* out) {
    if (!pool || !reqs || !host_table || !out || n < 1) return ODMA_ERR_INVALID;
    if (n > pool->alloc.config().max_batch) return ODMA_ERR_INVALID;
    int32_t rc = gather_batch(pool, reqs, n_new, n);
    if (rc != ODMA_OK) return rc;
    PlanInput in;
    in.n = n;
    in.kv_heads = pool->kv_heads;
    in.n_ctas = pool->plan_ctas;
    in.base = pool->v_base.data();
    in.cap = pool->v_cap.data();
    in.len = pool->v_len.data();
    in.n_new = n_new;
    odma_pool::PlanCache& pc = pool->plan_cache;
    if (!n_new && static_cast<uint64_t>(pc.desc.words) * 4 <= table_bytes) {
        int64_t kv_tokens = 0;
        if (plan_reusable(pool, reqs, n, &kv_tokens)) {
            std::copy(pc.table.begin(), pc.table.begin() + pc.desc.words, host_table);
            std::copy(pool->v_len.begin(), pool->v_len.end(), host_table + pc.desc.off_len);
            for (size_t k = 0; k < pc.end_word.size(); ++k)
                host_table[pc.end_word[k]] = pool->v_len[pc.end_req[k]] - pc.end_tok0[k];
            *out = pc.desc;
            out->kv_tokens = kv_tokens;
            out->epoch = pool->alloc.epoch();
            return ODMA_OK;
        }
    }
    rc = plan_batch(in, host_table, static_cast<int64_t>(table_bytes / 4), out);
    if (rc != ODMA_OK) return rc;
    out->epoch = pool->alloc.epoch();
    pc.valid = false;
    if (!n_new) {
        pc.reqs.assign(reqs, reqs + n);
        pc.base = pool->v_base;
        pc.cap = pool->v_cap;
        pc.len0 = pool->v_len;
        pc.table.assign(host_table, host_table + out->words);
        pc.desc = *out;
        pc.end_word.clear();
        pc.end_req.clear();
        pc.end_tok0.clear();
        auto note = [&](int32_t word0) {             // word0: first word of an item (or of its copy)
            if (host_table[word0 + 4] & 2) {
                pc.end_word.push_back(word0 + 3);
                pc.end_req.push_back(host_table[word0]);
                pc.end_tok0.push_back(host_table[word0 + 2]);
            }
        };
        for (int32_t k = 0; k < out->n_items; ++k) note(out->off_items + 8 * k);
        for (int32_t c = 0; c < out->n_ctas; ++c) {  // the first item's copy in each CTA record
            const int32_t* rec = host_table + out->off_cta + 12 * c;
            if (rec[0] < rec[1]) note(out->off_cta + 12 * c + 4);
        }
        pc.valid = true;
        pc.gen += 1;
    }
    return ODMA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The device-side address of a page-locked (pinned or registered) host buffer, NULL for
// anything else (pageable host memory, device memory, managed memory).
const void* device_alias(const void* host) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

int32_t check_tables(const odma_pool* pool, const odma_tables* t) {
    if (!t || !t->d_table || t->n < 1 || t->n_items < 1 || t->n_ctas < 1) return ODMA_ERR_INVALID;
    if (t->n_items > pool->slots_max) return ODMA_ERR_INVALID;
    return ODMA_OK;
}

void fill_decode_params(const odma_pool* pool, int32_t layer, const void* q, int32_t q_heads,
                        const odma_tables* t, void* out, float* lse, DecodeParams* p) {
    const int32_t* tab = static_cast<const int32_t*>(t->d_table);
    p->base = tab + t->off_base;
    p->cap = tab + t->off_cap;
    p->len = tab + t->off_len;
    p->cta = reinterpret_cast<const int4*>(tab + t->off_cta);
    p->items = reinterpret_cast<const int4*>(tab + t->off_items);
    p->combine = reinterpret_cast<const int4*>(tab + t->off_combine);
    p->counters = pool->alloc.config().fused_combine ? pool->d_counters : nullptr;
    p->q = q;
    p->out = out;
    p->lse = lse;
    p->part_o = pool->part_o;
    p->part_ml = pool->part_ml;
    p->pool = pool->dev_base;
    p->rows_per_array = pool->rows_per_array;
    p->layer = layer;
    p->q_heads = q_heads;
    p->kv_heads = pool->kv_heads;
    p->group = q_heads / pool->kv_heads;
    tc_shape(pool->head_dim, p->group, &p->stages, &p->q_slots);
    p->head_dim = pool->head_dim;
    p->scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(pool->head_dim)));
    p->status = pool->d_status;
    p->k_new = nullptr;
    p->v_new = nullptr;
    p->page_table = nullptr;
    p->max_pages = 0;
    p->wait_limit_ns = kDefaultWaitLimitNs;
    p->chained = 0;
    p->early_ok = 0;
    p->n_layers = 1;
    p->kv_fp8 = pool->dtype == ODMA_DTYPE_FP8_E4M3 ? 1 : 0;
    p->k_scale = p->v_scale = p->k_inv = p->v_inv = 1.f;
    if (p->kv_fp8) {
        p->k_scale = pool->k_scale[layer];
        p->v_scale = pool->v_scale[layer];
        p->k_inv = 1.0f / p->k_scale;
        p->v_inv = 1.0f / p->v_scale;
    }
}

int32_t check_decode_args(const odma_pool* pool, int32_t layer, const void* q, int32_t q_heads,
                          const odma_tables* t, const void* out) {
    if (!pool || !pool->dev_base) return ODMA_ERR_INVALID;
    if (layer < 0 || layer >= pool->layers || !q || !out || !aligned16(q) || !aligned16(out))
        return ODMA_ERR_INVALID;
    if (q_heads < pool->kv_heads || q_heads % pool->kv_heads != 0) return ODMA_ERR_INVALID;
    if (q_heads / pool->kv_heads > pool->alloc.config().max_group) return ODMA_ERR_INVALID;
    if (pool->dtype == ODMA_DTYPE_FP8_E4M3 && !umma_supported(pool->head_dim, q_heads / pool->kv_heads, true))
        return ODMA_ERR_INVALID;
    return check_tables(pool, t);
}

}  // namespace

extern "C" {

void odma_config_default(odma_config* cfg) {
    if (!cfg) return;
    std::memset(cfg, 0, sizeof *cfg);
    cfg->safety_pct = 10;
    cfg->max_len = 32768;
    cfg->granule = 16;
    cfg->window = 10000;
    cfg->refresh = 1000;
    cfg->n_levels = 4;
    for (int i = 0; i < 4; ++i) cfg->p_num[i] = i + 1;
    cfg->p_den = 4;
    cfg->gamma_permille = 200;
    cfg->tau_permille = 800;
    cfg->growth = 2;
    cfg->large_fixed = 0;
    cfg->max_batch = 1024;
    cfg->max_group = 8;
    cfg->plan_ctas = 0;
    cfg->fused_combine = 1;
    cfg->fused_append = 1;
    cfg->decode_kernel = ODMA_DECODE_AUTO;
    cfg->chain_launches = 1;
    cfg->span_layers = 1;
    cfg->async_recal = 0;
    cfg->cluster_observe = 0;
    cfg->readout = ODMA_READOUT_AUTO;
}

const char* odma_strerror(int32_t code) {
    switch (code) {
        case ODMA_OK: return "ok";
        case ODMA_ERR_INVALID: return "invalid argument";
        case ODMA_ERR_NOMEM: return "no free run of the needed size";
        case ODMA_ERR_UNKNOWN_REQ: return "unknown request";
        case ODMA_ERR_DUP_REQ: return "request already live";
        case ODMA_ERR_OVERFLOW: return "length beyond capacity";
        case ODMA_ERR_CUDA: return "CUDA call failed";
        case ODMA_ERR_TIMEOUT: return "device-side wait timed out";
        case ODMA_ERR_TOO_LARGE: return "batch beyond the fixed scratch array of odma_decode_attention_static";
    }
    return "unknown status";
}

int32_t odma_pool_create(void* dev_base, uint64_t bytes, int32_t layers, int32_t kv_heads,
                         int32_t head_dim, int32_t dtype, const odma_config* cfg_in, odma_pool** out) {
    if (!out) return ODMA_ERR_INVALID;
    *out = nullptr;
    if (dtype != ODMA_DTYPE_F32 && dtype != ODMA_DTYPE_BF16 && dtype != ODMA_DTYPE_FP8_E4M3) return ODMA_ERR_INVALID;
    odma_config cfg;
    if (cfg_in) cfg = *cfg_in; else odma_config_default(&cfg);
    const int32_t esz = dtype == ODMA_DTYPE_F32 ? 4 : dtype == ODMA_DTYPE_BF16 ? 2 : 1;
    const int32_t iosz = dtype == ODMA_DTYPE_F32 ? 4 : 2;
    if (layers < 1 || kv_heads < 1 || head_dim < 1 || (static_cast<int64_t>(head_dim) * esz) % 16 != 0)
        return ODMA_ERR_INVALID;
    if (cfg.max_batch < 1 || cfg.max_group < 1 || cfg.plan_ctas < 0) return ODMA_ERR_INVALID;
    if (cfg.decode_kernel < ODMA_DECODE_AUTO || cfg.decode_kernel > ODMA_DECODE_MMA_SYNC) return ODMA_ERR_INVALID;
    if (dev_base && (reinterpret_cast<uintptr_t>(dev_base) & 255u) != 0) return ODMA_ERR_INVALID;
    // an 8-bit pool is served by the tcgen05 kernel alone
    if (dtype == ODMA_DTYPE_FP8_E4M3 &&
        (!umma_supported(head_dim, 1, true) || cfg.decode_kernel == ODMA_DECODE_MMA_SYNC || cfg.max_group > 8))
        return ODMA_ERR_INVALID;

    odma_pool* p = new (std::nothrow) odma_pool();
    if (!p) return ODMA_ERR_NOMEM;
    int32_t rc = p->alloc.init(bytes, layers, kv_heads, head_dim, esz, cfg);
    if (rc != ODMA_OK) {
        delete p;
        return rc;
    }
    p->dev_base = dev_base;
    p->bytes = bytes;
    p->layers = layers;
    p->kv_heads = kv_heads;
    p->head_dim = head_dim;
    p->dtype = dtype;
    p->elem_bytes = esz;
    p->io_bytes = iosz;
    p->io_dtype = dtype == ODMA_DTYPE_F32 ? ODMA_DTYPE_F32 : ODMA_DTYPE_BF16;
    p->k_scale.assign(layers, 1.f);
    p->v_scale.assign(layers, 1.f);
    p->rows_per_array = p->alloc.T() * kv_heads;
    if (p->rows_per_array * layers * 2 >= (int64_t(1) << 31)) {
        delete p;
        return ODMA_ERR_INVALID;
    }
    p->plan_ctas = cfg.plan_ctas > 0 ? cfg.plan_ctas : 148;
    if (dev_base) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            delete p;
            return ODMA_ERR_CUDA;
        }
        if (cfg.plan_ctas == 0) p->plan_ctas = sms;
    }
    p->slots_max = static_cast<int64_t>(cfg.max_batch) * kv_heads + p->plan_ctas;
    p->table_words_max = plan_table_words(cfg.max_batch, kv_heads, p->plan_ctas);
    if (dev_base) {
        const size_t po = static_cast<size_t>(p->slots_max) * cfg.max_group * head_dim * 4;
        const size_t pm = static_cast<size_t>(p->slots_max) * cfg.max_group * 2 * 4;
        const size_t qb = static_cast<size_t>(cfg.max_batch) * kv_heads * cfg.max_group * head_dim * iosz;
        const size_t kb = static_cast<size_t>(cfg.max_batch) * kv_heads * head_dim * iosz;
        bool ok = cudaMalloc(&p->part_o, 2 * po) == cudaSuccess && cudaMalloc(&p->part_ml, 2 * pm) == cudaSuccess &&
                  cudaMalloc(&p->d_status, 4) == cudaSuccess && cudaMalloc(&p->d_q, qb) == cudaSuccess &&
                  cudaMalloc(&p->d_counters, static_cast<size_t>(p->slots_max) * 8) == cudaSuccess &&
                  cudaMemset(p->d_counters, 0, static_cast<size_t>(p->slots_max) * 8) == cudaSuccess &&
                  cudaMalloc(&p->d_out, qb) == cudaSuccess && cudaMalloc(&p->d_k_new, kb) == cudaSuccess &&
                  cudaMalloc(&p->d_v_new, kb) == cudaSuccess &&
                  cudaMalloc(&p->d_step_table, static_cast<size_t>(p->table_words_max) * 4) == cudaSuccess &&
                  cudaMemset(p->d_status, 0, 4) == cudaSuccess;
        if (ok) {
            p->part_o_floats = po / 4;
            p->part_ml_floats = pm / 4;
            p->part_o2 = p->part_o + p->part_o_floats;
            p->part_ml2 = p->part_ml + p->part_ml_floats;
            p->d_counters2 = p->d_counters + p->slots_max;
        }
        for (auto& s : p->staging) {
            ok = ok && cudaMallocHost(&s.host, static_cast<size_t>(p->table_words_max) * 4) == cudaSuccess &&
                 cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming) == cudaSuccess;
        }
        if (ok && ((dtype == ODMA_DTYPE_BF16 && tc_supported(head_dim, 1)) || dtype == ODMA_DTYPE_FP8_E4M3)) {
            ok = make_tensor_maps(dev_base, p->rows_per_array * layers * 2, head_dim, esz, &p->maps) == ODMA_OK;
            p->has_maps = ok;
        }
        if (!ok) {
            free_device_side(p);
            delete p;
            return ODMA_ERR_CUDA;
        }
    }
    *out = p;
    return ODMA_OK;
}

int32_t odma_pool_destroy(odma_pool* pool) {
    if (!pool) return ODMA_ERR_INVALID;
    if (pool->dev_base) free_device_side(pool);
    delete pool;
    return ODMA_OK;
}

int32_t odma_recal_flush(odma_pool* pool) {
    if (!pool) return ODMA_ERR_INVALID;
    pool->alloc.flush();
    return ODMA_OK;
}

int32_t odma_drain_observations(odma_pool* pool, int32_t* out, int32_t cap, int32_t* n) {
    return pool ? pool->alloc.drain(out, cap, n) : ODMA_ERR_INVALID;
}

int32_t odma_observe(odma_pool* pool, const int32_t* lengths, int32_t n) {
    return pool ? pool->alloc.observe(lengths, n) : ODMA_ERR_INVALID;
}

int32_t odma_set_kv_scales(odma_pool* pool, const float* k_scale, const float* v_scale) {
    if (!pool || !k_scale || !v_scale || pool->dtype != ODMA_DTYPE_FP8_E4M3) return ODMA_ERR_INVALID;
    for (int32_t l = 0; l < pool->layers; ++l)
        if (!(k_scale[l] > 0.f) || !(v_scale[l] > 0.f) || !std::isfinite(k_scale[l]) || !std::isfinite(v_scale[l]))
            return ODMA_ERR_INVALID;
    pool->k_scale.assign(k_scale, k_scale + pool->layers);
    pool->v_scale.assign(v_scale, v_scale + pool->layers);
    return ODMA_OK;
}

int32_t odma_set_buckets(odma_pool* pool, const int32_t* boundaries, int32_t n) {
    return pool ? pool->alloc.set_buckets(boundaries, n) : ODMA_ERR_INVALID;
}

int32_t odma_get_buckets(const odma_pool* pool, int32_t* boundaries, int32_t* n, uint64_t* epoch) {
    return pool ? pool->alloc.get_buckets(boundaries, n, epoch) : ODMA_ERR_INVALID;
}

int32_t odma_alloc(odma_pool* pool, uint64_t req, int32_t predicted_len, odma_slab* out) {
    return pool ? pool->alloc.reserve(req, predicted_len, out) : ODMA_ERR_INVALID;
}

int32_t odma_alloc_uncertain(odma_pool* pool, uint64_t req, int32_t l_hat, int32_t u_permille,
                             odma_slab* out) {
    return pool ? pool->alloc.reserve_uncertain(req, l_hat, u_permille, out) : ODMA_ERR_INVALID;
}

int32_t odma_ensure_capacity(odma_pool* pool, uint64_t req, int32_t needed_len, void* stream,
                             odma_slab* out, int32_t* migrated) {
    if (!pool) return ODMA_ERR_INVALID;
    Migration mig{};
    int32_t did = 0;
    int32_t rc = pool->alloc.ensure(req, needed_len, out, &did, &mig);
    if (migrated) *migrated = did;
    if (rc != ODMA_OK || !did || !pool->dev_base || mig.len == 0) return rc;
    MigrateParams mp;
    mp.pool = pool->dev_base;
    mp.rows_per_array = pool->rows_per_array;
    mp.src_base = mig.src_base;
    mp.src_cap = mig.src_cap;
    mp.dst_base = mig.dst_base;
    mp.dst_cap = mig.dst_cap;
    mp.len = mig.len;
    mp.arrays = pool->layers * 2;
    mp.kv_heads = pool->kv_heads;
    mp.row_vecs = pool->head_dim * pool->elem_bytes / 16;
    pool->decode_was_last = false;
    pool->last_fused_tensor = false;
    ProfScope ps(pool, ODMA_K_MIGRATE, as_stream(stream));
    return launch_migrate(mp, as_stream(stream)) == cudaSuccess ? ODMA_OK : ODMA_ERR_CUDA;
}

int32_t odma_free(odma_pool* pool, uint64_t req) {
    return pool ? pool->alloc.release(req) : ODMA_ERR_INVALID;
}

int32_t odma_commit_step(odma_pool* pool, const uint64_t* reqs, int32_t n, const int32_t* n_new) {
    return pool ? pool->alloc.commit(reqs, n, n_new) : ODMA_ERR_INVALID;
}

int32_t odma_get_slab(const odma_pool* pool, uint64_t req, odma_slab* out, int32_t* len) {
    if (!pool) return ODMA_ERR_INVALID;
    const Request* r = pool->alloc.find(req);
    if (!r) return ODMA_ERR_UNKNOWN_REQ;
    if (out) {
        out->base_tok = static_cast<int32_t>(r->base);
        out->cap_tok = static_cast<int32_t>(r->cap);
        out->pool_id = r->pool;
        out->bucket_id = r->bucket;
        out->epoch = pool->alloc.epoch();
    }
    if (len) *len = static_cast<int32_t>(r->len);
    return ODMA_OK;
}

int32_t odma_get_stats(const odma_pool* pool, odma_stats* out) {
    if (!pool || !out) return ODMA_ERR_INVALID;
    pool->alloc.stats(out);
    return ODMA_OK;
}

uint64_t odma_tables_bytes(const odma_pool* pool, int32_t n) {
    if (!pool || n < 1) return 0;
    return static_cast<uint64_t>(plan_table_words(n, pool->kv_heads, pool->plan_ctas)) * 4u;
}

int32_t odma_plan_host(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                       int32_t* host_table, uint64_t table_bytes, odma_tables* out) {
    return plan_into(pool, reqs, n_new, n, host_table, table_bytes, out);
}

int32_t odma_build_tables(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                          void* d_table, uint64_t table_bytes, void* stream, odma_tables* out) {
    if (!pool || !pool->dev_base || !d_table || !aligned16(d_table)) return ODMA_ERR_INVALID;
    if (n < 1 || table_bytes < odma_tables_bytes(pool, n)) return ODMA_ERR_INVALID;
    Staging& st = pool->staging[pool->staging_next];
    pool->staging_next = (pool->staging_next + 1) % kStagingSlots;
    if (st.in_flight && cudaEventSynchronize(st.done) != cudaSuccess) return ODMA_ERR_CUDA;
    st.in_flight = false;
    int32_t rc = plan_into(pool, reqs, n_new, n, st.host, static_cast<uint64_t>(pool->table_words_max) * 4, out);
    if (rc != ODMA_OK) return rc;
    if (cudaMemcpyAsync(d_table, st.host, static_cast<size_t>(out->words) * 4, cudaMemcpyHostToDevice,
                        as_stream(stream)) != cudaSuccess ||
        cudaEventRecord(st.done, as_stream(stream)) != cudaSuccess)
        return ODMA_ERR_CUDA;
    st.in_flight = true;
    out->d_table = d_table;
    return ODMA_OK;
}

int32_t odma_build_prefill_tables(odma_pool* pool, const uint64_t* reqs, const int32_t* n_new, int32_t n,
                                  void* d_table, uint64_t table_bytes, void* stream, odma_tables* out) {
    if (!pool || !pool->dev_base || !d_table || !aligned16(d_table) || !reqs || !n_new || !out || n < 1)
        return ODMA_ERR_INVALID;
    // one stream per new token: the owner's slab, read up to and including the token itself
    int64_t total = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (n_new[i] < 1) return ODMA_ERR_INVALID;
        total += n_new[i];
    }
    if (total > pool->alloc.config().max_batch || table_bytes < odma_tables_bytes(pool, static_cast<int32_t>(total)))
        return ODMA_ERR_INVALID;
    pool->v_base.clear();
    pool->v_cap.clear();
    pool->v_len.clear();
    for (int32_t i = 0; i < n; ++i) {
        const Request* r = pool->alloc.find(reqs[i]);
        if (!r) return ODMA_ERR_UNKNOWN_REQ;
        if (r->len + n_new[i] > r->cap) return ODMA_ERR_OVERFLOW;
        for (int32_t j = 0; j < n_new[i]; ++j) {
            pool->v_base.push_back(static_cast<int32_t>(r->base));
            pool->v_cap.push_back(static_cast<int32_t>(r->cap));
            pool->v_len.push_back(static_cast<int32_t>(r->len + j + 1));
        }
    }
    Staging& st = pool->staging[pool->staging_next];
    pool->staging_next = (pool->staging_next + 1) % kStagingSlots;
    if (st.in_flight && cudaEventSynchronize(st.done) != cudaSuccess) return ODMA_ERR_CUDA;
    st.in_flight = false;
    PlanInput in;
    in.n = static_cast<int32_t>(total);
    in.kv_heads = pool->kv_heads;
    in.n_ctas = pool->plan_ctas;
    in.base = pool->v_base.data();
    in.cap = pool->v_cap.data();
    in.len = pool->v_len.data();
    in.n_new = nullptr;
    pool->plan_cache.valid = false;                  // the scratch vectors no longer describe the cached batch
    int32_t rc = plan_batch(in, st.host, pool->table_words_max, out);
    if (rc != ODMA_OK) return rc;
    out->epoch = pool->alloc.epoch();
    out->n_new_total = 0;                            // nothing to append through this descriptor
    out->one_new_each = 0;
    if (cudaMemcpyAsync(d_table, st.host, static_cast<size_t>(out->words) * 4, cudaMemcpyHostToDevice,
                        as_stream(stream)) != cudaSuccess ||
        cudaEventRecord(st.done, as_stream(stream)) != cudaSuccess)
        return ODMA_ERR_CUDA;
    st.in_flight = true;
    out->d_table = d_table;
    return ODMA_OK;
}

int32_t odma_append_kv(odma_pool* pool, int32_t layer, const odma_tables* tables, const void* k_new,
                       const void* v_new, void* stream) {
    if (!pool || !pool->dev_base || layer < 0 || layer >= pool->layers) return ODMA_ERR_INVALID;
    if (!tables || !tables->d_table || tables->n < 1) return ODMA_ERR_INVALID;
    if (tables->n_new_total == 0) return ODMA_OK;
    if (!k_new || !v_new || !aligned16(k_new) || !aligned16(v_new)) return ODMA_ERR_INVALID;
    const int32_t* tab = static_cast<const int32_t*>(tables->d_table);
    AppendParams ap;
    ap.base = tab + tables->off_base;
    ap.cap = tab + tables->off_cap;
    ap.len = tab + tables->off_len;
    ap.cu_new = tab + tables->off_cu_new;
    ap.pool = pool->dev_base;
    ap.k_new = k_new;
    ap.v_new = v_new;
    ap.rows_per_array = pool->rows_per_array;
    ap.layer = layer;
    ap.n = tables->n;
    ap.kv_heads = pool->kv_heads;
    ap.n_new_total = tables->n_new_total;
    ap.row_vecs = pool->head_dim * pool->elem_bytes / 16;
    ap.one_new_each = tables->one_new_each;
    ap.quantize = pool->dtype == ODMA_DTYPE_FP8_E4M3 ? 1 : 0;
    ap.k_inv = ap.quantize ? 1.0f / pool->k_scale[layer] : 1.f;
    ap.v_inv = ap.quantize ? 1.0f / pool->v_scale[layer] : 1.f;
    pool->decode_was_last = false;
    pool->last_fused_tensor = false;
    ProfScope ps(pool, ODMA_K_APPEND, as_stream(stream));
    return launch_append(ap, as_stream(stream)) == cudaSuccess ? ODMA_OK : ODMA_ERR_CUDA;
}

}  // extern "C"

namespace {

// True when the bf16 tensor-core kernel serves this pool and group size (the kernel that can
// take the step's append along).
bool uses_tc(const odma_pool* pool, int32_t q_heads) {
    return pool->has_maps && tc_supported(pool->head_dim, q_heads / pool->kv_heads);
}

// Which of the two tensor-core kernels runs a launch.  ODMA_DECODE_AUTO: the tcgen05 kernel for a
// launch that can chain to the decode launch before it (the layers of a step over several layers,
// consecutive steps on different layers: it then runs without a dependency wait, measured 3 to 13 %
// faster), the mma.sync kernel for launches that have to wait (3 to 4 % faster there: its last
// tile and hand-over are a shorter chain).  8-bit pools: the tcgen05 kernel always.
bool uses_umma(const odma_pool* pool, int32_t group, bool chains) {
    const int32_t want = pool->alloc.config().decode_kernel;
    if (pool->dtype == ODMA_DTYPE_FP8_E4M3) return true;
    if (want == ODMA_DECODE_MMA_SYNC || !umma_supported(pool->head_dim, group, false)) return false;
    return want == ODMA_DECODE_TCGEN05 || chains;
}

// The tcgen05 kernel has a variant that reads an item's result out of tensor memory one step late,
// under the softmax of the lane's next item.  It pays where a CTA works through many short items
// per launch (measured on 1,024 streams of one or two tiles, all layers in one launch: 12.2 -> 11.2
// us per layer) and costs on longer ones (512 streams of ~300 tokens: 15.9 -> 16.4 us; 276 pieces
// of ~500 tokens: 14.0 -> 15.3 us), so a launch picks by the plan's counts unless the
// configuration says which.
constexpr int64_t kLateItemsPerCta = 3;      // items a CTA walks in the launch, at least
constexpr int64_t kLateTokensPerItem = 128;  // tokens per item on average, at most

cudaError_t launch_tensor_decode(const odma_pool* pool, const TensorMaps& maps, const DecodeParams& p, int mode,
                                 const odma_tables* t, cudaStream_t stream, const InlineLens* lens, bool umma,
                                 const SpanParams* span = nullptr) {
    const int n_ctas = t->n_ctas;
    const int32_t want = pool->alloc.config().readout;
    bool defer = want == ODMA_READOUT_LATE;
    if (want == ODMA_READOUT_AUTO)
        defer = static_cast<int64_t>(p.n_layers) * t->n_items >= kLateItemsPerCta * n_ctas &&
                t->kv_tokens * pool->kv_heads <= kLateTokensPerItem * t->n_items;
    defer = defer && mode == kModeSlab && !p.kv_fp8;
    return umma ? launch_decode_umma(maps, p, mode, n_ctas, stream, lens, span, defer)
                : launch_decode_tc(maps, p, mode, n_ctas, stream, lens);
}

// odma_decode_attention; with k_new / v_new the tensor-core kernel also appends the step's
// token (one per request) instead of finding it in the slab.
int32_t decode_attention_impl(odma_pool* pool, int32_t layer, const void* q, int32_t q_heads,
                              const odma_tables* tables, void* out, float* lse, void* stream,
                              const void* k_new, const void* v_new, const InlineLens* lens = nullptr,
                              int32_t chain_pos = -1, int32_t span = 1) {
    int32_t rc = check_decode_args(pool, layer, q, q_heads, tables, out);
    if (rc != ODMA_OK) return rc;
    DecodeParams p;
    fill_decode_params(pool, layer, q, q_heads, tables, out, lse, &p);
    if (k_new) {
        if (!uses_tc(pool, q_heads) || !tables->one_new_each || !v_new) return ODMA_ERR_INVALID;
        p.k_new = k_new;
        p.v_new = v_new;
    }
    cudaError_t e;
    bool fused = false;
    p.early_ok = pool->decode_was_last ? 1 : 0;
    pool->decode_was_last = true;
    {
        ProfScope ps(pool, ODMA_K_DECODE, as_stream(stream));
        if (pool->has_maps && tc_supported(pool->head_dim, p.group)) {
            if (p.stages < 2) return ODMA_ERR_INVALID;
            fused = p.counters != nullptr;
            // A launch whose predecessor on the stream is a fused decode launch of this pool on ANOTHER
            // layer has nothing to wait for: other K/V arrays, other outputs, inputs that were complete
            // when it was issued (they are not the predecessor's outputs: see the header), and the
            // other scratch set.  The layers of a step over several layers chain that way, and so do
            // consecutive steps on different layers.  Only the tcgen05 kernel runs without its
            // dependency wait.  (Anything else enqueued in between - a table copy, the caller's own
            // kernels - makes the launch wait for that operation to complete before it starts.)
            static thread_local SpanParams sp;          // filled for a launch over several layers only
            const bool disjoint = layer + span <= pool->last_lo || layer >= pool->last_hi;
            const bool can_chain = span == 1 && pool->alloc.config().chain_launches && fused && k_new != nullptr &&
                                   p.early_ok && pool->last_fused_tensor && pool->last_stream == stream && disjoint;
            const bool umma = uses_umma(pool, p.group, chain_pos >= 0 || can_chain || span > 1);
            if (span > 1) {
                // One launch for `span` layers of a step (the caller has checked that the tcgen05 kernel
                // serves it and that the scratch of all layers fits): the CTAs walk layer after layer over
                // the same plan; CTAs drift apart by whole layers, so every layer has its own partial
                // results and counters, laid one after the other across both scratch halves.  It waits for
                // the launch before it (the previous step touched the same layers) and nothing chains to it.
                const size_t n = static_cast<size_t>(tables->n);
                p.n_layers = span;
                sp.q_stride = sp.out_stride = static_cast<int64_t>(n * q_heads * pool->head_dim * pool->io_bytes);
                sp.new_stride = static_cast<int64_t>(n * pool->kv_heads * pool->head_dim * pool->io_bytes);
                sp.lse_stride = static_cast<int64_t>(n * q_heads);
                sp.part_o_stride = static_cast<int64_t>(tables->n_items) * p.group * pool->head_dim;
                sp.part_ml_stride = static_cast<int64_t>(tables->n_items) * p.group * 2;
                sp.counter_stride = tables->n_combine;
                if (p.kv_fp8)
                    for (int32_t l = 0; l < span; ++l)
                        sp.scales[l] = make_float4(pool->k_scale[layer + l], pool->v_scale[layer + l],
                                                       1.0f / pool->k_scale[layer + l], 1.0f / pool->v_scale[layer + l]);
            } else if (fused) {
                pool->scratch_parity ^= 1u;              // scratch sets alternate from launch to launch
                if (pool->scratch_parity) {
                    p.part_o = pool->part_o2;
                    p.part_ml = pool->part_ml2;
                    p.counters = pool->d_counters2;
                }
            }
            p.chained = umma && can_chain ? 1 : 0;     // the mma.sync kernel always waits (a late trigger from its
                                                       // producer warp was measured: 15.9 against 15.3 us waiting)
            pool->last_fused_tensor = span == 1 && fused && k_new != nullptr;
            pool->last_lo = layer;
            pool->last_hi = layer + span;
            pool->last_stream = stream;
            e = launch_tensor_decode(pool, pool->maps, p, kModeSlab, tables, as_stream(stream), lens, umma,
                                     span > 1 ? &sp : nullptr);
        } else if (generic_supported(pool->head_dim)) {
            pool->last_fused_tensor = false;
            p.counters = nullptr;
            e = launch_decode_generic(p, pool->dtype, tables->n_ctas, as_stream(stream));
        } else {
            return ODMA_ERR_INVALID;
        }
    }
    if (e != cudaSuccess) return ODMA_ERR_CUDA;
    if (tables->n_combine > 0 && !fused) {
        ProfScope ps(pool, ODMA_K_COMBINE, as_stream(stream));
        const int32_t* tab = static_cast<const int32_t*>(tables->d_table);
        e = launch_combine(reinterpret_cast<const int4*>(tab + tables->off_combine), tables->n_combine,
                           pool->part_o, pool->part_ml, out, lse, p.group, pool->head_dim, q_heads,
                           pool->io_dtype, as_stream(stream));
        if (e != cudaSuccess) return ODMA_ERR_CUDA;
    }
    return ODMA_OK;
}

}  // namespace

extern "C" {

int32_t odma_decode_attention(odma_pool* pool, int32_t layer, const void* q, int32_t q_heads,
                              const odma_tables* tables, void* out, float* lse, void* stream) {
    return decode_attention_impl(pool, layer, q, q_heads, tables, out, lse, stream, nullptr, nullptr);
}

int32_t odma_decode_step(odma_pool* pool, int32_t layer, int32_t n_layers, int32_t q_heads,
                         const uint64_t* reqs, int32_t n, const void* d_q, const void* d_k_new,
                         const void* d_v_new, void* d_out, float* lse, void* stream,
                         odma_tables* tables_out) {
    if (!pool || !pool->dev_base || !d_q || !d_k_new || !d_v_new || !d_out) return ODMA_ERR_INVALID;
    if (n_layers < 1 || layer < 0 || layer + n_layers > pool->layers) return ODMA_ERR_INVALID;
    if (!reqs || n < 1 || n > pool->alloc.config().max_batch) return ODMA_ERR_INVALID;
    const size_t qb = static_cast<size_t>(n) * q_heads * pool->head_dim * pool->io_bytes;
    const size_t kb = static_cast<size_t>(n) * pool->kv_heads * pool->head_dim * pool->io_bytes;
    // on the tensor-core path the append rides in the decode kernel: one launch per layer
    const bool fuse = pool->alloc.config().fused_append && q_heads >= pool->kv_heads &&
                      q_heads % pool->kv_heads == 0 && uses_tc(pool, q_heads) && aligned16(d_k_new) && aligned16(d_v_new);
    // With the append fused, nothing but that kernel reads the step's lengths, and it can take
    // them with its arguments: when the plan of an earlier step still serves (same requests,
    // same slabs, grown a little) and its table is the one in device memory, this step needs
    // no table copy at all.
    odma_tables t;
    static thread_local InlineLens lens;
    const bool inline_lens = fuse && n <= kInlineLens;
    bool reused = false;
    int32_t rc;
    if (inline_lens) {
        rc = gather_batch(pool, reqs, nullptr, n);
        if (rc != ODMA_OK) return rc;
        int64_t kv_tokens = 0;
        if (pool->step_table_gen != 0 && pool->step_table_gen == pool->plan_cache.gen &&
            plan_reusable(pool, reqs, n, &kv_tokens)) {
            t = pool->plan_cache.desc;
            t.d_table = pool->d_step_table;
            t.kv_tokens = kv_tokens;
            t.epoch = pool->alloc.epoch();
            reused = true;
        }
    }
    if (!reused) {
        rc = odma_build_tables(pool, reqs, nullptr, n, pool->d_step_table,
                               static_cast<uint64_t>(pool->table_words_max) * 4, stream, &t);
        if (rc != ODMA_OK) return rc;
        pool->step_table_gen = pool->plan_cache.valid ? pool->plan_cache.gen : 0;
    }
    if (inline_lens) {
        lens.n = n;
        std::copy(pool->v_len.begin(), pool->v_len.begin() + n, lens.len);
    }
    // All layers in ONE launch of the tcgen05 kernel when it serves this pool and the partial results
    // of every layer's split streams fit the scratch (a plan without split streams needs none).
    const int32_t group = q_heads / pool->kv_heads;
    const bool span_fits =
        t.n_combine == 0 ||
        (static_cast<size_t>(n_layers) * t.n_items * group * pool->head_dim <= 2 * pool->part_o_floats &&
         static_cast<size_t>(n_layers) * t.n_items * group * 2 <= 2 * pool->part_ml_floats &&
         static_cast<size_t>(n_layers) * t.n_combine <= 2 * static_cast<size_t>(pool->slots_max));
    if (fuse && n_layers > 1 && pool->alloc.config().fused_combine && pool->alloc.config().span_layers &&
        pool->alloc.config().decode_kernel != ODMA_DECODE_MMA_SYNC &&
        umma_supported(pool->head_dim, group, pool->dtype == ODMA_DTYPE_FP8_E4M3) && span_fits &&
        (pool->dtype != ODMA_DTYPE_FP8_E4M3 || n_layers <= kMaxSpanScales)) {
        rc = decode_attention_impl(pool, layer, d_q, q_heads, &t, d_out, lse, stream, d_k_new, d_v_new,
                                   inline_lens ? &lens : nullptr, 0, n_layers);
        if (rc != ODMA_OK) return rc;
        if (tables_out) *tables_out = t;
        return ODMA_OK;
    }
    for (int32_t l = 0; l < n_layers; ++l) {
        const uint8_t* kn = static_cast<const uint8_t*>(d_k_new) + l * kb;
        const uint8_t* vn = static_cast<const uint8_t*>(d_v_new) + l * kb;
        if (!fuse) {
            rc = odma_append_kv(pool, layer + l, &t, kn, vn, stream);
            if (rc != ODMA_OK) return rc;
        }
        rc = decode_attention_impl(pool, layer + l, static_cast<const uint8_t*>(d_q) + l * qb, q_heads, &t,
                                   static_cast<uint8_t*>(d_out) + l * qb,
                                   lse ? lse + static_cast<size_t>(l) * n * q_heads : nullptr, stream,
                                   fuse ? kn : nullptr, fuse ? vn : nullptr, inline_lens ? &lens : nullptr,
                                   fuse && n_layers > 1 ? l : -1);
        if (rc != ODMA_OK) return rc;
    }
    if (tables_out) *tables_out = t;
    return ODMA_OK;
}

int32_t odma_decode_step_host(odma_pool* pool, int32_t layer, int32_t q_heads, const uint64_t* reqs,
                              int32_t n, const void* h_q, const void* h_k_new, const void* h_v_new,
                              void* h_out, void* stream) {
    if (!pool || !pool->dev_base || !h_q || !h_k_new || !h_v_new || !h_out) return ODMA_ERR_INVALID;
    if (!reqs || n < 1 || n > pool->alloc.config().max_batch) return ODMA_ERR_INVALID;
    if (q_heads < pool->kv_heads || q_heads % pool->kv_heads != 0 ||
        q_heads / pool->kv_heads > pool->alloc.config().max_group)
        return ODMA_ERR_INVALID;
    const size_t qb = static_cast<size_t>(n) * q_heads * pool->head_dim * pool->io_bytes;
    const size_t kb = static_cast<size_t>(n) * pool->kv_heads * pool->head_dim * pool->io_bytes;
    cudaStream_t s = as_stream(stream);
    // Page-locked buffers are addressable from the device: the kernel then takes the queries
    // and the new rows straight from host memory (one bulk copy per stream, issued by the
    // producer while the KV tiles stream) and writes the result there, and the step is a single
    // launch with no staging copy on either side.
    {
        const void* dq = device_alias(h_q);
        const void* dk = device_alias(h_k_new);
        const void* dv = device_alias(h_v_new);
        void* dout = const_cast<void*>(device_alias(h_out));
        if (dq && dk && dv && dout && aligned16(dq) && aligned16(dk) && aligned16(dv) && aligned16(dout))
            return odma_decode_step(pool, layer, 1, q_heads, reqs, n, dq, dk, dv, dout, nullptr, stream, nullptr);
    }
    if (cudaMemcpyAsync(pool->d_q, h_q, qb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(pool->d_k_new, h_k_new, kb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(pool->d_v_new, h_v_new, kb, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return ODMA_ERR_CUDA;
    // the step itself is the device-buffer one (same plan reuse, same fused append)
    int32_t rc = odma_decode_step(pool, layer, 1, q_heads, reqs, n, pool->d_q, pool->d_k_new, pool->d_v_new,
                                  pool->d_out, nullptr, stream, nullptr);
    if (rc != ODMA_OK) return rc;
    if (cudaMemcpyAsync(h_out, pool->d_out, qb, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return ODMA_ERR_CUDA;
    return ODMA_OK;
}


int32_t odma_decode_attention_static(const odma_pool* pool, const void* dev_base, int32_t layer,
                                     const void* q, int32_t q_heads, const odma_tables* tables,
                                     void* out, float* lse, void* stream) {
    if (!pool || !dev_base || !q || !out || !tables || !tables->d_table) return ODMA_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(dev_base) & 255u) != 0 || !aligned16(q) || !aligned16(out) ||
        !aligned16(tables->d_table))
        return ODMA_ERR_INVALID;
    if (layer < 0 || layer >= pool->layers) return ODMA_ERR_INVALID;
    if (q_heads < pool->kv_heads || q_heads % pool->kv_heads != 0) return ODMA_ERR_INVALID;
    if (tables->n < 1 || tables->n_items < 1 || tables->n_ctas < 1) return ODMA_ERR_INVALID;
    if (!generic_supported(pool->head_dim) || pool->dtype == ODMA_DTYPE_FP8_E4M3) return ODMA_ERR_INVALID;
    const int32_t group = q_heads / pool->kv_heads;
    if (tables->n_items > kStaticSlots || group > kStaticGroup || pool->head_dim > kStaticHeadDim)
        return ODMA_ERR_TOO_LARGE;
    DecodeParams p;
    fill_decode_params(pool, layer, q, q_heads, tables, out, lse, &p);
    p.pool = dev_base;
    p.status = nullptr;       // the kernels of this path wait on nothing
    const int32_t* tab = static_cast<const int32_t*>(tables->d_table);
    cudaError_t e = launch_decode_static(p, pool->dtype, tables->n_ctas,
                                         reinterpret_cast<const int4*>(tab + tables->off_combine),
                                         tables->n_combine, as_stream(stream));
    return e == cudaSuccess ? ODMA_OK : ODMA_ERR_CUDA;
}

int32_t odma_check_status(odma_pool* pool, void* stream) {
    if (!pool || !pool->dev_base) return ODMA_ERR_INVALID;
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return ODMA_ERR_CUDA;
    uint32_t word = 0;
    if (cudaMemcpy(&word, pool->d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return ODMA_ERR_CUDA;
    if (word != 0) {
        // a kernel that gave up may have left split streams half counted
        if (cudaMemset(pool->d_status, 0, 4) != cudaSuccess ||
            cudaMemset(pool->d_counters, 0, static_cast<size_t>(pool->slots_max) * 8) != cudaSuccess)
            return ODMA_ERR_CUDA;
    }
    return (word & kStatusTimeout) ? ODMA_ERR_TIMEOUT : ODMA_OK;
}

int32_t odma_read_probe(odma_pool* pool, int32_t layer, int32_t q_heads, const odma_tables* tables,
                        void* stream) {
    if (!pool || !pool->dev_base || !pool->has_maps || layer < 0 || layer >= pool->layers)
        return ODMA_ERR_INVALID;
    if (pool->dtype != ODMA_DTYPE_BF16) return ODMA_ERR_INVALID;      // the probe is the mma.sync kernel's
    if (q_heads < pool->kv_heads || q_heads % pool->kv_heads != 0) return ODMA_ERR_INVALID;
    int32_t rc = check_tables(pool, tables);
    if (rc != ODMA_OK) return rc;
    DecodeParams p;
    // the probe moves the query bytes too; any valid device memory of that size will do
    fill_decode_params(pool, layer, pool->d_q, q_heads, tables, pool->d_out, nullptr, &p);
    if (!tc_supported(pool->head_dim, p.group) || p.group > pool->alloc.config().max_group || p.stages < 2)
        return ODMA_ERR_INVALID;
    pool->decode_was_last = false;
    pool->last_fused_tensor = false;
    ProfScope ps(pool, ODMA_K_PROBE, as_stream(stream));
    return launch_decode_tc(pool->maps, p, kModeProbe, tables->n_ctas, as_stream(stream)) == cudaSuccess
               ? ODMA_OK
               : ODMA_ERR_CUDA;
}

int32_t odma_profile_enable(odma_pool* pool, int32_t on) {
    if (!pool || !pool->dev_base) return ODMA_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) return ODMA_ERR_CUDA;
    clear_profile(pool);
    pool->profiling = on != 0;
    return ODMA_OK;
}

int32_t odma_profile_read(odma_pool* pool, int32_t kernel, double* total_ms, int64_t* launches) {
    if (!pool || !pool->dev_base || kernel < 0 || kernel >= ODMA_K_COUNT) return ODMA_ERR_INVALID;
    double ms = 0.0;
    int64_t count = 0;
    for (auto& r : pool->prof) {
        if (r.kernel != kernel) continue;
        if (cudaEventSynchronize(r.stop) != cudaSuccess) return ODMA_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.start, r.stop) != cudaSuccess) return ODMA_ERR_CUDA;
        ms += t;
        count += 1;
    }
    if (total_ms) *total_ms = ms;
    if (launches) *launches = count;
    return ODMA_OK;
}

/* Launches a one-thread kernel whose only wait can never be satisfied and must give up after
 * limit_ms; odma_check_status then reports ODMA_ERR_TIMEOUT.  Shows that a lost signal ends in
 * an error code, not in a hung GPU. */
int32_t odma_selftest_timeout(odma_pool* pool, int32_t limit_ms, void* stream) {
    if (!pool || !pool->dev_base || limit_ms < 1 || limit_ms > 1000) return ODMA_ERR_INVALID;
    return launch_wait_selftest(pool->d_status, static_cast<int64_t>(limit_ms) * 1000000ll,
                                as_stream(stream)) == cudaSuccess
               ? ODMA_OK
               : ODMA_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// page-16 ablation
// ---------------------------------------------------------------------------------------------

int32_t odma_paged_create(odma_pool* pool, void* d_pages, uint64_t bytes, odma_paged** out) {
    if (!out) return ODMA_ERR_INVALID;
    *out = nullptr;
    if (!pool || !pool->dev_base || !d_pages || (reinterpret_cast<uintptr_t>(d_pages) & 255u) != 0)
        return ODMA_ERR_INVALID;
    if (pool->dtype == ODMA_DTYPE_FP8_E4M3) return ODMA_ERR_INVALID;  // the ablation exists for 16- and 32-bit pools
    const uint64_t page_bytes = static_cast<uint64_t>(pool->layers) * 2u * pool->kv_heads * 16u *
                                pool->head_dim * pool->elem_bytes;
    const int64_t n_pages = static_cast<int64_t>(bytes / page_bytes);
    if (n_pages < 1 || n_pages * pool->kv_heads * 16 * pool->layers * 2 >= (int64_t(1) << 31))
        return ODMA_ERR_INVALID;
    odma_paged* pg = new (std::nothrow) odma_paged();
    if (!pg) return ODMA_ERR_NOMEM;
    pg->pool = pool;
    pg->d_pages = d_pages;
    pg->n_pages = n_pages;
    if (pool->has_maps) {
        if (make_tensor_maps(d_pages, n_pages * pool->kv_heads * 16 * pool->layers * 2, pool->head_dim,
                             pool->elem_bytes, &pg->maps) != ODMA_OK) {
            delete pg;
            return ODMA_ERR_CUDA;
        }
        pg->has_maps = true;
    }
    *out = pg;
    return ODMA_OK;
}

int32_t odma_paged_destroy(odma_paged* paged) {
    if (!paged) return ODMA_ERR_INVALID;
    if (paged->pinned) cudaFreeHost(paged->pinned);
    delete paged;
    return ODMA_OK;
}

int32_t odma_paged_build(odma_paged* paged, const odma_tables* tables, const int32_t* host_len,
                         uint64_t shuffle_seed, int32_t* d_page_table, int32_t max_pages, void* stream) {
    if (!paged || !tables || !tables->d_table || !host_len || !d_page_table || max_pages < 1)
        return ODMA_ERR_INVALID;
    odma_pool* pool = paged->pool;
    const int32_t n = tables->n;
    int64_t need = 0;
    int32_t longest = 0;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t pages = (host_len[i] + 15) / 16;
        if (host_len[i] < 1 || pages > max_pages) return ODMA_ERR_INVALID;
        need += pages;
        longest = std::max(longest, host_len[i]);
    }
    if (need > paged->n_pages) return ODMA_ERR_NOMEM;
    // page ids: 0,1,2,... in request order, or a seeded permutation of all pages of the buffer
    std::vector<int32_t> ids(static_cast<size_t>(shuffle_seed ? paged->n_pages : need));
    for (size_t i = 0; i < ids.size(); ++i) ids[i] = static_cast<int32_t>(i);
    if (shuffle_seed) {
        uint64_t s = shuffle_seed;
        auto next = [&s]() {                 // splitmix64
            uint64_t z = (s += 0x9E3779B97F4A7C15ull);
            z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
            z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
            return z ^ (z >> 31);
        };
        for (size_t i = ids.size() - 1; i > 0; --i) std::swap(ids[i], ids[next() % (i + 1)]);
    }
    const int64_t words = static_cast<int64_t>(n) * max_pages;
    if (words > paged->pinned_words) {
        if (paged->pinned) cudaFreeHost(paged->pinned);
        paged->pinned = nullptr;
        if (cudaMallocHost(&paged->pinned, static_cast<size_t>(words) * 4) != cudaSuccess) return ODMA_ERR_CUDA;
        paged->pinned_words = words;
    }
    std::fill(paged->pinned, paged->pinned + words, 0);
    size_t k = 0;
    for (int32_t i = 0; i < n; ++i)
        for (int32_t pg = 0; pg < (host_len[i] + 15) / 16; ++pg)
            paged->pinned[static_cast<size_t>(i) * max_pages + pg] = ids[k++];
    cudaStream_t s = as_stream(stream);
    if (cudaMemcpyAsync(d_page_table, paged->pinned, static_cast<size_t>(words) * 4, cudaMemcpyHostToDevice, s) !=
        cudaSuccess)
        return ODMA_ERR_CUDA;
    const int32_t* tab = static_cast<const int32_t*>(tables->d_table);
    ScatterPagesParams sp;
    sp.base = tab + tables->off_base;
    sp.cap = tab + tables->off_cap;
    sp.len = tab + tables->off_len;
    sp.page_table = d_page_table;
    sp.pool = pool->dev_base;
    sp.pages = paged->d_pages;
    sp.rows_per_array = pool->rows_per_array;
    sp.n_pages = paged->n_pages;
    sp.n = n;
    sp.max_pages = max_pages;
    sp.arrays = pool->layers * 2;
    sp.kv_heads = pool->kv_heads;
    sp.row_vecs = pool->head_dim * pool->elem_bytes / 16;
    if (launch_scatter_pages(sp, longest, s) != cudaSuccess) return ODMA_ERR_CUDA;
    // the pinned table is reused by the next call: wait for the copy
    return cudaStreamSynchronize(s) == cudaSuccess ? ODMA_OK : ODMA_ERR_CUDA;
}

int32_t odma_decode_attention_paged(odma_paged* paged, int32_t layer, const void* q, int32_t q_heads,
                                    const odma_tables* tables, const int32_t* d_page_table,
                                    int32_t max_pages, void* out, float* lse, void* stream) {
    if (!paged || !paged->has_maps || !d_page_table || max_pages < 1) return ODMA_ERR_INVALID;
    odma_pool* pool = paged->pool;
    int32_t rc = check_decode_args(pool, layer, q, q_heads, tables, out);
    if (rc != ODMA_OK) return rc;
    DecodeParams p;
    fill_decode_params(pool, layer, q, q_heads, tables, out, lse, &p);
    if (!tc_supported(pool->head_dim, p.group) || p.stages < 2) return ODMA_ERR_INVALID;
    p.pool = paged->d_pages;
    p.rows_per_array = paged->n_pages * pool->kv_heads * 16;
    p.page_table = d_page_table;
    p.max_pages = max_pages;
    pool->decode_was_last = false;        // nothing chains to, or starts early behind, a launch of the ablation
    pool->last_fused_tensor = false;
    cudaError_t e;
    {
        ProfScope ps(pool, ODMA_K_DECODE, as_stream(stream));
        e = launch_tensor_decode(pool, paged->maps, p, kModePaged, tables, as_stream(stream), nullptr,
                                 uses_umma(pool, p.group, false));
    }
    if (e != cudaSuccess) return ODMA_ERR_CUDA;
    if (tables->n_combine > 0 && p.counters == nullptr) {
        ProfScope ps(pool, ODMA_K_COMBINE, as_stream(stream));
        const int32_t* tab = static_cast<const int32_t*>(tables->d_table);
        e = launch_combine(reinterpret_cast<const int4*>(tab + tables->off_combine), tables->n_combine,
                           pool->part_o, pool->part_ml, out, lse, p.group, pool->head_dim, q_heads,
                           pool->io_dtype, as_stream(stream));
        if (e != cudaSuccess) return ODMA_ERR_CUDA;
    }
    return ODMA_OK;
}

int32_t odma_sim_run(odma_pool* pool, const odma_sim_params* params, const odma_sim_request* reqs, int32_t n,
                     odma_sim_result* out) {
    if (!pool || !params) return ODMA_ERR_INVALID;
    odma_stats st;
    pool->alloc.stats(&st);
    if (st.live != 0) return ODMA_ERR_INVALID;
    pool->plan_cache.valid = false;
    return simulate(pool->alloc, *params, reqs, n, out);
}

}  // extern "C"
