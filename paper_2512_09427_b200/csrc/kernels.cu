// CUDA kernels of libodma for sm_100a.
//
//  append_kv_kernel        writes the step's new K/V rows behind each request's tokens
//  migrate_copy_kernel     slab -> slab copy of one request (allocate-and-copy migration)
//  decode_tc_kernel        split decode attention, bf16: TMA-staged slab streams, GQA heads
//                          packed into the M dimension of mma.sync tiles, fp32 online softmax
//  decode_generic_kernel   same result for any dtype / group size on the plain ALUs (fp32 path)
//  combine_kernel          log-sum-exp merge of the partial results of split streams
//  scatter_pages_kernel    re-lays slabs into 16-token pages (ablation input)
//
// The decode kernels are persistent: CTA c works through items [cta_begin[c], cta_begin[c+1])
// of the host-built plan; an item is a run of tokens of one (request, KV head) stream.
#include "kernels.hpp"

#include <cuda_bf16.h>

#include <algorithm>

#include "odma.h"

#pragma nv_diag_suppress 128   // the probe instantiation leaves the merge code unreachable

namespace odma {
namespace {

// =============================================================================================
// small PTX wrappers
// =============================================================================================

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}

// Every wait in this file is bounded: when `limit_ns` passes without the barrier completing,
// the waiter raises the CTA's abort flag and the timeout bit of the status word and gives up;
// every other waiter of the CTA sees the flag and gives up too.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            uint32_t* status, int64_t limit_ns) {
    uint64_t t0 = 0;
    for (uint32_t i = 1;; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 63u) == 0u) {
            if (abort_flag && *abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (static_cast<int64_t>(now - t0) > limit_ns) {
                if (abort_flag) *abort_flag = 1;
                atomicOr(status, kStatusTimeout);
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* status, int64_t limit_ns) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, limit_ns);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x,
                                            int32_t y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes,
                                          uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// =============================================================================================
// decode attention, tensor-core path (bf16, head_dim 64 or 128, group <= 16)
// =============================================================================================
//
// Roles: warps 0..3 consume, warp 4 (one lane) produces.  A pipeline stage holds one tile of 64
// keys and 64 values of one stream, written by TMA with the 128-byte swizzle so that ldmatrix
// reads are conflict-free.  Consumer warp w owns keys [16w, 16w+16) of every tile and keeps its
// own running (max, sum, output); the four are merged through shared memory when the item ends.
//
// The contraction is arranged with the KEYS on the M side of the MMA tiles and the query heads
// of the GQA group on the N side (8 heads per n-tile, rows >= group are zero):
//     S^T[16 keys x 8 heads]  = K[16 keys x D]   . Q^T[D x 8 heads]
//     O^T[D x 8 heads]       += V^T[D x 16 keys] . P^T[16 keys x 8 heads]
// so a group of 7 heads wastes one column in eight instead of nine rows in sixteen, and the
// softmax weights go from the first product's accumulator to the second product's B operand
// with one 8x8 register transpose (movmatrix) per eight keys.

constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kTcThreads = kConsumerThreads + 32;
constexpr int kTile = 64;
constexpr int kMaxStages = 8;

template <int D, int NT>
struct TcConfig {
    static constexpr int kRows = NT * 8;
    static constexpr int kKvTileBytes = kTile * D * 2;
    static constexpr int kStageBytes = 2 * kKvTileBytes;
    static constexpr int kQBytes = kRows * D * 2;
    static constexpr int kMoStride = D + 4;
    static constexpr int kMergeFloats = kConsumerWarps * kRows * kMoStride;
    static constexpr int kMlFloats = kConsumerWarps * kRows * 2;
    static constexpr int kFixedBytes =
        2 * kQBytes + (kMergeFloats + kMlFloats) * 4 + 2 * 8 * 4 /*desc*/ + (2 * kMaxStages + 8) * 8 /*barriers*/ + 64;
    static constexpr int kAlignSlack = 1024;
    static int smem_bytes(int stages) { return stages * kStageBytes + kFixedBytes + kAlignSlack; }
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ void store4(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, float a, float b, float c, float d) {
    *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf16(a, b), pack_bf16(c, d));
}

// Log-sum-exp merge of the `ns` partial results of one (request, KV head) stream, slots
// [slot0, slot0+ns): out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), M = max_s m_s.
// Thread `tid` of `nthreads` takes two groups of four output elements of one query head.
// Partials are read through L2 (they may have been written by other SMs a moment ago).
template <typename T>
__device__ __forceinline__ void combine_stream(const float* part_o, const float* part_ml, int slot0,
                                               int ns, int req, int head, int group, int D,
                                               int q_heads, T* out, float* lse, int tid, int nthreads) {
    const int per_row = D >> 3;
    for (int idx = tid; idx < group * per_row; idx += nthreads) {
        const int r = idx / per_row, c = idx - r * per_row;
        const int d0 = c * 4, d1 = (D >> 1) + c * 4;
        float M = -INFINITY;
#pragma unroll 4
        for (int s = 0; s < ns; ++s)
            M = fmaxf(M, __ldcg(part_ml + (static_cast<size_t>(slot0 + s) * group + r) * 2));
        float L = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll 2
        for (int s = 0; s < ns; ++s) {
            const size_t prow = static_cast<size_t>(slot0 + s) * group + r;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + prow * 2));
            const float e = ml.x == -INFINITY ? 0.f : exp2f(ml.x - M);
            const float4 x = ldcg4(part_o + prow * D + d0), y = ldcg4(part_o + prow * D + d1);
            L = fmaf(ml.y, e, L);
            a.x = fmaf(x.x, e, a.x); a.y = fmaf(x.y, e, a.y); a.z = fmaf(x.z, e, a.z); a.w = fmaf(x.w, e, a.w);
            b.x = fmaf(y.x, e, b.x); b.y = fmaf(y.y, e, b.y); b.z = fmaf(y.z, e, b.z); b.w = fmaf(y.w, e, b.w);
        }
        const float inv = 1.f / L;
        const size_t row = static_cast<size_t>(req) * q_heads + static_cast<size_t>(head) * group + r;
        store4(out + row * D + d0, a.x * inv, a.y * inv, a.z * inv, a.w * inv);
        store4(out + row * D + d1, b.x * inv, b.y * inv, b.z * inv, b.w * inv);
        if (c == 0 && lse) lse[row] = (M + log2f(L)) * 0.6931471805599453f;
    }
}

template <int D, int NT, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tm_big,
                 const __grid_constant__ CUtensorMap tm_small, const DecodeParams p) {
    using Cfg = TcConfig<D, NT>;
    constexpr int ROWS = Cfg::kRows;
    constexpr int HALVES = D / 64;                 // 128-byte column blocks per row
    constexpr int HALF_BYTES = kTile * 128;
    constexpr int MO = Cfg::kMoStride;
    const int STAGES = p.stages;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* kv = smem;
    uint8_t* qbuf = kv + STAGES * Cfg::kStageBytes;
    float* mrg_o = reinterpret_cast<float*>(qbuf + 2 * Cfg::kQBytes);
    float* mrg_ml = mrg_o + Cfg::kMergeFloats;
    int* desc = reinterpret_cast<int*>(mrg_ml + Cfg::kMlFloats);
    uint64_t* bars = reinterpret_cast<uint64_t*>(desc + 16);
    volatile int* flags = reinterpret_cast<volatile int*>(bars + 2 * kMaxStages + 8);
    volatile int* abort_flag = flags;            // flags[0]: a wait timed out somewhere in the CTA
    volatile int* last_flag = flags + 1;         // flags[1]: this CTA completes a split stream

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (kMaxStages + s); };
    auto qfull_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + s); };
    auto qempty_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + 2 + s); };
    const uint32_t mready_bar = bar0 + 8u * (2 * kMaxStages + 4);
    const uint32_t mdone_bar = bar0 + 8u * (2 * kMaxStages + 5);
    const uint32_t cfence_bar = bar0 + 8u * (2 * kMaxStages + 6);
    const uint32_t cflag_bar = bar0 + 8u * (2 * kMaxStages + 7);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int64_t limit = p.wait_limit_ns;
    const int cta = blockIdx.x;

    // the producer's first loads are in flight while the barriers are being set up
    int4 rec = make_int4(0, 0, 0, 0), first_a = rec, first_b = rec;
    if (tid == kConsumerThreads) {
        const int4* r = p.cta + 3 * cta;
        rec = __ldg(r);
        first_a = __ldg(r + 1);
        first_b = __ldg(r + 2);
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_big)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_small)) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), kConsumerWarps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(qfull_bar(s), 1);
            mbar_init(qempty_bar(s), kConsumerWarps);
        }
        mbar_init(mready_bar, kConsumerWarps);
        mbar_init(mdone_bar, kConsumerWarps);
        mbar_init(cfence_bar, kConsumerWarps);
        mbar_init(cflag_bar, kConsumerWarps);
        flags[0] = 0;
        flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // query rows >= group stay zero for the whole kernel; the bulk copy only writes rows < group
    for (int i = tid; i < 2 * Cfg::kQBytes / 16; i += kTcThreads)
        reinterpret_cast<uint4*>(qbuf)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    const uint32_t kv_u32 = smem_u32(kv);
    const uint32_t q_u32 = smem_u32(qbuf);

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const int it_begin = rec.x, it_end = rec.y;
            uint32_t stage = 0, phase = 0;
            uint32_t issued_any = 0, issued_odd = 0;     // per stage: loads issued at all / an odd number
            bool ok = true;
            const int64_t k_array = static_cast<int64_t>(p.layer) * 2 * p.rows_per_array;
            const int64_t v_array = k_array + p.rows_per_array;
            uint32_t k_item = 0;
            for (int it = it_begin; ok; ++it, ++k_item) {
                const uint32_t qs = k_item & 1u;
                ok = mbar_wait(qempty_bar(qs), ((k_item >> 1) & 1u) ^ 1u, abort_flag, p.status, limit);
                if (!ok) break;
                int* dsc = desc + qs * 8;
                if (it >= it_end) {                      // end marker
                    dsc[2] = 0;
                    mbar_arrive(qfull_bar(qs));
                    break;
                }
                int4 a = first_a, b = first_b;
                if (it != it_begin) {
                    a = __ldg(p.items + 2 * it);
                    b = __ldg(p.items + 2 * it + 1);
                }
                const int req = a.x, head = a.y, tok0 = a.z, ntok = a.w;
                dsc[0] = req;
                dsc[1] = head;
                dsc[2] = ntok;
                dsc[3] = b.x;     // direct
                dsc[4] = b.y;     // slot
                dsc[5] = b.w;     // combine record
                const uint32_t q_bytes = static_cast<uint32_t>(p.group) * D * 2u;
                mbar_expect_tx(qfull_bar(qs), q_bytes);
                bulk_load(q_u32 + qs * Cfg::kQBytes,
                          static_cast<const uint8_t*>(p.q) +
                              (static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * p.group) * D * 2,
                          q_bytes, qfull_bar(qs));
                const int64_t row = b.z;
                const int32_t* pages = nullptr;
                if (MODE == kModePaged)
                    pages = p.page_table + static_cast<size_t>(req) * p.max_pages + tok0 / 16;
                const int ntiles = (ntok + kTile - 1) / kTile;
                for (int t = 0; t < ntiles; ++t) {
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, limit);
                    if (!ok) break;
                    const int valid = min(kTile, ntok - t * kTile);
                    const uint32_t kdst = kv_u32 + stage * Cfg::kStageBytes;
                    const uint32_t vdst = kdst + Cfg::kKvTileBytes;
                    if (MODE != kModePaged && valid == kTile) {
                        mbar_expect_tx(full_bar(stage), Cfg::kStageBytes);
                        const int32_t ky = static_cast<int32_t>(k_array + row + t * kTile);
                        const int32_t vy = static_cast<int32_t>(v_array + row + t * kTile);
#pragma unroll
                        for (int h = 0; h < HALVES; ++h) {
                            tma_load_2d(kdst + h * HALF_BYTES, &tm_big, h * 64, ky, full_bar(stage));
                            tma_load_2d(vdst + h * HALF_BYTES, &tm_big, h * 64, vy, full_bar(stage));
                        }
                    } else {
                        const int nb = (valid + 15) >> 4;     // 16-row boxes; never past ceil16(len)
                        mbar_expect_tx(full_bar(stage), static_cast<uint32_t>(nb) * 16u * D * 2u * 2u);
                        for (int bx = 0; bx < nb; ++bx) {
                            int32_t ky, vy;
                            if (MODE == kModePaged) {
                                const int64_t prow =
                                    (static_cast<int64_t>(pages[t * 4 + bx]) * p.kv_heads + head) * 16;
                                ky = static_cast<int32_t>(k_array + prow);
                                vy = static_cast<int32_t>(v_array + prow);
                            } else {
                                ky = static_cast<int32_t>(k_array + row + t * kTile + bx * 16);
                                vy = static_cast<int32_t>(v_array + row + t * kTile + bx * 16);
                            }
#pragma unroll
                            for (int h = 0; h < HALVES; ++h) {
                                tma_load_2d(kdst + h * HALF_BYTES + bx * 2048, &tm_small, h * 64, ky,
                                            full_bar(stage));
                                tma_load_2d(vdst + h * HALF_BYTES + bx * 2048, &tm_small, h * 64, vy,
                                            full_bar(stage));
                            }
                        }
                    }
                    issued_any |= 1u << stage;
                    issued_odd ^= 1u << stage;
                    if (++stage == static_cast<uint32_t>(STAGES)) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // Something timed out.  Before the CTA's shared memory can be handed to another
                // CTA, wait (bounded, ignoring the abort flag) for the loads already in flight.
                for (int s = 0; s < STAGES; ++s)
                    if ((issued_any >> s) & 1u)      // parity of the stage's latest phase
                        mbar_wait_slow(full_bar(s), ((issued_odd >> s) & 1u) ^ 1u, nullptr, p.status,
                                       limit / 4 + 1);
            }
        }
        __syncwarp();
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int qd = lane >> 2, qt = lane & 3;          // row within 8, position within the quad
    const int mi = lane >> 3, r8 = lane & 7;          // ldmatrix: matrix id, row within it
    // K tile as the A operand: matrices (keys 0-7, d 0-7) (keys 8-15, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 8-15)
    const uint32_t k_lane_off = (warp * 16 + (mi & 1) * 8 + r8) * 128;
    const uint32_t xk = (mi >> 1) ^ r8;
    // V tile, transposed on load, as the A operand: (keys 0-7, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 0-7) (keys 8-15, d 8-15)
    const uint32_t v_lane_off = (warp * 16 + (mi >> 1) * 8 + r8) * 128;
    const uint32_t xv = (mi & 1) ^ r8;
    // Q as the B operand: four consecutive 16-byte chunks of head r8
    const uint32_t q_lane_off = r8 * (D * 2) + mi * 16;
    const int key_lo = warp * 16 + qd;                // the thread's two key rows: key_lo, key_lo + 8
    const int vkey0 = warp * 16 + qt * 2;             // keys of its value fragments: vkey0, +1, +8, +9
    const float scale = p.scale_log2;
    const int group = p.group;

    uint32_t stage = 0, phase = 0, n_split = 0;
    bool ok = true;
    for (uint32_t k_item = 0; ok; ++k_item) {
        const uint32_t qs = k_item & 1u;
        ok = mbar_wait(qfull_bar(qs), (k_item >> 1) & 1u, abort_flag, p.status, limit);
        if (!ok) break;
        const int* dsc = desc + qs * 8;
        const int req = dsc[0], head = dsc[1], ntok = dsc[2], direct = dsc[3], slot = dsc[4], comb = dsc[5];
        if (ntok == 0) break;

        uint32_t qb[NT][D / 16][2];
        if (MODE != kModeProbe) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int j = 0; j < D / 32; ++j) {
                    uint32_t r[4];
                    ldmatrix_x4(r, q_u32 + qs * Cfg::kQBytes + nt * 8 * (D * 2) + q_lane_off + j * 64);
                    qb[nt][2 * j][0] = r[0];
                    qb[nt][2 * j][1] = r[1];
                    qb[nt][2 * j + 1][0] = r[2];
                    qb[nt][2 * j + 1][1] = r[3];
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(qempty_bar(qs));

        float o[NT][D / 16][4];
        float m_run[NT][2], l_run[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int i = 0; i < D / 16; ++i) o[nt][i][0] = o[nt][i][1] = o[nt][i][2] = o[nt][i][3] = 0.f;
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
        }

        const int ntiles = (ntok + kTile - 1) / kTile;
        for (int t = 0; t < ntiles; ++t) {
            ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, limit);
            if (!ok) break;
            const int valid = min(kTile, ntok - t * kTile);
            if (MODE != kModeProbe && warp * 16 < valid) {
                const uint32_t kbase = kv_u32 + stage * Cfg::kStageBytes;
                const uint32_t vbase = kbase + Cfg::kKvTileBytes;
                // ---- S^T = K Q^T for this warp's 16 keys; two accumulators shorten the chain
                float s[NT][4], s2[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) s[nt][i] = s2[nt][i] = 0.f;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    uint32_t a[4];
                    ldmatrix_x4(a, kbase + (kk >> 2) * HALF_BYTES + k_lane_off + ((((kk & 3) * 2) ^ xk) << 4));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        if (kk & 1)
                            mma_bf16(s2[nt], a[0], a[1], a[2], a[3], qb[nt][kk][0], qb[nt][kk][1]);
                        else
                            mma_bf16(s[nt], a[0], a[1], a[2], a[3], qb[nt][kk][0], qb[nt][kk][1]);
                    }
                }
                // ---- keys at or beyond the item's end: scores are selected to -inf (never
                //      added to), value rows are zeroed in registers below
                const bool ragged = valid < kTile;
                const bool in_lo = key_lo < valid, in_hi = key_lo + 8 < valid;
                uint32_t vm0 = 0xFFFFFFFFu, vm1 = 0xFFFFFFFFu;
                if (ragged) {
                    vm0 = (vkey0 < valid ? 0x0000FFFFu : 0u) | (vkey0 + 1 < valid ? 0xFFFF0000u : 0u);
                    vm1 = (vkey0 + 8 < valid ? 0x0000FFFFu : 0u) | (vkey0 + 9 < valid ? 0xFFFF0000u : 0u);
                }
                // ---- online softmax, fp32; a head's maximum is shared by the eight lanes that
                //      hold its keys (shuffles over the lane bits that select the key row)
                uint32_t pb[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    float c0 = s[nt][0] + s2[nt][0], c1 = s[nt][1] + s2[nt][1];
                    float c2 = s[nt][2] + s2[nt][2], c3 = s[nt][3] + s2[nt][3];
                    if (!in_lo) c0 = c1 = -INFINITY;
                    if (!in_hi) c2 = c3 = -INFINITY;
                    float mx0 = fmaxf(c0, c2), mx1 = fmaxf(c1, c3);
#pragma unroll
                    for (int off = 4; off < 32; off <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, off));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, off));
                    }
                    const float mn0 = fmaxf(m_run[nt][0], mx0 * scale), mn1 = fmaxf(m_run[nt][1], mx1 * scale);
                    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
                    const float corr0 = exp2f(m_run[nt][0] - mu0), corr1 = exp2f(m_run[nt][1] - mu1);
                    const float p0 = exp2f(fmaf(c0, scale, -mu0)), p1 = exp2f(fmaf(c1, scale, -mu1));
                    const float p2 = exp2f(fmaf(c2, scale, -mu0)), p3 = exp2f(fmaf(c3, scale, -mu1));
                    l_run[nt][0] = fmaf(l_run[nt][0], corr0, p0 + p2);
                    l_run[nt][1] = fmaf(l_run[nt][1], corr1, p1 + p3);
                    m_run[nt][0] = mn0;
                    m_run[nt][1] = mn1;
#pragma unroll
                    for (int i = 0; i < D / 16; ++i) {
                        o[nt][i][0] *= corr0;
                        o[nt][i][1] *= corr1;
                        o[nt][i][2] *= corr0;
                        o[nt][i][3] *= corr1;
                    }
                    // P[key][head] -> P^T fragments: (head qd; keys 2qt, 2qt+1) and (+8, +9)
                    pb[nt][0] = movmatrix_trans(pack_bf16(p0, p1));
                    pb[nt][1] = movmatrix_trans(pack_bf16(p2, p3));
                }
                // ---- O^T += V^T P^T
#pragma unroll
                for (int dt = 0; dt < D / 16; ++dt) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, vbase + (dt >> 2) * HALF_BYTES + v_lane_off + ((((dt & 3) * 2) ^ xv) << 4));
                    if (ragged) {
                        a[0] &= vm0;
                        a[1] &= vm0;
                        a[2] &= vm1;
                        a[3] &= vm1;
                    }
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        mma_bf16(o[nt][dt], a[0], a[1], a[2], a[3], pb[nt][0], pb[nt][1]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(stage));
            if (++stage == static_cast<uint32_t>(STAGES)) {
                stage = 0;
                phase ^= 1u;
            }
        }
        if (!ok) break;
        if (MODE == kModeProbe) continue;

        // ---- merge the four warps' partial results and write the item's result
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l_run[nt][0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[nt][0], off);
                l_run[nt][1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[nt][1], off);
            }
        if (k_item > 0) {
            ok = mbar_wait(mdone_bar, (k_item - 1u) & 1u, abort_flag, p.status, limit);
            if (!ok) break;
        }
        float* mo = mrg_o + warp * ROWS * MO;
        float* mml = mrg_ml + warp * ROWS * 2;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int h0 = nt * 8 + qt * 2;
#pragma unroll
            for (int dt = 0; dt < D / 16; ++dt) {
                const int d = dt * 16 + qd;
                mo[h0 * MO + d] = o[nt][dt][0];
                mo[(h0 + 1) * MO + d] = o[nt][dt][1];
                mo[h0 * MO + d + 8] = o[nt][dt][2];
                mo[(h0 + 1) * MO + d + 8] = o[nt][dt][3];
            }
            if (qd == 0) {
                mml[h0 * 2] = m_run[nt][0];
                mml[h0 * 2 + 1] = l_run[nt][0];
                mml[h0 * 2 + 2] = m_run[nt][1];
                mml[h0 * 2 + 3] = l_run[nt][1];
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(mready_bar);
        ok = mbar_wait(mready_bar, k_item & 1u, abort_flag, p.status, limit);
        if (!ok) break;
        constexpr int PER_ROW = D / 8;
        for (int idx = tid; idx < group * PER_ROW; idx += kConsumerThreads) {
            const int r = idx / PER_ROW, c = idx - r * PER_ROW;
            const int d0 = c * 4, d1 = D / 2 + c * 4;
            float mw[kConsumerWarps], M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                mw[w] = mrg_ml[(w * ROWS + r) * 2];
                M = fmaxf(M, mw[w]);
            }
            float L = 0.f;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const float e = mw[w] == -INFINITY ? 0.f : exp2f(mw[w] - M);   // warps without keys
                const float4 x = *reinterpret_cast<const float4*>(mrg_o + (w * ROWS + r) * MO + d0);
                const float4 y = *reinterpret_cast<const float4*>(mrg_o + (w * ROWS + r) * MO + d1);
                L = fmaf(mrg_ml[(w * ROWS + r) * 2 + 1], e, L);
                a.x = fmaf(x.x, e, a.x); a.y = fmaf(x.y, e, a.y); a.z = fmaf(x.z, e, a.z); a.w = fmaf(x.w, e, a.w);
                b.x = fmaf(y.x, e, b.x); b.y = fmaf(y.y, e, b.y); b.z = fmaf(y.z, e, b.z); b.w = fmaf(y.w, e, b.w);
            }
            if (direct) {
                const float inv = 1.f / L;
                const size_t row = static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * group + r;
                __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
                store4(out + row * D + d0, a.x * inv, a.y * inv, a.z * inv, a.w * inv);
                store4(out + row * D + d1, b.x * inv, b.y * inv, b.z * inv, b.w * inv);
                if (c == 0 && p.lse) p.lse[row] = (M + log2f(L)) * 0.6931471805599453f;
            } else {
                const size_t prow = static_cast<size_t>(slot) * group + r;
                *reinterpret_cast<float4*>(p.part_o + prow * D + d0) = a;
                *reinterpret_cast<float4*>(p.part_o + prow * D + d1) = b;
                if (c == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(M, L);
            }
        }
        if (!direct && p.counters != nullptr) {
            // ---- the CTA that delivers a split stream's last piece merges all of them: every
            //      thread's partial stores are fenced, one thread counts this piece in, and the
            //      CTA that sees the count complete reads the pieces back through L2
            __threadfence();
            __syncwarp();
            if (lane == 0) mbar_arrive(cfence_bar);
            ok = mbar_wait(cfence_bar, n_split & 1u, abort_flag, p.status, limit);
            if (!ok) break;
            const int4 cr = __ldg(p.combine + comb);         // {request, head, first slot, pieces}
            if (tid == 0) {
                const uint32_t seen = atomicAdd(p.counters + comb, 1u);
                const int last = seen + 1u == static_cast<uint32_t>(cr.w);
                if (last) p.counters[comb] = 0u;              // ready for the next launch
                *last_flag = last;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(cflag_bar);
            ok = mbar_wait(cflag_bar, n_split & 1u, abort_flag, p.status, limit);
            if (!ok) break;
            ++n_split;
            if (*last_flag) {
                __threadfence();
                combine_stream(p.part_o, p.part_ml, cr.z, cr.w, cr.x, cr.y, group, D, p.q_heads,
                               reinterpret_cast<__nv_bfloat16*>(p.out), p.lse, tid, kConsumerThreads);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(mdone_bar);
    }
}

// =============================================================================================
// decode attention, generic path (fp32 or bf16 storage, any group size, plain ALUs, fp32 math)
// =============================================================================================

template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
    static constexpr int kElems = 4;
    __device__ static void unpack(const uint4& v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x);
        x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z);
        x[3] = __uint_as_float(v.w);
    }
};
template <>
struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void unpack(const uint4& v, float (&x)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

constexpr int kGenericHeads = 8;    // query heads handled per pass over an item
constexpr int kGenericWarps = 4;

template <typename T, int DPL>      // head_dim = 32 * DPL
__global__ void __launch_bounds__(kGenericWarps * 32)
decode_generic_kernel(const DecodeParams p) {
    constexpr int D = 32 * DPL;
    constexpr int GC = kGenericHeads;
    constexpr int VE = Vec16<T>::kElems;
    __shared__ float q_s[GC][D];
    __shared__ float p_s[kGenericWarps][GC][32];
    __shared__ float mrg_o[kGenericWarps][GC][D];
    __shared__ float mrg_ml[kGenericWarps][GC][2];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const T* pool = static_cast<const T*>(p.pool);
    const T* qg = static_cast<const T*>(p.q);
    T* outg = static_cast<T*>(p.out);
    const float scale = p.scale_log2;

    const int4 rec = __ldg(p.cta + 3 * cta);
    for (int it = rec.x; it < rec.y; ++it) {
        const int4 a = p.items[2 * it], b = p.items[2 * it + 1];
        const int req = a.x, head = a.y, tok0 = a.z, ntok = a.w, direct = b.x, slot = b.y;
        const int64_t row0 = static_cast<int64_t>(p.base[req]) * p.kv_heads +
                             static_cast<int64_t>(head) * p.cap[req] + tok0;
        const T* K = pool + (static_cast<int64_t>(p.layer) * 2 * p.rows_per_array + row0) * D;
        const T* V = K + p.rows_per_array * D;

        for (int h0 = 0; h0 < p.group; h0 += GC) {
            const int gc = min(GC, p.group - h0);
            __syncthreads();
            for (int idx = tid; idx < gc * D; idx += kGenericWarps * 32) {
                const int r = idx / D, d = idx - r * D;
                q_s[r][d] = to_float(
                    qg[(static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * p.group + h0 + r) * D + d]);
            }
            __syncthreads();

            float m[GC], l[GC], o[GC][DPL];
#pragma unroll
            for (int r = 0; r < GC; ++r) {
                m[r] = -INFINITY;
                l[r] = 0.f;
#pragma unroll
                for (int c = 0; c < DPL; ++c) o[r][c] = 0.f;
            }
            for (int j0 = warp * 32; j0 < ntok; j0 += kGenericWarps * 32) {
                const int j = j0 + lane;
                const bool valid = j < ntok;
                float s[GC];
#pragma unroll
                for (int r = 0; r < GC; ++r) s[r] = 0.f;
                if (valid) {
                    const uint4* kp = reinterpret_cast<const uint4*>(K + static_cast<int64_t>(j) * D);
#pragma unroll 2
                    for (int v = 0; v < D / VE; ++v) {
                        float x[VE];
                        Vec16<T>::unpack(kp[v], x);
#pragma unroll
                        for (int e = 0; e < VE; ++e)
#pragma unroll
                            for (int r = 0; r < GC; ++r)
                                if (r < gc) s[r] = fmaf(q_s[r][v * VE + e], x[e], s[r]);
                    }
                }
#pragma unroll
                for (int r = 0; r < GC; ++r) {
                    if (r >= gc) continue;          // uniform across the warp
                    const float sv = valid ? s[r] * scale : -INFINITY;
                    float mx = sv;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1)
                        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
                    const float m_new = fmaxf(m[r], mx);      // finite: lane 0 is always valid
                    const float pr = exp2f(sv - m_new);
                    const float corr = exp2f(m[r] - m_new);
                    float ps = pr;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xFFFFFFFFu, ps, off);
                    l[r] = fmaf(l[r], corr, ps);
                    m[r] = m_new;
#pragma unroll
                    for (int c = 0; c < DPL; ++c) o[r][c] *= corr;
                    p_s[warp][r][lane] = pr;
                }
                __syncwarp();
                const int cnt = min(32, ntok - j0);
                for (int jj = 0; jj < cnt; ++jj) {
                    float v[DPL];
#pragma unroll
                    for (int c = 0; c < DPL; ++c)
                        v[c] = to_float(V[static_cast<int64_t>(j0 + jj) * D + lane + 32 * c]);
#pragma unroll
                    for (int r = 0; r < GC; ++r) {
                        if (r >= gc) continue;
                        const float pr = p_s[warp][r][jj];
#pragma unroll
                        for (int c = 0; c < DPL; ++c) o[r][c] = fmaf(pr, v[c], o[r][c]);
                    }
                }
                __syncwarp();
            }
#pragma unroll
            for (int r = 0; r < GC; ++r) {
                if (r >= gc) continue;
#pragma unroll
                for (int c = 0; c < DPL; ++c) mrg_o[warp][r][lane + 32 * c] = o[r][c];
                if (lane == 0) {
                    mrg_ml[warp][r][0] = m[r];
                    mrg_ml[warp][r][1] = l[r];
                }
            }
            __syncthreads();
            for (int idx = tid; idx < gc * D; idx += kGenericWarps * 32) {
                const int r = idx / D, d = idx - r * D;
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < kGenericWarps; ++w) M = fmaxf(M, mrg_ml[w][r][0]);
                float L = 0.f, O = 0.f;
#pragma unroll
                for (int w = 0; w < kGenericWarps; ++w) {
                    const float e = exp2f(mrg_ml[w][r][0] - M);
                    L = fmaf(mrg_ml[w][r][1], e, L);
                    O = fmaf(mrg_o[w][r][d], e, O);
                }
                if (direct) {
                    const size_t row = static_cast<size_t>(req) * p.q_heads +
                                       static_cast<size_t>(head) * p.group + h0 + r;
                    store_out(outg + row * D + d, O / L);
                    if (d == 0 && p.lse) p.lse[row] = (M + log2f(L)) * 0.6931471805599453f;
                } else {
                    const size_t prow = static_cast<size_t>(slot) * p.group + h0 + r;
                    p.part_o[prow * D + d] = O;
                    if (d == 0) {
                        p.part_ml[prow * 2] = M;
                        p.part_ml[prow * 2 + 1] = L;
                    }
                }
            }
        }
    }
}

// =============================================================================================
// combine: out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M),  M = max_s m_s
// =============================================================================================

template <typename T>
__global__ void __launch_bounds__(128)
combine_kernel(const int4* __restrict__ combine, const float* __restrict__ part_o,
               const float* __restrict__ part_ml, T* __restrict__ out, float* __restrict__ lse,
               int group, int D, int q_heads) {
    const int4 rec = combine[blockIdx.x];
    combine_stream(part_o, part_ml, rec.z, rec.w, rec.x, rec.y, group, D, q_heads, out, lse,
                   static_cast<int>(threadIdx.x), static_cast<int>(blockDim.x));
}

// =============================================================================================
// append / migrate / page scatter: 16-byte vector copies
// =============================================================================================

__global__ void __launch_bounds__(256) append_kv_kernel(const AppendParams p) {
    const int64_t vecs_per_tok = static_cast<int64_t>(p.kv_heads) * p.row_vecs;
    const int64_t total = static_cast<int64_t>(p.n_new_total) * vecs_per_tok * 2;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    uint4* pool = static_cast<uint4*>(p.pool);
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int kv = static_cast<int>(i / (static_cast<int64_t>(p.n_new_total) * vecs_per_tok));
        const int64_t rem = i - kv * static_cast<int64_t>(p.n_new_total) * vecs_per_tok;
        const int tok = static_cast<int>(rem / vecs_per_tok);
        const int within = static_cast<int>(rem - tok * vecs_per_tok);
        const int head = within / p.row_vecs, vec = within - head * p.row_vecs;
        // request owning new token `tok`: last r with cu_new[r] <= tok (tok itself when every
        // request appends exactly one token, the decode case)
        int req = tok;
        if (!p.one_new_each) {
            int lo = 0, hi = p.n;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (p.cu_new[mid] <= tok) lo = mid; else hi = mid;
            }
            req = lo;
        }
        const int n_new = p.cu_new[req + 1] - p.cu_new[req];
        const int pos = p.len[req] - n_new + (tok - p.cu_new[req]);
        const int64_t row = static_cast<int64_t>(p.base[req]) * p.kv_heads +
                            static_cast<int64_t>(head) * p.cap[req] + pos;
        const int64_t array = static_cast<int64_t>(p.layer) * 2 + kv;
        const uint4* src = static_cast<const uint4*>(kv ? p.v_new : p.k_new);
        pool[(array * p.rows_per_array + row) * p.row_vecs + vec] = src[rem];
    }
}

__global__ void __launch_bounds__(256) migrate_copy_kernel(const MigrateParams p) {
    // blockIdx.y = array * kv_heads + head: one contiguous run of len rows each
    const int array = blockIdx.y / p.kv_heads, head = blockIdx.y - array * p.kv_heads;
    uint4* pool = static_cast<uint4*>(p.pool);
    const int64_t src = (array * p.rows_per_array + p.src_base * p.kv_heads + head * p.src_cap) * p.row_vecs;
    const int64_t dst = (array * p.rows_per_array + p.dst_base * p.kv_heads + head * p.dst_cap) * p.row_vecs;
    const int64_t total = p.len * p.row_vecs;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride)
        pool[dst + i] = pool[src + i];
}

__global__ void __launch_bounds__(256) scatter_pages_kernel(const ScatterPagesParams p) {
    // grid: x over vectors of one (request, array, head) run, y = array*kv_heads + head, z = request
    const int req = blockIdx.z;
    const int array = blockIdx.y / p.kv_heads, head = blockIdx.y - array * p.kv_heads;
    const int len = p.len[req];
    const uint4* pool = static_cast<const uint4*>(p.pool);
    uint4* pages = static_cast<uint4*>(p.pages);
    const int64_t src = (array * p.rows_per_array + static_cast<int64_t>(p.base[req]) * p.kv_heads +
                         static_cast<int64_t>(head) * p.cap[req]) * p.row_vecs;
    const int64_t total = static_cast<int64_t>(len) * p.row_vecs;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int tok = static_cast<int>(i / p.row_vecs), vec = static_cast<int>(i - static_cast<int64_t>(tok) * p.row_vecs);
        const int64_t page = p.page_table[static_cast<size_t>(req) * p.max_pages + tok / 16];
        const int64_t drow = ((array * p.n_pages + page) * p.kv_heads + head) * 16 + (tok & 15);
        pages[drow * p.row_vecs + vec] = pool[src + i];
    }
}

__global__ void wait_selftest_kernel(uint32_t* status, int64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // nobody ever arrives on `bar`: the wait must give up after limit_ns
        mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
    }
}

// ---------------------------------------------------------------------------------------------
// launch helpers
// ---------------------------------------------------------------------------------------------

constexpr int kSmemPerSm = 233472;        // shared memory of one SM
constexpr int kSmemPerCtaMax = 232448;    // most one CTA may ask for
constexpr int kSmemCtaReserve = 1024;     // what the system keeps per resident CTA

template <int D, int NT, int MODE>
cudaError_t launch_tc_inst(const TensorMaps& maps, const DecodeParams& p, int n_ctas, cudaStream_t stream) {
    using Cfg = TcConfig<D, NT>;
    static bool configured = false;
    auto kern = decode_tc_kernel<D, NT, MODE>;
    const int smem = Cfg::smem_bytes(p.stages);
    if (p.stages < 2 || p.stages > kMaxStages || smem > kSmemPerCtaMax) return cudaErrorInvalidValue;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCtaMax);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<n_ctas, kTcThreads, smem, stream>>>(maps.big, maps.small, p);
    return cudaGetLastError();
}

template <int D, int NT>
cudaError_t launch_tc_mode(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas, cudaStream_t s) {
    switch (mode) {
        case kModeSlab: return launch_tc_inst<D, NT, kModeSlab>(maps, p, n_ctas, s);
        case kModePaged: return launch_tc_inst<D, NT, kModePaged>(maps, p, n_ctas, s);
        case kModeProbe: return launch_tc_inst<D, NT, kModeProbe>(maps, p, n_ctas, s);
    }
    return cudaErrorInvalidValue;
}

template <int D, int NT>
int32_t tc_stages_inst(int32_t ctas_per_sm) {
    using Cfg = TcConfig<D, NT>;
    const int budget = std::min(kSmemPerSm / ctas_per_sm - kSmemCtaReserve, kSmemPerCtaMax);
    const int n = (budget - Cfg::kFixedBytes - Cfg::kAlignSlack) / Cfg::kStageBytes;
    return n < 2 ? 0 : (n > kMaxStages ? kMaxStages : n);
}

template <typename T>
cudaError_t launch_generic_t(const DecodeParams& p, int n_ctas, cudaStream_t s) {
    switch (p.head_dim) {
        case 32: decode_generic_kernel<T, 1><<<n_ctas, kGenericWarps * 32, 0, s>>>(p); break;
        case 64: decode_generic_kernel<T, 2><<<n_ctas, kGenericWarps * 32, 0, s>>>(p); break;
        case 128: decode_generic_kernel<T, 4><<<n_ctas, kGenericWarps * 32, 0, s>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

bool tc_supported(int32_t head_dim, int32_t group) {
    return (head_dim == 64 || head_dim == 128) && group >= 1 && group <= 16;
}

bool generic_supported(int32_t head_dim) { return head_dim == 32 || head_dim == 64 || head_dim == 128; }

int32_t tc_stages(int32_t head_dim, int32_t group, int32_t ctas_per_sm) {
    if (!tc_supported(head_dim, group) || ctas_per_sm < 1) return 0;
    const bool two = group > 8;
    if (head_dim == 128) return two ? tc_stages_inst<128, 2>(ctas_per_sm) : tc_stages_inst<128, 1>(ctas_per_sm);
    return two ? tc_stages_inst<64, 2>(ctas_per_sm) : tc_stages_inst<64, 1>(ctas_per_sm);
}

cudaError_t launch_decode_tc(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                             cudaStream_t stream) {
    const bool two = p.group > 8;
    if (p.head_dim == 128)
        return two ? launch_tc_mode<128, 2>(maps, p, mode, n_ctas, stream)
                   : launch_tc_mode<128, 1>(maps, p, mode, n_ctas, stream);
    if (p.head_dim == 64)
        return two ? launch_tc_mode<64, 2>(maps, p, mode, n_ctas, stream)
                   : launch_tc_mode<64, 1>(maps, p, mode, n_ctas, stream);
    return cudaErrorInvalidValue;
}

cudaError_t launch_decode_generic(const DecodeParams& p, int dtype, int n_ctas, cudaStream_t stream) {
    return dtype == ODMA_DTYPE_F32 ? launch_generic_t<float>(p, n_ctas, stream)
                                   : launch_generic_t<__nv_bfloat16>(p, n_ctas, stream);
}

cudaError_t launch_combine(const int4* combine, int n_combine, const float* part_o,
                           const float* part_ml, void* out, float* lse, int group, int head_dim,
                           int q_heads, int dtype, cudaStream_t stream) {
    if (n_combine <= 0) return cudaSuccess;
    if (dtype == ODMA_DTYPE_F32)
        combine_kernel<float><<<n_combine, 128, 0, stream>>>(combine, part_o, part_ml,
                                                             static_cast<float*>(out), lse, group,
                                                             head_dim, q_heads);
    else
        combine_kernel<__nv_bfloat16><<<n_combine, 128, 0, stream>>>(
            combine, part_o, part_ml, static_cast<__nv_bfloat16*>(out), lse, group, head_dim, q_heads);
    return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t stream) {
    if (p.n_new_total <= 0) return cudaSuccess;
    const int64_t total = static_cast<int64_t>(p.n_new_total) * p.kv_heads * p.row_vecs * 2;
    const int64_t blocks = (total + 255) / 256;
    const int grid = static_cast<int>(blocks < 148 * 16 ? blocks : 148 * 16);
    append_kv_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_migrate(const MigrateParams& p, cudaStream_t stream) {
    if (p.len <= 0) return cudaSuccess;
    const int64_t total = p.len * p.row_vecs;
    const int64_t blocks = (total + 255) / 256;
    dim3 grid(static_cast<unsigned>(blocks < 64 ? blocks : 64), static_cast<unsigned>(p.arrays * p.kv_heads));
    migrate_copy_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_scatter_pages(const ScatterPagesParams& p, int64_t max_len, cudaStream_t stream) {
    const int64_t total = max_len * p.row_vecs;
    const int64_t blocks = (total + 255) / 256;
    dim3 grid(static_cast<unsigned>(blocks < 32 ? (blocks > 0 ? blocks : 1) : 32),
              static_cast<unsigned>(p.arrays * p.kv_heads), static_cast<unsigned>(p.n));
    scatter_pages_kernel<<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// decode attention with the split partials in a fixed device array instead of allocated scratch
// ---------------------------------------------------------------------------------------------

// One array per GPU that loads the library, held until the process exits: room for
// kStaticSlots pieces of kStaticGroup query heads, each head_dim outputs plus (max, sum).
constexpr int kStaticFloats = kStaticSlots * kStaticGroup * (kStaticHeadDim + 2);
static __device__ __align__(256) float g_static_partials[kStaticFloats];

cudaError_t launch_decode_static(DecodeParams p, int dtype, int n_ctas, const int4* combine,
                                 int n_combine, cudaStream_t stream) {
    // In host code the array's name is not a device address; the address is asked for once
    // per device, with that device current, and kept.
    static float* scratch_of_device[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!scratch_of_device[dev]) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_partials);
        if (e != cudaSuccess) return e;
        scratch_of_device[dev] = ptr;
    }
    // partial outputs first, then the (max, sum) pairs; every slot a launch reads it has
    // written itself, so nothing has to start at zero
    p.part_o = scratch_of_device[dev];
    p.part_ml = scratch_of_device[dev] + static_cast<size_t>(kStaticSlots) * kStaticGroup * kStaticHeadDim;
    p.counters = nullptr;
    e = launch_decode_generic(p, dtype, n_ctas, stream);
    if (e != cudaSuccess) return e;
    return launch_combine(combine, n_combine, p.part_o, p.part_ml, p.out, p.lse, p.group, p.head_dim,
                          p.q_heads, dtype, stream);
}

cudaError_t launch_wait_selftest(uint32_t* status, int64_t limit_ns, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace odma
