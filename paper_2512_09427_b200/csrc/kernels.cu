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

#include "odma.h"

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
// The query heads of the group are the M rows of the MMA tiles (rows >= group are zero).

constexpr int kConsumerWarps = 4;
constexpr int kTcThreads = (kConsumerWarps + 1) * 32;
constexpr int kTile = 64;

template <int D, bool HI>
struct TcConfig {
    static constexpr int kRows = HI ? 16 : 8;
    static constexpr int kKvTileBytes = kTile * D * 2;
    static constexpr int kStageBytes = 2 * kKvTileBytes;
    static constexpr int kQBytes = 16 * D * 2;
    static constexpr int kMoStride = D + 8;
    static constexpr int kMergeBytes = kConsumerWarps * kRows * (kMoStride + 2) * 4;
    static constexpr int kFixedBytes = 2 * kQBytes + kMergeBytes + 64 /*desc*/ + 256 /*barriers*/;
    static constexpr int kBudget = 227 * 1024 - 1024 /*alignment slack*/;
    static constexpr int kStagesFit = (kBudget - kFixedBytes) / kStageBytes;
    static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
    static constexpr int kSmemBytes = kStages * kStageBytes + kFixedBytes + 1024;
};

template <int D, bool HI, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tm_big,
                 const __grid_constant__ CUtensorMap tm_small, const DecodeParams p) {
    using Cfg = TcConfig<D, HI>;
    constexpr int STAGES = Cfg::kStages;
    constexpr int ROWS = Cfg::kRows;
    constexpr int HALVES = D / 64;                 // 128-byte column blocks per row
    constexpr int HALF_BYTES = kTile * 128;
    constexpr int MO_STRIDE = Cfg::kMoStride;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* kv = smem;
    uint8_t* qbuf = kv + STAGES * Cfg::kStageBytes;
    float* mrg_o = reinterpret_cast<float*>(qbuf + 2 * Cfg::kQBytes);
    float* mrg_ml = mrg_o + kConsumerWarps * ROWS * MO_STRIDE;
    int* desc = reinterpret_cast<int*>(mrg_ml + kConsumerWarps * ROWS * 2);
    uint64_t* bars = reinterpret_cast<uint64_t*>(desc + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 6);

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (STAGES + s); };
    auto qfull_bar = [&](uint32_t s) { return bar0 + 8u * (2 * STAGES + s); };
    auto qempty_bar = [&](uint32_t s) { return bar0 + 8u * (2 * STAGES + 2 + s); };
    const uint32_t mready_bar = bar0 + 8u * (2 * STAGES + 4);
    const uint32_t mdone_bar = bar0 + 8u * (2 * STAGES + 5);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int64_t limit = p.wait_limit_ns;

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
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // query rows >= group stay zero for the whole kernel; TMA only ever writes rows < group
    for (int i = tid; i < 2 * Cfg::kQBytes / 16; i += kTcThreads)
        reinterpret_cast<uint4*>(qbuf)[i] = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    const int cta = blockIdx.x;
    const int it_begin = p.cta_begin[cta], it_end = p.cta_begin[cta + 1];
    const uint32_t kv_u32 = smem_u32(kv);
    const uint32_t q_u32 = smem_u32(qbuf);

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // loads issued per stage (drain on abort)
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
                    dsc[3] = 0;
                    mbar_arrive(qfull_bar(qs));
                    break;
                }
                const int4 a = p.items[2 * it], b = p.items[2 * it + 1];
                const int req = a.x, head = a.y, tok0 = a.z, ntok = a.w;
                dsc[0] = req;
                dsc[1] = head;
                dsc[2] = tok0;
                dsc[3] = ntok;
                dsc[4] = b.x;
                dsc[5] = b.y;
                const uint32_t q_bytes = static_cast<uint32_t>(p.group) * D * 2u;
                mbar_expect_tx(qfull_bar(qs), q_bytes);
                bulk_load(q_u32 + qs * Cfg::kQBytes,
                          static_cast<const uint8_t*>(p.q) +
                              (static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * p.group) * D * 2,
                          q_bytes, qfull_bar(qs));
                int64_t row = 0;
                const int32_t* pages = nullptr;
                if (MODE == kModePaged) {
                    pages = p.page_table + static_cast<size_t>(req) * p.max_pages + tok0 / 16;
                } else {
                    row = static_cast<int64_t>(p.base[req]) * p.kv_heads +
                          static_cast<int64_t>(head) * p.cap[req] + tok0;
                }
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
                    issued[stage] += 1;
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // Something timed out.  Before the CTA's shared memory can be handed to another
                // CTA, wait (bounded, ignoring the abort flag) for the loads already in flight.
                for (int s = 0; s < STAGES; ++s)
                    if (issued[s])
                        mbar_wait_slow(full_bar(s), (issued[s] - 1u) & 1u, nullptr, p.status,
                                       limit / 4 + 1);
            }
        }
        __syncwarp();
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int qd = lane >> 2, qt = lane & 3;          // row within 8, position within the quad
    const int mi = lane >> 3, r8 = lane & 7;          // ldmatrix: matrix id, row within it
    const uint32_t k_lane_off = (warp * 16 + (mi >> 1) * 8 + r8) * 128;
    const uint32_t xk = (mi & 1) ^ r8;
    const uint32_t v_lane_off = (warp * 16 + (mi & 1) * 8 + r8) * 128;
    const uint32_t xv = (mi >> 1) ^ r8;
    const uint32_t q_lane_off = ((mi & 1) * 8 + r8) * (D * 2) + (mi >> 1) * 16;
    const int kidx0 = warp * 16 + qt * 2;             // first of this thread's key columns
    const float scale = p.scale_log2;
    const int group = p.group;

    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (uint32_t k_item = 0; ok; ++k_item) {
        const uint32_t qs = k_item & 1u;
        ok = mbar_wait(qfull_bar(qs), (k_item >> 1) & 1u, abort_flag, p.status, limit);
        if (!ok) break;
        const int* dsc = desc + qs * 8;
        const int req = dsc[0], head = dsc[1], ntok = dsc[3], direct = dsc[4], slot = dsc[5];
        if (ntok == 0) break;

        uint32_t qa[D / 16][4];
        if (MODE != kModeProbe) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
                ldmatrix_x4(qa[kk], q_u32 + qs * Cfg::kQBytes + q_lane_off + kk * 32);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(qempty_bar(qs));

        float o[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

        const int ntiles = (ntok + kTile - 1) / kTile;
        for (int t = 0; t < ntiles; ++t) {
            ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, limit);
            if (!ok) break;
            const int valid = min(kTile, ntok - t * kTile);
            if (MODE != kModeProbe && warp * 16 < valid) {
                const uint32_t kbase = kv_u32 + stage * Cfg::kStageBytes;
                const uint32_t vbase = kbase + Cfg::kKvTileBytes;
                // ---- S = Q K^T for this warp's 16 keys (two n-tiles of 8 keys)
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    uint32_t b[4];
                    ldmatrix_x4(b, kbase + (kk >> 2) * HALF_BYTES + k_lane_off +
                                       ((((kk & 3) * 2) ^ xk) << 4));
                    mma_bf16(s0, qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b[0], b[1]);
                    mma_bf16(s1, qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b[2], b[3]);
                }
                // ---- keys at or beyond the item's end: scores are selected to -inf (never
                //      added to), value rows are zeroed in registers below
                uint32_t vm0 = 0xFFFFFFFFu, vm1 = 0xFFFFFFFFu;
                const bool ragged = valid < kTile;
                if (ragged) {
                    const bool in0 = kidx0 < valid, in1 = kidx0 + 1 < valid;
                    const bool in8 = kidx0 + 8 < valid, in9 = kidx0 + 9 < valid;
                    if (!in0) s0[0] = s0[2] = -INFINITY;
                    if (!in1) s0[1] = s0[3] = -INFINITY;
                    if (!in8) s1[0] = s1[2] = -INFINITY;
                    if (!in9) s1[1] = s1[3] = -INFINITY;
                    vm0 = (in0 ? 0x0000FFFFu : 0u) | (in1 ? 0xFFFF0000u : 0u);
                    vm1 = (in8 ? 0x0000FFFFu : 0u) | (in9 ? 0xFFFF0000u : 0u);
                }
                // ---- online softmax, fp32, row max shared across the quad by shuffles
                uint32_t pa0, pa1 = 0u, pa2, pa3 = 0u;
                {
                    float mx = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
                    const float m_new = fmaxf(m_lo, mx * scale);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                    const float corr = exp2f(m_lo - m_use);
                    const float p0 = exp2f(fmaf(s0[0], scale, -m_use));
                    const float p1 = exp2f(fmaf(s0[1], scale, -m_use));
                    const float p2 = exp2f(fmaf(s1[0], scale, -m_use));
                    const float p3 = exp2f(fmaf(s1[1], scale, -m_use));
                    l_lo = fmaf(l_lo, corr, (p0 + p1) + (p2 + p3));
                    m_lo = m_new;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        o[i][0] *= corr;
                        o[i][1] *= corr;
                    }
                    pa0 = pack_bf16(p0, p1);
                    pa2 = pack_bf16(p2, p3);
                }
                if (HI) {
                    float mx = fmaxf(fmaxf(s0[2], s0[3]), fmaxf(s1[2], s1[3]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
                    const float m_new = fmaxf(m_hi, mx * scale);
                    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                    const float corr = exp2f(m_hi - m_use);
                    const float p0 = exp2f(fmaf(s0[2], scale, -m_use));
                    const float p1 = exp2f(fmaf(s0[3], scale, -m_use));
                    const float p2 = exp2f(fmaf(s1[2], scale, -m_use));
                    const float p3 = exp2f(fmaf(s1[3], scale, -m_use));
                    l_hi = fmaf(l_hi, corr, (p0 + p1) + (p2 + p3));
                    m_hi = m_new;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        o[i][2] *= corr;
                        o[i][3] *= corr;
                    }
                    pa1 = pack_bf16(p0, p1);
                    pa3 = pack_bf16(p2, p3);
                }
                // ---- O += P V
#pragma unroll
                for (int jj = 0; jj < D / 16; ++jj) {
                    uint32_t b[4];
                    ldmatrix_x4_trans(b, vbase + (jj >> 2) * HALF_BYTES + v_lane_off +
                                             ((((jj & 3) * 2) ^ xv) << 4));
                    if (ragged) {
                        b[0] &= vm0;
                        b[1] &= vm1;
                        b[2] &= vm0;
                        b[3] &= vm1;
                    }
                    mma_bf16(o[2 * jj], pa0, pa1, pa2, pa3, b[0], b[1]);
                    mma_bf16(o[2 * jj + 1], pa0, pa1, pa2, pa3, b[2], b[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(stage));
            if (++stage == STAGES) {
                stage = 0;
                phase ^= 1u;
            }
        }
        if (!ok) break;
        if (MODE == kModeProbe) continue;

        // ---- merge the four warps' partial results and write the item's result
        l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
        if (HI) {
            l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
            l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);
        }
        if (k_item > 0) {
            ok = mbar_wait(mdone_bar, (k_item - 1u) & 1u, abort_flag, p.status, limit);
            if (!ok) break;
        }
        float* mo = mrg_o + warp * ROWS * MO_STRIDE;
        float* mml = mrg_ml + warp * ROWS * 2;
        if (qd < group) {
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2*>(mo + qd * MO_STRIDE + i * 8 + qt * 2) =
                    make_float2(o[i][0], o[i][1]);
            if (qt == 0) {
                mml[qd * 2] = m_lo;
                mml[qd * 2 + 1] = l_lo;
            }
        }
        if (HI && qd + 8 < group) {
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2*>(mo + (qd + 8) * MO_STRIDE + i * 8 + qt * 2) =
                    make_float2(o[i][2], o[i][3]);
            if (qt == 0) {
                mml[(qd + 8) * 2] = m_hi;
                mml[(qd + 8) * 2 + 1] = l_hi;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(mready_bar);
        ok = mbar_wait(mready_bar, k_item & 1u, abort_flag, p.status, limit);
        if (!ok) break;
        for (int idx = tid; idx < group * D; idx += kConsumerWarps * 32) {
            const int r = idx / D, d = idx - r * D;
            float mw[kConsumerWarps], M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                mw[w] = mrg_ml[(w * ROWS + r) * 2];
                M = fmaxf(M, mw[w]);
            }
            float L = 0.f, O = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const float e = exp2f(mw[w] - M);       // exp2(-inf) = 0 for warps without keys
                L = fmaf(mrg_ml[(w * ROWS + r) * 2 + 1], e, L);
                O = fmaf(mrg_o[(w * ROWS + r) * MO_STRIDE + d], e, O);
            }
            if (direct) {
                const size_t row = static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * group + r;
                reinterpret_cast<__nv_bfloat16*>(p.out)[row * D + d] = __float2bfloat16_rn(O / L);
                if (d == 0 && p.lse) p.lse[row] = (M + log2f(L)) * 0.6931471805599453f;
            } else {
                const size_t prow = static_cast<size_t>(slot) * group + r;
                p.part_o[prow * D + d] = O;
                if (d == 0) {
                    p.part_ml[prow * 2] = M;
                    p.part_ml[prow * 2 + 1] = L;
                }
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

    for (int it = p.cta_begin[cta]; it < p.cta_begin[cta + 1]; ++it) {
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
    const int req = rec.x, head = rec.y, slot0 = rec.z, ns = rec.w;
    for (int idx = threadIdx.x; idx < group * D; idx += blockDim.x) {
        const int r = idx / D, d = idx - r * D;
        float M = -INFINITY;
        for (int s = 0; s < ns; ++s)
            M = fmaxf(M, part_ml[(static_cast<size_t>(slot0 + s) * group + r) * 2]);
        float L = 0.f, O = 0.f;
        for (int s = 0; s < ns; ++s) {
            const size_t prow = static_cast<size_t>(slot0 + s) * group + r;
            const float e = exp2f(part_ml[prow * 2] - M);
            L = fmaf(part_ml[prow * 2 + 1], e, L);
            O = fmaf(part_o[prow * D + d], e, O);
        }
        const size_t row = static_cast<size_t>(req) * q_heads + static_cast<size_t>(head) * group + r;
        store_out(out + row * D + d, O / L);
        if (d == 0 && lse) lse[row] = (M + log2f(L)) * 0.6931471805599453f;
    }
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
        // request owning new token `tok`: last r with cu_new[r] <= tok
        int lo = 0, hi = p.n;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.cu_new[mid] <= tok) lo = mid; else hi = mid;
        }
        const int req = lo;
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

template <int D, bool HI, int MODE>
cudaError_t launch_tc_inst(const TensorMaps& maps, const DecodeParams& p, int n_ctas, cudaStream_t stream) {
    using Cfg = TcConfig<D, HI>;
    static bool configured = false;
    auto kern = decode_tc_kernel<D, HI, MODE>;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<n_ctas, kTcThreads, Cfg::kSmemBytes, stream>>>(maps.big, maps.small, p);
    return cudaGetLastError();
}

template <int D, bool HI>
cudaError_t launch_tc_mode(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas, cudaStream_t s) {
    switch (mode) {
        case kModeSlab: return launch_tc_inst<D, HI, kModeSlab>(maps, p, n_ctas, s);
        case kModePaged: return launch_tc_inst<D, HI, kModePaged>(maps, p, n_ctas, s);
        case kModeProbe: return launch_tc_inst<D, HI, kModeProbe>(maps, p, n_ctas, s);
    }
    return cudaErrorInvalidValue;
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

cudaError_t launch_decode_tc(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                             cudaStream_t stream) {
    const bool hi = p.group > 8;
    if (p.head_dim == 128)
        return hi ? launch_tc_mode<128, true>(maps, p, mode, n_ctas, stream)
                  : launch_tc_mode<128, false>(maps, p, mode, n_ctas, stream);
    if (p.head_dim == 64)
        return hi ? launch_tc_mode<64, true>(maps, p, mode, n_ctas, stream)
                  : launch_tc_mode<64, false>(maps, p, mode, n_ctas, stream);
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

cudaError_t launch_wait_selftest(uint32_t* status, int64_t limit_ns, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace odma
