// CUDA kernels of libodma for sm_100a.
//
//  append_kv_kernel        writes the step's new K/V rows behind each request's tokens (an 8-bit
//                          pool: quantised to E4M3 on the way)
//  migrate_copy_kernel     slab -> slab copy of one request (allocate-and-copy migration)
//  decode_tc_kernel        split decode attention, bf16: TMA-staged slab streams, keys on the M
//                          side and the GQA group's heads on the N side of mma.sync tiles, fp32
//                          online softmax; can take the step's append and the merge of split
//                          streams along
//  decode_generic_kernel   same result for any dtype / group size on the plain ALUs (fp32 path)
//  combine_kernel          log-sum-exp merge of the partial results of split streams
//  scatter_pages_kernel    re-lays slabs into 16-token pages (ablation input)
//
// The decode kernels are persistent: CTA c works through the items of its record in the
// host-built plan; an item is a run of tokens of one (request, KV head) stream.
#include "kernels.hpp"

#include <cuda_bf16.h>

#include <algorithm>

#include "device_utils.cuh"
#include "odma.h"

#pragma nv_diag_suppress 128   // the probe instantiation leaves the merge code unreachable

namespace odma {
namespace {

using namespace dev;

// =============================================================================================
// decode attention, tensor-core path (bf16, head_dim 64 or 128, group <= 16)
// =============================================================================================
//
// Roles: warps 0..7 consume (two groups of four), warp 8 produces, warps 9.. finish.  A
// pipeline stage holds one tile of 64 keys and 64 values of one stream, written by TMA with the
// 128-byte swizzle so that ldmatrix reads are conflict-free.  The CTA's items go to the two
// consumer groups in turn (short items are latency chains; two in flight hide each other, and
// one group's hand-over runs under the other's streaming); a stream of 16 tiles or more is
// worked on by both groups, its tiles going to them in turn (two tiles in flight).
// Warp w of a group owns keys [16w, 16w+16) of every tile of the group's item and keeps its own
// running (max, sum, output): the four warps sit on the four schedulers of the SM.  A warp's
// work on 16 keys is a chain of dependent steps (ldmatrix, mma chains of 21 cycles a link,
// shuffles, ex2, movmatrix, mma: 770 cycles), so spreading a tile over four warps is what
// keeps a tile's latency short (0.4 us against 1.3 us for one warp on all 64 keys).
// When an item ends the four warps drop their partial results into the group's merge buffer
// and go straight on to the group's next item; the finisher warps merge the four, write the
// item's result (or partial result) to global memory and, for a split stream, count the piece
// in and merge all pieces if it was the last one.  Queries, item descriptors and (with the
// append fused in) the stream's new K and V rows travel through a ring of 4..8 slots so the
// producer can run several short items ahead of the consumers.
//
// A query slot is refilled by bulk copies (async proxy) after generic-proxy reads of it: its
// release (mbarrier arrive) is preceded by fence.proxy.async.  Merge buffers are written and
// read through the generic proxy only; arrive (release) and wait (acquire) order them.
//
// The contraction is arranged with the KEYS on the M side of the MMA tiles and the query heads
// of the GQA group on the N side (8 heads per n-tile; columns >= group hold whatever the
// query slot holds and are never written out: a column of the product depends on that column
// of the B operand only):
//     S^T[16 keys x 8 heads]  = K[16 keys x D]   . Q^T[D x 8 heads]
//     O^T[D x 8 heads]       += V^T[D x 16 keys] . P^T[16 keys x 8 heads]
// so a group of 7 heads wastes one column in eight instead of nine rows in sixteen, and the
// softmax weights go from the first product's accumulator to the second product's B operand
// with one 8x8 register transpose (movmatrix) per eight keys.

constexpr int kConsumerWarps = 4;                 // per consumer group: one tile is shared by four warps
constexpr int kConsumerGroups = 2;                // items go to the groups in turn
constexpr int kConsumerThreads = kConsumerGroups * kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerGroups * kConsumerWarps;
constexpr int kFinisherWarp0 = kProducerWarp + 1;
constexpr int kFinisherWarps = 3;                 // 12 warps in all: three per scheduler, 168 registers each
constexpr int kFinisherThreads = kFinisherWarps * 32;
constexpr int kTcThreads = kConsumerThreads + 32 + kFinisherThreads;
constexpr int kTile = 64;
constexpr int kMaxStages = 8;
constexpr int kMinQSlots = 4, kMaxQSlots = 8;
constexpr int kMergeBufs = 2;
constexpr int kBothGroupsTiles = 16;              // streams this long are worked on by both consumer groups at once                // tiles each consumer warp asks into L2 at the start of the kernel
constexpr int kNumBars = 2 * kMaxStages + 2 * kMaxQSlots + 2 * kMergeBufs + 2;

template <int D, int NT>
struct TcConfig {
    static constexpr int kRows = NT * 8;
    static constexpr int kKvTileBytes = kTile * D * 2;
    static constexpr int kStageBytes = 2 * kKvTileBytes;
    static constexpr int kQBytes = kRows * D * 2;
    static constexpr int kNewBytes = 2 * D * 2;            // the step's new K row and V row of the item's stream
    static constexpr int kQSlotBytes = kQBytes + kNewBytes;
    static constexpr int kMoStride = D + 4;
    static constexpr int kMergeFloats = kConsumerWarps * kRows * kMoStride;
    static constexpr int kMlFloats = kConsumerWarps * kRows * 2;
    // merge buffers (+ their item headers), descriptor ring, barriers, flags
    static constexpr int kFixedBytes = kMergeBufs * ((kMergeFloats + kMlFloats) * 4 + 32) +
                                       kMaxQSlots * 32 + kNumBars * 8 + 64;
    static constexpr int kAlignSlack = 1024;
    static int smem_bytes(int stages, int q_slots) {
        return stages * kStageBytes + q_slots * kQSlotBytes + kFixedBytes + kAlignSlack;
    }
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// Log-sum-exp merge of the `ns` partial results of one (request, KV head) stream, slots
// [slot0, slot0+ns): out = sum_s o_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), M = max_s m_s.
// Thread `tid` of `nthreads` takes groups of four output elements of one query head.
// Partials are read through L2 (they may have been written by other SMs a moment ago).
template <typename T>
__device__ __forceinline__ void combine_stream(const float* part_o, const float* part_ml, int slot0,
                                               int ns, int req, int head, int group, int D,
                                               int q_heads, T* out, float* lse, int tid, int nthreads) {
    const int per_row = D >> 2;
    for (int idx = tid; idx < group * per_row; idx += nthreads) {
        const int r = idx / per_row, d0 = (idx - r * per_row) * 4;
        float M = -INFINITY, L = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int s = 0; s < ns; ++s) {
            const size_t prow = static_cast<size_t>(slot0 + s) * group + r;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + prow * 2));
            const float4 x = ldcg4(part_o + prow * D + d0);
            lse_fold(M, L, a, ml.x, ml.y, x);
        }
        const float inv = fast_rcp(L);
        const size_t row = static_cast<size_t>(req) * q_heads + static_cast<size_t>(head) * group + r;
        store4(out + row * D + d0, a.x * inv, a.y * inv, a.z * inv, a.w * inv);
        if (d0 == 0 && lse) lse[row] = (M + fast_log2(L)) * 0.6931471805599453f;
    }
}

template <int D, int NT, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ TensorMaps tm, const DecodeParams p,
                 const __grid_constant__ InlineLens lens) {
    using Cfg = TcConfig<D, NT>;
    constexpr int ROWS = Cfg::kRows;
    constexpr int HALVES = D / 64;                 // 128-byte column blocks per row
    constexpr int HALF_BYTES = kTile * 128;
    constexpr int MO = Cfg::kMoStride;
    const uint32_t STAGES = static_cast<uint32_t>(p.stages);
    const uint32_t QSLOTS = static_cast<uint32_t>(p.q_slots);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* kv = smem;
    uint8_t* qbuf = kv + STAGES * Cfg::kStageBytes;
    float* mrg_o = reinterpret_cast<float*>(qbuf + QSLOTS * Cfg::kQSlotBytes);
    float* mrg_ml = mrg_o + kMergeBufs * Cfg::kMergeFloats;
    int* mrg_hdr = reinterpret_cast<int*>(mrg_ml + kMergeBufs * Cfg::kMlFloats);   // 8 ints per buffer
    int* desc = mrg_hdr + kMergeBufs * 8;                                           // 8 ints per slot
    uint64_t* bars = reinterpret_cast<uint64_t*>(desc + kMaxQSlots * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + kNumBars);
    volatile int* last_flag = abort_flag + 1;    // finishers: this CTA delivered a stream's last piece

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar0 + 8u * (kMaxStages + s); };
    auto qfull_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + s); };
    auto qempty_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + kMaxQSlots + s); };
    auto mready_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + 2 * kMaxQSlots + s); };
    auto mdone_bar = [&](uint32_t s) { return bar0 + 8u * (2 * kMaxStages + 2 * kMaxQSlots + kMergeBufs + s); };
    const uint32_t fstored_bar = bar0 + 8u * (2 * kMaxStages + 2 * kMaxQSlots + 2 * kMergeBufs);
    const uint32_t fcounted_bar = fstored_bar + 8u;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int64_t limit = p.wait_limit_ns;
    const int cta = blockIdx.x;

    // the producer's first loads are in flight while the barriers are being set up
    int4 rec = make_int4(0, 0, 0, 0), first_a = rec, first_b = rec;
    int4 mine_a = rec, mine_b = rec;                 // producer: descriptor of item `lane` of the CTA's current 32
    if (warp == kProducerWarp) {
        const int4* r = p.cta + 3 * cta;
        rec = __ldg(r);
        first_a = __ldg(r + 1);
        first_b = __ldg(r + 2);
        if (lane < 4)
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.box[lane])) : "memory");
    } else if (warp >= kFinisherWarp0 && lane == 0) {
        rec = __ldg(p.cta + 3 * cta);
    }
    if (tid < kNumBars) {                            // one barrier per thread
        constexpr uint32_t all_consumers = kConsumerGroups * kConsumerWarps;
        const uint32_t b = static_cast<uint32_t>(tid);
        const uint32_t count = b < kMaxStages                        ? 1u               // full
                               : b < 2 * kMaxStages                  ? all_consumers    // empty
                               : b < 2 * kMaxStages + kMaxQSlots     ? 1u               // query slot full
                               : b < 2 * kMaxStages + 2 * kMaxQSlots ? all_consumers    // query slot empty
                               : b < 2 * kMaxStages + 2 * kMaxQSlots + kMergeBufs
                                   ? static_cast<uint32_t>(kConsumerWarps)              // merge buffer ready
                                   : static_cast<uint32_t>(kFinisherWarps);             // done / stored / counted
        mbar_init(bar0 + 8u * b, count);
        if (tid == 0) {
            *abort_flag = 0;
            *last_flag = 0;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch.  Everything above (barrier set-up, the CTA's record from
    // the step's table, which no kernel writes) may run while the previous kernel of the stream
    // is still draining; so may the producer's early loads below.  Everything else comes after
    // the dependency wait.  The next kernel of the stream is let go only AFTER this wait: when
    // its CTAs run their own early part, the kernel before this one is then known to be
    // complete, so the only kernel a CTA can overlap with is its immediate predecessor.
    if (warp != kProducerWarp) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    const uint32_t kv_u32 = smem_u32(kv);
    const uint32_t q_u32 = smem_u32(qbuf);

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer
        // Every lane fetches item descriptors (32 at a time, one per lane) and works out its
        // item's rows; the values reach all lanes by shuffles.  Waits are taken by the whole
        // warp; lane 0 arms the barriers; a tile's copies (one per 128-byte column block of K
        // and of V) are issued by as many lanes at once, so are the copies of an item's
        // queries and new K / V rows: the time the warp spends per copy is what bounds the
        // rate of short items.
        const int it_begin = rec.x, it_end = rec.y;       // every lane read the record
        uint32_t issued_any = 0, issued_odd = 0;     // per stage: loads issued at all / an odd number
        bool ok = true;
        const int64_t k_array = static_cast<int64_t>(p.layer) * 2 * p.rows_per_array;
        const int64_t v_array = k_array + p.rows_per_array;
        constexpr int COPIES = 2 * HALVES;            // copies per box position: K and V, each column block

        // An item's rows as this step sees them.  A piece that ends its stream ends where the
        // stream ends NOW (the plan may be an earlier step's, made when the stream was a little
        // shorter).  With the append fused in, the stream's last token is not in the slab yet:
        // it is not streamed (a consumer warp takes it from k_new / v_new and writes it there).
        // `safe` = rows that no kernel still running can be writing: the previous kernel of the
        // stream (the only one that can overlap with this one) may be this kernel one step
        // earlier, whose new token is the stream's last row but one; the last row is this
        // step's own.
        struct Rows {
            int ntok, safe;
            bool has_new;
        };
        auto rows_of = [&](const int4& a, const int4& b) {
            Rows r;
            const bool ends = (b.x & 2) != 0;
            const int ntok_now = (lens.n > 0 && ends) ? lens.len[a.x] - a.z : a.w;
            r.has_new = p.k_new != nullptr && ends;
            r.ntok = ntok_now - (r.has_new ? 1 : 0);
            r.safe = ends ? ntok_now - 2 : ntok_now;
            return r;
        };
        // One tile of a slab stream = up to four groups of 16 rows, fetched with one copy per
        // 128-byte column block of K and of V (a box of 16, 32, 48 or 64 rows; never past
        // ceil16 of the stream's length).  part 0: the whole tile; part 1: only the groups that
        // lie wholly in the safe rows, with the barrier told to expect the whole tile; part 2:
        // the rest of a tile whose part 1 is under way.  Called by the whole warp.
        auto issue_slab_tile = [&](uint32_t stage, int64_t row, int t, int ntok, int safe, int part) {
            const int r0 = t * kTile;
            const int nb = (min(kTile, ntok - r0) + 15) >> 4;
            const int ge = min(nb, max(safe - r0, 0) >> 4);
            const int g0 = part == 2 ? ge : 0, g1 = part == 1 ? ge : nb;
            if (part != 2) {
                if (lane == 0) mbar_expect_tx(full_bar(stage), static_cast<uint32_t>(nb) * 16u * D * 2u * 2u);
                issued_any |= 1u << stage;
                issued_odd ^= 1u << stage;
                __syncwarp();
            }
            if (g1 <= g0 || lane >= COPIES) return;
            const int h = lane >> 1, kv = lane & 1;
            const uint32_t dst = kv_u32 + stage * Cfg::kStageBytes + kv * Cfg::kKvTileBytes + g0 * 2048 + h * HALF_BYTES;
            const int32_t y = static_cast<int32_t>((kv ? v_array : k_array) + row + r0 + g0 * 16);
            tma_load_2d(dst, &tm.box[g1 - g0 - 1], h * 64, y, full_bar(stage));
        };

        // descriptors of the CTA's first 32 items (the very first came with the record), each
        // lane's resolved on the spot: n_tokens becomes the rows to stream, the combine word's
        // place is kept, and the safe row count travels in a register of its own
        int mine_safe = 0;
        auto resolve_mine = [&]() {
            const Rows r = rows_of(mine_a, mine_b);
            mine_a.w = r.ntok;
            mine_safe = r.safe;
        };
        if (it_begin + lane < it_end) {
            mine_a = __ldg(p.items + 2 * (it_begin + lane));
            mine_b = __ldg(p.items + 2 * (it_begin + lane) + 1);
            resolve_mine();
        }
        const Rows first_r = rows_of(first_a, first_b);
        auto item_of = [&](int j, int4& a, int4& b, int& safe) {     // item held by lane j, to all lanes
            a.x = __shfl_sync(0xFFFFFFFFu, mine_a.x, j);
            a.y = __shfl_sync(0xFFFFFFFFu, mine_a.y, j);
            a.z = __shfl_sync(0xFFFFFFFFu, mine_a.z, j);
            a.w = __shfl_sync(0xFFFFFFFFu, mine_a.w, j);
            b.x = __shfl_sync(0xFFFFFFFFu, mine_b.x, j);
            b.y = __shfl_sync(0xFFFFFFFFu, mine_b.y, j);
            b.z = __shfl_sync(0xFFFFFFFFu, mine_b.z, j);
            b.w = __shfl_sync(0xFFFFFFFFu, mine_b.w, j);
            safe = __shfl_sync(0xFFFFFFFFu, mine_safe, j);
        };
        // Early start: the safe rows of the CTA's first tiles (one per pipeline stage) are
        // requested before the dependency wait, so that HBM is already streaming while the
        // previous grid finishes; queries, new tokens and the rows in flux come after it.
        int n_early = 0;
        if (MODE != kModePaged && p.early_ok) {
            for (int j = 0; j < 32 && it_begin + j < it_end && n_early < static_cast<int>(STAGES); ++j) {
                int4 a = first_a, b = first_b;
                int safe = first_r.safe;
                a.w = first_r.ntok;
                if (j > 0) item_of(j, a, b, safe);
                const int ntiles = (a.w + kTile - 1) / kTile;
                for (int t = 0; t < ntiles && n_early < static_cast<int>(STAGES); ++t, ++n_early)
                    issue_slab_tile(static_cast<uint32_t>(n_early), b.z, t, a.w, safe, 1);
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

        uint32_t stage = 0, phase = 0, qs = 0, qphase = 0;
        int n_tile = 0;                               // tiles issued so far (the first n_early only need their rest)
        for (int it = it_begin;; ++it) {
            const int j = (it - it_begin) & 31;
            if (j == 0 && it != it_begin && it + lane < it_end) {
                mine_a = __ldg(p.items + 2 * (it + lane));
                mine_b = __ldg(p.items + 2 * (it + lane) + 1);
                resolve_mine();
            }
            int4 a = first_a, b = first_b;
            int safe = first_r.safe;
            a.w = first_r.ntok;
            if (it != it_begin) item_of(j, a, b, safe);
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(qempty_bar(qs), qphase ^ 1u, abort_flag, p.status, limit));
            if (!ok) break;
            int* dsc = desc + qs * 8;
            if (it >= it_end) {                          // end marker
                if (lane == 0) {
                    dsc[6] = 0;
                    mbar_arrive(qfull_bar(qs));
                }
                break;
            }
            const int req = a.x, head = a.y, tok0 = a.z, ntok = a.w;
            const bool has_new = p.k_new != nullptr && (b.x & 2);
            const uint32_t q_bytes = static_cast<uint32_t>(p.group) * D * 2u;
            if (lane == 0) {
                dsc[0] = req;
                dsc[1] = head;
                dsc[2] = ntok;
                dsc[3] = b.x & 1;                        // direct
                dsc[4] = b.y;                            // slot
                dsc[5] = b.w;                            // combine record
                dsc[6] = 1;                              // a real item
                dsc[7] = has_new ? b.z + ntok : -1;      // pool row of the new token
                mbar_expect_tx(qfull_bar(qs), q_bytes + (has_new ? Cfg::kNewBytes : 0));
            }
            __syncwarp();
            if (lane == 0) {
                bulk_load(q_u32 + qs * Cfg::kQSlotBytes,
                          static_cast<const uint8_t*>(p.q) +
                              (static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * p.group) * D * 2,
                          q_bytes, qfull_bar(qs));
            } else if (lane < 3 && has_new) {            // the new token's K and V rows ride behind the queries
                const size_t nrow = (static_cast<size_t>(req) * p.kv_heads + head) * D * 2;
                const uint8_t* src = static_cast<const uint8_t*>(lane == 1 ? p.k_new : p.v_new) + nrow;
                bulk_load(q_u32 + qs * Cfg::kQSlotBytes + Cfg::kQBytes + (lane - 1) * D * 2, src, D * 2, qfull_bar(qs));
            }
            if (++qs == QSLOTS) {
                qs = 0;
                qphase ^= 1u;
            }
            const int64_t row = b.z;
            const int ntiles = (ntok + kTile - 1) / kTile;
            for (int t = 0; t < ntiles; ++t, ++n_tile) {
                if (n_tile < n_early) {                  // first use of the stage, part 1 under way
                    issue_slab_tile(stage, row, t, ntok, safe, 2);
                } else {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, limit));
                    if (!ok) break;
                    if (MODE != kModePaged) {
                        issue_slab_tile(stage, row, t, ntok, safe, 0);
                    } else {                             // one 16-row box per page, all of them at once
                        const int nb = (min(kTile, ntok - t * kTile) + 15) >> 4;
                        if (lane == 0) mbar_expect_tx(full_bar(stage), static_cast<uint32_t>(nb) * 16u * D * 2u * 2u);
                        issued_any |= 1u << stage;
                        issued_odd ^= 1u << stage;
                        __syncwarp();
                        const int bx = lane / COPIES, w = lane - bx * COPIES;
                        if (bx < nb) {
                            const int h = w >> 1, kv = w & 1;
                            const int32_t page = p.page_table[static_cast<size_t>(req) * p.max_pages + tok0 / 16 + t * 4 + bx];
                            const int64_t prow = (static_cast<int64_t>(page) * p.kv_heads + head) * 16;
                            tma_load_2d(kv_u32 + stage * Cfg::kStageBytes + kv * Cfg::kKvTileBytes + h * HALF_BYTES + bx * 2048,
                                        &tm.box[0], h * 64, static_cast<int32_t>((kv ? v_array : k_array) + prow),
                                        full_bar(stage));
                        }
                    }
                }
                if (++stage == STAGES) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (!ok) break;
        }
        if (lane == 0 && !ok) {
            // Something timed out.  Before the CTA's shared memory can be handed to another
            // CTA, wait (bounded, ignoring the abort flag) for the loads already in flight.
            for (uint32_t s = 0; s < STAGES; ++s)
                if ((issued_any >> s) & 1u)      // parity of the stage's latest phase
                    mbar_wait_slow(full_bar(s), ((issued_odd >> s) & 1u) ^ 1u, nullptr, p.status,
                                   limit / 4 + 1);
        }
        return;
    }

    if (warp >= kFinisherWarp0) {
        // ------------------------------------------------------------------ finishers
        if (MODE == kModeProbe) return;
        const int ftid = tid - kFinisherWarp0 * 32;
        constexpr int fthreads = kFinisherThreads;
        const int n_items = __shfl_sync(0xFFFFFFFFu, rec.y - rec.x, 0);
        const int group = p.group;
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
        constexpr int PER_ROW = D / 4;                   // float4 chunks per head
        const int total = group * PER_ROW;
        // CH = chunks of four output elements per thread; every thread computes CH chunks
        // (indices past the end are clamped, their results dropped) so the code is branch-free
        constexpr int CH = (ROWS * PER_ROW + kFinisherThreads - 1) / kFinisherThreads;
        {
            uint32_t n_split = 0;
            uint32_t handed = 0;                         // per merge buffer: parity of its next hand-over
            for (int k = 0; k < n_items; ++k) {
                // the item's start group first, then (long streams) the other one
                const uint32_t g0 = static_cast<uint32_t>(k) & 1u;
                if (!mbar_wait(mready_bar(g0), (handed >> g0) & 1u, abort_flag, p.status, limit)) return;
                handed ^= 1u << g0;
                const int* hdr = mrg_hdr + g0 * 8;
                const int req = hdr[0], head = hdr[1], direct = hdr[2], slot = hdr[3], comb = hdr[4];
                const int parts = hdr[5] ? 2 : 1;
                const bool count_in = !direct && p.counters != nullptr;
                int4 cr = make_int4(0, 0, 0, 0);         // {request, head, first slot, pieces}
                if (count_in) cr = __ldg(p.combine + comb);
                float4 acc[CH];
                float acc_m[CH], acc_l[CH];
                int rr[CH], dd[CH];
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    const int idx = min(ftid + i * fthreads, total - 1);
                    rr[i] = idx / PER_ROW;
                    dd[i] = (idx - rr[i] * PER_ROW) * 4;
                    acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    acc_m[i] = -INFINITY;
                    acc_l[i] = 0.f;
                }
                for (int part = 0; part < parts; ++part) {
                    const uint32_t g = g0 ^ static_cast<uint32_t>(part);
                    if (part == 1) {
                        if (!mbar_wait(mready_bar(g), (handed >> g) & 1u, abort_flag, p.status, limit)) return;
                        handed ^= 1u << g;
                    }
                    const float* bo = mrg_o + g * Cfg::kMergeFloats;
                    const float* bml = mrg_ml + g * Cfg::kMlFloats;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {      // a warp without keys left max = -inf
#pragma unroll
                        for (int i = 0; i < CH; ++i) {
                            const float2 ml = *reinterpret_cast<const float2*>(bml + (w * ROWS + rr[i]) * 2);
                            const float4 x = *reinterpret_cast<const float4*>(bo + (w * ROWS + rr[i]) * MO + dd[i]);
                            lse_fold(acc_m[i], acc_l[i], acc[i], ml.x, ml.y, x);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(mdone_bar(g));        // the buffer may be refilled
                }
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    if (ftid + i * fthreads >= total) continue;
                    const int r = rr[i], d0 = dd[i];
                    if (direct) {
                        const float inv = fast_rcp(acc_l[i]);
                        const size_t row = static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * group + r;
                        store4(out + row * D + d0, acc[i].x * inv, acc[i].y * inv, acc[i].z * inv, acc[i].w * inv);
                        if (d0 == 0 && p.lse) p.lse[row] = (acc_m[i] + fast_log2(acc_l[i])) * 0.6931471805599453f;
                    } else {
                        const size_t prow = static_cast<size_t>(slot) * group + r;
                        *reinterpret_cast<float4*>(p.part_o + prow * D + d0) = acc[i];
                        if (d0 == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(acc_m[i], acc_l[i]);
                    }
                }
                __syncwarp();
                if (lane == 0 && count_in) mbar_arrive(fstored_bar);
                if (!count_in) continue;
                // The CTA that delivers a split stream's last piece merges all of them.  Once
                // every finisher thread has issued its partial stores, one thread fences them,
                // counts this piece in and tells the rest whether the count is complete; if so
                // each thread folds all pieces in slot order, its own from the registers it
                // still holds, the others read back through L2.
                if (!mbar_wait(fstored_bar, n_split & 1u, abort_flag, p.status, limit)) return;
                if (ftid == 0) {
                    __threadfence();
                    const uint32_t seen = atomicAdd(p.counters + comb, 1u);
                    const int last = seen + 1u == static_cast<uint32_t>(cr.w);
                    if (last) p.counters[comb] = 0u;      // ready for the next launch
                    *last_flag = last;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(fcounted_bar);
                if (!mbar_wait(fcounted_bar, n_split & 1u, abort_flag, p.status, limit)) return;
                ++n_split;
                if (!*last_flag) continue;
                __threadfence();
                const size_t orow0 = static_cast<size_t>(cr.x) * p.q_heads + static_cast<size_t>(cr.y) * group;
                float fm[CH], fl[CH];
                float4 fa[CH];
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    fm[i] = -INFINITY;
                    fl[i] = 0.f;
                    fa[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                for (int s = 0; s < cr.w; ++s) {
                    if (cr.z + s == slot) {               // this CTA's own piece
#pragma unroll
                        for (int i = 0; i < CH; ++i) lse_fold(fm[i], fl[i], fa[i], acc_m[i], acc_l[i], acc[i]);
                        continue;
                    }
                    float2 ml[CH];
                    float4 x[CH];
#pragma unroll
                    for (int i = 0; i < CH; ++i) {        // all loads of the piece first
                        const size_t prow = static_cast<size_t>(cr.z + s) * group + rr[i];
                        ml[i] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + prow * 2));
                        x[i] = ldcg4(p.part_o + prow * D + dd[i]);
                    }
#pragma unroll
                    for (int i = 0; i < CH; ++i) lse_fold(fm[i], fl[i], fa[i], ml[i].x, ml[i].y, x[i]);
                }
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    if (ftid + i * fthreads >= total) continue;
                    const float inv = fast_rcp(fl[i]);
                    store4(out + (orow0 + rr[i]) * D + dd[i], fa[i].x * inv, fa[i].y * inv, fa[i].z * inv, fa[i].w * inv);
                    if (dd[i] == 0 && p.lse) p.lse[orow0 + rr[i]] = (fm[i] + fast_log2(fl[i])) * 0.6931471805599453f;
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int qd = lane >> 2, qt = lane & 3;          // row within 8, position within the quad
    const int mi = lane >> 3, r8 = lane & 7;          // ldmatrix: matrix id, row within it
    // K tile as the A operand: matrices (keys 0-7, d 0-7) (keys 8-15, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 8-15)
    const int cw = warp & (kConsumerWarps - 1);       // warp within its group
    const uint32_t grp = static_cast<uint32_t>(warp) / kConsumerWarps;
    const uint32_t k_lane_off = (cw * 16 + (mi & 1) * 8 + r8) * 128;
    const uint32_t xk = (mi >> 1) ^ r8;
    // V tile, transposed on load, as the A operand: (keys 0-7, d 0-7) (keys 0-7, d 8-15) (keys 8-15, d 0-7) (keys 8-15, d 8-15)
    const uint32_t v_lane_off = (cw * 16 + (mi >> 1) * 8 + r8) * 128;
    const uint32_t xv = (mi & 1) ^ r8;
    // Q as the B operand: four consecutive 16-byte chunks of head r8
    const uint32_t q_lane_off = r8 * (D * 2) + mi * 16;
    const int key_lo = cw * 16 + qd;                // the thread's two key rows: key_lo, key_lo + 8
    const int vkey0 = cw * 16 + qt * 2;             // keys of its value fragments: vkey0, +1, +8, +9
    const float scale = p.scale_log2;

    uint32_t stage = 0, phase = 0, qs = 0, qphase = 0;
    uint32_t n_dep = 0;                               // partial results this group has left for the finishers
    bool ok = true;
    for (uint32_t k_item = 0; ok; ++k_item) {
        ok = mbar_wait(qfull_bar(qs), qphase, abort_flag, p.status, limit);
        if (!ok) break;
        const int* dsc = desc + qs * 8;
        const int req = dsc[0], head = dsc[1], ntok = dsc[2], direct = dsc[3], slot = dsc[4], comb = dsc[5];
        const int new_row = dsc[7];
        if (dsc[6] == 0) break;
        const int ntiles = (ntok + kTile - 1) / kTile;
        // Items go to the two groups in turn: while one group hands an item over and starts its
        // next one, the other is in the middle of its own.  A long stream is worked on by both
        // groups, its tiles going to them in turn from the start group (two tiles in flight:
        // there the hand-over is a small part, and the tile rate is what counts).
        const bool starts = (k_item & 1u) == grp;
        const bool both = ntiles >= kBothGroupsTiles;
        if (!starts && !both) {
            // Nothing of this item is this group's: let go of the slot and walk over its tiles in step with
            // the ring.  A barrier's parity tells apart only two consecutive phases, so neither
            // group may fall a whole phase behind or run one ahead of any stage: every warp of
            // both groups waits for each tile to land and signs the stage off, the owners after
            // using it, the others at once.
            __syncwarp();
            if (lane == 0) mbar_arrive(qempty_bar(qs));
            if (++qs == QSLOTS) {
                qs = 0;
                qphase ^= 1u;
            }
            for (int t = 0; t < ntiles; ++t) {
                ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, limit);
                if (!ok) break;
                if (lane == 0) mbar_arrive(empty_bar(stage));
                if (++stage == STAGES) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            continue;
        }

        uint32_t qb[NT][D / 16][2];
        if (MODE != kModeProbe) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int j = 0; j < D / 32; ++j) {
                    uint32_t r[4];
                    ldmatrix_x4(r, q_u32 + qs * Cfg::kQSlotBytes + nt * 8 * (D * 2) + q_lane_off + j * 64);
                    qb[nt][2 * j][0] = r[0];
                    qb[nt][2 * j][1] = r[1];
                    qb[nt][2 * j + 1][0] = r[2];
                    qb[nt][2 * j + 1][1] = r[3];
                }
        }
        float o[NT][D / 16][4];
        float m_run[NT][2], l_run[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int i = 0; i < D / 16; ++i) o[nt][i][0] = o[nt][i][1] = o[nt][i][2] = o[nt][i][3] = 0.f;
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
        }
        // (which warp: the group's last one when the stream is so short that this warp has no keys
        // of its own, 48 tokens or fewer; else the first)
        const int new_cw = ntok <= kTile - 16 ? kConsumerWarps - 1 : 0;
        if (MODE == kModeSlab && new_row >= 0 && cw == new_cw && starts) {
            // The token appended this step (the piece ends its stream and the append is fused
            // in): its K and V rows sit behind the queries in the slot.  The group's first warp
            // starts from it instead of from nothing: running maximum = its score, sum = 1,
            // output = its value row; and it writes the two rows into the slab for the steps
            // to come.  Each lane holds, of head qd, elements kk*16 + 2qt + {0, 1, 8, 9} of the
            // query: it adds up its part of the score, the quad completes it.
            const uint8_t* nk = qbuf + qs * Cfg::kQSlotBytes + Cfg::kQBytes;
            const uint8_t* nv = nk + D * 2;
            float dot[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) dot[nt] = 0.f;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t k0 = *reinterpret_cast<const uint32_t*>(nk + (kk * 16 + qt * 2) * 2);
                const uint32_t k1 = *reinterpret_cast<const uint32_t*>(nk + (kk * 16 + qt * 2 + 8) * 2);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint32_t q0 = qb[nt][kk][0], q1 = qb[nt][kk][1];
                    dot[nt] = fmaf(__uint_as_float(q0 << 16), __uint_as_float(k0 << 16), dot[nt]);
                    dot[nt] = fmaf(__uint_as_float(q0 & 0xFFFF0000u), __uint_as_float(k0 & 0xFFFF0000u), dot[nt]);
                    dot[nt] = fmaf(__uint_as_float(q1 << 16), __uint_as_float(k1 << 16), dot[nt]);
                    dot[nt] = fmaf(__uint_as_float(q1 & 0xFFFF0000u), __uint_as_float(k1 & 0xFFFF0000u), dot[nt]);
                }
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                dot[nt] += __shfl_xor_sync(0xFFFFFFFFu, dot[nt], 1);
                dot[nt] += __shfl_xor_sync(0xFFFFFFFFu, dot[nt], 2);
                // the accumulator columns of this lane are heads 2qt and 2qt + 1
                m_run[nt][0] = __shfl_sync(0xFFFFFFFFu, dot[nt], qt * 8) * scale;
                m_run[nt][1] = __shfl_sync(0xFFFFFFFFu, dot[nt], qt * 8 + 4) * scale;
                l_run[nt][0] = l_run[nt][1] = qd == 0 ? 1.f : 0.f;      // summed over qd when the item ends
#pragma unroll
                for (int dt = 0; dt < D / 16; ++dt) {
                    const uint32_t lo = *reinterpret_cast<const uint16_t*>(nv + (dt * 16 + qd) * 2);
                    const uint32_t hi = *reinterpret_cast<const uint16_t*>(nv + (dt * 16 + qd + 8) * 2);
                    o[nt][dt][0] = o[nt][dt][1] = __uint_as_float(lo << 16);
                    o[nt][dt][2] = o[nt][dt][3] = __uint_as_float(hi << 16);
                }
            }
            constexpr int ROW_VECS = D * 2 / 16;
            if (lane < 2 * ROW_VECS) {                   // K row, then V row, 16 bytes per lane
                const int kv = lane / ROW_VECS, vec = lane - kv * ROW_VECS;
                uint4* dst = reinterpret_cast<uint4*>(const_cast<void*>(p.pool)) +
                             ((static_cast<int64_t>(p.layer) * 2 + kv) * p.rows_per_array + new_row) * ROW_VECS + vec;
                *dst = *reinterpret_cast<const uint4*>(nk + lane * 16);
            }
        }
        // The slot is refilled by a bulk copy (async proxy) the moment its last reader lets go of it;
        // the reads above went through the generic proxy.  The cross-proxy fence orders them
        // before the arrive that licenses the refill.
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(qempty_bar(qs));
        if (++qs == QSLOTS) {
            qs = 0;
            qphase ^= 1u;
        }

        for (int t = 0; t < ntiles; ++t) {
            ok = mbar_wait(full_bar(stage), phase, abort_flag, p.status, limit);
            if (!ok) break;
            const int valid = min(kTile, ntok - t * kTile);
            const bool mine = !both || ((t & 1) == 0) == starts;     // of a shared stream, even tiles are the start group's
            if (MODE != kModeProbe && mine && cw * 16 < valid) {
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
                    const float corr0 = fast_exp2(m_run[nt][0] - mu0), corr1 = fast_exp2(m_run[nt][1] - mu1);
                    const float p0 = fast_exp2(fmaf(c0, scale, -mu0)), p1 = fast_exp2(fmaf(c1, scale, -mu1));
                    const float p2 = fast_exp2(fmaf(c2, scale, -mu0)), p3 = fast_exp2(fmaf(c3, scale, -mu1));
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
            if (++stage == STAGES) {
                stage = 0;
                phase ^= 1u;
            }
        }
        if (!ok) break;
        if (MODE == kModeProbe) continue;

        // ---- hand the warp's partial result to the finishers and move on
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l_run[nt][0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[nt][0], off);
                l_run[nt][1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[nt][1], off);
            }
        const uint32_t mb = grp;                      // each group has its own buffer
        if (n_dep > 0) {                              // the finishers are done with what the group left there last
            ok = mbar_wait(mdone_bar(mb), (n_dep - 1u) & 1u, abort_flag, p.status, limit);
            if (!ok) break;
        }
        ++n_dep;
        float* mo = mrg_o + mb * Cfg::kMergeFloats + cw * ROWS * MO;
        float* mml = mrg_ml + mb * Cfg::kMlFloats + cw * ROWS * 2;
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
        if (cw == 0 && lane == 0) {
            int* hdr = mrg_hdr + mb * 8;
            hdr[0] = req;
            hdr[1] = head;
            hdr[2] = direct;
            hdr[3] = slot;
            hdr[4] = comb;
            hdr[5] = both;                            // the other group leaves a partial result too
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(mready_bar(mb));
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
        const int req = a.x, head = a.y, tok0 = a.z, ntok = a.w, direct = b.x & 1, slot = b.y;
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

template <bool QUANT>
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
        if (QUANT) {
            // a stored vector of 16 codes comes from two vectors of eight bf16 numbers
            const float inv = kv ? p.v_inv : p.k_inv;
            const uint2 a = quantize8_e4m3(src[2 * rem], inv), b = quantize8_e4m3(src[2 * rem + 1], inv);
            pool[(array * p.rows_per_array + row) * p.row_vecs + vec] = make_uint4(a.x, a.y, b.x, b.y);
        } else {
            pool[(array * p.rows_per_array + row) * p.row_vecs + vec] = src[rem];
        }
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
cudaError_t launch_tc_inst(const TensorMaps& maps, const DecodeParams& p, int n_ctas, cudaStream_t stream,
                           const InlineLens& lens) {
    using Cfg = TcConfig<D, NT>;
    static bool configured[64] = {false};          // the opt-in to large shared memory is per device
    auto kern = decode_tc_kernel<D, NT, MODE>;
    const int smem = Cfg::smem_bytes(p.stages, p.q_slots);
    if (p.stages < 2 || p.stages > kMaxStages || p.q_slots < kMinQSlots || p.q_slots > kMaxQSlots ||
        smem > kSmemPerCtaMax)
        return cudaErrorInvalidValue;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCtaMax);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas));
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(smem);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, maps, p, lens);
}

template <int D, int NT>
cudaError_t launch_tc_mode(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas, cudaStream_t s,
                           const InlineLens& lens) {
    switch (mode) {
        case kModeSlab: return launch_tc_inst<D, NT, kModeSlab>(maps, p, n_ctas, s, lens);
        case kModePaged: return launch_tc_inst<D, NT, kModePaged>(maps, p, n_ctas, s, lens);
        case kModeProbe: return launch_tc_inst<D, NT, kModeProbe>(maps, p, n_ctas, s, lens);
    }
    return cudaErrorInvalidValue;
}

// Pipeline depth and query-ring depth that fit when `ctas_per_sm` CTAs share an SM: as many
// stages as possible on top of the smallest ring, then the ring grows into what is left.
template <int D, int NT>
void tc_shape_inst(int32_t ctas_per_sm, int32_t* stages, int32_t* q_slots) {
    using Cfg = TcConfig<D, NT>;
    const int budget = std::min(kSmemPerSm / ctas_per_sm - kSmemCtaReserve, kSmemPerCtaMax);
    const int room = budget - Cfg::kFixedBytes - Cfg::kAlignSlack - kMinQSlots * Cfg::kQSlotBytes;
    int n = room / Cfg::kStageBytes;
    n = n > kMaxStages ? kMaxStages : n;
    if (n < 2) {
        *stages = *q_slots = 0;
        return;
    }
    const int extra = (room - n * Cfg::kStageBytes) / Cfg::kQSlotBytes;
    *stages = n;
    *q_slots = std::min(kMaxQSlots, kMinQSlots + extra);
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

void tc_shape(int32_t head_dim, int32_t group, int32_t* stages, int32_t* q_slots) {
    const int32_t ctas_per_sm = 1;
    *stages = *q_slots = 0;
    if (!tc_supported(head_dim, group)) return;
    const bool two = group > 8;
    if (head_dim == 128)
        two ? tc_shape_inst<128, 2>(ctas_per_sm, stages, q_slots) : tc_shape_inst<128, 1>(ctas_per_sm, stages, q_slots);
    else
        two ? tc_shape_inst<64, 2>(ctas_per_sm, stages, q_slots) : tc_shape_inst<64, 1>(ctas_per_sm, stages, q_slots);
}

cudaError_t launch_decode_tc(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                             cudaStream_t stream, const InlineLens* lens_in) {
    static const InlineLens no_lens{};                 // n = 0: lengths as planned
    const InlineLens& lens = lens_in ? *lens_in : no_lens;
    const bool two = p.group > 8;
    if (p.head_dim == 128)
        return two ? launch_tc_mode<128, 2>(maps, p, mode, n_ctas, stream, lens)
                   : launch_tc_mode<128, 1>(maps, p, mode, n_ctas, stream, lens);
    if (p.head_dim == 64)
        return two ? launch_tc_mode<64, 2>(maps, p, mode, n_ctas, stream, lens)
                   : launch_tc_mode<64, 1>(maps, p, mode, n_ctas, stream, lens);
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
    if (p.quantize)
        append_kv_kernel<true><<<grid, 256, 0, stream>>>(p);
    else
        append_kv_kernel<false><<<grid, 256, 0, stream>>>(p);
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
