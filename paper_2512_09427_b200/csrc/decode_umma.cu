// Split decode attention on the fifth-generation tensor cores (tcgen05 / tensor memory): bf16
// slabs, and slabs of E4M3 codes (one byte per element) with bf16 queries and output.
//
// Same contract as decode_tc_kernel (kernels.cu): persistent CTAs walk the items of the
// host-built plan; an item is a run of tokens of one (request, KV head) stream; K and V tiles
// of 64 tokens arrive by TMA in the 128-byte-swizzled layout.  Here the two products of a tile
// are issued as tcgen05.mma instructions that read K, V, Q and P straight from shared memory
// and accumulate in tensor memory:
//     S[heads x 64 keys] = Q[heads x D]   . K[64 keys x D]^T      A, B K-major
//     O[heads x D]      += P[heads x 64]  . V[64 keys x D]        A K-major, B MN-major
// The GQA group's query heads are the first rows of an M = 64 operand.  A row of the result
// depends on that row of A only, so the other rows of the A descriptors (whatever shared memory
// follows the real rows) cost nothing but tensor throughput, of which this path uses little.
// With M = 64, rows 0..15 of an accumulator live in lanes 0..15 of tensor memory, which warps
// 0 and 4 of a CTA can read.
//
// Two items are in flight per CTA ("lanes": items go to them in turn), each with its own
// softmax warp, two S buffers and one O accumulator in tensor memory and two P buffers in
// shared memory, so one item's hand-over runs under the other's streaming.  Warp roles:
//     0, 4   (0, 5 in the late-read-out variant, whose second products of lane 0 are issued by warp 4)
//            softmax + finish of lane 0 / 1: S from tensor memory (one thread holds 16 keys of
//            one head), masking, running reference maximum, P = 2^(s - m) to shared memory; on
//            an item's last tile the value rows between the item's end and the next multiple of
//            16 are zeroed (the second product runs over whole groups of 16 keys); when the item
//            ends, O from tensor memory, normalise, write out (or leave a partial result and,
//            for the last piece of a split stream, merge all pieces).  With the append fused in,
//            the step's new token never enters the tensor-core path: its score is a dot product
//            on the plain ALUs and its value row is added when the item ends.
//     2      MMA issue of the first products, both lanes, in ring order (one elected lane of the
//            converged warp); S(t+1) is issued as soon as S(t-1) has been read out, so the
//            softmax of the next tile overlaps the second product of this one
//     5, 6   MMA issue of the second products of lane 0 / 1; tcgen05.commit releases pipeline
//            stages, query slots and buffers
//     1      producer: TMA loads of K/V tiles into the stage ring
//     3      query loader: the group's query rows, global -> swizzled shared memory; the step's
//            new K/V rows to a side buffer and into the slab
//
// A parity wait can tell apart only the current phase of a barrier and the one before, so every
// barrier here is waited on, phase after phase, by ONE role that sees each of its phases: the
// stage ring by warp 2 (which therefore issues the first products in ring order), the per-lane
// barriers by that lane's softmax warp, by warp 2 or by the lane's second-product warp, a query
// slot (slot = item number mod 8, so a slot always serves the same lane) by warp 2 and that
// lane's softmax warp.  Roles that need ring positions (which stage a tile sits in) count tiles
// over the CTA's whole item list.
//
// The softmax keeps a reference m per head that is the maximum seen when the item started and
// is raised only when a tile's maximum exceeds it by more than 2^8: P stays below 256, which
// bf16 and the fp32 accumulator hold without loss, and the accumulator in tensor memory is
// rescaled (read, multiplied, written back) only on that rare path.  (m, l, O) with such a
// reference is a valid partial result for the log-sum-exp merge.
//
// 8-bit slabs (F8): K and V tiles are E4M3 codes, 128 bytes per row, and both products are
// kind::f8f6f4 instructions (E4M3 x E4M3, fp32 accumulation, K = 32), so the A operands must be
// E4M3 as well.  Neither the queries nor the probabilities are rounded to 3 mantissa bits for
// that: each is split into two E4M3 terms, x = hi + lo / 16, which occupy rows h and h + 8 of
// the A operand (at most 8 heads per group), and the two result rows are added when they are
// read from tensor memory (one thread holds rows h and h + 8 of its columns).  A bf16 query
// times a power of two that brings its row's largest element into [128, 256) splits exactly
// (8 significant bits = 4 + 4); a probability splits with a relative error of 2^-8, what
// rounding it to bf16 costs the 16-bit kernel.  Probabilities are kept below 16 (reference
// raised when a tile's maximum passes it by 2^4) and multiplied by 16 before the split, so
// that the small ones stay normal numbers.  The key scale goes into the score factor, the
// value scale onto the result; the step's new token is quantised by the query loader (codes to
// the slab and to the side buffer) and used, like every other token, as its code's value.
#include <algorithm>

#include "device_utils.cuh"
#include "odma.h"

namespace odma {
namespace {

using namespace dev;

constexpr int kTile = 64;
constexpr int kUmmaWarps = 8;
constexpr int kUmmaThreads = kUmmaWarps * 32;
constexpr int kMaxStages = 12;
constexpr int kQSlots = 8;
constexpr int kLanes = 2;
constexpr int kBothTiles = 4;             // 8-bit slabs: items of this many tiles or more are worked on by both lanes
constexpr float kRescaleAbove = 8.f;      // log2 units a tile's maximum may pass the reference by (16-bit slabs)
constexpr float kRescaleAbove8 = 4.f;     // 8-bit slabs: P < 16
constexpr int kMaxStages16 = 8;           // stage-ring depth limits: 16-bit slabs / 8-bit slabs (kMaxStages)

// barrier indices
constexpr int kBarFull = 0, kBarEmpty = kMaxStages;
constexpr int kBarQFull = 2 * kMaxStages, kBarQEmpty = kBarQFull + kQSlots;
constexpr int kBarLane0 = kBarQEmpty + kQSlots;
constexpr int kBarPerLane = 12;           // s_full[2] s_empty[2] p_full[2] p_empty[2] o_full o_empty x_full x_empty
constexpr int kBarDrain = kBarLane0 + kLanes * kBarPerLane;
constexpr int kNumBars = kBarDrain + 3;

constexpr int kTmemCols = 512;            // all of it: one CTA per SM
constexpr int kTmemLaneCols = 256;        // per lane: S0 at +0, S1 at +64, O at +128

template <int D, int NT, bool F8>
struct UmmaConfig {
    static constexpr int kElem = F8 ? 1 : 2;               // bytes of a stored K/V element
    static constexpr int kRowGroups = F8 ? 2 : NT;         // groups of 8 rows of the A operands (F8: hi and lo terms)
    static constexpr int kHalves = D * kElem / 128;        // 128-byte column blocks per row
    static constexpr int kKvTileBytes = kTile * D * kElem;
    static constexpr int kStageBytes = 2 * kKvTileBytes;
    static constexpr int kQHalfBytes = kRowGroups * 1024;  // rows of 128 bytes
    static constexpr int kQSlotBytes = kHalves * kQHalfBytes;
    static constexpr int kPBufBytes = kRowGroups * 1024;   // rows of 64 keys (F8: 64 of a row's 128 bytes used)
    static constexpr int kPBytes = kLanes * 2 * kPBufBytes;
    static constexpr int kQBytes = kQSlots * kQSlotBytes;
    // the step's new K row and V row of an item's stream (as stored); F8: and the score factor of each head
    static constexpr int kNewBytes = 2 * D * kElem + (F8 ? 64 : 0);
    static constexpr int kNewBufBytes = ((kQSlots * kNewBytes + 1023) / 1024) * 1024;
    static constexpr int kXchgBytes = kLanes * 16 * 2 * 4;  // per lane and head: (reference maximum, sum) of a helper lane
    static constexpr int kTailBytes = kNumBars * 8 + 64 + kXchgBytes;
    static constexpr int kAlignSlack = 1024;
    static constexpr int kStagesMax = F8 ? kMaxStages : kMaxStages16;
    static int smem_bytes(int stages) {
        return kNewBufBytes + kPBytes + kQBytes + stages * kStageBytes + kTailBytes + kAlignSlack;
    }
};

// ---- tcgen05 wrappers -------------------------------------------------------------------------

// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, A K-major.
__host__ __device__ constexpr uint32_t umma_idesc(int m, int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

// Instruction descriptor of kind::f8f6f4: fp32 accumulator, E4M3 A and B (format 0), A K-major.
__host__ __device__ constexpr uint32_t umma_idesc8(int m, int n, bool b_mn_major) {
    return (1u << 4) | (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(m >> 4) << 24);
}

template <bool F8>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    if (F8)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(d_tmem),
            "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(d_tmem),
            "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
}

// The barrier receives one arrival once every tcgen05.mma this thread has issued is complete.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 lanes x 64 columns of 32 bits: lane t of the warp receives, in register 4i + j, row
// t/4 + 8 (j/2), column 8i + 2 (t%4) + (j%2) (the accumulator layout of m16n8 tiles, repeated
// along the columns).
__device__ __forceinline__ void tmem_ld_x8(uint32_t addr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr)
        : "memory");
}
// 16 lanes x 32 columns
__device__ __forceinline__ void tmem_ld_x4(uint32_t addr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(addr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_x4(uint32_t addr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(addr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- items ------------------------------------------------------------------------------------

// What an item of the plan means in this step.  A piece that ends its stream ends where the
// stream ends NOW (the plan may be an earlier step's, made when the stream was a little
// shorter).  With the append fused in, the stream's last token is not in the slab yet: it is
// not streamed; the softmax warp takes it from k_new / v_new.
struct Item {
    int req, head, tok0;
    int n_slab;       // rows streamed from the slab
    int tiles;        // ceil(n_slab / 64); 0 when the item is nothing but the new token
    int safe;         // rows of the piece that no kernel still running can be writing
    int row0;         // first row of the piece inside one K (or V) array of the pool
    int direct, slot, comb;
    bool has_new;
};

__device__ __forceinline__ Item item_of(const int4& a, const int4& b, const InlineLens& lens, bool fused) {
    Item it;
    const bool ends = (b.x & 2) != 0;
    it.req = a.x;
    it.head = a.y;
    it.tok0 = a.z;
    const int n_keys = (lens.n > 0 && ends) ? lens.len[a.x] - a.z : a.w;
    it.has_new = fused && ends;
    it.n_slab = n_keys - (it.has_new ? 1 : 0);
    it.tiles = (it.n_slab + kTile - 1) / kTile;
    // the previous kernel of the stream (the only one that can overlap with this one) may be
    // this kernel one step earlier, whose new token is the stream's last row but one
    it.safe = ends ? n_keys - 2 : n_keys;
    it.row0 = b.z;
    it.direct = b.x & 1;
    it.slot = b.y;
    it.comb = b.w;
    return it;
}

template <int D, int NT, int MODE, bool F8, bool DEFER>
__global__ void __launch_bounds__(kUmmaThreads, 1)
decode_umma_kernel(const __grid_constant__ TensorMaps tm, const DecodeParams p,
                   const __grid_constant__ InlineLens lens, const __grid_constant__ SpanParams sp) {
    using Cfg = UmmaConfig<D, NT, F8>;
    static_assert(!F8 || (D == 128 && NT == 1 && MODE == kModeSlab), "8-bit slabs: head_dim 128, group <= 8, slab mode");
    static_assert(!DEFER || (!F8 && MODE == kModeSlab), "late read-out: 16-bit slabs");
    constexpr int ES = Cfg::kElem;
    constexpr int HALVES = Cfg::kHalves;
    constexpr int HALF_BYTES = kTile * 128;           // one 128-byte column block of a K or V tile
    constexpr int ROW_CHUNKS = D * 2 / 16;            // 16-byte chunks per row of q, k_new, v_new (bf16)
    constexpr int KV_CHUNKS = D * ES / 16;            // 16-byte chunks per stored row
    constexpr int QK_STEPS = D * ES / 32;             // 32 bytes of a row per instruction (K = 16 or 32)
    constexpr int PV_KEYS = 16 * (2 / ES);            // keys per instruction of the second product
    constexpr float RESCALE_ABOVE = F8 ? kRescaleAbove8 : kRescaleAbove;
    const uint32_t STAGES = static_cast<uint32_t>(p.stages);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    // New-row buffers, P buffers and query slots come first: an M = 64 descriptor reads 8 KB
    // from its base, and what follows the last of them is the stage ring.
    uint8_t* newbuf = smem;
    uint8_t* pbuf = newbuf + Cfg::kNewBufBytes;
    uint8_t* qbuf = pbuf + Cfg::kPBytes;
    uint8_t* kv = qbuf + Cfg::kQBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(kv + STAGES * Cfg::kStageBytes);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + kNumBars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(abort_flag) + 1);
    float* xchg = reinterpret_cast<float*>(const_cast<int*>(abort_flag) + 16);   // [lane][head][2]

    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int idx) { return bar0 + 8u * static_cast<uint32_t>(idx); };
    auto lane_bar = [&](int L, int idx) { return bar0 + 8u * static_cast<uint32_t>(kBarLane0 + L * kBarPerLane + idx); };
    enum { S_FULL = 0, S_EMPTY = 2, P_FULL = 4, P_EMPTY = 6, O_FULL = 8, O_EMPTY = 9, X_FULL = 10, X_EMPTY = 11 };
    // 8-bit slabs: the softmax warp is the slowest role (a tile arrives in half the time), so an item of
    // kBothTiles tiles or more is worked on by both lanes, its tiles going to them in turn
    constexpr bool BOTH = F8;
    // The late-read-out variant puts the two softmax warps on different schedulers (both lanes are at
    // work most of the time there, and on one scheduler each slows the other down).  Tensor-memory
    // lanes 0..31 belong to warps 0 and 4, lanes 32..63 to warps 1 and 5; an M = 64 accumulator keeps
    // rows 16..31 in lanes 32..47.  So lane 1's A operands (queries, P) are described from 2 KB (16
    // rows) before their first row: its heads are rows 16.. of its products, and warp 5 reads them.
    // (Rows 0..15 are then whatever lies there; they are never looked at.)  Measured with the read-out
    // at once, the same arrangement lost 3 % on long streams, and the 8-bit kernel needs both softmax
    // warps on lanes 0..15 (a home lane reads the helper lane's accumulator): both keep warps 0 and 4.
    constexpr bool SPLIT = DEFER;
    constexpr int W_SOFT1 = SPLIT ? 5 : 4, W_PV0 = SPLIT ? 4 : 5, W_PV1 = 6;
    constexpr uint32_t ROWS16 = 16u * 128u;            // bytes of 16 operand rows

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int64_t limit = p.wait_limit_ns;
    const int cta = blockIdx.x;
    const bool fused = p.k_new != nullptr;
    // The CTA's record and its first item (the record carries a copy) are asked for before anything
    // else: the set-up below runs under their latency, and no role starts with a load that depends
    // on another (a chained CTA's first tile is requested one L2 round trip earlier).
    const int4 rec = __ldg(p.cta + 3 * cta);
    const int4 first_a = __ldg(p.cta + 3 * cta + 1), first_b = __ldg(p.cta + 3 * cta + 2);

    // a query slot is handed back by the MMA thread and the lane's softmax warp (BOTH: and the other lane's,
    // which takes the heads' score factors from it when it helps with the item)
    if (tid < kNumBars) mbar_init(bar(tid), (tid >= kBarQEmpty && tid < kBarQEmpty + kQSlots) ? (BOTH ? 3u : 2u) : 1u);
    if (tid == 0) {
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // rows of the query slots beyond the group stay zero for the whole kernel
    for (int i = tid; i < Cfg::kQBytes / 16; i += kUmmaThreads)
        reinterpret_cast<uint4*>(qbuf)[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async();
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(static_cast<uint32_t>(kTmemCols))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int it_begin = rec.x, it_end = rec.y;
    // A launch may span several layers of a step: every role walks the CTA's items once per layer, in
    // one sequence x = 0 .. n_layers * n_it - 1 (item it_begin + x mod n_it of layer x div n_it); ring
    // positions, buffer parities and query slots simply run on across the layers.
    const int n_it = it_end - it_begin;
    const int total = n_it * p.n_layers;
    const bool span = p.n_layers > 1;
    // the walk: item `it` of layer `li`, advanced by every role at the end of each turn of its loop
    int it = it_begin, li = 0;
    auto advance = [&]() {
        if (++it == it_end) {
            it = it_begin;
            ++li;
        }
    };
    auto next_item = [&]() { return it + 1 < it_end ? it + 1 : (li + 1 < p.n_layers ? it_begin : it_end); };
    const uint32_t kv_u32 = smem_u32(kv);
    const uint32_t q_u32 = smem_u32(qbuf);
    const uint32_t p_u32 = smem_u32(pbuf);

    // Programmatic dependent launch: all of the above may run while the previous kernel of the
    // stream drains, and so may the producer's first loads of rows nobody can be writing; the
    // rest comes after the dependency wait.  The next kernel is let go only after this wait (by
    // warp 7, which does nothing else), so a kernel can overlap with its immediate predecessor
    // only.  A chained launch follows a decode launch of the same pool on ANOTHER layer (the next
    // layer of a step, or a step on another layer): other K/V arrays, other outputs, the other
    // scratch set, inputs that were complete when it was issued; none of its roles waits, and its
    // CTAs do real work on every SM the predecessor's CTAs have left.  (Warp 7 still waits before letting the next
    // launch go: the kernel two launches back, which used the same scratch set, is complete
    // before any CTA of this one starts.)
    const bool chained = p.chained != 0;
    if (warp == 3 && !chained) {
        // Before the wait nothing may be READ that the previous kernel could still be writing,
        // but a line may be asked into L2 (the point of coherence: a later write lands in the
        // same line): the queries and new rows of the CTA's first items, so that the loads after
        // the wait are L2 hits.
        for (int it = it_begin + (lane >> 2); it < it_end && it < it_begin + kQSlots; it += 8) {
            const int4 a = __ldg(p.items + 2 * it), b = __ldg(p.items + 2 * it + 1);
            const Item im = item_of(a, b, lens, fused);
            const uint8_t* src = static_cast<const uint8_t*>(p.q) +
                                 (static_cast<size_t>(im.req) * p.q_heads + static_cast<size_t>(im.head) * p.group) * D * 2;
            for (int off = (lane & 3) * 128; off < p.group * D * 2; off += 512)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(src + off) : "memory");
            if (im.has_new && (lane & 3) < 2) {
                const size_t nrow = (static_cast<size_t>(im.req) * p.kv_heads + im.head) * D * 2;
                const uint8_t* nsrc = static_cast<const uint8_t*>((lane & 1) ? p.v_new : p.k_new) + nrow;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nsrc) : "memory");
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nsrc + 128) : "memory");
            }
        }
    }
    if (warp == 7) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    } else if (warp != 1 && !chained) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    // item walk shared by the roles: descriptor of item `it`, the next one already on its way
    int4 nxt_a = make_int4(0, 0, 0, 0), nxt_b = nxt_a;
    auto fetch = [&](int it) {
        if (it == it_begin) {                          // the copy in the CTA's record
            nxt_a = first_a;
            nxt_b = first_b;
        } else if (it < it_end) {
            nxt_a = __ldg(p.items + 2 * it);
            nxt_b = __ldg(p.items + 2 * it + 1);
        }
    };

    bool ok = true;
    if (warp == 1) {
        // ------------------------------------------------------------------ producer
        uint32_t issued_any = 0, issued_odd = 0;     // per stage: loads issued at all / an odd number of times
        int64_t k_array = static_cast<int64_t>(p.layer) * 2 * p.rows_per_array;      // of the layer being issued
        int64_t v_array = k_array + p.rows_per_array;
        constexpr int COPIES = 2 * HALVES;            // copies per box position: K and V, each column block
        // One tile of a slab stream = up to four groups of 16 rows, fetched with one copy per
        // 128-byte column block of K and of V (a box of 16, 32, 48 or 64 rows; never past
        // ceil16 of the rows to stream).  part 0: the whole tile; part 1: only the groups that
        // lie wholly in the safe rows, with the barrier told to expect the whole tile; part 2:
        // the rest of a tile whose part 1 is under way.  Called by the whole warp.
        auto issue_tile = [&](uint32_t stage, const Item& im, int t, int part) {
            const int r0 = t * kTile;
            const int nb = (min(kTile, im.n_slab - r0) + 15) >> 4;
            const int ge = min(nb, max(im.safe - r0, 0) >> 4);
            const int g0 = part == 2 ? ge : 0, g1 = part == 1 ? ge : nb;
            if (part != 2) {
                if (lane == 0) mbar_expect_tx(bar(kBarFull + stage), static_cast<uint32_t>(nb) * 16u * D * ES * 2u);
                issued_any |= 1u << stage;
                issued_odd ^= 1u << stage;
                __syncwarp();
            }
            if (MODE == kModePaged) {                 // one 16-row box per page, all of them at once
                const int bx = lane / COPIES, w = lane - bx * COPIES;
                if (bx < nb) {
                    const int h = w >> 1, kvsel = w & 1;
                    const int32_t page = p.page_table[static_cast<size_t>(im.req) * p.max_pages + im.tok0 / 16 + t * 4 + bx];
                    const int64_t prow = (static_cast<int64_t>(page) * p.kv_heads + im.head) * 16;
                    tma_load_2d(kv_u32 + stage * Cfg::kStageBytes + kvsel * Cfg::kKvTileBytes + h * HALF_BYTES + bx * 2048,
                                &tm.box[0], h * 64, static_cast<int32_t>((kvsel ? v_array : k_array) + prow),
                                bar(kBarFull + stage));
                }
                return;
            }
            if (g1 <= g0 || lane >= COPIES) return;
            const int h = lane >> 1, kvsel = lane & 1;
            const uint32_t dst = kv_u32 + stage * Cfg::kStageBytes + kvsel * Cfg::kKvTileBytes + g0 * 2048 + h * HALF_BYTES;
            const int32_t y = static_cast<int32_t>((kvsel ? v_array : k_array) + im.row0 + r0 + g0 * 16);
            tma_load_2d(dst, &tm.box[g1 - g0 - 1], h * 64, y, bar(kBarFull + stage));
        };
        if (lane < 4)
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.box[lane])) : "memory");
        // Early start: the safe rows of the CTA's first tiles (one per pipeline stage) are
        // requested before the dependency wait, so that HBM is already streaming while the
        // previous grid finishes.
        int n_early = 0;
        if (MODE != kModePaged && !chained && p.early_ok) {
            int4 a = first_a, b = first_b;
            for (int it = it_begin; it < it_end && n_early < static_cast<int>(STAGES); ++it) {
                if (it != it_begin) {
                    a = __ldg(p.items + 2 * it);
                    b = __ldg(p.items + 2 * it + 1);
                }
                const Item im = item_of(a, b, lens, fused);
                for (int t = 0; t < im.tiles && n_early < static_cast<int>(STAGES); ++t, ++n_early)
                    issue_tile(static_cast<uint32_t>(n_early), im, t, 1);
            }
        }
        if (!chained) asm volatile("griddepcontrol.wait;" ::: "memory");

        uint32_t g = 0;                               // tiles issued so far
        fetch(it_begin);
        for (int x = 0; x < total && ok; ++x, advance()) {
            const Item im = item_of(nxt_a, nxt_b, lens, fused);
            fetch(next_item());
            k_array = static_cast<int64_t>(p.layer + li) * 2 * p.rows_per_array;
            v_array = k_array + p.rows_per_array;
            for (int t = 0; t < im.tiles; ++t, ++g) {
                const uint32_t stage = g % STAGES, phase = (g / STAGES) & 1u;
                if (g < static_cast<uint32_t>(n_early)) {        // first use of the stage, part 1 under way
                    issue_tile(stage, im, t, 2);
                    continue;
                }
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(kBarEmpty + stage), phase ^ 1u, abort_flag, p.status, limit));
                if (!ok) break;
                issue_tile(stage, im, t, 0);
            }
        }
        if (lane == 0 && (!ok || *abort_flag)) {
            // Something timed out.  Before the CTA's shared memory can be handed to another
            // CTA, wait (bounded, ignoring the abort flag) for the loads already in flight.
            for (uint32_t s = 0; s < STAGES; ++s)
                if ((issued_any >> s) & 1u)      // parity of the stage's latest phase
                    mbar_wait_slow(bar(kBarFull + s), ((issued_odd >> s) & 1u) ^ 1u, nullptr, p.status, limit / 4 + 1);
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ query loader
        // chunk c (16 bytes) of head r of the group goes to row r of column block c / 8, at the
        // swizzled position (c % 8) ^ (r % 8) of that row; the new K and V rows go, as they
        // are, to the slot's side buffer and to the slab
        const uint8_t* qg = static_cast<const uint8_t*>(p.q);
        constexpr int Q_LOADS = (NT * 8 * ROW_CHUNKS + 31) / 32;
        fetch(it_begin);
        for (int x = 0; x < total; ++x, advance()) {
            const int k = x;
            const Item im = item_of(nxt_a, nxt_b, lens, fused);
            fetch(next_item());
            const uint32_t slot = static_cast<uint32_t>(k) % kQSlots, use = static_cast<uint32_t>(k) / kQSlots;
            const uint8_t* src = qg + (span ? li * sp.q_stride : 0) +
                                 (static_cast<size_t>(im.req) * p.q_heads + static_cast<size_t>(im.head) * p.group) * D * 2;
            const uint8_t* new_k = static_cast<const uint8_t*>(p.k_new) + (span ? li * sp.new_stride : 0);
            const uint8_t* new_v = static_cast<const uint8_t*>(p.v_new) + (span ? li * sp.new_stride : 0);
            const int64_t layer_l = p.layer + li;
            // this layer's scales of an 8-bit pool
            const float4 sc4 = (F8 && span) ? sp.scales[li] : make_float4(p.k_scale, p.v_scale, p.k_inv, p.v_inv);
            uint4 v[Q_LOADS];
#pragma unroll
            for (int i = 0; i < Q_LOADS; ++i) {
                const int idx = lane + 32 * i;
                v[i] = make_uint4(0u, 0u, 0u, 0u);
                if (idx < p.group * ROW_CHUNKS) v[i] = __ldg(reinterpret_cast<const uint4*>(src) + idx);
            }
            uint4 nv = make_uint4(0u, 0u, 0u, 0u);
            const bool mine = im.has_new && lane < 2 * ROW_CHUNKS;
            const int kvsel = lane / ROW_CHUNKS, c_new = lane - kvsel * ROW_CHUNKS;
            if (mine) {
                const size_t nrow = (static_cast<size_t>(im.req) * p.kv_heads + im.head) * ROW_CHUNKS;
                nv = __ldg(reinterpret_cast<const uint4*>(kvsel ? new_v : new_k) + nrow + c_new);
            }
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(kBarQEmpty + slot), (use & 1u) ^ 1u, abort_flag, p.status, limit));
            if (!ok) break;
            uint8_t* dst = qbuf + slot * Cfg::kQSlotBytes;
            if (F8) {
                // A row of D bf16 numbers is 16 chunks: lanes 0..15 hold row 2i, lanes 16..31 row 2i + 1
                // of load i.  Per row: the power of two that brings the largest element into [128, 256),
                // then x * 2^e = hi + lo / 16 in E4M3 (exact for all but elements 2^13 below the largest),
                // hi to row r, lo to row r + 8 of the slot; the score factor 2^-e * k_scale * log2(e) /
                // sqrt(D) of the row goes to the side buffer.
                float* qf = reinterpret_cast<float*>(newbuf + slot * Cfg::kNewBytes + 2 * D);
#pragma unroll
                for (int i = 0; i < Q_LOADS; ++i) {
                    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                    uint32_t amax = 0;                   // as bits: the order of non-negative floats
#pragma unroll
                    for (int j = 0; j < 4; ++j) amax = max(amax, max((w[j] << 16) & 0x7FFFFFFFu, w[j] & 0x7FFF0000u));
#pragma unroll
                    for (int sh = 1; sh < 16; sh <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, sh));
                    const int ex = static_cast<int>(amax >> 23);                 // biased exponent of the largest element
                    const int e = (ex == 0 || ex == 255) ? 0 : min(134 - ex, 120);  // 2^e * largest in [128, 256)
                    const float up = __uint_as_float(static_cast<uint32_t>(e + 127) << 23);
                    const int r = (lane + 32 * i) / ROW_CHUNKS, c = (lane + 32 * i) % ROW_CHUNKS;
                    if (r < p.group) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float x0 = __uint_as_float(w[j] << 16) * up, x1 = __uint_as_float(w[j] & 0xFFFF0000u) * up;
                            hi[j] = pack_e4m3(x0, x1);
                            const float2 h = unpack_e4m3(hi[j]);
                            lo[j] = pack_e4m3((x0 - h.x) * 16.f, (x1 - h.y) * 16.f);
                        }
                        uint8_t* row = dst + r * 128 + ((((c >> 1) ^ r) & 7) << 4) + (c & 1) * 8;
                        *reinterpret_cast<uint2*>(row) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
                        *reinterpret_cast<uint2*>(row + 1024) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
                        if (c == 0) qf[r] = __uint_as_float(static_cast<uint32_t>(127 - e) << 23) * (sc4.x * p.scale_log2);
                    }
                }
                if (mine) {
                    // the new rows as the slab will hold them: eight codes from this lane's eight numbers
                    const uint2 codes = quantize8_e4m3(nv, kvsel ? sc4.w : sc4.z);
                    *reinterpret_cast<uint2*>(newbuf + slot * Cfg::kNewBytes + lane * 8) = codes;
                    uint2* slab = reinterpret_cast<uint2*>(const_cast<void*>(p.pool)) +
                                  ((layer_l * 2 + kvsel) * p.rows_per_array + im.row0 + im.n_slab) * (D / 8) + c_new;
                    *slab = codes;
                }
            } else {
#pragma unroll
                for (int i = 0; i < Q_LOADS; ++i) {
                    const int idx = lane + 32 * i;
                    if (idx < p.group * ROW_CHUNKS) {
                        const int r = idx / ROW_CHUNKS, c = idx - r * ROW_CHUNKS;
                        *reinterpret_cast<uint4*>(dst + (c >> 3) * Cfg::kQHalfBytes + (r >> 3) * 1024 + (r & 7) * 128 +
                                                  (((c & 7) ^ (r & 7)) << 4)) = v[i];
                    }
                }
                if (mine) {
                    *reinterpret_cast<uint4*>(newbuf + slot * Cfg::kNewBytes + lane * 16) = nv;
                    uint4* slab = reinterpret_cast<uint4*>(const_cast<void*>(p.pool)) +
                                  ((layer_l * 2 + kvsel) * p.rows_per_array + im.row0 + im.n_slab) * ROW_CHUNKS + c_new;
                    *slab = nv;
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQFull + slot));
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ MMA issue, first products
        // In ring order: a tile's stage has landed, its lane's S buffer has been read out, and for
        // an item's first tile its queries are there.  The whole warp runs the loop and one
        // elected lane issues: tcgen05 instructions issued from a converged warp cost a third of
        // what they cost a lone thread of a diverged one.
        uint32_t elected;
        asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xFFFFFFFF;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(elected));
        constexpr uint32_t IDESC_QK = F8 ? umma_idesc8(64, kTile, false) : umma_idesc(64, kTile, false);
        uint32_t c[kLanes] = {0, 0};                  // tiles of each lane issued so far
        uint32_t g = 0;
        fetch(it_begin);
        for (int x = 0; x < total && ok; ++x, advance()) {
            const int k = x;
            const Item im = item_of(nxt_a, nxt_b, lens, fused);
            fetch(next_item());
            const bool both = BOTH && im.tiles >= kBothTiles;
            const uint32_t slot = static_cast<uint32_t>(k) % kQSlots, use = static_cast<uint32_t>(k) / kQSlots;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(kBarQFull + slot), use & 1u, abort_flag, p.status, limit));
            if (!ok) break;
            if (im.tiles == 0) {
                // nothing but the step's new token: no product; the slot is signed off (after it was
                // filled, not before: its previous use must be over)
                if (elected) mbar_arrive(bar(kBarQEmpty + slot));
                continue;
            }
            const uint32_t qb = q_u32 + slot * Cfg::kQSlotBytes;
            const uint32_t qb1 = qb - ROWS16;            // lane 1 (SPLIT): the heads as rows 16..
            for (int t = 0; t < im.tiles; ++t, ++g) {
                const uint32_t stage = g % STAGES, phase = (g / STAGES) & 1u;
                const int L = (both ? k + t : k) & 1;
                const uint32_t cc = L ? c[1] : c[0], b = cc & 1u, u = cc >> 1;
                // both barriers are looked at before either answer is needed; the slow path only when one is not ready
                const bool f_ok = mbar_try(bar(kBarFull + stage), phase), e_ok = mbar_try(lane_bar(L, S_EMPTY + b), (u & 1u) ^ 1u);
                if (!__all_sync(0xFFFFFFFFu, f_ok && e_ok)) {
                    bool good = f_ok || mbar_wait_slow(bar(kBarFull + stage), phase, abort_flag, p.status, limit);
                    if (good && !e_ok) good = mbar_wait_slow(lane_bar(L, S_EMPTY + b), (u & 1u) ^ 1u, abort_flag, p.status, limit);
                    ok = __all_sync(0xFFFFFFFFu, good);
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t kbase = kv_u32 + stage * Cfg::kStageBytes;
                const uint32_t t_s = tmem + static_cast<uint32_t>(L * kTmemLaneCols) + b * 64u;
                if (elected) {
#pragma unroll
                    for (int ks = 0; ks < QK_STEPS; ++ks)
                        umma<F8>(t_s, smem_desc((SPLIT && L ? qb1 : qb) + (ks >> 2) * Cfg::kQHalfBytes + (ks & 3) * 32, 16, 1024),
                                  smem_desc(kbase + (ks >> 2) * HALF_BYTES + (ks & 3) * 32, 16, 1024), IDESC_QK, ks > 0 ? 1u : 0u);
                    umma_commit(lane_bar(L, S_FULL + b));
                    if (t == im.tiles - 1) umma_commit(bar(kBarQEmpty + slot));
                }
                __syncwarp();
                if (L) ++c[1]; else ++c[0];
            }
        }
        // nothing may still be running when tensor memory is given back
        if (elected) umma_commit(bar(kBarDrain));
        __syncwarp();
        mbar_wait_slow(bar(kBarDrain), 0, nullptr, p.status, limit / 4 + 1);
    } else if (warp == W_PV0 || warp == W_PV1) {
        // ------------------------------------------------------------------ MMA issue, second products of one lane
        // A tile's P has been written (and, for an item's first tile, the lane's O of the item
        // before has been read out); the commits hand the stage back to the producer and the P
        // buffer to the softmax warp, and after an item's last tile tell it that O is complete.
        const int L = warp == W_PV0 ? 0 : 1;
        uint32_t elected;
        asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xFFFFFFFF;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(elected));
        constexpr uint32_t IDESC_PV = F8 ? umma_idesc8(64, D, true) : umma_idesc(64, D, true);
        const uint32_t t_o = tmem + static_cast<uint32_t>(L * kTmemLaneCols) + 128u;
        uint32_t c = 0, j = 0, g = 0;                 // the lane's tiles and items (with tiles) so far; ring position
        fetch(it_begin);
        for (int x = 0; x < total && ok; ++x, advance()) {
            const int k = x;
            const Item im = item_of(nxt_a, nxt_b, lens, fused);
            fetch(next_item());
            const uint32_t g0 = g;
            g += static_cast<uint32_t>(im.tiles);
            // the lane's tiles of the item: all of them, or every second one when both lanes work on it
            const bool both = BOTH && im.tiles >= kBothTiles;
            if ((!both && (k & 1) != L) || im.tiles == 0) continue;
            const int t_first = both ? (L ^ k) & 1 : 0, t_step = both ? 2 : 1;
            for (int t = t_first; t < im.tiles; t += t_step, ++c) {
                const uint32_t b = c & 1u, u = c >> 1, st = (g0 + static_cast<uint32_t>(t)) % STAGES;
                bool good = mbar_wait_spin(lane_bar(L, P_FULL + b), u & 1u, abort_flag, p.status, limit);
                if (good && t == t_first) good = mbar_wait(lane_bar(L, O_EMPTY), (j & 1u) ^ 1u, abort_flag, p.status, limit);
                ok = __all_sync(0xFFFFFFFFu, good);
                if (!ok) break;
                tc_fence_after();
                const bool last = t + t_step >= im.tiles;                      // the lane's last tile of the item
                const int ksteps = (t == im.tiles - 1 ? im.n_slab - t * kTile + PV_KEYS - 1 : kTile) / PV_KEYS;
                const uint32_t vbase = kv_u32 + st * Cfg::kStageBytes + Cfg::kKvTileBytes;
                const uint32_t pb = p_u32 + static_cast<uint32_t>((L * 2 + static_cast<int>(b)) * Cfg::kPBufBytes) -
                                    (SPLIT && L ? ROWS16 : 0u);
                if (elected) {
                    for (int ks = 0; ks < ksteps; ++ks)
                        umma<F8>(t_o, smem_desc(pb + ks * 32, 16, 1024), smem_desc(vbase + ks * (PV_KEYS * 128), HALF_BYTES, 1024), IDESC_PV,
                                  (t == t_first && ks == 0) ? 0u : 1u);
                    umma_commit(bar(kBarEmpty + st));
                    umma_commit(lane_bar(L, P_EMPTY + b));
                    if (last) umma_commit(lane_bar(L, O_FULL));
                }
                __syncwarp();
            }
            ++j;
        }
        if (elected) umma_commit(bar(kBarDrain + 1 + L));
        __syncwarp();
        mbar_wait_slow(bar(kBarDrain + 1 + L), 0, nullptr, p.status, limit / 4 + 1);
    } else if (warp == 0 || warp == W_SOFT1) {
        // ------------------------------------------------------------------ softmax + finish
        const int L = warp == 0 ? 0 : 1;
        // (SPLIT: lane 1's rows are in tensor-memory lanes 32.., the lane field of the address is bits 16..)
        const uint32_t t_s = tmem + static_cast<uint32_t>(L * kTmemLaneCols) + (SPLIT && L ? (32u << 16) : 0u), t_o = t_s + 128u;
        uint8_t* p_lane = pbuf + L * 2 * Cfg::kPBufBytes;
        const int hq = lane >> 2, kq = (lane & 3) * 2;      // head row within 8; first of the thread's two keys within 8
        const float scale = p.scale_log2;
        const int group = p.group;
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
        uint32_t c = 0, j = 0, g = 0;                       // the lane's tiles and items so far; ring position
        uint32_t n_helped = 0, n_merged = 0;                // items this lane helped with / merged the other lane's part of
        float* x_mine = xchg + L * 32;                      // where this lane leaves (m, l) per head as a helper
        const float* x_other = xchg + (L ^ 1) * 32;

        // ---- an item's result: O from tensor memory, then out / partial / merge.  `fli` is the layer
        // the item belongs to (its outputs and scratch), `both` whether the other lane helped with it.
        auto finish = [&](const Item& im, int fli, bool both, float (&m_ref)[NT], float (&l_acc)[NT],
                          const float (&s_new)[NT], const uint32_t (&v_new)[D / 8]) {
            __nv_bfloat16* out_l = out + (span ? fli * (sp.out_stride / 2) : 0);
            float* lse_l = p.lse ? p.lse + (span ? fli * sp.lse_stride : 0) : nullptr;
            float* part_o_l = p.part_o + (span ? fli * sp.part_o_stride : 0);
            float* part_ml_l = p.part_ml + (span ? fli * sp.part_ml_stride : 0);
            uint32_t* counters_l = p.counters ? p.counters + (span ? static_cast<size_t>(fli) * sp.counter_stride : 0) : nullptr;
            float oo[NT][D / 4];                          // [rs][2i + e]: head hq + 8 rs, element 8i + kq + e
            if (im.tiles > 0) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait_spin(lane_bar(L, O_FULL), j & 1u, abort_flag, p.status, limit));
                if (!ok) return;
                tc_fence_after();
#pragma unroll
                for (int blk = 0; blk < D / 64; ++blk) {
                    uint32_t r[32];
                    tmem_ld_x8(t_o + blk * 64u, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
#pragma unroll
                        for (int rs = 0; rs < NT; ++rs) {
                            if (F8) {                     // (hi row + lo row / 16) / 16: P went in times 16
                                oo[0][2 * (8 * blk + i)] = fmaf(__uint_as_float(r[4 * i + 2]), 0.0625f, __uint_as_float(r[4 * i])) * 0.0625f;
                                oo[0][2 * (8 * blk + i) + 1] =
                                    fmaf(__uint_as_float(r[4 * i + 3]), 0.0625f, __uint_as_float(r[4 * i + 1])) * 0.0625f;
                            } else {
                                oo[rs][2 * (8 * blk + i)] = __uint_as_float(r[4 * i + 2 * rs]);
                                oo[rs][2 * (8 * blk + i) + 1] = __uint_as_float(r[4 * i + 2 * rs + 1]);
                            }
                        }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(lane_bar(L, O_EMPTY));
                ++j;
            } else {
#pragma unroll
                for (int rs = 0; rs < NT; ++rs)
#pragma unroll
                    for (int i = 0; i < D / 4; ++i) oo[rs][i] = 0.f;
            }
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) {
                l_acc[rs] += __shfl_xor_sync(0xFFFFFFFFu, l_acc[rs], 1);
                l_acc[rs] += __shfl_xor_sync(0xFFFFFFFFu, l_acc[rs], 2);
            }
            if (BOTH && both) {
                // the helper lane's part: its (m, l) from shared memory, its accumulator from its
                // columns of tensor memory; both are signed off on its behalf
                const int LO = L ^ 1;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(lane_bar(LO, X_FULL), n_merged & 1u, abort_flag, p.status, limit));
                if (!ok) return;
                ++n_merged;
                tc_fence_after();
                const float2 ml = *reinterpret_cast<const float2*>(x_other + hq * 2);
                const float mn = fmaxf(m_ref[0], ml.x);
                const float e_mine = fast_exp2(m_ref[0] - mn), w_other = fast_exp2(ml.x - mn);
                const float e_other = w_other * 0.0625f;     // its accumulator still carries the factor 16 of P
                l_acc[0] = fmaf(l_acc[0], e_mine, ml.y * w_other);
                m_ref[0] = mn;
                const uint32_t t_o_other = tmem + static_cast<uint32_t>(LO * kTmemLaneCols) + 128u;
#pragma unroll
                for (int blk = 0; blk < D / 64; ++blk) {
                    uint32_t r[32];
                    tmem_ld_x8(t_o_other + blk * 64u, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {          // (hi row + lo row / 16) / 16, as in the lane's own read-out
                        float& a0 = oo[0][2 * (8 * blk + i)];
                        float& a1 = oo[0][2 * (8 * blk + i) + 1];
                        a0 = fmaf(a0, e_mine, fmaf(__uint_as_float(r[4 * i + 2]), 0.0625f, __uint_as_float(r[4 * i])) * e_other);
                        a1 = fmaf(a1, e_mine, fmaf(__uint_as_float(r[4 * i + 3]), 0.0625f, __uint_as_float(r[4 * i + 1])) * e_other);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(lane_bar(LO, O_EMPTY));
                    mbar_arrive(lane_bar(LO, X_EMPTY));
                }
            }
            if (im.has_new) {
#pragma unroll
                for (int rs = 0; rs < NT; ++rs) {
                    const float pn = fast_exp2(s_new[rs] - m_ref[rs]);
                    l_acc[rs] += pn;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        const float2 vv = F8 ? unpack_e4m3(v_new[i])
                                             : make_float2(__uint_as_float(v_new[i] << 16), __uint_as_float(v_new[i] & 0xFFFF0000u));
                        oo[rs][2 * i] = fmaf(pn, vv.x, oo[rs][2 * i]);
                        oo[rs][2 * i + 1] = fmaf(pn, vv.y, oo[rs][2 * i + 1]);
                    }
                }
            }
            if (F8) {                                      // codes to values
                const float v_scale = span ? sp.scales[fli].y : p.v_scale;
#pragma unroll
                for (int i = 0; i < D / 4; ++i) oo[0][i] *= v_scale;
            }
            auto write_out = [&](int req, int head, int rs, float M, float Lsum, const float (&x)[D / 4]) {
                const int h = hq + 8 * rs;
                if (h >= group) return;
                const float inv = fast_rcp(Lsum);
                const size_t row = static_cast<size_t>(req) * p.q_heads + static_cast<size_t>(head) * group + h;
                __nv_bfloat16* dst = out_l + row * D + kq;
#pragma unroll
                for (int i = 0; i < D / 8; ++i)
                    *reinterpret_cast<uint32_t*>(dst + 8 * i) = pack_bf16(x[2 * i] * inv, x[2 * i + 1] * inv);
                if ((lane & 3) == 0 && lse_l) lse_l[row] = (M + fast_log2(Lsum)) * 0.6931471805599453f;
            };
            if (im.direct) {
#pragma unroll
                for (int rs = 0; rs < NT; ++rs) write_out(im.req, im.head, rs, m_ref[rs], l_acc[rs], oo[rs]);
                return;
            }
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) {
                const int h = hq + 8 * rs;
                if (h >= group) continue;
                const size_t prow = static_cast<size_t>(im.slot) * group + h;
                float* po = part_o_l + prow * D + kq;
#pragma unroll
                for (int i = 0; i < D / 8; ++i) *reinterpret_cast<float2*>(po + 8 * i) = make_float2(oo[rs][2 * i], oo[rs][2 * i + 1]);
                if ((lane & 3) == 0) *reinterpret_cast<float2*>(part_ml_l + prow * 2) = make_float2(m_ref[rs], l_acc[rs]);
            }
            if (counters_l == nullptr) return;             // a combine kernel follows
            // The CTA that delivers a split stream's last piece merges all of them, in slot
            // order (so the result does not depend on which CTA that is), reading them back
            // through L2 (its own included), the next piece's loads in flight while one is folded.
            const int4 cr = __ldg(p.combine + im.comb);   // {request, head, first slot, pieces}
            __syncwarp();
            int is_last = 0;
            if (lane == 0) {
                __threadfence();
                const uint32_t seen = atomicAdd(counters_l + im.comb, 1u);
                is_last = seen + 1u == static_cast<uint32_t>(cr.w);
                if (is_last) counters_l[im.comb] = 0u;     // ready for the next launch
            }
            is_last = __shfl_sync(0xFFFFFFFFu, is_last, 0);
            if (!is_last) return;
            __threadfence();
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) {
                const int h = hq + 8 * rs;
                if (h >= group) continue;
                float fm = -INFINITY, fl = 0.f, fa[D / 4];
#pragma unroll
                for (int i = 0; i < D / 4; ++i) fa[i] = 0.f;
                auto load = [&](int s, float2& ml, float2 (&x)[D / 8]) {
                    const size_t prow = static_cast<size_t>(cr.z + s) * group + h;
                    ml = __ldcg(reinterpret_cast<const float2*>(part_ml_l + prow * 2));
                    const float* po = part_o_l + prow * D + kq;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) x[i] = __ldcg(reinterpret_cast<const float2*>(po + 8 * i));
                };
                auto fold = [&](const float2& ml, const float2 (&x)[D / 8]) {
                    const float mn = fmaxf(fm, ml.x);
                    const float e0 = fm == -INFINITY ? 0.f : fast_exp2(fm - mn);
                    const float e1 = ml.x == -INFINITY ? 0.f : fast_exp2(ml.x - mn);
                    fl = fmaf(fl, e0, ml.y * e1);
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        fa[2 * i] = fmaf(fa[2 * i], e0, x[i].x * e1);
                        fa[2 * i + 1] = fmaf(fa[2 * i + 1], e0, x[i].y * e1);
                    }
                    fm = mn;
                };
                float2 ml_a, ml_b, x_a[D / 8], x_b[D / 8];
                load(0, ml_a, x_a);
                for (int s = 0; s < cr.w; s += 2) {
                    if (s + 1 < cr.w) load(s + 1, ml_b, x_b);
                    fold(ml_a, x_a);
                    if (s + 1 < cr.w) {
                        if (s + 2 < cr.w) load(s + 2, ml_a, x_a);
                        fold(ml_b, x_b);
                    }
                }
                write_out(cr.x, cr.y, rs, fm, fl, fa);
            }
        };

        // DEFER (launches in which a lane works through several short items): an item's result is
        // taken from tensor memory one step late.  Once an item's last P is handed over, the warp
        // goes on to the lane's NEXT item (its new token's score, the softmax of its first tile) and
        // only then reads out and stores the earlier item, whose second products have run meanwhile.
        // (Only the first tile: the next item's second products cannot start before the accumulator
        // is read out.)  The loop takes one turn more than there are items, for the last result.
        Item pd_im = {};
        int pd_li = 0;
        bool pd_valid = false;
        float pd_m[NT], pd_l[NT], pd_s[NT];
        uint32_t pd_v[D / 8];
        fetch(it_begin);
        for (int x = 0; x < total + (DEFER ? 1 : 0) && ok; ++x, advance()) {
            const int k = x;
            const bool have = x < total;
            Item im = item_of(nxt_a, nxt_b, lens, fused);
            if (have) {
                fetch(next_item());
            } else {
                im.tiles = 0;
                im.has_new = false;
            }
            const uint32_t g0 = g;
            g += static_cast<uint32_t>(im.tiles);
            // BOTH: an item of kBothTiles tiles or more is worked on by both lanes, its tiles going to
            // them in turn from its home lane (item number mod 2).  The other lane is the helper: it
            // leaves its accumulator in tensor memory and its (m, l) in shared memory, and the home
            // lane merges the two parts and finishes the item.  Every item's query slot is visited by
            // both softmax warps (each sees every phase of the slot's barriers, and a helper takes the
            // heads' score factors from it).
            const bool both = BOTH && im.tiles >= kBothTiles, home = (k & 1) == L;
            if (!BOTH && !home && have) continue;
            const int t_first = both ? (L ^ k) & 1 : 0, t_step = both ? 2 : 1;
            const uint32_t slot = static_cast<uint32_t>(k) % kQSlots, use = static_cast<uint32_t>(k) / kQSlots;
            float s_new[NT];
            uint32_t v_new[D / 8];
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) s_new[rs] = -INFINITY;
            float qfac = scale;                            // F8: the head's score factor (query power of two, key scale)
            if (have) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(kBarQFull + slot), use & 1u, abort_flag, p.status, limit));
                if (!ok) break;
                if (!both && !home) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarQEmpty + slot));
                    continue;
                }
                // The token appended this step: its scaled score per head from the query rows and the
                // new K row in shared memory (each thread adds up the elements it will also hold of the
                // output, the quad completes the sum); its value row, packed, for when the item ends.
                if (F8) qfac = reinterpret_cast<const float*>(newbuf + slot * Cfg::kNewBytes + 2 * D)[hq];
                if (im.has_new && home && F8) {
                    // queries as hi + lo / 16 from rows hq and hq + 8 of the slot, the new rows as codes
                    const uint8_t* qs = qbuf + slot * Cfg::kQSlotBytes + hq * 128;
                    const uint8_t* nk = newbuf + slot * Cfg::kNewBytes;
                    float dot = 0.f;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        const float2 kk = unpack_e4m3(*reinterpret_cast<const uint16_t*>(nk + 8 * i + kq));
                        v_new[i] = *reinterpret_cast<const uint16_t*>(nk + D + 8 * i + kq);
                        const int off = (((i >> 1) ^ hq) << 4) + (i & 1) * 8 + kq;
                        const float2 qh = unpack_e4m3(*reinterpret_cast<const uint16_t*>(qs + off));
                        const float2 ql = unpack_e4m3(*reinterpret_cast<const uint16_t*>(qs + 1024 + off));
                        dot = fmaf(fmaf(ql.x, 0.0625f, qh.x), kk.x, dot);
                        dot = fmaf(fmaf(ql.y, 0.0625f, qh.y), kk.y, dot);
                    }
                    dot += __shfl_xor_sync(0xFFFFFFFFu, dot, 1);
                    dot += __shfl_xor_sync(0xFFFFFFFFu, dot, 2);
                    s_new[0] = dot * qfac;
                } else if (im.has_new && home) {
                    const uint8_t* qs = qbuf + slot * Cfg::kQSlotBytes;
                    const uint8_t* nk = newbuf + slot * Cfg::kNewBytes;
                    const uint8_t* nvp = nk + D * 2;
                    float dot[NT];
#pragma unroll
                    for (int rs = 0; rs < NT; ++rs) dot[rs] = 0.f;
#pragma unroll
                    for (int i = 0; i < D / 8; ++i) {
                        const uint32_t kk = *reinterpret_cast<const uint32_t*>(nk + (8 * i + kq) * 2);
                        v_new[i] = *reinterpret_cast<const uint32_t*>(nvp + (8 * i + kq) * 2);
#pragma unroll
                        for (int rs = 0; rs < NT; ++rs) {
                            const uint32_t qq = *reinterpret_cast<const uint32_t*>(
                                qs + (i >> 3) * Cfg::kQHalfBytes + rs * 1024 + hq * 128 + (((i & 7) ^ hq) << 4) + kq * 2);
                            dot[rs] = fmaf(__uint_as_float(qq << 16), __uint_as_float(kk << 16), dot[rs]);
                            dot[rs] = fmaf(__uint_as_float(qq & 0xFFFF0000u), __uint_as_float(kk & 0xFFFF0000u), dot[rs]);
                        }
                    }
#pragma unroll
                    for (int rs = 0; rs < NT; ++rs) {
                        dot[rs] += __shfl_xor_sync(0xFFFFFFFFu, dot[rs], 1);
                        dot[rs] += __shfl_xor_sync(0xFFFFFFFFu, dot[rs], 2);
                        s_new[rs] = dot[rs] * scale;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarQEmpty + slot));
            }

            float m_ref[NT], l_acc[NT];
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) {
                m_ref[rs] = s_new[rs];
                l_acc[rs] = 0.f;
            }
            // one tile of the item (`first`: the lane's first tile of it); false when a wait ran out
            auto do_tile = [&](int t, bool first) -> bool {
                const uint32_t b = c & 1u, u = c >> 1;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait_spin(lane_bar(L, S_FULL + b), u & 1u, abort_flag, p.status, limit));
                if (!ok) return false;
                tc_fence_after();
                uint32_t r[32];
                tmem_ld_x8(t_s + b * 64u, r);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(lane_bar(L, S_EMPTY + b));
                const int valid = min(kTile, im.n_slab - t * kTile);
                // scaled scores, keys at or beyond the item's end selected to -inf; tile maximum per head
                float sc[NT][16], mx[NT];
#pragma unroll
                for (int rs = 0; rs < NT; ++rs) {
                    mx[rs] = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float s = F8 ? fmaf(__uint_as_float(r[4 * i + 2 + e]), 0.0625f, __uint_as_float(r[4 * i + e])) * qfac
                                         : __uint_as_float(r[4 * i + 2 * rs + e]) * scale;
                            if (8 * i + kq + e >= valid) s = -INFINITY;
                            sc[rs][2 * i + e] = s;
                            mx[rs] = fmaxf(mx[rs], s);
                        }
                    mx[rs] = fmaxf(mx[rs], __shfl_xor_sync(0xFFFFFFFFu, mx[rs], 1));
                    mx[rs] = fmaxf(mx[rs], __shfl_xor_sync(0xFFFFFFFFu, mx[rs], 2));
                }
                if (first) {
#pragma unroll
                    for (int rs = 0; rs < NT; ++rs) m_ref[rs] = fmaxf(m_ref[rs], mx[rs]);
                } else {
                    bool grow = false;
#pragma unroll
                    for (int rs = 0; rs < NT; ++rs) grow = grow || mx[rs] > m_ref[rs] + RESCALE_ABOVE;
                    if (__any_sync(0xFFFFFFFFu, grow)) {
                        // Rare: raise the reference of the heads that need it and rescale their
                        // rows of the accumulator.  Every second product issued so far must be
                        // complete (the previous tile's releases its P buffer when it is); none
                        // can be issued before this tile's P is handed over.
                        const uint32_t pc = c - 1u;
                        ok = __all_sync(0xFFFFFFFFu, mbar_wait(lane_bar(L, P_EMPTY + (pc & 1u)), (pc >> 1) & 1u, abort_flag,
                                                              p.status, limit));
                        if (!ok) return false;
                        tc_fence_after();
                        float f[2] = {1.f, 1.f};
#pragma unroll
                        for (int rs = 0; rs < NT; ++rs) {
                            const float mn = mx[rs] > m_ref[rs] + RESCALE_ABOVE ? mx[rs] : m_ref[rs];
                            f[rs] = fast_exp2(m_ref[rs] - mn);
                            l_acc[rs] *= f[rs];
                            m_ref[rs] = mn;
                        }
                        if (F8) f[1] = f[0];             // rows h and h + 8 are the two terms of one head
#pragma unroll
                        for (int blk = 0; blk < D / 32; ++blk) {
                            uint32_t o[16];
                            tmem_ld_x4(t_o + blk * 32u, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                o[4 * i] = __float_as_uint(__uint_as_float(o[4 * i]) * f[0]);
                                o[4 * i + 1] = __float_as_uint(__uint_as_float(o[4 * i + 1]) * f[0]);
                                o[4 * i + 2] = __float_as_uint(__uint_as_float(o[4 * i + 2]) * f[1]);
                                o[4 * i + 3] = __float_as_uint(__uint_as_float(o[4 * i + 3]) * f[1]);
                            }
                            tmem_st_x4(t_o + blk * 32u, o);
                        }
                        tmem_wait_st();
                        tc_fence_before();
                    }
                }
                // P = 2^(s - m) as bf16, 64 keys per head row, in the K-major swizzled layout; the row sums stay fp32
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(lane_bar(L, P_EMPTY + b), (u & 1u) ^ 1u, abort_flag, p.status, limit));
                if (!ok) return false;
                uint8_t* pb = p_lane + b * Cfg::kPBufBytes;
#pragma unroll
                for (int rs = 0; rs < NT; ++rs) {
                    float sum = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float p0 = fast_exp2(sc[rs][2 * i] - m_ref[rs]), p1 = fast_exp2(sc[rs][2 * i + 1] - m_ref[rs]);
                        sum += p0 + p1;
                        if (F8) {
                            // 16 P = hi + lo / 16: hi to row hq, lo to row hq + 8; keys 8i + kq, + 1 are bytes of the row
                            const float y0 = p0 * 16.f, y1 = p1 * 16.f;
                            const uint32_t hi = pack_e4m3(y0, y1);
                            const float2 h = unpack_e4m3(hi);
                            const uint32_t lo = pack_e4m3((y0 - h.x) * 16.f, (y1 - h.y) * 16.f);
                            uint8_t* dst = pb + hq * 128 + (((i >> 1) ^ hq) << 4) + (i & 1) * 8 + kq;
                            *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(hi);
                            *reinterpret_cast<uint16_t*>(dst + 1024) = static_cast<uint16_t>(lo);
                        } else {
                            *reinterpret_cast<uint32_t*>(pb + rs * 1024 + hq * 128 + ((i ^ hq) << 4) + kq * 2) = pack_bf16(p0, p1);
                        }
                    }
                    l_acc[rs] += sum;
                }
                if (valid & (PV_KEYS - 1)) {
                    // the second product takes whole groups of 16 (8-bit slabs: 32) keys: value rows between
                    // the item's end and the end of its last group are zeroed (P is zero there; the rows hold
                    // whatever the slab or the stage did, which may not be a finite number)
                    uint8_t* vt = kv + ((g0 + static_cast<uint32_t>(t)) % STAGES) * Cfg::kStageBytes + Cfg::kKvTileBytes;
                    const int zero_rows = PV_KEYS - (valid & (PV_KEYS - 1));
                    for (int idx = lane; idx < zero_rows * KV_CHUNKS; idx += 32) {
                        const int zr = valid + idx / KV_CHUNKS, cc = idx % KV_CHUNKS;
                        *reinterpret_cast<uint4*>(vt + (cc >> 3) * HALF_BYTES + zr * 128 + (((cc & 7) ^ (zr & 7)) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(lane_bar(L, P_FULL + b));
                ++c;
                return true;
            };
            int t = t_first;
            if (DEFER && t < im.tiles) {
                if (!do_tile(t, true)) break;
                t += t_step;
            }
            if (DEFER && pd_valid) {
                finish(pd_im, pd_li, false, pd_m, pd_l, pd_s, pd_v);
                pd_valid = false;
                if (!ok) break;
            }
            for (; t < im.tiles; t += t_step)
                if (!do_tile(t, !DEFER && t == t_first)) break;
            if (!ok || !have) break;
            if (BOTH && !home) {
                // helper: once its accumulator is complete, (m, l) per head goes to shared memory;
                // the home lane reads the accumulator itself and signs it off
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(lane_bar(L, O_FULL), j & 1u, abort_flag, p.status, limit));
                if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(lane_bar(L, X_EMPTY), (n_helped & 1u) ^ 1u, abort_flag, p.status, limit));
                if (!ok) break;
                ++j;
                ++n_helped;
                l_acc[0] += __shfl_xor_sync(0xFFFFFFFFu, l_acc[0], 1);
                l_acc[0] += __shfl_xor_sync(0xFFFFFFFFu, l_acc[0], 2);
                if ((lane & 3) == 0) *reinterpret_cast<float2*>(x_mine + hq * 2) = make_float2(m_ref[0], l_acc[0]);
                __syncwarp();
                if (lane == 0) mbar_arrive(lane_bar(L, X_FULL));
                continue;
            }

            if (!DEFER) {
                finish(im, li, both, m_ref, l_acc, s_new, v_new);
                if (!ok) break;
                continue;
            }
            pd_im = im;
            pd_li = li;
            pd_valid = true;
#pragma unroll
            for (int rs = 0; rs < NT; ++rs) {
                pd_m[rs] = m_ref[rs];
                pd_l[rs] = l_acc[rs];
                pd_s[rs] = s_new[rs];
            }
            if (im.has_new) {
#pragma unroll
                for (int i = 0; i < D / 8; ++i) pd_v[i] = v_new[i];
            }
        }
    }

    // ---- tear-down: every role comes here, on every path, and tensor memory is given back
    if (!ok) *abort_flag = 1;
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(static_cast<uint32_t>(kTmemCols))
                     : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// launch
// ---------------------------------------------------------------------------------------------

constexpr int kSmemPerCtaMax = 232448;    // most dynamic shared memory one CTA may ask for
constexpr int kMaxDevices = 64;

template <int D, int NT, bool F8>
int umma_stages() {
    using Cfg = UmmaConfig<D, NT, F8>;
    const int n = (kSmemPerCtaMax - Cfg::smem_bytes(0)) / Cfg::kStageBytes;
    return std::min(n, Cfg::kStagesMax);
}

template <int D, int NT, int MODE, bool F8, bool DEFER>
cudaError_t launch_umma_inst(const TensorMaps& maps, DecodeParams p, int n_ctas, cudaStream_t stream,
                             const InlineLens& lens, const SpanParams& sp) {
    using Cfg = UmmaConfig<D, NT, F8>;
    static bool configured[kMaxDevices] = {false};     // the opt-in to large shared memory is per device
    auto kern = decode_umma_kernel<D, NT, MODE, F8, DEFER>;
    p.stages = umma_stages<D, NT, F8>();
    if (p.stages < 2) return cudaErrorInvalidValue;
    const int smem = Cfg::smem_bytes(p.stages);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCtaMax);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas));
    cfg.blockDim = dim3(kUmmaThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(smem);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, maps, p, lens, sp);
}

template <int D, int NT>
cudaError_t launch_umma_mode(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas, cudaStream_t s,
                             const InlineLens& lens, const SpanParams& sp, bool defer) {
    switch (mode) {
        case kModeSlab:
            return defer ? launch_umma_inst<D, NT, kModeSlab, false, true>(maps, p, n_ctas, s, lens, sp)
                         : launch_umma_inst<D, NT, kModeSlab, false, false>(maps, p, n_ctas, s, lens, sp);
        case kModePaged: return launch_umma_inst<D, NT, kModePaged, false, false>(maps, p, n_ctas, s, lens, sp);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool umma_supported(int32_t head_dim, int32_t group, bool kv_fp8) {
    if (kv_fp8) return head_dim == 128 && group >= 1 && group <= 8;
    return (head_dim == 64 || head_dim == 128) && group >= 1 && group <= 16;
}

cudaError_t launch_decode_umma(const TensorMaps& maps, const DecodeParams& p, int mode, int n_ctas,
                               cudaStream_t stream, const InlineLens* lens_in, const SpanParams* span_in, bool defer) {
    static const InlineLens no_lens{};                 // n = 0: lengths as planned
    static const SpanParams no_span{};                 // never read by a one-layer launch
    const InlineLens& lens = lens_in ? *lens_in : no_lens;
    if (p.n_layers > 1 && !span_in) return cudaErrorInvalidValue;
    const SpanParams& sp = span_in ? *span_in : no_span;
    if (p.kv_fp8) {
        if (!umma_supported(p.head_dim, p.group, true) || mode != kModeSlab) return cudaErrorInvalidValue;
        return launch_umma_inst<128, 1, kModeSlab, true, false>(maps, p, n_ctas, stream, lens, sp);
    }
    const bool two = p.group > 8;
    if (p.head_dim == 128)
        return two ? launch_umma_mode<128, 2>(maps, p, mode, n_ctas, stream, lens, sp, defer)
                   : launch_umma_mode<128, 1>(maps, p, mode, n_ctas, stream, lens, sp, defer);
    if (p.head_dim == 64)
        return two ? launch_umma_mode<64, 2>(maps, p, mode, n_ctas, stream, lens, sp, defer)
                   : launch_umma_mode<64, 1>(maps, p, mode, n_ctas, stream, lens, sp, defer);
    return cudaErrorInvalidValue;
}

}  // namespace odma
