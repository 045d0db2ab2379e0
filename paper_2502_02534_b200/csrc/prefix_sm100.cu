// Prefix stage: every sample's query rows of one KV head, batched against the shared
// prompt K/V, on the 5th-generation tensor cores (tcgen05) with accumulators in tensor
// memory (TMEM) and operands brought in by TMA.
//
// Arithmetic: the paper's attn Task 2 recurrence (deferred division).  For one key tile
// with raw scores s = q.k and c = sm_scale * log2(e):
//     m' = max(m, max_j c*s_j),  p_j = 2^(c*s_j - m'),  l' = l * 2^(m - m') + sum_j p_j,
//     O' = O * 2^(m - m') + P V,      and at the end  out = O / l,  lse = (m + log2 l) ln 2.
// The reference maximum is only moved when a tile's maximum exceeds it by more than 2^8
// (the result is unchanged: the factor cancels between O and l), so the accumulator in
// TMEM is almost never rescaled.
//
// One thread block = one work item = (kv head, up to 256 query rows, a range of keys); thread = TMEM lane =
// query row.  Per key tile and row tile:  S = Q K^T (SS MMA, K-major operands, 128-byte swizzle) -> the softmax
// warpgroup reads S from TMEM and writes P (bf16) back to TMEM -> O += P V (TS MMA, P from TMEM, V as MN-major B
// operand).  K/V are read from HBM/L2 once per item.  Three shapes of block, chosen per launch from the plan:
//   two row tiles (some item has > 128 rows), 11 warps, 128-key tiles, ring of 5 tiles:
//     warps 0-3 / 4-7  softmax warpgroup of row tile 0 / 1
//     warp 8           TMA producer: Q once, then K and V tiles through a ring of buffers
//     warp 9           MMA issuer (one lane) and owner of the TMEM allocation
//     warp 10          watcher (one lane): waits for the K/V tiles of each key tile to land and adds its arrival to
//                      the P barrier of row tile 0, so that the issuer polls one barrier per row tile and key tile
//     The two row tiles alternate on the tensor pipe (one tile's softmax overlaps the other's MMAs); P is written
//     over S.  TMEM: S0 S1 at columns 0 / 128, O0 O1 at 256 / 256 + D.
//   one row tile, small (<= 128 rows; short items, or enough rows not to be purely HBM-bound), 8 warps:
//     0-3 softmax, 4 producer, 5 issuer of QK^T, 6 issuer of PV, 7 watcher.  The issuing thread is a serial
//     bottleneck -- between two batches of MMAs it polls barriers and commits, a few hundred cycles of scalar code
//     per tile during which the tensor pipe drains -- so the two kinds of MMA have an issuer each, whose waits
//     overlap the other's MMAs.  <= 144 registers, 129 KB of shared memory: ONE SUFFIX BLOCK FITS BESIDE IT
//     on the SM.  64-key tiles through a ring of 6 (three tiles of look-ahead in 96 KB); S0/S1 alternate by key
//     tile so that QK^T of tile j+1 runs under the softmax of tile j; P has TMEM columns of its own (384..511),
//     which keeps S intact and makes the common softmax a single pass against the current reference maximum.
//   one row tile, long (<= 64 rows and long items: HBM-bound): the same with 128-key tiles, a ring of 6 and no
//     watcher (7 warps); owns the SM.
// The epilogue sends O / l through a padded staging tile laid over the idle ring, so that every global store
// instruction writes one full row.  Launched as a programmatic dependent: set-up (barriers, TMEM) overlaps the
// tail of the preceding kernel, `griddepcontrol.wait` precedes the first memory access, and the suffix stage is
// released to run beside this grid.
//
// Causal mode (prefill: the "samples" of an item are consecutive prompt tokens, its keys the prompt up to the
// item's last token): row r sees key c only if c's packed token index <= the row's own, a per-row bound on the
// valid keys of a tile, so only an item's diagonal tiles leave the unmasked fast path.  A row that has seen no
// key yet keeps m = -inf, l = 0; exponents are taken against 0 instead of -inf, and l = 0 ends as out = 0,
// lse = -inf, which the merge stage ignores.
//
// Every wait on an mbarrier is bounded: when the limit passes, the block raises
// PSA_ERR_TIMEOUT in the status word, stops storing results, and drains to a normal exit
// (TMEM freed) instead of spinning.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr float kRescaleThreshold = 8.f; // log2 units
// bf16 by truncation, unbiased: exponentiate x + log2(1 + 2^-9), truncate, and divide the row sum by (1 + 2^-9) at the end
constexpr float kTruncBias = 0.0028150156f;      // log2(1 + 2^-9)
constexpr float kTruncUnbias = 0.99805068f;      // 1 / (1 + 2^-9)
constexpr float kTileSumLimit = 64.f * 256.f * 1.01f;   // 64 exponentials of at most 2^8 (times the factor above)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit passed or another thread already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs)
{
#pragma unroll 1
    for (int i = 0; i < 64; ++i)   // the common case ends here, without reading the (slow) global timer
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One lane of a converged warp.  Code guarded by this (rather than by a test of the lane index) is known to the
// compiler to run on a single lane, so descriptors and addresses stay in the uniform datapath the tensor-core
// instructions take their operands from; guarded by `lane == 0` every tcgen05.mma cost the issuing thread 90-130
// cycles of register shuffling, more than the 64 cycles the instruction needs to execute.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// D[tmem] (+)= A * B with A from shared memory (mma_ss) or from tensor memory (mma_ts), B from shared memory.
// Shared-memory descriptors are 64-bit values: the high word holds layout constants, the low word the address
// (in 16-byte units), so stepping through a tile is one add.  kAcc: accumulate onto D (compile-time: the predicate
// operand is then an immediate); mma_ts_p takes the flag at run time.
template <bool kAcc>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc)
{
    if constexpr (kAcc)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t db, uint32_t idesc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(db), "r"(idesc) : "memory");
}
__device__ __forceinline__ void mma_ts_p(uint32_t d_tmem, uint32_t a_tmem, uint64_t db, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread = lane (row), register i = column i
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 2^x without the special-function unit: x = n + f with n the nearest integer (magic-number rounding) and f in
// [-0.5, 0.5], a minimax cubic for 2^f (relative error below 7.5e-5, mean error 5e-6), and n added to the exponent bits.
// Three adds, three FMAs, a maximum and two integer operations: more instructions than one ex2, but on pipes that are
// idle while the special-function unit, one exponential per score, is the scarce resource of the softmax pass.
__device__ __forceinline__ float poly_exp2(float x)
{
    x = fmaxf(x, -126.f);                        // below that the result is zero for every purpose here
    const float t = x + 12582912.f;              // 1.5 * 2^23: n lands in the low mantissa bits
    const float f = x - (t - 12582912.f);
    float p = fmaf(f, 0.0551716648f, 0.2426111251f);
    p = fmaf(p, f, 0.6932609677f);
    p = fmaf(p, f, 0.9999280572f);
    // at the clamp (masked keys arrive as -inf) the value is a denormal just below 2^-126: a flushing multiply by one
    // turns it into the exact zero that ex2 returns there
    float r;
    asm("mul.ftz.f32 %0, %1, 0f3F800000;" : "=f"(r) : "f"(__uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23))));
    return r;
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor (tcgen05): start address, leading / stride byte offsets (all in 16-byte units),
// descriptor version 1, 128-byte swizzle.
// The descriptor's two words: only the low one depends on the address, and moving the start by `bytes` adds
// bytes / 16 to it (tiles lie in the low 256 KB of the shared window, so the 14-bit field cannot overflow).
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t addr, uint32_t lbo_bytes) { return ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16); }
__host__ __device__ constexpr uint32_t smem_desc_hi(uint32_t sbo_bytes) { return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29); }
// Instruction descriptor for kind::f16: bf16 x bf16 -> f32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major)
{
    return (1u << 4) /* D = f32 */ | (1u << 7) /* A = bf16 */ | (1u << 10) /* B = bf16 */ |
           (uint32_t(b_mn_major) << 16) | (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

// Shared-memory plan of one block.  kTwo: two row tiles (two Q tiles, 11 warps); otherwise one row
// tile (one Q tile, 7 or 8 warps).
constexpr int kMaxRing = 6;
// Ring length per block shape: 5 x 32 KB beside two Q tiles, else 6 (never fewer buffers than the epilogue
// staging tile needs).
template <int D, bool kTwo, bool kLowReg>
__host__ __device__ constexpr int prefix_ring() { return (kTwo && D == 128) ? 5 : kMaxRing; }
// Keys per tile: 128, except in the small block, whose 96 KB ring then holds six 64-key tiles (three tiles of
// look-ahead) instead of three 128-key tiles (none: every load would wait for the previous tile's MMA).
template <bool kLowReg>
__host__ __device__ constexpr int prefix_tile_keys() { return kLowReg ? 64 : kPrefixTileKeys; }
template <int D, bool kTwo, int kKeys>
struct PrefixSmem {
    static constexpr int kHalves = D / 64;
    static constexpr int kQHalfBytes = kPrefixTileRows * 128;         // one TMA box of Q: 128 rows x 64 bf16
    static constexpr int kQTileBytes = kHalves * kQHalfBytes;
    static constexpr int kHalfBytes = kKeys * 128;                    // one TMA box of K or V: kKeys rows x 64 bf16
    static constexpr int kTileBytes = kHalves * kHalfBytes;           // a K or V tile
    static constexpr int kQTiles = kTwo ? 2 : 1;
    static constexpr int kBarOff = 0;                                 // barriers first, tiles after them
    static constexpr int kNumBars = 1 + 2 * kMaxRing + 4 + 2;         // q, full[], empty[], s_full[2], p_full[2], drain[2]
    static constexpr int kTmemPtrOff = kBarOff + 8 * kNumBars;
    static constexpr int kAbortOff = kTmemPtrOff + 4;
    static constexpr int kQOff = 1024;
    static constexpr int kRingOff = kQOff + kQTiles * kQTileBytes;
    static constexpr int kStageRowFloats = D + 4;                     // padded row of the epilogue staging tile
    static constexpr int kStageBytes = kPrefixTileRows * kStageRowFloats * 4;
    static constexpr int kTmemCols = 512;   // S0 S1 (128 each) at 0; O0 O1 (D each) at 256, or O at 256 and P0 P1 at 384
    __host__ __device__ static constexpr int total(int ring) { return kRingOff + ring * kTileBytes; }
    __host__ __device__ static constexpr int min_ring() { return (kQTiles * kStageBytes + kTileBytes - 1) / kTileBytes; }
};

template <int D, bool kTwo, bool kLowReg>
__device__ __forceinline__ void
prefix_body(const CUtensorMap *pmap_q, const CUtensorMap *pmap_k, const CUtensorMap *pmap_v,
            const PrefixItem *__restrict__ items, int group, int causal, float scale_log2,
            float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status, int *launch_counter,
            int *done_counter)
{
    constexpr int kKeys = prefix_tile_keys<kLowReg>();   // keys per tile
    using L = PrefixSmem<D, kTwo, kKeys>;
    constexpr int ring = prefix_ring<D, kTwo, kLowReg>();   // K/V tile buffers in flight
    constexpr int kSoftmaxWarps = kTwo ? 8 : 4;
    constexpr int kProducerWarp = kSoftmaxWarps, kMmaWarp = kSoftmaxWarps + 1, kMmaWarp2 = kSoftmaxWarps + 2;
    constexpr int kWatchWarp = kSoftmaxWarps + 3;   // one row tile only (with two row tiles the second issuer warp watches)
    // A watcher thread folds the "K/V tile landed" waits into the P barriers.  Measured: it pays in the two-row-tile
    // block (69 instead of 78 us on 2048 rows x 8192 keys x 8 heads) and in the small block that shares its SM with
    // a suffix block (whole step 59.1 instead of 61.6 us on 64 samples x 16384 + U[0,2048] tokens, although that
    // block alone gets 4 % slower); the long one-row-tile block is 4 % slower with it and goes without.
    constexpr bool kWatch = kTwo || kLowReg;
    constexpr int kKSteps = D / 16;                 // MMA k-steps of QK^T
    constexpr int kPSteps = kKeys / 16;   // MMA k-steps of PV
    constexpr uint32_t kIdescQK = make_idesc(kKeys, false);
    constexpr uint32_t kIdescPV = make_idesc(D, true);
    constexpr uint32_t kColS = 0, kColO = 256;   // S buffer b at column 128 b (kKeys of them in use)
    constexpr int kChunks = kKeys / 32;          // 32-column pieces of one S tile
    constexpr uint32_t kColP = 384;   // one row tile only: P0, P1 (64 columns each) behind O

    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {   // swizzled tiles need a 1024-byte aligned base; refuse to run rather than read garbage
        if (threadIdx.x == 0) atomicCAS(status, 0, int(PSA_ERR_BOUNDS));
        return;
    }
    const uint32_t bar0 = sbase + L::kBarOff;
    auto bar_q = [&]() { return bar0; };
    auto bar_full = [&](int i) { return bar0 + 8 * (1 + i); };
    auto bar_empty = [&](int i) { return bar0 + 8 * (1 + kMaxRing + i); };
    auto bar_s = [&](int b) { return bar0 + 8 * (1 + 2 * kMaxRing + b); };
    auto bar_p = [&](int b) { return bar0 + 8 * (3 + 2 * kMaxRing + b); };
    auto bar_drain = [&](int who) { return bar0 + 8 * (5 + 2 * kMaxRing + who); };   // error path only
    volatile uint32_t *tmem_ptr = reinterpret_cast<volatile uint32_t *>(smem + L::kTmemPtrOff);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kAbortOff);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // A counted launch (fused step) announces itself to the merge stage.  This may happen before the wait for the
    // preceding grid: if that grid is the previous step's merge stage, all of its warps have read the counters by
    // the time they let this grid start.  Doing it here hides the round trip behind the set-up.
    if (launch_counter != nullptr && blockIdx.x == 0 && threadIdx.x == 0)
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(launch_counter) : "memory");
    const int4 it0 = __ldg(reinterpret_cast<const int4 *>(items + blockIdx.x));
    const int4 it1 = __ldg(reinterpret_cast<const int4 *>(items + blockIdx.x) + 1);
    const int first_token = it0.x, n_keys = it0.y, kv = it0.z, first_sample = it0.w;
    const int n_rows = it1.x, prow0 = it1.y;
    const int n_tiles = (n_keys + kKeys - 1) / kKeys;
    const int n_rt = kTwo ? (n_rows > kPrefixTileRows ? 2 : 1) : 1;   // row tiles in use
    const int samples_per_tile = kPrefixTileRows / group;

    // Which S buffer / barrier phase serves (row tile t, key tile j):
    //   two row tiles: buffer t, one use per key tile;  one row tile: buffers alternate with j.
    auto sbuf = [&](int t, int j) { return kTwo ? t : (j & 1); };
    auto sphase = [&](int j) { return uint32_t(kTwo ? (j & 1) : ((j >> 1) & 1)); };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar_q(), 1);
        for (int i = 0; i < kMaxRing; ++i) { mbar_init(bar_full(i), 1); mbar_init(bar_empty(i), 1); }
        // p[t]: one arrival per softmax thread of row tile t; with two row tiles p[0] also takes the arrival of the
        // thread that watches the K/V tiles land (see the MMA issuers); with one row tile both p[] are per key tile
        // and both take it
        for (int t = 0; t < 2; ++t) { mbar_init(bar_s(t), 1); mbar_init(bar_p(t), 128 + ((kWatch && (!kTwo || t == 0)) ? 1 : 0)); }
        for (int t = 0; t < 2; ++t) mbar_init(bar_drain(t), 1);
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_ptr)), L::kTmemCols);
        tmem_relinquish();
    }
    if (warp == kProducerWarp && elect_one()) { prefetch_tensormap(pmap_q); prefetch_tensormap(pmap_k); prefetch_tensormap(pmap_v); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;
    // Launched as a programmatic dependent of whatever precedes it in the stream, this block did its set-up
    // while that kernel drained; from here on it reads inputs and (later) overwrites partial results, so the
    // predecessor must be complete.  Only then may our own dependent (the suffix stage) start beside us.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the announcement of a counted launch (see the top of the kernel) is visible before this block lets the suffix
    // grid -- and with it the merge grid -- start
    if (launch_counter != nullptr && blockIdx.x == 0 && threadIdx.x == 0) __threadfence();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            mbar_expect_tx(bar_q(), n_rt * L::kQTileBytes);
            for (int t = 0; t < n_rt; ++t)
                for (int h = 0; h < L::kHalves; ++h)
                    tma_load_4d(sbase + L::kQOff + t * L::kQTileBytes + h * L::kQHalfBytes, pmap_q, bar_q(), h * 64, 0, kv,
                                first_sample + t * samples_per_tile);
            // ring order: K0 V0 K1 V1 ...
            for (int i = 0; i < 2 * n_tiles; ++i) {
                const int slot = i % ring, use = i / ring;
                if (use > 0 && !mbar_wait(bar_empty(slot), (use - 1) & 1, abort_flag)) break;
                const int tok = first_token + (i >> 1) * kKeys;
                const CUtensorMap *map = (i & 1) ? pmap_v : pmap_k;
                mbar_expect_tx(bar_full(slot), L::kTileBytes);
                for (int h = 0; h < L::kHalves; ++h)
                    tma_load_3d(sbase + L::kRingOff + slot * L::kTileBytes + h * L::kHalfBytes, map, bar_full(slot), h * 64, kv, tok);
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp2) {
        // ------------------------------------------------------------ MMA issuers: one lane of each of two warps
        // A single issuing thread is a serial bottleneck: between two batches of MMAs it polls barriers and commits,
        // a few hundred cycles of scalar code each time, during which the tensor pipe drains and idles.  With two
        // issuers the waits of one overlap the MMAs of the other.
        //   two row tiles: thread 0 issues everything, thread 1 only watches the K/V tiles land (see there)
        //   one row tile:  issuer 0 issues every QK^T, issuer 1 every PV
        if (elect_one()) {
            const int who = warp - kMmaWarp;
            auto wait_entry = [&](int e) { return mbar_wait(bar_full(e % ring), (e / ring) & 1, abort_flag); };
            constexpr uint64_t kHi = uint64_t(smem_desc_hi(1024)) << 32;
            const uint64_t q_desc = kHi | smem_desc_lo(sbase + L::kQOff, 16);
            const uint64_t ring_k_desc = kHi | smem_desc_lo(sbase + L::kRingOff, 16);            // K tiles: K-major, no leading offset
            const uint64_t ring_v_desc = kHi | smem_desc_lo(sbase + L::kRingOff, L::kHalfBytes); // V tiles: MN-major, halves kHalfBytes apart
            auto issue_qk = [&](int t, int sb, int kslot) {   // S[sb] = Q_t K^T, K in ring slot `kslot`
                const uint64_t a = q_desc + uint32_t(t) * (L::kQTileBytes >> 4);
                const uint64_t b = ring_k_desc + uint32_t(kslot) * (L::kTileBytes >> 4);
                const uint32_t d = tmem_base + kColS + uint32_t(sb) * 128;
#pragma unroll
                for (int k = 0; k < kKSteps; ++k) {
                    const uint64_t ak = a + (((k / 4) * L::kQHalfBytes + (k % 4) * 32) >> 4);
                    const uint64_t bk = b + (((k / 4) * L::kHalfBytes + (k % 4) * 32) >> 4);
                    if (k == 0) mma_ss<false>(d, ak, bk, kIdescQK);
                    else mma_ss<true>(d, ak, bk, kIdescQK);
                }
            };
            auto issue_pv = [&](int t, uint32_t p_tmem, int vslot, bool first) {   // O_t += P V, V in ring slot `vslot`
                const uint64_t b = ring_v_desc + uint32_t(vslot) * (L::kTileBytes >> 4);
                const uint32_t d = tmem_base + kColO + t * D;
#pragma unroll
                for (int k = 0; k < kPSteps; ++k) {
                    if (k == 0) mma_ts_p(d, p_tmem, b, kIdescPV, first ? 0u : 1u);
                    else mma_ts(d, p_tmem + k * 8, b + ((k * 2048) >> 4), kIdescPV);
                }
            };
            auto next_slot = [&](int sl, int by) { sl += by; return sl >= ring ? sl - ring : sl; };
            if constexpr (kTwo) {
                // Two row tiles: ONE issuer, which alternates between the tiles (two threads issuing into the same
                // pipe measured slower here: 95 us instead of 77 us on 2048 rows x 8192 keys x 8 heads).  The second
                // thread only watches the K/V tiles land: per key tile j it waits for V_j and K_{j+1} and then adds
                // its arrival to p[0], so that the issuer, whose every poll costs the tensor pipe idle time, has one
                // wait per row tile and key tile (P ready, which now also says "operands landed") instead of three.
                if (who == 1) {
                    bool landed = true;
                    for (int j = 0; landed && j < n_tiles; ++j) {
                        if (j > 0) landed = mbar_wait(bar_p(0), sphase(j - 1), abort_flag);   // one arrival per phase of p[0]
                        if (landed) landed = wait_entry(2 * j + 1);                           // V_j
                        if (landed && j + 1 < n_tiles) landed = wait_entry(2 * j + 2);        // K_{j+1}
                        if (landed) mbar_arrive(bar_p(0));
                    }
                }
                bool ok = who == 0;
                if (ok) ok = mbar_wait(bar_q(), 0, abort_flag);
                if (ok) ok = wait_entry(0);   // K_0
                if (ok) {
                    tc_fence_after();
                    for (int t = 0; t < n_rt; ++t) { issue_qk(t, t, 0); tc_commit(bar_s(t)); }
                    tc_commit(bar_empty(0));                       // K_0 is free once both QK^T are done
                }
                int vslot = 1;   // ring slot of V_j; K_{j+1} is in the next one
                for (int j = 0; ok && j < n_tiles; ++j) {
                    const int kslot = next_slot(vslot, 1);
                    for (int t = 0; t < n_rt; ++t) {
                        // p[0] of tile j completes only after V_j and K_{j+1} have landed (the watcher's arrival)
                        if (!(ok = mbar_wait(bar_p(t), sphase(j), abort_flag))) break;
                        tc_fence_after();
                        issue_pv(t, tmem_base + kColS + t * 128 /* P over S */, vslot, j == 0);
                        if (t == n_rt - 1) tc_commit(bar_empty(vslot));
                        if (j + 1 < n_tiles) {
                            issue_qk(t, t, kslot);
                            tc_commit(bar_s(t));
                            if (t == n_rt - 1) tc_commit(bar_empty(kslot));
                        }
                    }
                    vslot = next_slot(vslot, 2);
                }
            } else if (who == 0) {
                // QK^T issuer.  S0/S1 alternate by key tile, so QK^T of tile j+1 runs under the softmax of tile j;
                // S[j & 1] may be overwritten (by tile j+2) once the softmax of tile j has handed over its P.
                bool ok = mbar_wait(bar_q(), 0, abort_flag);
                for (int j = 0; ok && j < 2 && j < n_tiles; ++j) {
                    if (!(ok = wait_entry(2 * j))) break;
                    tc_fence_after();
                    issue_qk(0, j & 1, (2 * j) % ring);
                    tc_commit(bar_s(j & 1));
                    tc_commit(bar_empty((2 * j) % ring));
                }
                int kslot = 4 % ring;   // ring slot of K_{j+2} = entry 2j+4
                for (int j = 0; ok && j + 2 < n_tiles; ++j) {
                    // p[j & 1] of tile j: P handed over and, with a watcher, V_j and K_{j+2} landed (its arrival)
                    if (!kWatch && !(ok = wait_entry(2 * j + 4))) break;
                    if (!(ok = mbar_wait(bar_p(j & 1), sphase(j), abort_flag))) break;
                    tc_fence_after();
                    issue_qk(0, j & 1, kslot);
                    tc_commit(bar_s(j & 1));
                    tc_commit(bar_empty(kslot));
                    kslot = next_slot(kslot, 2);
                }
            } else {
                // PV issuer
                bool ok = true;
                int vslot = 1 % ring;   // ring slot of V_j = entry 2j+1
                for (int j = 0; ok && j < n_tiles; ++j) {
                    if (!kWatch && !(ok = wait_entry(2 * j + 1))) break;
                    if (!(ok = mbar_wait(bar_p(j & 1), sphase(j), abort_flag))) break;
                    tc_fence_after();
                    issue_pv(0, tmem_base + kColP + (j & 1) * 64, vslot, j == 0);
                    tc_commit(bar_empty(vslot));
                    vslot = next_slot(vslot, 2);
                }
            }
        }
    } else if (!kTwo && kWatch && warp == kWatchWarp) {
        // ------------------------------------------------------------ watcher (one row tile): per key tile j it waits
        // for V_j and K_{j+2} to land and then adds its arrival to p[j & 1], so that the two issuers poll one barrier each
        if (elect_one()) {
            bool landed = true;
            for (int j = 0; landed && j < n_tiles; ++j) {
                if (j >= 2) landed = mbar_wait(bar_p(j & 1), sphase(j - 2), abort_flag);   // one arrival per phase
                if (landed) landed = mbar_wait(bar_full((2 * j + 1) % ring), ((2 * j + 1) / ring) & 1, abort_flag);
                if (landed && j + 2 < n_tiles) landed = mbar_wait(bar_full((2 * j + 4) % ring), ((2 * j + 4) / ring) & 1, abort_flag);
                if (landed) mbar_arrive(bar_p(j & 1));
            }
        }
    } else if (warp < 4 * n_rt) {
        // ------------------------------------------------------------ softmax + epilogue
        const int t = warp >> 2;                       // row tile
        const int row = (warp & 3) * 32 + lane;        // row inside the tile = TMEM lane
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        const uint32_t o_addr = tmem_base + lane_addr + kColO + t * D;
        float m_ref = -INFINITY, l_sum = 0.f;
        bool ok = true;
        uint32_t sreg[4][32];
        for (int j = 0; j < n_tiles; ++j) {
            const int b = sbuf(t, j);
            const uint32_t s_addr = tmem_base + lane_addr + kColS + b * 128;
            if (!(ok = mbar_wait(bar_s(b), sphase(j), abort_flag))) break;
            tc_fence_after();
            // keys of this tile the row may see: all that exist (< kKeys only on the last tile) and, under the causal
            // mask of a prefill, only those up to the row's own token (rows and keys share the packed token index)
            int valid = n_keys - j * kKeys;
            if (causal) valid = min(valid, first_sample + (t * kPrefixTileRows + row) / group - (first_token + j * kKeys) + 1);

            // Rescale the accumulator in TMEM by 2^(m_ref - m_new) for the rows whose reference maximum moves.
            // The whole warp comes here together because TMEM loads and stores are warp-collective.
            auto move_reference = [&](bool need, float m_new) -> bool {
                const float alpha = need ? fast_exp2(m_ref - m_new) : 1.f;   // 0 on the first tile
                if (j > 0) {
                    // O must be quiescent: PV of tile j-1 has to be complete, which is what releases the ring
                    // buffer of V_{j-1} (PV of tile j cannot start before this thread hands over P)
                    if (!mbar_wait(bar_empty((2 * j - 1) % ring), ((2 * j - 1) / ring) & 1, abort_flag)) return false;
                    tc_fence_after();
                    uint32_t oreg[32];
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        tmem_ld32(o_addr + c * 32, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) oreg[i] = __float_as_uint(__uint_as_float(oreg[i]) * alpha);
                        tmem_st32(o_addr + c * 32, oreg);
                    }
                    tmem_wait_st();
                }
                l_sum *= alpha;
                if (need) m_ref = m_new;
                return true;
            };

            float tile_sum = 0.f;   // the row's sum over this tile (times 1 + 2^-9, see exp_in_place)
            if constexpr (kTwo) {
                // ---- S in registers; P (bf16) is written back over the first 64 columns of S.
                // Common case: ONE pass that exponentiates against the current reference maximum while tracking the
                // largest exponent.  Only if that exceeds the threshold (or on a row's first visible keys) is S read
                // again from tensor memory -- P has not been stored yet, so it is still there -- and the tile redone
                // the classic way: maximum, move the reference (rescaling O), exponentials.
                auto load_s = [&]() {
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, sreg[c]);
                    tmem_wait_ld();
                    if (valid < kKeys) {   // last tile of a ragged prompt, or the diagonal of a prefill: masked keys become -inf
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (c * 32 + i >= valid) sreg[c][i] = 0xff800000u;
                    }
                };
                // sreg: 128 scores -> 64 words of packed bf16 P (in sreg[0], sreg[1]); returns the row's sum of the tile.
                // bf16 by truncation (a byte permute on the integer pipe: the special-function unit does the
                // exponentials and nothing else), unbiased by exponentiating x + log2(1 + 2^-9); no running maximum: a
                // tile sum above kKeys * 2^8 is what tells that some exponent exceeded the threshold.
                auto exp_in_place = [&]() -> float {
                    const float off = kTruncBias - (m_ref == -INFINITY ? 0.f : m_ref);   // no key seen yet: exponentiate against 0
                    float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            const float p0 = fast_exp2(fmaf(__uint_as_float(sreg[c][i]), scale_log2, off));
                            const float p1 = fast_exp2(fmaf(__uint_as_float(sreg[c][i + 1]), scale_log2, off));
                            sum[(i >> 1) & 3] += p0 + p1;
                            sreg[c / 2][(c % 2) * 16 + i / 2] = __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
                        }
                    }
                    return (sum[0] + sum[1]) + (sum[2] + sum[3]);
                };
                load_s();
                bool redo = j == 0;   // nothing to exponentiate against yet
                if (j > 0) {
                    tile_sum = exp_in_place();
                    redo = __any_sync(0xffffffffu, !(tile_sum <= float(kKeys) * 256.f * 1.01f) || (m_ref == -INFINITY && valid > 0));
                    if (redo) load_s();
                }
                if (redo) {
                    float mx[8] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i) mx[i & 7] = fmaxf(mx[i & 7], __uint_as_float(sreg[c][i]));   // eight independent chains
                    const float tmax = scale_log2 * fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                    // move the reference maximum only when a logit exceeds it by more than the threshold
                    const bool need = tmax > m_ref + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, need)) {
                        if (!(ok = move_reference(need, tmax))) break;
                    }
                    tile_sum = exp_in_place();
                }
                tmem_st32(s_addr, sreg[0]);
                tmem_st32(s_addr + 32, sreg[1]);
            } else {
                // ---- one row tile: P has TMEM columns of its own, so S stays intact and the common case is a
                // single pass that exponentiates against the CURRENT reference maximum while tracking the
                // largest exponent; only if that exceeds the threshold (or on the first tile) is the tile redone
                // after moving the reference.  S is streamed 32 columns at a time (two chunks in flight).
                const uint32_t p_addr = tmem_base + lane_addr + kColP + b * 64;
                // P[b] was last read by the PV of tile j-2, which a different thread issues than the QK^T that made this S
                if (j >= 2 && !(ok = mbar_wait(bar_empty((2 * j - 3) % ring), ((2 * j - 3) / ring) & 1, abort_flag))) break;
                auto exp_pass = [&]() -> float {   // the same truncating, bias-cancelling form as above, 32 columns at a time
                    const float off = kTruncBias - (m_ref == -INFINITY ? 0.f : m_ref);   // no key seen yet: exponentiate against 0
                    uint32_t r[2][32];
                    float sum[4] = {0.f, 0.f, 0.f, 0.f};
                    tmem_ld32(s_addr, r[0]);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        if (c + 1 < kChunks) tmem_ld32(s_addr + (c + 1) * 32, r[(c + 1) & 1]);
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            float x0 = fmaf(__uint_as_float(r[c & 1][i]), scale_log2, off);
                            float x1 = fmaf(__uint_as_float(r[c & 1][i + 1]), scale_log2, off);
                            if (valid < kKeys) {   // masked keys of a ragged last tile
                                if (c * 32 + i >= valid) x0 = -INFINITY;
                                if (c * 32 + i + 1 >= valid) x1 = -INFINITY;
                            }
                            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                            sum[(i >> 1) & 3] += p0 + p1;
                            pk[i / 2] = __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
                        }
                        tmem_st16(p_addr + c * 16, pk);
                        tmem_wait_ld();
                    }
                    return (sum[0] + sum[1]) + (sum[2] + sum[3]);
                };
                bool redo = j == 0;   // nothing to exponentiate against yet
                if (j > 0) {
                    tile_sum = exp_pass();
                    // redo when an exponent exceeded the threshold (the sum tells) or a row meets its first visible key
                    redo = __any_sync(0xffffffffu, !(tile_sum <= float(kKeys) * 256.f * 1.01f) || (m_ref == -INFINITY && valid > 0));
                }
                if (redo) {
                    // the tile's maximum, then the classic update, then the exponentials again
                    uint32_t r[2][32];
                    float mx[2] = {-INFINITY, -INFINITY};
                    tmem_ld32(s_addr, r[0]);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        if (c + 1 < kChunks) tmem_ld32(s_addr + (c + 1) * 32, r[(c + 1) & 1]);
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (valid >= kKeys || c * 32 + i < valid) mx[i & 1] = fmaxf(mx[i & 1], __uint_as_float(r[c & 1][i]));
                        tmem_wait_ld();
                    }
                    const float tmax = scale_log2 * fmaxf(mx[0], mx[1]);
                    const bool need = tmax > m_ref + kRescaleThreshold;
                    if (!(ok = move_reference(need, tmax))) break;
                    tile_sum = exp_pass();
                }
            }
            l_sum += tile_sum;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p(b));
        }
        // ---- epilogue: out = O / l, lse = (m + log2 l) ln 2.  The tile goes through shared memory (the
        // ring is idle by now) so that every global store instruction writes one full 4*D-byte row.
        // The release of the last V buffer follows the last MMA of the block (of both row tiles): O is final
        // and nothing reads the ring any more, so the staging tile may overlay it.
        l_sum *= kTruncUnbias;   // the row sums carry the factor (1 + 2^-9) of the truncation trick
        if (ok) ok = mbar_wait(bar_empty((2 * n_tiles - 1) % ring), ((2 * n_tiles - 1) / ring) & 1, abort_flag);
        float *stage = reinterpret_cast<float *>(smem + L::kRingOff + t * L::kStageBytes);
        if (ok) {
            tc_fence_after();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;   // a row that saw no key in this item: O = 0, lse = -inf
            float *mine = stage + row * L::kStageRowFloats;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t oreg[32];
                tmem_ld32(o_addr + c * 32, oreg);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<float4 *>(mine + c * 32 + i) =
                        make_float4(__uint_as_float(oreg[i]) * inv, __uint_as_float(oreg[i + 1]) * inv,
                                    __uint_as_float(oreg[i + 2]) * inv, __uint_as_float(oreg[i + 3]) * inv);
            }
            const int r = t * kPrefixTileRows + row;
            if (r < n_rows) partial_lse[prow0 + r] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
        }
        // the four warps of this row tile meet (named barrier 1 + t), then write rows round-robin
        asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");
        if (!*abort_flag) {
            constexpr int kLanesPerRow = D / 4;                    // float4 per row: 32 or 16
            constexpr int kRowsPerInstr = 32 / kLanesPerRow;       // 1 or 2
            const int sub = lane / kLanesPerRow, col = (lane % kLanesPerRow) * 4;
            const int rows_here = min(kPrefixTileRows, n_rows - t * kPrefixTileRows);
            for (int r = (warp & 3) * kRowsPerInstr + sub; r < rows_here; r += 4 * kRowsPerInstr) {
                const float4 v = *reinterpret_cast<const float4 *>(stage + r * L::kStageRowFloats + col);
                *reinterpret_cast<float4 *>(partial_o + size_t(prow0 + t * kPrefixTileRows + r) * D + col) = v;
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicCAS(status, 0, int(PSA_ERR_TIMEOUT));
        // let copies that were already issued land before the block's shared memory is released
        if (warp == kProducerWarp && lane == 0) {
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 2000000ull) { }
        }
        // Tensor memory is freed below.  MMAs that an issuing thread had queued before it gave up may still be
        // running, so each issuing thread commits once more -- the commit completes when every tensor-core
        // operation that thread issued has retired -- and waits for that (bounded: 2 ms is thousands of times
        // the longest queue this block can hold; nothing waits on these two barriers otherwise).
        if ((warp == kMmaWarp || warp == kMmaWarp2) && elect_one()) {   // the lane that issued the MMAs
            const uint32_t bar = bar_drain(warp - kMmaWarp);
            tc_commit(bar);
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(bar, 0) && global_timer_ns() - t0 < 2000000ull) { }
        }
        __syncthreads();
    }
    // Every result of this block is stored (the barrier above): count the block off for the merge stage of a fused
    // step, which is ordered behind the suffix grid only.
    if (done_counter != nullptr && threadIdx.x == 0)   // a release reduction: nothing comes back, the thread does not wait
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(done_counter) : "memory");
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, L::kTmemCols);
    }
}

template <int D>
__global__ void __launch_bounds__(352, 1)
prefix_kernel_two(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const PrefixItem *__restrict__ items, int group, int causal,
                  float scale_log2, float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status,
                   int *launch_counter, int *done_counter)
{
    prefix_body<D, true, false>(&map_q, &map_k, &map_v, items, group, causal, scale_log2, partial_o, partial_lse, status, launch_counter,
                           done_counter);
}

// At most 144 registers per thread: two of these warps and one suffix warp (208) fit the 512 registers per lane of
// an SM sub-partition, which is what lets a suffix block run beside this block.
template <int D>
__global__ void __maxnreg__(144)
prefix_kernel_one(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const PrefixItem *__restrict__ items, int group, int causal,
                  float scale_log2, float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status,
                   int *launch_counter, int *done_counter)
{
    prefix_body<D, false, true>(&map_q, &map_k, &map_v, items, group, causal, scale_log2, partial_o, partial_lse, status, launch_counter,
                           done_counter);
}

// One row tile, long items: the block owns the SM anyway (long ring), so S stays in registers.
template <int D>
__global__ void __launch_bounds__(224, 1)
prefix_kernel_one_long(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const PrefixItem *__restrict__ items, int group, int causal,
                       float scale_log2, float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status,
                        int *launch_counter, int *done_counter)
{
    prefix_body<D, false, false>(&map_q, &map_k, &map_v, items, group, causal, scale_log2, partial_o, partial_lse, status, launch_counter,
                            done_counter);
}

// ---------------------------------------------------------------------------------------------------------------
// Decoupled block: two softmax warpgroups ("streams") whose score tiles are produced TWO steps ahead.
//
// The blocks above make a stream's next score tile only after its current probabilities have been consumed (P is
// written over S and there is one S buffer per stream), so every key tile costs a stream the whole chain
// S ready -> softmax pass -> P ready -> PV -> QK^T -> S ready, and the tensor pipe idles for the part of it that the
// other stream's work does not cover.  Here a key tile has 64 keys, which leaves tensor memory for TWO S buffers per
// stream (4 x 64 columns) beside the two accumulators (2 x D columns): QK^T of step j + 2 is issued right behind PV
// of step j, so that S of step j + 1 is already complete when a warpgroup finishes step j.  The warpgroups then run
// their passes back to back and the issuing thread finds P waiting: the block is bound by the tensor pipe (8 SS MMAs
// of 48 cycles + 4 TS MMAs of 64 cycles per 128 rows x 64 keys) instead of by the chain.
//
// Two forms of "stream":
//   kPing == false  two ROW tiles of 128 rows share every K/V tile (items of up to 256 rows): stream t = row tile t.
//   kPing == true   ONE row tile (items of up to 128 rows), the streams take alternate KEY tiles (stream t: tiles
//                   t, t + 2, ...), each with its own accumulator and running (m, l); the two are combined in the
//                   epilogue (the same identity the merge stage uses).  Both warpgroups work for every row count.
// K and V tiles travel through a ring each; the producer issues K `kLead` tiles ahead of V (the distance between a
// tile's QK^T and its PV).  11 warps: 0-3 / 4-7 softmax warpgroups, 8 TMA producer, 9 / 10 MMA issuer of stream 0 / 1
// (warp 9 owns the tensor memory allocation).  The block owns its SM (all 227 KB of shared memory at head dimension 128).
template <int D, bool kPing>
struct PrefixSmem2 {
    static constexpr int kKeys = 64;
    static constexpr int kHalves = D / 64;
    static constexpr int kQTiles = kPing ? 1 : 2;
    static constexpr int kQHalfBytes = kPrefixTileRows * 128;
    static constexpr int kQTileBytes = kHalves * kQHalfBytes;
    static constexpr int kHalfBytes = kKeys * 128;                    // one TMA box of K or V: 64 rows x 64 bf16
    static constexpr int kTileBytes = kHalves * kHalfBytes;
    // Ring lengths: all of the 227 KB, a tile takes 1.5-2 us to arrive.  With alternate key tiles the lengths must be
    // EVEN, so that a slot only ever holds tiles of one stream: that stream's issuer then waits on every phase of the
    // slot's "landed" barrier in turn.  With an odd length a slot would alternate between the streams, each issuer
    // would see only every other phase, and a parity wait two phases ahead of the barrier reads as satisfied -- the
    // issuer would run ahead of a tile of the other stream that is still in flight (seen as a launch failure when
    // the block shared the memory system with a bandwidth-bound grid and tiles landed far out of order).
    static constexpr int kRK = 6, kRV = kPing ? 6 : 4;
    static constexpr int kLead = kPing ? 4 : 2;                       // K tiles issued before the first V tile
    // barriers (8 bytes each)
    static constexpr int kBarQ = 0, kBarKFull = 1, kBarKEmpty = kBarKFull + kRK, kBarVFull = kBarKEmpty + kRK,
                         kBarVEmpty = kBarVFull + kRV, kBarS = kBarVEmpty + kRV, kBarP = kBarS + 4, kBarPV = kBarP + 4,
                         kBarDone = kBarPV + 4, kBarDrain = kBarDone + 1, kNumBars = kBarDrain + 2;
    static constexpr int kTmemPtrOff = 8 * kNumBars;
    static constexpr int kAbortOff = kTmemPtrOff + 4;
    static constexpr int kExchangeOff = 1024;                         // kPing: (m, l) of every row of both streams, 2 KB
    static constexpr int kQOff = 3072;
    static constexpr int kKRingOff = kQOff + kQTiles * kQTileBytes;
    static constexpr int kVRingOff = kKRingOff + kRK * kTileBytes;
    static constexpr int kTotal = kVRingOff + kRV * kTileBytes;
    static constexpr int kStageRowFloats = D + 4;
    static constexpr int kStageBytes = kPrefixTileRows * kStageRowFloats * 4;   // staging tile(s) overlay Q and the rings
    static constexpr int kTmemCols = 512;                             // S[t][b] at 64 (2 t + b); O[t] at 256 + t D
    static_assert(kAbortOff + 4 <= kExchangeOff && kTotal <= 227 * 1024 && kQTiles * kStageBytes <= kTotal - kQOff, "shared memory plan");
    static_assert(!kPing || (kRK % 2 == 0 && kRV % 2 == 0), "a ring slot must belong to one stream");
};

template <int D, bool kPing>
__device__ __forceinline__ void
prefix_body2(const CUtensorMap *pmap_q, const CUtensorMap *pmap_k, const CUtensorMap *pmap_v,
             const PrefixItem *__restrict__ items, int group, int causal, float scale_log2,
             float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status, int *launch_counter,
             int *done_counter)
{
    using L = PrefixSmem2<D, kPing>;
    constexpr int kKeys = L::kKeys;
    constexpr int kProducerWarp = 8, kMmaWarp = 9;
    constexpr int kKSteps = D / 16, kPSteps = kKeys / 16;
    constexpr uint32_t kIdescQK = make_idesc(kKeys, false);
    constexpr uint32_t kIdescPV = make_idesc(D, true);
    constexpr uint32_t kColO = 256;

    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {   // swizzled tiles need a 1024-byte aligned base; refuse to run rather than read garbage
        if (threadIdx.x == 0) atomicCAS(status, 0, int(PSA_ERR_BOUNDS));
        return;
    }
    auto bar = [&](int i) { return sbase + 8 * i; };
    auto bar_s = [&](int t, int b) { return bar(L::kBarS + 2 * t + b); };     // S[t][b] complete (tcgen05.commit)
    auto bar_p = [&](int t, int b) { return bar(L::kBarP + 2 * t + b); };     // P written over S[t][b] (128 softmax threads)
    auto bar_pv = [&](int t, int b) { return bar(L::kBarPV + 2 * t + b); };   // the PV that read that P is complete: O[t] quiescent
    volatile uint32_t *tmem_ptr = reinterpret_cast<volatile uint32_t *>(smem + L::kTmemPtrOff);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + L::kAbortOff);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (launch_counter != nullptr && blockIdx.x == 0 && threadIdx.x == 0)
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(launch_counter) : "memory");
    const int4 it0 = __ldg(reinterpret_cast<const int4 *>(items + blockIdx.x));
    const int4 it1 = __ldg(reinterpret_cast<const int4 *>(items + blockIdx.x) + 1);
    const int first_token = it0.x, n_keys = it0.y, kv = it0.z, first_sample = it0.w;
    const int n_rows = it1.x, prow0 = it1.y;
    const int n_tiles = (n_keys + kKeys - 1) / kKeys;
    const int samples_per_tile = kPrefixTileRows / group;
    // stream t, step j  ->  key tile, and how many steps the stream has
    const int n_streams = kPing ? (n_tiles > 1 ? 2 : 1) : (n_rows > kPrefixTileRows ? 2 : 1);
    auto key_tile = [&](int t, int j) { return kPing ? 2 * j + t : j; };
    auto n_steps = [&](int t) { return t >= n_streams ? 0 : (kPing ? (n_tiles - t + 1) / 2 : n_tiles); };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar(L::kBarQ), 1);
        // a ring slot is free again when every stream that reads the tile has consumed it: both row tiles, or the
        // one stream an alternate key tile belongs to
        const int users = kPing ? 1 : n_streams;
        for (int i = 0; i < L::kRK; ++i) { mbar_init(bar(L::kBarKFull + i), 1); mbar_init(bar(L::kBarKEmpty + i), users); }
        for (int i = 0; i < L::kRV; ++i) { mbar_init(bar(L::kBarVFull + i), 1); mbar_init(bar(L::kBarVEmpty + i), users); }
        for (int i = 0; i < 4; ++i) { mbar_init(bar(L::kBarS + i), 1); mbar_init(bar(L::kBarP + i), 128); mbar_init(bar(L::kBarPV + i), 1); }
        mbar_init(bar(L::kBarDone), 2);   // one arrival per issuing thread
        mbar_init(bar(L::kBarDrain), 1);
        mbar_init(bar(L::kBarDrain + 1), 1);
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_ptr)), L::kTmemCols);
        tmem_relinquish();
    }
    if (warp == kProducerWarp && elect_one()) { prefetch_tensormap(pmap_q); prefetch_tensormap(pmap_k); prefetch_tensormap(pmap_v); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (launch_counter != nullptr && blockIdx.x == 0 && threadIdx.x == 0) __threadfence();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            const int q_tiles = kPing ? 1 : n_streams;
            mbar_expect_tx(bar(L::kBarQ), q_tiles * L::kQTileBytes);
            for (int t = 0; t < q_tiles; ++t)
                for (int h = 0; h < L::kHalves; ++h)
                    tma_load_4d(sbase + L::kQOff + t * L::kQTileBytes + h * L::kQHalfBytes, pmap_q, bar(L::kBarQ), h * 64, 0, kv,
                                first_sample + t * samples_per_tile);
            bool ok = true;
            auto load = [&](bool is_v, int i) {   // key tile i of K or V into its ring
                const int ring = is_v ? L::kRV : L::kRK;
                const int slot = i % ring, use = i / ring;
                const uint32_t full = bar((is_v ? L::kBarVFull : L::kBarKFull) + slot), empty = bar((is_v ? L::kBarVEmpty : L::kBarKEmpty) + slot);
                if (use > 0 && !(ok = mbar_wait(empty, (use - 1) & 1, abort_flag))) return;
                mbar_expect_tx(full, L::kTileBytes);
                const uint32_t dst = sbase + (is_v ? L::kVRingOff : L::kKRingOff) + slot * L::kTileBytes;
                for (int h = 0; h < L::kHalves; ++h)
                    tma_load_3d(dst + h * L::kHalfBytes, is_v ? pmap_v : pmap_k, full, h * 64, kv, first_token + i * kKeys);
            };
            for (int i = 0; ok && i < L::kLead && i < n_tiles; ++i) load(false, i);
            for (int i = 0; ok && i < n_tiles; ++i) {
                load(true, i);
                if (ok && i + L::kLead < n_tiles) load(false, i + L::kLead);
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // ------------------------------------------------------------ MMA issuers: one elected lane per stream.
        // A stream's issuer has about 640 tensor-pipe cycles of its own MMAs per step and the same again of the other
        // stream's to do its waits and commits in; one thread serving both streams could not keep up (a satisfied
        // barrier wait still costs it 100-200 cycles, and a step has three).
        const int t = warp - kMmaWarp;
        if (elect_one()) {
            constexpr uint64_t kHi = uint64_t(smem_desc_hi(1024)) << 32;
            const uint64_t q_desc = (kHi | smem_desc_lo(sbase + L::kQOff, 16)) + uint32_t(kPing ? 0 : t) * (L::kQTileBytes >> 4);
            const uint64_t k_desc = kHi | smem_desc_lo(sbase + L::kKRingOff, 16);              // K-major, no leading offset
            const uint64_t v_desc = kHi | smem_desc_lo(sbase + L::kVRingOff, L::kHalfBytes);   // MN-major, halves kHalfBytes apart
            const uint32_t o_tmem = tmem_base + kColO + t * D;
            auto wait_k = [&](int i) { return mbar_wait(bar(L::kBarKFull + i % L::kRK), (i / L::kRK) & 1, abort_flag); };
            auto wait_v = [&](int i) { return mbar_wait(bar(L::kBarVFull + i % L::kRV), (i / L::kRV) & 1, abort_flag); };
            auto issue_qk = [&](int b, int i) {   // S[t][b] = Q K_i^T
                const uint64_t kb = k_desc + uint32_t(i % L::kRK) * (L::kTileBytes >> 4);
                const uint32_t d = tmem_base + uint32_t(2 * t + b) * 64;
#pragma unroll
                for (int k = 0; k < kKSteps; ++k) {
                    const uint64_t ak = q_desc + (((k / 4) * L::kQHalfBytes + (k % 4) * 32) >> 4);
                    const uint64_t bk = kb + (((k / 4) * L::kHalfBytes + (k % 4) * 32) >> 4);
                    if (k == 0) mma_ss<false>(d, ak, bk, kIdescQK);
                    else mma_ss<true>(d, ak, bk, kIdescQK);
                }
                tc_commit(bar_s(t, b));
                tc_commit(bar(L::kBarKEmpty + i % L::kRK));
            };
            auto issue_pv = [&](int b, int i, bool first) {   // O[t] += P V_i, P in the first 32 columns of S[t][b]
                const uint64_t vb = v_desc + uint32_t(i % L::kRV) * (L::kTileBytes >> 4);
                const uint32_t p_tmem = tmem_base + uint32_t(2 * t + b) * 64;
#pragma unroll
                for (int k = 0; k < kPSteps; ++k) {
                    if (k == 0) mma_ts_p(o_tmem, p_tmem, vb, kIdescPV, first ? 0u : 1u);
                    else mma_ts(o_tmem, p_tmem + k * 8, vb + ((k * 2048) >> 4), kIdescPV);
                }
                tc_commit(bar_pv(t, b));
                tc_commit(bar(L::kBarVEmpty + i % L::kRV));
            };
            const int steps = n_steps(t);
            bool ok = steps > 0;
            if (ok) ok = mbar_wait(bar(L::kBarQ), 0, abort_flag);
            // prologue: the stream's first two score tiles
            for (int j = 0; ok && j < 2 && j < steps; ++j) {
                const int i = key_tile(t, j);
                if (!(ok = wait_k(i))) break;
                tc_fence_after();
                issue_qk(j, i);
            }
            for (int j = 0; ok && j < steps; ++j) {
                const int i = key_tile(t, j), b = j & 1;
                if (!(ok = wait_v(i))) break;
                if (!(ok = mbar_wait(bar_p(t, b), (j >> 1) & 1, abort_flag))) break;
                tc_fence_after();
                issue_pv(b, i, j == 0);
                if (j + 2 < steps) {
                    const int i2 = key_tile(t, j + 2);
                    if (!(ok = wait_k(i2))) break;
                    tc_fence_after();
                    issue_qk(b, i2);   // overwrites P of step j: ordered behind the PV just issued
                }
            }
            // when this barrier flips, every MMA of both issuers is complete
            if (ok && steps > 0) tc_commit(bar(L::kBarDone));
            else mbar_arrive(bar(L::kBarDone));
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------ softmax warpgroups + epilogue
        const int t = warp >> 2;                       // stream
        const int row = (warp & 3) * 32 + lane;        // row inside the row tile = TMEM lane
        const int row_tile = kPing ? 0 : t;
        const uint32_t lane_addr = uint32_t((warp & 3) * 32) << 16;
        const uint32_t o_addr = tmem_base + lane_addr + kColO + t * D;
        const int my_steps = n_steps(t);
        float m_ref = -INFINITY, l_sum = 0.f;
        bool ok = true;
        uint32_t sreg[2][32];
        for (int j = 0; j < my_steps; ++j) {
            const int b = j & 1, i = key_tile(t, j);
            const uint32_t s_addr = tmem_base + lane_addr + uint32_t(2 * t + b) * 64;
            if (!(ok = mbar_wait(bar_s(t, b), (j >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            int valid = n_keys - i * kKeys;
            if (causal) valid = min(valid, first_sample + (row_tile * kPrefixTileRows + row) / group - (first_token + i * kKeys) + 1);
            auto load_s = [&]() {
                tmem_ld32(s_addr, sreg[0]);
                tmem_ld32(s_addr + 32, sreg[1]);
                tmem_wait_ld();
                if (valid < kKeys) {   // ragged last tile, or the diagonal of a prefill: masked keys become -inf
#pragma unroll
                    for (int c = 0; c < 2; ++c)
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (c * 32 + e >= valid) sreg[c][e] = 0xff800000u;
                }
            };
            // 64 scores -> 32 words of packed bf16 P in sreg[0]; returns the row's sum of this tile.
            // The special-function unit is the scarce pipe here (one exponential per score), so nothing else may use
            // it: bf16 comes from TRUNCATING p (a byte permute on the integer pipe) instead of a rounding conversion,
            // and the bias of truncation (half a unit in the last place on average) is cancelled by exponentiating
            // x + log2(1 + 2^-9): every p -- and with it the row sum, which is corrected once in the epilogue --
            // carries the factor (1 + 2^-9).  No running maximum either: if every exponent is below the threshold the
            // tile sum is at most 64 * 2^8, so a sum above that bound is what sends the tile to the slow path.
            auto exp_in_place = [&]() -> float {
                const float off = kTruncBias - (m_ref == -INFINITY ? 0.f : m_ref);   // a row that has seen no key yet: exponentiate against 0
                float ps[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        // every third pair takes the polynomial: with two warps per scheduler the pass is bound by the
                        // special-function unit, and a third of the work is what the other pipes absorb for free
                        const bool poly = ((e >> 1) % 3) == 2;
                        const float x0 = fmaf(__uint_as_float(sreg[c][e]), scale_log2, off), x1 = fmaf(__uint_as_float(sreg[c][e + 1]), scale_log2, off);
                        const float p0 = poly ? poly_exp2(x0) : fast_exp2(x0), p1 = poly ? poly_exp2(x1) : fast_exp2(x1);
                        ps[(e >> 1) & 3] += p0 + p1;
                        sreg[0][c * 16 + e / 2] = __byte_perm(__float_as_uint(p0), __float_as_uint(p1), 0x7632);
                    }
                return (ps[0] + ps[1]) + (ps[2] + ps[3]);
            };
            auto move_reference = [&](bool need, float m_new) -> bool {
                const float alpha = need ? fast_exp2(m_ref - m_new) : 1.f;   // 0 on the stream's first tile
                if (j > 0) {
                    // O[t] must be quiescent: the PV of this stream's previous step has to be complete
                    if (!mbar_wait(bar_pv(t, (j - 1) & 1), ((j - 1) >> 1) & 1, abort_flag)) return false;
                    tc_fence_after();
                    uint32_t oreg[32];
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        tmem_ld32(o_addr + c * 32, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
                        tmem_st32(o_addr + c * 32, oreg);
                    }
                    tmem_wait_st();
                }
                l_sum *= alpha;
                if (need) m_ref = m_new;
                return true;
            };
            load_s();
            float tile_sum = 0.f;
            bool redo = j == 0;   // nothing to exponentiate against yet
            if (j > 0) {
                // common case: ONE pass against the current reference maximum; S is still intact (P not stored yet),
                // so a tile with an exponent above the threshold -- or a row's first visible key -- is simply done again
                tile_sum = exp_in_place();
                redo = __any_sync(0xffffffffu, !(tile_sum <= kTileSumLimit) || (m_ref == -INFINITY && valid > 0));
                if (redo) load_s();
            }
            if (redo) {
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e) mx[e & 3] = fmaxf(mx[e & 3], __uint_as_float(sreg[c][e]));
                const float tmax = scale_log2 * fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                const bool need = tmax > m_ref + kRescaleThreshold;
                if (__any_sync(0xffffffffu, need)) {
                    if (!(ok = move_reference(need, tmax))) break;
                }
                tile_sum = exp_in_place();
            }
            tmem_st32(s_addr, sreg[0]);
            l_sum += tile_sum;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p(t, b));
        }
        // ---- epilogue.  Every MMA of the block is complete (O final, Q and the rings idle): the staging tile(s) may
        // overlay them, so that every global store instruction writes one full row.
        l_sum *= kTruncUnbias;   // the row sums carry the factor (1 + 2^-9) of the truncation trick
        const bool active = kPing || t < n_streams;
        if (active) {
            if (ok) ok = mbar_wait(bar(L::kBarDone), 0, abort_flag);
            if (ok) tc_fence_after();
            float *stage = reinterpret_cast<float *>(smem + L::kQOff) + (kPing ? 0 : t * (L::kStageBytes / 4));
            float *mine = stage + row * L::kStageRowFloats;
            if constexpr (!kPing) {
                if (ok) {
                    const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;   // a row that saw no key in this item: O = 0, lse = -inf
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t oreg[32];
                        tmem_ld32(o_addr + c * 32, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            *reinterpret_cast<float4 *>(mine + c * 32 + e) =
                                make_float4(__uint_as_float(oreg[e]) * inv, __uint_as_float(oreg[e + 1]) * inv,
                                            __uint_as_float(oreg[e + 2]) * inv, __uint_as_float(oreg[e + 3]) * inv);
                    }
                    const int r = t * kPrefixTileRows + row;
                    if (r < n_rows) partial_lse[prow0 + r] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
                }
                asm volatile("bar.sync %0, 128;" ::"r"(1 + t) : "memory");   // the four warps of this row tile
            } else {
                // combine the two streams of a row: with M = max(m_0, m_1) and a_t = 2^(m_t - M),
                //   l = a_0 l_0 + a_1 l_1,   out = (a_0 O_0 + a_1 O_1) / l.
                // (m, l) cross through shared memory; stream t then finishes the column half t of every row, reading
                // both accumulators from tensor memory (a warp reaches the same 32 lanes in either).
                float2 *exch = reinterpret_cast<float2 *>(smem + L::kExchangeOff);
                exch[t * kPrefixTileRows + row] = make_float2(m_ref, l_sum);
                asm volatile("bar.sync 1, 256;" ::: "memory");
                const float2 other = exch[(1 - t) * kPrefixTileRows + row];
                const float m0 = t == 0 ? m_ref : other.x, l0 = t == 0 ? l_sum : other.y;
                const float m1 = t == 0 ? other.x : m_ref, l1 = t == 0 ? other.y : l_sum;
                const float top = fmaxf(m0, m1);
                const float a0 = m0 == -INFINITY ? 0.f : fast_exp2(m0 - top), a1 = m1 == -INFINITY ? 0.f : fast_exp2(m1 - top);
                const float l = a0 * l0 + a1 * l1;
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const bool have1 = n_streams > 1;    // otherwise O_1 was never written
                if (ok) {
                    const uint32_t o0 = tmem_base + lane_addr + kColO, o1 = o0 + D;
                    const float w0 = a0 * inv, w1 = a1 * inv;
#pragma unroll 1
                    for (int c = t * (D / 64); c < (t + 1) * (D / 64); ++c) {   // 32-column pieces of this stream's half
                        uint32_t r0[32], r1[32];
                        tmem_ld32(o0 + c * 32, r0);
                        if (have1) tmem_ld32(o1 + c * 32, r1);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            float v[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                v[u] = __uint_as_float(r0[e + u]) * w0;
                                if (have1) v[u] = fmaf(__uint_as_float(r1[e + u]), w1, v[u]);
                            }
                            *reinterpret_cast<float4 *>(mine + c * 32 + e) = make_float4(v[0], v[1], v[2], v[3]);
                        }
                    }
                    if (t == 0 && row < n_rows) partial_lse[prow0 + row] = l > 0.f ? (top + log2f(l)) * 0.6931471805599453f : -INFINITY;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            if (!*abort_flag) {
                constexpr int kLanesPerRow = D / 4;                    // float4 per row: 32 or 16
                constexpr int kRowsPerInstr = 32 / kLanesPerRow;       // 1 or 2
                const int sub = lane / kLanesPerRow, col = (lane % kLanesPerRow) * 4;
                const int tile_row0 = kPing ? 0 : t * kPrefixTileRows;
                const int rows_here = min(kPrefixTileRows, n_rows - tile_row0);
                const int n_writers = kPing ? 8 : 4, writer = kPing ? warp : (warp & 3);
                for (int r = writer * kRowsPerInstr + sub; r < rows_here; r += n_writers * kRowsPerInstr) {
                    const float4 v = *reinterpret_cast<const float4 *>(stage + r * L::kStageRowFloats + col);
                    *reinterpret_cast<float4 *>(partial_o + size_t(prow0 + tile_row0 + r) * D + col) = v;
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicCAS(status, 0, int(PSA_ERR_TIMEOUT));
        // let copies that were already issued land before the block's shared memory is released
        if (warp == kProducerWarp && lane == 0) {
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 2000000ull) { }
        }
        // MMAs queued before the issuing thread gave up may still run: one more commit completes when all of them
        // have retired; wait for it (bounded) before tensor memory is freed
        if ((warp == kMmaWarp || warp == kMmaWarp + 1) && elect_one()) {
            const uint32_t drain = bar(L::kBarDrain + warp - kMmaWarp);
            tc_commit(drain);
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(drain, 0) && global_timer_ns() - t0 < 2000000ull) { }
        }
        __syncthreads();
    }
    if (done_counter != nullptr && threadIdx.x == 0)
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(done_counter) : "memory");
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, L::kTmemCols);
    }
}

template <int D, bool kPing>
__global__ void __launch_bounds__(352, 1)
prefix_kernel_decoupled(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_v, const PrefixItem *__restrict__ items, int group, int causal,
                        float scale_log2, float *__restrict__ partial_o, float *__restrict__ partial_lse, int *__restrict__ status,
                        int *launch_counter, int *done_counter)
{
    prefix_body2<D, kPing>(&map_q, &map_k, &map_v, items, group, causal, scale_log2, partial_o, partial_lse, status, launch_counter,
                           done_counter);
}

// Self-test of the bounded wait: one block waits on a barrier that nothing ever arrives on.  The wait must give
// up after `limit_ns`, report PSA_ERR_TIMEOUT through the status word and let the block exit normally.
__global__ void bounded_wait_selftest_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicCAS(status, 0, int(PSA_ERR_TIMEOUT));
}

// ---------------------------------------------------------------- host side
using EncodeFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                              const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode_fn(std::string *err)
{
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    static cudaError_t rc = cudaSuccess;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        rc = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (rc == cudaSuccess && q == cudaDriverEntryPointSuccess) fn = reinterpret_cast<EncodeFn>(p);
    });
    if (!fn && err) *err = "cuTensorMapEncodeTiled is not available from the driver";
    return fn;
}

bool encode(EncodeFn fn, CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides_bytes,
            const cuuint32_t *box, std::string *err)
{
    cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, cuuint32_t(rank), const_cast<void *>(base), dims, strides_bytes, box,
                    elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (err) *err = "cuTensorMapEncodeTiled failed with code " + std::to_string(int(r));
        return false;
    }
    return true;
}

// kShape: 2 = two row tiles; 1 = one row tile, small block that can share the SM with a suffix block (short items,
// or enough rows per tile that the block is not purely HBM-bound); 0 = one row tile, long ring, owns the SM
template <int D, int kShape>
int launch_one(const PrefixArgs &a, const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, cudaStream_t st)
{
    constexpr bool kTwo = kShape == 2;
    using L = PrefixSmem<D, kTwo, prefix_tile_keys<kShape == 1>()>;
    auto kern = kShape == 2 ? prefix_kernel_two<D> : (kShape == 1 ? prefix_kernel_one<D> : prefix_kernel_one_long<D>);
    // ring length: enough buffers for the epilogue staging tile(s); short items of the one-row-tile
    // shape get the smallest block so that a suffix block fits beside it on the SM
    constexpr int ring = prefix_ring<D, kTwo, kShape == 1>();
    static_assert(L::total(ring) <= 227 * 1024 && L::min_ring() <= ring, "shared memory plan does not fit");
    static PerDeviceOnce once;   // per instantiation
    const int cfg_rc = once.ensure([&] {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::total(ring));
        // ask for the largest shared-memory carve-out so that a suffix block can share the SM
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return int(e);
    });
    if (cfg_rc != 0) return cfg_rc;
    const float scale_log2 = a.sm_scale * 1.4426950408889634f;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(a.num_items);
    lc.blockDim = dim3(kTwo ? 352 : (kShape == 1 ? 256 : 224));   // softmax warps, producer, two more single-thread warps (MMA issuers / watcher)
    lc.dynamicSmemBytes = L::total(ring);
    lc.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = 1;   // set-up may overlap the tail of the preceding kernel; the kernel waits before touching memory
    return int(cudaLaunchKernelEx(&lc, kern, mq, mk, mv, a.items, a.num_q_heads / a.num_kv_heads, int(a.causal), scale_log2, a.partial_o,
                                  a.partial_lse, a.status, a.launch_counter, a.done_counter));
}

template <int D, bool kPing>
int launch_decoupled(const PrefixArgs &a, const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, cudaStream_t st)
{
    using L = PrefixSmem2<D, kPing>;
    auto kern = prefix_kernel_decoupled<D, kPing>;
    static PerDeviceOnce once;   // per instantiation
    const int cfg_rc = once.ensure([&] {
        return int(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal));
    });
    if (cfg_rc != 0) return cfg_rc;
    const float scale_log2 = a.sm_scale * 1.4426950408889634f;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(a.num_items);
    lc.blockDim = dim3(352);   // two softmax warpgroups, producer, one MMA issuer per stream
    lc.dynamicSmemBytes = L::kTotal;
    lc.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = 1;
    return int(cudaLaunchKernelEx(&lc, kern, mq, mk, mv, a.items, a.num_q_heads / a.num_kv_heads, int(a.causal), scale_log2, a.partial_o,
                                  a.partial_lse, a.status, a.launch_counter, a.done_counter));
}

}  // namespace

int launch_bounded_wait_selftest(int32_t *status, unsigned long long limit_ns, void *stream)
{
    bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, limit_ns);
    return int(cudaGetLastError());
}

int launch_prefix(const PrefixArgs &a, void *stream, std::string *err)
{
    if (a.num_items == 0) return 0;
    const int G = a.num_q_heads / a.num_kv_heads;
    const int D = a.head_dim;
    // Block shape.  0: one row tile, long (HBM-bound items of few rows); 1: one row tile, small (shares its SM with a
    // suffix block); 2: two row tiles, coupled (kept for comparison); 3: decoupled, two row tiles; 4: decoupled, one
    // row tile with the streams on alternate key tiles.  a.kernel_choice forces one where the rows allow it.
    int shape;
    if (a.max_rows_per_item > kPrefixTileRows) shape = a.kernel_choice == PSA_PREFIX_KERNEL_COUPLED ? 2 : 3;
    else if (a.kernel_choice == PSA_PREFIX_KERNEL_SMALL) shape = 1;
    else if (a.kernel_choice == PSA_PREFIX_KERNEL_LONG) shape = 0;
    else if (a.kernel_choice == PSA_PREFIX_KERNEL_DECOUPLED) shape = 4;
    // no suffix stage in this plan (a prefix-only step): nothing to share the SM with, so rows that fill most of a
    // row tile take the decoupled block with its streams on alternate key tiles
    else if (a.no_suffix_stage && a.max_rows_per_item > 64 && a.max_tiles_per_item >= 2) shape = 4;
    else shape = (a.max_tiles_per_item <= 2 || a.max_rows_per_item > 64) ? 1 : 0;
    const int tile_keys = (shape == 0 || shape == 2) ? kPrefixTileKeys : 64;
    // The three tensor maps depend only on the buffers' addresses, the strides and a few plan constants, and a
    // decode loop presents the same few buffers step after step: encoding them (three driver calls, 2-3 us) is
    // done once per distinct key and kept in a small per-thread table.
    struct MapKey {
        const void *q, *k, *v;
        int64_t stride_tok, stride_head, total_tokens;
        int32_t num_samples, num_q_heads, num_kv_heads, head_dim, tile_keys, device;
        bool operator==(const MapKey &o) const
        {
            return q == o.q && k == o.k && v == o.v && stride_tok == o.stride_tok && stride_head == o.stride_head &&
                   total_tokens == o.total_tokens && num_samples == o.num_samples && num_q_heads == o.num_q_heads &&
                   num_kv_heads == o.num_kv_heads && head_dim == o.head_dim && tile_keys == o.tile_keys && device == o.device;
        }
    };
    struct MapEntry { MapKey key; CUtensorMap mq, mk, mv; bool valid; };
    constexpr int kMapCache = 16;
    thread_local MapEntry cache[kMapCache] = {};
    thread_local int next_victim = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) dev = -1;
    const MapKey key{a.q, a.k, a.v, a.stride_tok, a.stride_head, a.total_tokens, a.num_samples, a.num_q_heads, a.num_kv_heads,
                     a.head_dim, tile_keys, dev};
    MapEntry *hit = nullptr;
    for (int i = 0; i < kMapCache && !hit; ++i)
        if (cache[i].valid && cache[i].key == key) hit = &cache[i];
    if (!hit) {
        EncodeFn fn = get_encode_fn(err);
        if (!fn) return int(cudaErrorNotSupported);
        MapEntry e{};
        e.key = key;
        {   // Q as (d, g, kv head, sample): a box of (64, G, 1, 128/G) lands as 128 rows ordered sample-major, g fastest
            const cuuint64_t dims[4] = {cuuint64_t(D), cuuint64_t(G), cuuint64_t(a.num_kv_heads), cuuint64_t(a.num_samples)};
            const cuuint64_t strides[3] = {cuuint64_t(D) * 2, cuuint64_t(G) * D * 2, cuuint64_t(a.num_q_heads) * D * 2};
            const cuuint32_t box[4] = {64, cuuint32_t(G), 1, cuuint32_t(kPrefixTileRows / G)};
            if (!encode(fn, &e.mq, a.q, 4, dims, strides, box, err)) return int(cudaErrorInvalidValue);
        }
        {   // K and V as (d, kv head, token): a box of (64, 1, tile_keys) is one 64-wide half of a key tile
            const cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(a.num_kv_heads), cuuint64_t(a.total_tokens)};
            const cuuint64_t strides[2] = {cuuint64_t(a.stride_head) * 2, cuuint64_t(a.stride_tok) * 2};
            const cuuint32_t box[3] = {64, 1, cuuint32_t(tile_keys)};
            if (!encode(fn, &e.mk, a.k, 3, dims, strides, box, err)) return int(cudaErrorInvalidValue);
            if (!encode(fn, &e.mv, a.v, 3, dims, strides, box, err)) return int(cudaErrorInvalidValue);
        }
        e.valid = true;
        hit = &cache[next_victim];
        next_victim = (next_victim + 1) % kMapCache;
        *hit = e;
    }
    const CUtensorMap &mq = hit->mq, &mk = hit->mk, &mv = hit->mv;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc;
    if (shape == 3) rc = D == 128 ? launch_decoupled<128, false>(a, mq, mk, mv, st) : launch_decoupled<64, false>(a, mq, mk, mv, st);
    else if (shape == 4) rc = D == 128 ? launch_decoupled<128, true>(a, mq, mk, mv, st) : launch_decoupled<64, true>(a, mq, mk, mv, st);
    else if (shape == 2) rc = D == 128 ? launch_one<128, 2>(a, mq, mk, mv, st) : launch_one<64, 2>(a, mq, mk, mv, st);
    else if (shape == 1) rc = D == 128 ? launch_one<128, 1>(a, mq, mk, mv, st) : launch_one<64, 1>(a, mq, mk, mv, st);
    else rc = D == 128 ? launch_one<128, 0>(a, mq, mk, mv, st) : launch_one<64, 0>(a, mq, mk, mv, st);
    if (rc != 0 && err) *err = std::string("prefix launch: ") + cudaGetErrorString(cudaError_t(rc));
    return rc;
}

}  // namespace psa
