// Full-history prompt scores: s_t = (1/G) sum_g sum_{tau >= t} lambda^(T-1-tau) a^(tau)_{g,t},
// a^(tau) the causal softmax row of prompt query tau (App. B with the window taken as the whole
// prompt; Eq. (score) unrolled).  A dense T x T x d contraction done twice on the tensor cores:
//   pass 1  row statistics: log-sum-exp of every query's causal row (skipped when the caller
//           hands in the values its own prefill attention produced);
//   pass 2  column sums: for a block of 128 keys, over every later query tile and every query
//           head of the group, exp(logit - lse) weighted by the decay.
// Both passes are one kernel.  A 128-row block of one operand (queries in pass 1, keys in pass 2)
// stays in shared memory; 128-row tiles of the other stream through a two-stage ring, brought in
// by TMA (cp.async.bulk.tensor, 128-byte swizzle) and announced on an mbarrier per stage.  One thread issues
// tcgen05.mma: 128 x 128 x d logits per tile, both operands from shared memory, the fp32
// accumulator in tensor memory, two accumulators so that the next tile's product runs under this
// tile's exponentials.
//
// Two CTAs share an SM (two tile stages and 256 of the 512 tensor-memory columns each), so one
// CTA's waits -- for a product, for an accumulator load -- are covered by the other's arithmetic.
// Per CTA one warp requests the tiles and issues the products, one (pass 2) prepares each query's
// exponent offset, and eight only read accumulators and do the exponentials.
// Accumulator: row i of the product is lane i of tensor memory, column j is column j.  A warp can
// read the 32 lanes of its quadrant (warp % 4), so the eight warps share a tile as 4 row quadrants
// x 2 column halves: a thread reads two blocks of 32 columns of one resident row per tile
// (tcgen05.ld.32x32b.x32) and keeps that row's running max / sum or column sum over its columns;
// the two partial results of a row are folded through shared memory once, at the end.
// (Measured on the way here, c4 shape, per layer: 4 epilogue warps, one CTA per SM, tiles staged
// with 16-byte cp.async into an unswizzled layout 90.7 ms; 16 warps 75.9; TMA tiles 58.2; a warp
// of its own for requests and products 47.1, another for the offsets 41.6; mbarriers instead of a
// block barrier per tile 39.2; two CTAs of 8 epilogue warps per SM 32.3.)
//
// Every wait is bounded; a thread that gives up records ZSM_ERR_TIMEOUT and every thread still
// reaches the end of the kernel, where the tensor memory is released.
#include "zsm_prefill_full.cuh"

#include <cuda.h>

#include <type_traits>

namespace zsm {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

constexpr int kTcRows = 128;      // resident rows = streamed rows per tile = M = N of one step
constexpr int kTcEpiThreads = 256;             // 4 row quadrants x 2 column halves of the accumulator
constexpr int kTcColParts = kTcEpiThreads / 128; // column parts; a thread reads 128 / parts columns per tile
constexpr int kTcThreads = kTcEpiThreads + 64;  // + a warp that requests tiles and issues products
                                                // + a warp that prepares the exponent offsets
constexpr int kTcStages = 2;      // streamed tiles in shared memory (two CTAs share an SM)
constexpr int kTcOffRing = 8;     // per-query exponent offsets: entries of the items in flight
constexpr int kTcTmemCols = 256;  // two 128-column accumulators
constexpr int kTcKBlock = 64;     // elements of the head dimension per 128-byte swizzled row

enum : int32_t { WF_MMA = 41, WF_TILE = 42, WF_RESIDENT = 43, WF_ACC = 44 };

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 2^x for a pair of exponents x <= 0 without the special-function unit: x = n + f with n = round(x)
// (adding 1.5 * 2^23 leaves n in the low mantissa bits), a degree-4 polynomial for 2^f on
// |f| <= 1/2 (interpolation at the Chebyshev nodes, relative error 3.6e-6) and n added into the
// exponent field.  Results below 2^-125 (also x = -inf) come out as 2^-125.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
    constexpr float kMagic = 12582912.f;
    x.x = fmaxf(x.x, -125.f);
    x.y = fmaxf(x.y, -125.f);
    const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 nf = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __ffma2_rn(nf, make_float2(-1.f, -1.f), x);
    float2 r = __ffma2_rn(f, make_float2(0.00966636836528778f, 0.00966636836528778f),
                          make_float2(0.055921975523233414f, 0.055921975523233414f));
    r = __ffma2_rn(r, f, make_float2(0.2402234971523285f, 0.2402234971523285f));
    r = __ffma2_rn(r, f, make_float2(0.6931210160255432f, 0.6931210160255432f));
    r = __ffma2_rn(r, f, make_float2(1.0f, 1.0f));
    r.x = __uint_as_float(__float_as_uint(r.x) + (__float_as_uint(t.x) << 23));
    r.y = __uint_as_float(__float_as_uint(r.y) + (__float_as_uint(t.y) << 23));
    return r;
}
// Share of the scoring passes' exponentials that takes that route (the rest: one `ex2` each, 16
// per clock per SM, which is what bounds those passes): a quarter.  B200, c4 shape, per layer,
// first call on an idle box: column pass 14.7 -> 14.0 ms, row pass 15.0 -> 14.3 ms (2 % under the
// power cap); a half makes the row pass slower again.
constexpr int kPolyPairsOf8 = 2;

// Shared-memory matrix descriptor of a K-major operand stored as rows of 128 bytes with the
// 128-byte swizzle (what the tensor map writes): start address in 16-byte units, stride byte
// offset = 8 rows x 128 bytes, descriptor version 1, layout type 2 (128-byte swizzle).  The
// leading byte offset is not used for this layout.
__device__ __forceinline__ uint64_t umma_desc_sw128(const void *smem_ptr) {
    const uint64_t a = (smem_u32(smem_ptr) >> 4) & 0x3fffu;
    return a | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void umma_f16_ss(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
        "}\n"
        :
        : "r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
          "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Eight columns of this thread's lane.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Sixteen columns of this thread's lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One box of a 3-D tensor map (head dimension, position, head) into this CTA's shared memory.
// x is a multiple of 64 elements, so the copy starts on a 128-byte boundary of the row.
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *map, int x, int y, int z,
                                            uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y),
        "r"(z)
        : "memory");
}

template <int D>
struct TcSmem {
    static constexpr int KB = D / kTcKBlock;                 // 128-byte-row blocks per tile
    static constexpr int KBLOCK = kTcRows * 128;             // bytes of one block: 128 rows x 128 B
    static constexpr int TILE = KB * KBLOCK;                 // one operand tile
    static constexpr int a = 0;
    static constexpr int b = TILE;
    static constexpr int off = TILE * (1 + kTcStages);
    static constexpr int comb = off + kTcOffRing * kTcRows * 4;  // [4][128] float2: partial results
    static constexpr int bars = comb + 4 * kTcRows * 8;          // full[3], mma[2], resident, slot, flag
    static constexpr int total = bars + 128 + 1024;              // + slack to align the base to 1 KiB
};

template <typename T, int D, bool COLSUM>
__global__ void __launch_bounds__(kTcThreads, 2)
    full_pass_tc_kernel(const FullScoreParams p, const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_q) {
    using L = TcSmem<D>;
    constexpr int KS = D / 16;  // tensor-core steps along the head dimension
    extern __shared__ uint8_t smem_raw[];
    // the swizzle pattern repeats every 1024 bytes: tiles start on such a boundary
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    float *off_s = reinterpret_cast<float *>(smem + L::off);
    float2 *comb = reinterpret_cast<float2 *>(smem + L::comb);
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L::bars);  // [3] tile landed
    uint64_t *mma_bar = full_bar + kTcStages;                            // [2] product finished
    uint64_t *res_bar = mma_bar + 2;                                     // resident block landed
    uint64_t *acc_free = res_bar + 1;                                    // [2] accumulator read
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_free + 2);
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(tmem_slot + 2);
    // accumulators picked up so far, counted per epilogue warp (paces the offset warp)
    uint32_t *picked = reinterpret_cast<uint32_t *>(tmem_slot + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Tn = p.T, G = p.G;
    const int nb = (Tn + kTcRows - 1) / kTcRows;
    // the longest blocks first: pass 2 walks nb - rb tiles, pass 1 rb + 1
    const int rb = COLSUM ? blockIdx.x : nb - 1 - blockIdx.x;
    int b, hk, hq = 0;
    if (COLSUM) {
        b = blockIdx.y / p.n_kv_heads;
        hk = blockIdx.y % p.n_kv_heads;
    } else {
        b = blockIdx.y / (p.n_kv_heads * G);
        hq = blockIdx.y % (p.n_kv_heads * G);
        hk = hq / G;
    }
    const int zk = b * p.n_kv_heads + hk;           // head coordinate in the K map
    const int zq0 = b * p.n_kv_heads * G + hk * G;  // first query head of the group in the Q map
    const CUtensorMap *map_res = COLSUM ? &map_k : &map_q;
    const CUtensorMap *map_str = COLSUM ? &map_q : &map_k;
    const int z_res = COLSUM ? zk : b * p.n_kv_heads * G + hq;

    const int first = COLSUM ? rb : 0;
    const int per = COLSUM ? nb - rb : rb + 1;
    const int items = COLSUM ? per * G : per;
    const float scale2 = p.scale * kLog2e;
    const float l2lam = log2f(p.lambda);
    const int quad = warp & 3, cq = warp >> 2;  // accumulator lanes 32 quad.., columns 32 cq..
    const int rloc = quad * 32 + lane;
    const int row = rb * kTcRows + rloc;         // the resident row this thread works on

    if (tid == 0) {
        // a stage is full when its tile has landed and (pass 2) its offsets are written
        for (int s = 0; s < kTcStages; ++s) mbar_init(&full_bar[s], COLSUM ? 2 : 1);
        *picked = 0;
        mbar_init(&mma_bar[0], 1);
        mbar_init(&mma_bar[1], 1);
        mbar_init(res_bar, 1);
        mbar_init(&acc_free[0], kTcEpiThreads / 32);
        mbar_init(&acc_free[1], kTcEpiThreads / 32);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(tmem_slot)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // exponent offset of query q of head g: decay lambda^(T-1-q) and the row's normaliser
    // Tile of item i.  Pass 2 walks the query tiles from the last one down: the blocks of a head
    // start together, so they then ask for the same tiles at about the same time and all but the
    // first get them from L2.
    auto tile_of = [&](int i) -> int { return COLSUM ? first + per - 1 - i % per : i; };
    // (offset warp) the 128 exponent offsets of an item (head g, query tile jb) into ring entry e:
    // the rows' log-sum-exp are fetched one item ahead of where they are written
    auto fetch_lse = [&](int g, int jb, float (&l)[kTcRows / 32]) {
#pragma unroll
        for (int k = 0; k < kTcRows / 32; ++k) {
            const int q = jb * kTcRows + k * 32 + lane;
            l[k] = (g < G && q < Tn) ? p.lse[((size_t)zq0 + g) * Tn + q] : 0.f;
        }
    };
    auto put_offsets = [&](int e, int jb, const float (&l)[kTcRows / 32]) {
#pragma unroll
        for (int k = 0; k < kTcRows / 32; ++k) {
            const int q = jb * kTcRows + k * 32 + lane;
            float o = -INFINITY;
            if (q < Tn) {
                const float dec = (q == Tn - 1) ? 0.f : static_cast<float>(Tn - 1 - q) * l2lam;
                o = dec - l[k] * kLog2e;
            }
            off_s[e * kTcRows + k * 32 + lane] = o;
        }
    };
    // (one thread) request item i's tile
    auto load_item = [&](int i) {
        if (i >= items) return;
        const int s = i % kTcStages;
        const int jb = tile_of(i);
        const int z = COLSUM ? zq0 + i / per : zk;
        mbar_arrive_expect_tx(&full_bar[s], L::TILE);
#pragma unroll
        for (int kb = 0; kb < L::KB; ++kb)
            tma_load_3d(smem + L::b + s * L::TILE + kb * L::KBLOCK, map_str, kb * kTcKBlock, jb * kTcRows, z,
                        &full_bar[s]);
    };

    const bool producer = warp == kTcEpiThreads / 32;
    const bool offsetter = warp == kTcEpiThreads / 32 + 1;
    // offset warp: the item whose log-sum-exp it holds (head og, tile ojb, ring entry oe)
    float lse_ahead[kTcRows / 32] = {0.f, 0.f, 0.f, 0.f};
    int og = 0, ojb = first + per - 1, oe = 0;
    auto next_item = [&]() {
        if (--ojb < first) {
            ojb = first + per - 1;
            ++og;
        }
        if (++oe == kTcOffRing) oe = 0;
    };
    if (offsetter && COLSUM) {
        for (int i = 0; i < kTcStages && i < items; ++i) {
            fetch_lse(og, ojb, lse_ahead);
            put_offsets(oe, ojb, lse_ahead);
            next_item();
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[i]);
        }
        fetch_lse(og, ojb, lse_ahead);
    }
    if (producer) {
        if (lane == 0) {
            mbar_arrive_expect_tx(res_bar, L::TILE);
#pragma unroll
            for (int kb = 0; kb < L::KB; ++kb)
                tma_load_3d(smem + L::a + kb * L::KBLOCK, map_res, kb * kTcKBlock, rb * kTcRows, z_res, res_bar);
            for (int i = 0; i < kTcStages; ++i) load_item(i);
        }
    }

    const uint32_t idesc = (1u << 4) | ((Elem<T>::kIsBf16 ? 1u : 0u) << 7) |
                           ((Elem<T>::kIsBf16 ? 1u : 0u) << 10) | ((kTcRows >> 3) << 17) |
                           ((kTcRows >> 4) << 24);

    float m = -INFINITY, z = 0.f, colsum = 0.f;
    bool ok = true;
    // everything a thread does with the finished product of item j
    auto epilogue = [&](int j) {
        const int buf = j & 1;
        if (!mbar_wait_bounded(&mma_bar[buf], (j >> 1) & 1u, abort_flag, p.status, WF_MMA)) {
            ok = false;
            return;
        }
        tc_fence_after();
        const int jb = tile_of(j);
        const bool diag = jb == rb;
        const float *off = off_s + (j % kTcOffRing) * kTcRows;
        constexpr int CH = 4 / kTcColParts;  // 32-column chunks per thread
#pragma unroll 1
        for (int c = 0; c < CH; ++c) {
        const int ch = cq * CH + c;
        uint32_t v[32];
        tmem_ld32(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kTcRows + ch * 32, v);
        if (c == CH - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&acc_free[buf]);  // this warp is done with the accumulator
                if (COLSUM) atomicAdd(picked, 1u);
            }
        }
        const int col0 = jb * kTcRows + ch * 32;
        if (!COLSUM) {
            float bm = -INFINITY;
            if (diag) {  // only the tile on the diagonal needs the causal mask (warp-uniform branch)
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    float x = __uint_as_float(v[e]) * scale2;
                    if (col0 + e > row) x = -INFINITY;  // keep key <= query
                    v[e] = __float_as_uint(x);
                    bm = fmaxf(bm, x);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float x = __uint_as_float(v[e]) * scale2;
                    v[e] = __float_as_uint(x);
                    bm = fmaxf(bm, x);
                }
            }
            const float mn = fmaxf(m, bm);
            const float mu = mn == -INFINITY ? 0.f : mn;
            float sum = z * ex2(m - mu), sum1 = 0.f;  // two chains of additions
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                if ((e / 2) % 8 < kPolyPairsOf8) {
                    const float2 y = ex2_poly2(make_float2(__uint_as_float(v[e]) - mu, __uint_as_float(v[e + 1]) - mu));
                    sum += y.x;
                    sum1 += y.y;
                } else {
                    sum += ex2(__uint_as_float(v[e]) - mu);
                    sum1 += ex2(__uint_as_float(v[e + 1]) - mu);
                }
            }
            z = sum + sum1;
            m = mn;
        } else {
            if (diag) {  // only the tile on the diagonal needs the causal mask (warp-uniform branch)
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                    const float4 o = *reinterpret_cast<const float4 *>(off + ch * 32 + e4 * 4);
                    const float oo[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float x = ex2(fmaf(__uint_as_float(v[e4 * 4 + e]), scale2, oo[e]));
                        if (col0 + e4 * 4 + e < row) x = 0.f;  // keep query >= key
                        colsum += x;
                    }
                }
            } else {
                float cs1 = 0.f;  // two chains of additions
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                    const float4 o = *reinterpret_cast<const float4 *>(off + ch * 32 + e4 * 4);
                    if (e4 % 4 < kPolyPairsOf8) {  // the first pair of two groups in four: a quarter
                        const float2 y = ex2_poly2(make_float2(fmaf(__uint_as_float(v[e4 * 4]), scale2, o.x),
                                                               fmaf(__uint_as_float(v[e4 * 4 + 1]), scale2, o.y)));
                        colsum += y.x;
                        cs1 += y.y;
                    } else {
                        colsum += ex2(fmaf(__uint_as_float(v[e4 * 4]), scale2, o.x));
                        cs1 += ex2(fmaf(__uint_as_float(v[e4 * 4 + 1]), scale2, o.y));
                    }
                    colsum += ex2(fmaf(__uint_as_float(v[e4 * 4 + 2]), scale2, o.z));
                    cs1 += ex2(fmaf(__uint_as_float(v[e4 * 4 + 3]), scale2, o.w));
                }
                colsum += cs1;
            }
        }
        }
    };

    // Three roles, tied by mbarriers only (no block-wide barrier per tile):
    //   mma_bar[b]   producer -> everyone: the product in accumulator b is complete
    //   acc_free[b]  16 epilogue warps -> producer, offset warp: accumulator b has been read into
    //                registers (so the exponentials of the item before it are finished too)
    const bool epi = warp < kTcEpiThreads / 32;
    if (producer) {
        if (lane == 0) {
            for (int i = 0; i < items && ok; ++i) {
                bool ready = i > 0 || mbar_wait_bounded(res_bar, 0, abort_flag, p.status, WF_RESIDENT);
                if (i >= 2)  // item i - 2 has left this accumulator
                    ready = ready && mbar_wait_bounded(&acc_free[i & 1], ((i - 2) >> 1) & 1u, abort_flag,
                                                       p.status, WF_ACC);
                ready = ready && mbar_wait_bounded(&full_bar[i % kTcStages], (i / kTcStages) & 1u, abort_flag,
                                                   p.status, WF_TILE);
                if (!ready) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint8_t *bt = smem + L::b + (i % kTcStages) * L::TILE;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int o = (ks / 4) * L::KBLOCK + (ks % 4) * 32;  // 16 elements = 32 bytes on
                    umma_f16_ss(tmem_base + (i & 1) * kTcRows, umma_desc_sw128(smem + L::a + o),
                                umma_desc_sw128(bt + o), idesc, ks > 0);
                }
                umma_commit(&mma_bar[i & 1]);
                if (i >= 1) {
                    // item i - 1's product frees its stage: request the tile three items on
                    if (mbar_wait_bounded(&mma_bar[(i - 1) & 1], ((i - 1) >> 1) & 1u, abort_flag, p.status, WF_MMA))
                        load_item(i - 1 + kTcStages);
                    else
                        ok = false;
                }
            }
        }
    } else if (offsetter) {
        if (COLSUM) {
            // entry of item i + 2, once every epilogue warp has picked up item i - 1 (ring of 8:
            // the entry's previous owner, item i - 6, was finished long before)
            for (int i = 1; i - 1 + kTcStages < items && ok; ++i) {
                // a count, not a barrier phase: the epilogue warps may be two items on by now
                const uint32_t need = static_cast<uint32_t>(i) * (kTcEpiThreads / 32);
                const uint64_t t0 = global_timer_ns();
                while (*reinterpret_cast<volatile uint32_t *>(picked) < need) {
                    __nanosleep(64);
                    if (*abort_flag || global_timer_ns() - t0 > kWaitLimitNs) {
                        if (!*abort_flag && lane == 0) dev_set_status(p.status, DEV_ERR_TIMEOUT, WF_ACC, blockIdx.x);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                }
                if (!ok) break;
                put_offsets(oe, ojb, lse_ahead);
                next_item();
                fetch_lse(og, ojb, lse_ahead);
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[(i - 1 + kTcStages) % kTcStages]);
            }
        }
    } else {
        for (int j = 0; j < items && ok; ++j) epilogue(j);
    }

    // fold the four column blocks' partial results of each row
    __syncwarp();
    if (epi) comb[cq * kTcRows + rloc] = COLSUM ? make_float2(colsum, 0.f) : make_float2(m, z);
    tc_fence_before();
    if (__syncthreads_or(!ok)) ok = false;
    if (ok && epi && cq == 0 && row < Tn) {
        if (!COLSUM) {
            float mm = -INFINITY;
#pragma unroll
            for (int k = 0; k < kTcColParts; ++k) mm = fmaxf(mm, comb[k * kTcRows + rloc].x);
            float zz = 0.f;
#pragma unroll
            for (int k = 0; k < kTcColParts; ++k) {
                const float2 t = comb[k * kTcRows + rloc];
                zz += t.y * ex2(t.x - mm);  // a block that saw no key has sum 0 and max -inf
            }
            p.lse_out[((size_t)b * p.n_kv_heads * G + hq) * Tn + row] = (mm + log2f(zz)) * kLn2;
        } else {
            float v = 0.f;
#pragma unroll
            for (int k = 0; k < kTcColParts; ++k) v += comb[k * kTcRows + rloc].x;
            p.scores[((size_t)b * p.n_kv_heads + hk) * Tn + row] = v * (1.0f / static_cast<float>(G));
        }
    }
    if (!ok && producer && lane == 0) {
        // copies that were requested may still land: give them time before the memory goes away
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    __syncwarp();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"(kTcTmemCols)
                     : "memory");
}

// A whole accumulator row: 128 columns of this thread's lane in one load, then the wait.
__device__ __forceinline__ void tmem_ld128(uint32_t taddr, uint32_t (&v)[128]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x128.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
        "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
        "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, "
        "%64, %65, %66, %67, %68, %69, %70, %71, %72, %73, %74, %75, %76, %77, %78, %79, "
        "%80, %81, %82, %83, %84, %85, %86, %87, %88, %89, %90, %91, %92, %93, %94, %95, "
        "%96, %97, %98, %99, %100, %101, %102, %103, %104, %105, %106, %107, %108, %109, %110, %111, "
        "%112, %113, %114, %115, %116, %117, %118, %119, %120, %121, %122, %123, %124, %125, %126, %127}, [%128];\n\t"
        "tcgen05.wait::ld.sync.aligned;\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31]),
          "=r"(v[32]), "=r"(v[33]), "=r"(v[34]), "=r"(v[35]), "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]),
          "=r"(v[40]), "=r"(v[41]), "=r"(v[42]), "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]),
          "=r"(v[48]), "=r"(v[49]), "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]),
          "=r"(v[56]), "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63]),
          "=r"(v[64]), "=r"(v[65]), "=r"(v[66]), "=r"(v[67]), "=r"(v[68]), "=r"(v[69]), "=r"(v[70]), "=r"(v[71]),
          "=r"(v[72]), "=r"(v[73]), "=r"(v[74]), "=r"(v[75]), "=r"(v[76]), "=r"(v[77]), "=r"(v[78]), "=r"(v[79]),
          "=r"(v[80]), "=r"(v[81]), "=r"(v[82]), "=r"(v[83]), "=r"(v[84]), "=r"(v[85]), "=r"(v[86]), "=r"(v[87]),
          "=r"(v[88]), "=r"(v[89]), "=r"(v[90]), "=r"(v[91]), "=r"(v[92]), "=r"(v[93]), "=r"(v[94]), "=r"(v[95]),
          "=r"(v[96]), "=r"(v[97]), "=r"(v[98]), "=r"(v[99]), "=r"(v[100]), "=r"(v[101]), "=r"(v[102]), "=r"(v[103]),
          "=r"(v[104]), "=r"(v[105]), "=r"(v[106]), "=r"(v[107]), "=r"(v[108]), "=r"(v[109]), "=r"(v[110]), "=r"(v[111]),
          "=r"(v[112]), "=r"(v[113]), "=r"(v[114]), "=r"(v[115]), "=r"(v[116]), "=r"(v[117]), "=r"(v[118]), "=r"(v[119]),
          "=r"(v[120]), "=r"(v[121]), "=r"(v[122]), "=r"(v[123]), "=r"(v[124]), "=r"(v[125]), "=r"(v[126]), "=r"(v[127])
        : "r"(taddr)
        : "memory");
}

// Sixteen 32-bit columns of this thread's lane (32 packed 16-bit weights) into tensor memory.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n"
        :
        : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// Thirty-two 32-bit columns of this thread's lane into tensor memory.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
        :
        : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// Product with the M x K operand in tensor memory (lane = row, a 32-bit column holds two
// consecutive 16-bit elements of the row) and the N x K operand through a shared-memory descriptor.
__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t"
        "}\n"
        :
        : "r"(tmem_d), "r"(tmem_a), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// ---------------------------------------------------------------------------
// Causal attention of the prompt in one pass: o_tau = sum_{t <= tau} a^(tau)_t v_t [Eq. (att_score)]
// and the log-sum-exp of every query's row.  Per CTA two blocks of 128 queries of one head are
// resident, each with a group of four warps of its own; every key and value tile up to the
// diagonal is fetched once and serves both blocks.  For block g and key tile j
//   product 1   S_g = Q_g K_j^T      (tcgen05.mma, both operands from shared memory, 128 fp32
//                                     columns of tensor memory per block)
//   weights     a thread owns one query row: P_g = exp2(S_g * scale - m_ref) as 16-bit values,
//               written back into the columns S_g came from (two weights per 32-bit column; bf16
//               storage: the high parts in the first 64 columns, the remainders in the other 64),
//               and their fp32 sum.  m_ref follows the row's running maximum lazily: it moves
//               only when a tile's maximum exceeds it by more than 8 (weights stay below 2^8),
//               and then the thread rescales its row of O_g in tensor memory and its sum
//   product 2   O_g += P_g V_j       (tcgen05.mma with the M x K operand in tensor memory; V's tile,
//               rows = keys, is the N x K operand in "MN-major" form: N = head dimension contiguous)
// At the end o = O_g / sum and lse = m_ref + log2(sum).  The weights never pass through shared
// memory, and the two groups work on different products at any time: while one group's
// exponentials run, the tensor cores multiply for the other.  The products of one block follow one
// another in issue order on the tensor pipe, which is what lets S_g(j + 1) overwrite the columns
// P_g(j) was read from, and what makes O_g quiescent between "S_g(j) complete" and this group's
// "weights written".  One thread requests tiles and issues every product.  2 x 128 (S) + 2 x d (O)
// tensor-memory columns: one CTA per SM.
// ---------------------------------------------------------------------------
constexpr int kAoThreads = kTcEpiThreads + 32;
constexpr int kAoKStages = 3;  // key tiles in shared memory
constexpr int kAoVStages = 2;  // value tiles
enum : int32_t { WA_S = 51, WA_P = 52, WA_K = 54, WA_V = 55, WA_VFREE = 56, WA_O = 58, WA_Q = 59 };

template <int D>
struct AoSmem {
    static constexpr int KB = D / kTcKBlock;
    static constexpr int KBLOCK = kTcRows * 128;
    static constexpr int TILE = KB * KBLOCK;          // Q, K or V tile
    static constexpr int q = 0;                       // two query blocks
    static constexpr int k = 2 * TILE;
    static constexpr int v = k + kAoKStages * TILE;
    static constexpr int bars = v + kAoVStages * TILE;
    static constexpr int total = bars + 256 + 1024;   // + slack to align the base to 1 KiB
    static constexpr int tmem_cols = 512;             // 2 x 128 (S) + 2 x D (O), a power of two
};

// V tile as the N x K operand with N (head dimension) contiguous: 64 elements per 128-byte row,
// 8 keys per swizzle atom; the other 64 elements of d one block on (leading offset), the next 8
// keys 1024 bytes on (stride offset).  `kstep`: 16 keys = two atoms.
template <int D>
__device__ __forceinline__ uint64_t umma_desc_v_mn(const uint8_t *tile, int kstep) {
    const uint64_t a = ((smem_u32(tile) + static_cast<uint32_t>(kstep) * 2048u) >> 4) & 0x3fffu;
    return a | (static_cast<uint64_t>(AoSmem<D>::KBLOCK >> 4) << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

template <typename T, int D>
__global__ void __launch_bounds__(kAoThreads, 1)
    attn_out_tc_kernel(const FullScoreParams p, void *out_ptr, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q) {
    using L = AoSmem<D>;
    using E = Elem<T>;
    constexpr int KS = D / 16;
    // bf16 keeps 8 bits of a weight: it is written as a high part and a remainder (two products
    // per step), which brings the weights to 16 bits; fp16's 11 bits are enough for a 16-bit output
    constexpr bool kSplitW = E::kIsBf16;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t *q_bar = reinterpret_cast<uint64_t *>(smem + L::bars);
    uint64_t *k_full = q_bar + 1;               // [3] key tile landed
    uint64_t *v_full = k_full + kAoKStages;     // [2] value tile landed
    uint64_t *v_free = v_full + kAoVStages;     // [2] both blocks' product 2 done with the value tile
    uint64_t *s_ready = v_free + kAoVStages;    // [2] block g's product 1 complete
    uint64_t *p_ready = s_ready + 2;            // [2] block g's weights written by its four warps
    uint64_t *o_done = p_ready + 2;             // [2] block g's last product complete
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(o_done + 2);
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(tmem_slot + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Tn = p.T, G = p.G;
    const int nb = (Tn + kTcRows - 1) / kTcRows;
    const int nb2 = (nb + 1) / 2;
    const int rb2 = nb2 - 1 - blockIdx.x;  // the longest pairs of blocks first
    const int b = blockIdx.y / (p.n_kv_heads * G);
    const int hq = blockIdx.y % (p.n_kv_heads * G);
    const int zk = b * p.n_kv_heads + hq / G;
    const int zq = b * p.n_kv_heads * G + hq;
    // block g holds queries 128 (2 rb2 + g) ..; it walks the key tiles 0 .. 2 rb2 + g.  The second
    // block of the last pair may lie past the prompt's end: then it has no tile at all.
    const int n0 = 2 * rb2 + 1;
    const int n1 = (2 * rb2 + 1 < nb) ? 2 * rb2 + 2 : 0;
    const int nmax = n1 > n0 ? n1 : n0;
    const float scale2 = p.scale * kLog2e;

    if (tid == 0) {
        mbar_init(q_bar, 1);
        for (int s = 0; s < kAoKStages; ++s) mbar_init(&k_full[s], 1);
        for (int s = 0; s < kAoVStages; ++s) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_free[s], 1);
        }
        for (int g = 0; g < 2; ++g) {
            mbar_init(&s_ready[g], 1);
            mbar_init(&p_ready[g], 4);
            mbar_init(&o_done[g], 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(tmem_slot)),
                     "r"(L::tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 2 * kTcRows;  // O_g at tmem_o + g * D

    const uint32_t f = E::kIsBf16 ? 1u : 0u;
    const uint32_t idesc_s = (1u << 4) | (f << 7) | (f << 10) | ((kTcRows >> 3) << 17) | ((kTcRows >> 4) << 24);
    // product 2: B (the value tile) is "MN-major" (bit 16), N = D
    const uint32_t idesc_o = (1u << 4) | (f << 7) | (f << 10) | (1u << 16) | ((static_cast<uint32_t>(D) >> 3) << 17) |
                             ((kTcRows >> 4) << 24);
    bool ok = true;
    const bool producer = warp == kTcEpiThreads / 32;

    if (producer) {
        if (lane == 0) {
            auto load_tile = [&](uint8_t *dst, const CUtensorMap *map, int z, int jb, uint64_t *bar) {
                mbar_arrive_expect_tx(bar, L::TILE);
#pragma unroll
                for (int kb = 0; kb < L::KB; ++kb)
                    tma_load_3d(dst + kb * L::KBLOCK, map, kb * kTcKBlock, jb * kTcRows, z, bar);
            };
            // both query blocks on one barrier (rows past the prompt's end read as zero)
            mbar_arrive_expect_tx(q_bar, 2 * L::TILE);
            for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int kb = 0; kb < L::KB; ++kb)
                    tma_load_3d(smem + L::q + g * L::TILE + kb * L::KBLOCK, &map_q, kb * kTcKBlock,
                                (2 * rb2 + g) * kTcRows, zq, q_bar);
            for (int i = 0; i < kAoKStages && i < nmax; ++i)
                load_tile(smem + L::k + i * L::TILE, &map_k, zk, i, &k_full[i]);
            for (int i = 0; i < kAoVStages && i < nmax; ++i)
                load_tile(smem + L::v + i * L::TILE, &map_v, zk, i, &v_full[i]);
            // product 1 of block g with key tile j (its stage has landed)
            auto issue_s = [&](int g, int j) {
                const uint8_t *kt = smem + L::k + (j % kAoKStages) * L::TILE;
                const uint8_t *qt = smem + L::q + g * L::TILE;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int o = (ks / 4) * L::KBLOCK + (ks % 4) * 32;  // 16 elements = 32 bytes on
                    umma_f16_ss(tmem_base + g * kTcRows, umma_desc_sw128(qt + o), umma_desc_sw128(kt + o), idesc_s,
                                ks > 0);
                }
                umma_commit(&s_ready[g]);
            };
            // product 2 of block g with value tile j: the weights sit where S_g was
            auto issue_pv = [&](int g, int j) {
                const uint8_t *vt = smem + L::v + (j % kAoVStages) * L::TILE;
                const uint32_t pw = tmem_base + g * kTcRows;
#pragma unroll
                for (int ks = 0; ks < kTcRows / 16; ++ks) {  // 16 keys = 8 columns of packed weights
                    umma_f16_ts(tmem_o + g * D, pw + ks * 8, umma_desc_v_mn<D>(vt, ks), idesc_o,
                                (j > 0 || ks > 0) ? 1u : 0u);
                    if constexpr (kSplitW)
                        umma_f16_ts(tmem_o + g * D, pw + 64 + ks * 8, umma_desc_v_mn<D>(vt, ks), idesc_o, 1u);
                }
            };
            ok = mbar_wait_bounded(q_bar, 0, abort_flag, p.status, WA_Q) &&
                 mbar_wait_bounded(&k_full[0], 0, abort_flag, p.status, WA_K);
            if (ok) {
                tc_fence_after();
                issue_s(0, 0);
                if (n1 > 0) issue_s(1, 0);
            }
            for (int j = 0; j < nmax && ok; ++j) {
                if (j >= 1) {
                    // the products of tile j - 1 are done with their value stage: tile j + 1 goes there
                    ok = mbar_wait_bounded(&v_free[(j - 1) % kAoVStages], ((j - 1) / kAoVStages) & 1u, abort_flag,
                                           p.status, WA_VFREE);
                    if (ok && j + 1 < nmax)
                        load_tile(smem + L::v + ((j + 1) % kAoVStages) * L::TILE, &map_v, zk, j + 1,
                                  &v_full[(j + 1) % kAoVStages]);
                }
                if (ok)
                    ok = mbar_wait_bounded(&v_full[j % kAoVStages], (j / kAoVStages) & 1u, abort_flag, p.status, WA_V);
                bool k_next = false;
                for (int g = 0; g < 2 && ok; ++g) {
                    const int n = g ? n1 : n0;
                    if (j >= n) continue;
                    ok = mbar_wait_bounded(&p_ready[g], j & 1u, abort_flag, p.status, WA_P);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(g, j);
                    if (j + 1 == n) umma_commit(&o_done[g]);
                    if (j + 1 < n) {
                        if (!k_next) {
                            ok = mbar_wait_bounded(&k_full[(j + 1) % kAoKStages], ((j + 1) / kAoKStages) & 1u,
                                                   abort_flag, p.status, WA_K);
                            if (!ok) break;
                            tc_fence_after();
                            k_next = true;
                        }
                        issue_s(g, j + 1);
                    }
                }
                if (!ok) break;
                umma_commit(&v_free[j % kAoVStages]);
                // both blocks have turned S(j) into weights, so product 1 of tile j is complete and
                // its key stage is free
                if (j + kAoKStages < nmax)
                    load_tile(smem + L::k + (j % kAoKStages) * L::TILE, &map_k, zk, j + kAoKStages,
                              &k_full[j % kAoKStages]);
            }
            if (!ok) {
                // copies that were requested may still land: give them time before the memory goes away
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else {
        // two groups of four warps: group g owns query block g; accumulator lanes 32 quad ..
        const int g = warp >> 2, quad = warp & 3;
        const int n = g ? n1 : n0;
        const int qt = 2 * rb2 + g;  // this block's query tile = its diagonal key tile
        const int rloc = quad * 32 + lane;
        const int row = qt * kTcRows + rloc;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t s_addr = lane_base + g * kTcRows;
        const uint32_t o_addr = lane_base + 2 * kTcRows + g * D;
        // Running softmax of this thread's row, log2 domain: the weights are taken against `m_ref`,
        // which follows the row's maximum lazily -- it moves only when a tile's maximum exceeds it
        // by more than 2^8 (so weights stay below 256, within fp16), and then the row of O and
        // the running sum are rescaled.  After the first tiles that is rare.
        float m_ref = -INFINITY, l0 = 0.f, l1 = 0.f;
        for (int j = 0; j < n && ok; ++j) {
            if (!mbar_wait_bounded(&s_ready[g], j & 1u, abort_flag, p.status, WA_S)) {
                ok = false;
                break;
            }
            // product 1 of tile j was issued behind product 2 of tile j - 1, so O_g is at rest
            // until this group announces its weights
            tc_fence_after();
            uint32_t v[128];  // this thread's row of S: 128 keys
            tmem_ld128(s_addr, v);
            // only the tile on the diagonal needs the causal mask: a warp-uniform branch between
            // two copies of the loops.  Keys past `lim` (tile-relative) are masked.
            const bool diag = j == qt;
            const int lim = row - j * kTcRows;
            float mx = -INFINITY, mx1 = -INFINITY;
            if (diag || scale2 <= 0.f) {
#pragma unroll
                for (int e = 0; e < 128; ++e) {
                    float x = __uint_as_float(v[e]) * scale2;
                    if (diag && e > lim) x = -INFINITY;  // keep key <= query
                    v[e] = __float_as_uint(x);
                    mx = fmaxf(mx, x);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 128; e += 2) {
                    mx = fmaxf(mx, __uint_as_float(v[e]));
                    mx1 = fmaxf(mx1, __uint_as_float(v[e + 1]));
                }
                mx = fmaxf(mx, mx1) * scale2;
            }
            const bool move = mx > m_ref + 8.f;  // always on the first tile
            if (__any_sync(0xffffffffu, move)) {
                const float m_new = move ? mx : m_ref;
                const float fac = !move ? 1.f : (m_ref == -INFINITY ? 0.f : ex2(m_ref - m_new));
                l0 *= fac;
                l1 *= fac;
                m_ref = m_new;
                if (j > 0) {
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(o_addr + c * 32, o);
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * fac);
                        tmem_st32(o_addr + c * 32, o);
                    }
                }
            }
            auto weights = [&](auto scaled) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t w[16];                  // 32 weights, packed in pairs
                    [[maybe_unused]] uint32_t wl[kSplitW ? 16 : 1];   // their remainders
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float x0, x1;
                        if constexpr (decltype(scaled)::value) {  // v holds scaled, masked logits
                            x0 = ex2(__uint_as_float(v[c * 32 + e]) - m_ref);
                            x1 = ex2(__uint_as_float(v[c * 32 + e + 1]) - m_ref);
                        } else {
                            x0 = ex2(fmaf(__uint_as_float(v[c * 32 + e]), scale2, -m_ref));
                            x1 = ex2(fmaf(__uint_as_float(v[c * 32 + e + 1]), scale2, -m_ref));
                        }
                        l0 += x0;
                        l1 += x1;
                        if constexpr (E::kIsBf16) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
                            const float2 hb = __bfloat1622float2(h);
                            const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - hb.x, x1 - hb.y);
                            w[e / 2] = *reinterpret_cast<const uint32_t *>(&h);
                            wl[e / 2] = *reinterpret_cast<const uint32_t *>(&l);
                        } else {
                            const __half2 h = __floats2half2_rn(x0, x1);
                            w[e / 2] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                    }
                    // the whole row is in registers, so its columns can be overwritten
                    tmem_st16(s_addr + c * 16, w);
                    if constexpr (kSplitW) tmem_st16(s_addr + 64 + c * 16, wl);
                }
            };
            if (diag || scale2 <= 0.f)
                weights(std::true_type{});
            else
                weights(std::false_type{});
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_ready[g]);
        }
        if (n > 0 && ok && mbar_wait_bounded(&o_done[g], 0, abort_flag, p.status, WA_O)) {
            tc_fence_after();
            const float l = l0 + l1;
            const float inv = 1.0f / l;  // the key at position 0 is visible to every query: l > 0
            if (row < Tn) p.lse_out[(size_t)zq * Tn + row] = (m_ref + log2f(l)) * kLn2;
            T *orow = static_cast<T *>(out_ptr) + ((size_t)zq * Tn + row) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(o_addr + c * 32, o);
                if (row < Tn) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t pk[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float a0 = __uint_as_float(o[e + 2 * k]) * inv;
                            const float a1 = __uint_as_float(o[e + 2 * k + 1]) * inv;
                            if constexpr (E::kIsBf16) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(a0, a1);
                                pk[k] = *reinterpret_cast<const uint32_t *>(&h);
                            } else {
                                const __half2 h = __floats2half2_rn(a0, a1);
                                pk[k] = *reinterpret_cast<const uint32_t *>(&h);
                            }
                        }
                        *reinterpret_cast<uint4 *>(orow + c * 32 + e) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(L::tmem_cols)
                     : "memory");
}

// ---------------------------------------------------------------------------
// Window scoring of the prompt pass (App. B: the last W prompt queries score the keys) on tcgen05:
// the scaled, causally masked logits of a unit's G*W window queries against every key, fp32
// [G*W][T], and per 128-key chunk each query row's (max, sum exp) -- the same outputs as the
// warp-level kernel of the prompt pass, for windows of G*W = 32, 64, 96 or 128 rows.
// Persistent CTAs, grid (CTAs per unit, units): CTA x takes the unit's chunks x, x + gridDim.x, ...
// The window's queries are resident in shared memory (one TMA box of G*W rows); 128-key chunks
// stream through a two-stage ring (TMA, 128-byte swizzle).  One thread requests chunks and issues
// the products: positions are the M side (a chunk's 128 keys = the 128 tensor-memory lanes), the
// window's rows the N side, two accumulators of G*W columns so the next chunk's product runs under
// this chunk's write-out.  Write-out, 32 query rows at a time: the NW warps move their lanes'
// columns (128 / NW each) into a shared tile [row][position], then take 32 / NW rows each -- a lane
// handles positions lane, lane + 32, ... -- which gives coalesced row writes and the row's
// (max, sum exp) of the chunk by warp shuffles; two tiles taken in turn, one named barrier per
// round.  Two CTAs share an SM for windows of up to 64 rows.
// ---------------------------------------------------------------------------
// NW write-out warps (8 for windows of up to 64 rows, where two CTAs share an SM; 16 beyond, where the
// CTA has the SM to itself) + the warp that requests and issues
constexpr int kWlStages = 2;
constexpr int kWlLT = kTcRows + 4;  // padded row of the shared tile (floats)
enum : int32_t { WW_Q = 61, WW_K = 62, WW_ACC = 63, WW_MMA = 64 };

template <int D>
struct WlSmem {
    static constexpr int KB = D / kTcKBlock;
    static constexpr int KBLOCK = kTcRows * 128;
    static constexpr int TILE = KB * KBLOCK;  // a chunk of keys
    static constexpr int k = 0;
    static constexpr int q = kWlStages * TILE;  // up to 128 query rows
    static __host__ __device__ constexpr int lt(int GW) { return q + KB * GW * 128; }
    static __host__ __device__ constexpr int bars(int GW) { return lt(GW) + 2 * 32 * kWlLT * 4; }  // two tiles
    static __host__ __device__ constexpr int total(int GW) { return bars(GW) + 128 + 1024; }
};

template <typename T, int D, int NW>
__global__ void __launch_bounds__(NW * 32 + 32, NW == 8 ? 2 : 1)
    window_logits_tc_kernel(const WindowLogitsParams p, const __grid_constant__ CUtensorMap map_k,
                            const __grid_constant__ CUtensorMap map_q) {
    using L = WlSmem<D>;
    constexpr int KS = D / 16;
    constexpr int CH = kTcRows;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int GW = p.G * p.W;
    float *lt = reinterpret_cast<float *>(smem + L::lt(GW));
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L::bars(GW));  // [2] chunk landed
    uint64_t *mma_bar = full_bar + kWlStages;                               // [2] product finished
    uint64_t *acc_free = mma_bar + 2;                                       // [2] accumulator read
    uint64_t *q_bar = acc_free + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_bar + 1);
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(tmem_slot + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ul = blockIdx.y;
    const int b = ul / p.n_kv_heads, h = ul % p.n_kv_heads;
    const int T_len = p.T, W = p.W;
    const int n_chunks = (T_len + CH - 1) / CH;
    const int n_my = blockIdx.x < n_chunks ? (n_chunks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    // tensor-memory columns: two accumulators of GW columns, rounded up to a power of two
    const uint32_t tmem_cols = GW <= 32 ? 64u : (GW <= 64 ? 128u : 256u);

    if (tid == 0) {
        for (int s = 0; s < kWlStages; ++s) mbar_init(&full_bar[s], 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&mma_bar[s], 1);
            mbar_init(&acc_free[s], 4);
        }
        mbar_init(q_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;

    if (warp == NW) {
        if (lane == 0 && n_my > 0) {
            auto load_chunk = [&](int i) {  // this CTA's i-th chunk into stage i % 2
                const int s = i % kWlStages;
                const int c = blockIdx.x + i * gridDim.x;
                mbar_arrive_expect_tx(&full_bar[s], L::TILE);
#pragma unroll
                for (int kb = 0; kb < L::KB; ++kb)
                    tma_load_3d(smem + L::k + s * L::TILE + kb * L::KBLOCK, &map_k, kb * kTcKBlock, c * CH, ul,
                                &full_bar[s]);
            };
            // the unit's window: rows (b, h G .. h G + G - 1, 0 .. W - 1) are consecutive
            mbar_arrive_expect_tx(q_bar, L::KB * GW * 128);
#pragma unroll
            for (int kb = 0; kb < L::KB; ++kb)
                tma_load_3d(smem + L::q + kb * GW * 128, &map_q, kb * kTcKBlock,
                            (b * p.n_kv_heads + h) * GW, 0, q_bar);
            for (int i = 0; i < kWlStages && i < n_my; ++i) load_chunk(i);
            const uint32_t f = Elem<T>::kIsBf16 ? 1u : 0u;
            const uint32_t idesc = (1u << 4) | (f << 7) | (f << 10) | ((static_cast<uint32_t>(GW) >> 3) << 17) |
                                   ((kTcRows >> 4) << 24);
            ok = mbar_wait_bounded(q_bar, 0, abort_flag, p.status, WW_Q);
            for (int i = 0; i < n_my && ok; ++i) {
                const int s = i % kWlStages, buf = i & 1;
                ok = mbar_wait_bounded(&full_bar[s], (i / kWlStages) & 1u, abort_flag, p.status, WW_K);
                if (ok && i >= 2)
                    ok = mbar_wait_bounded(&acc_free[buf], ((i - 2) >> 1) & 1u, abort_flag, p.status, WW_ACC);
                if (!ok) break;
                tc_fence_after();
                const uint8_t *kt = smem + L::k + s * L::TILE;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int ko = (ks / 4) * L::KBLOCK + (ks % 4) * 32;   // 16 elements = 32 bytes on
                    const int qo = (ks / 4) * GW * 128 + (ks % 4) * 32;
                    umma_f16_ss(tmem_base + buf * GW, umma_desc_sw128(kt + ko), umma_desc_sw128(smem + L::q + qo),
                                idesc, ks > 0);
                }
                umma_commit(&mma_bar[buf]);
                // the finished product frees the chunk's stage: request the chunk two on
                if (i + kWlStages < n_my) {
                    ok = mbar_wait_bounded(&mma_bar[buf], (i >> 1) & 1u, abort_flag, p.status, WW_MMA);
                    if (ok) load_chunk(i + kWlStages);
                }
            }
            if (!ok) {
                // copies that were requested may still land: give them time before the memory goes away
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else {
        float *logits = p.logits + (size_t)ul * GW * T_len;
        float2 *partial = p.partial + (size_t)ul * GW * n_chunks;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        int rounds = 0;
        for (int i = 0; i < n_my; ++i) {
            const int buf = i & 1;
            const int chunk = blockIdx.x + i * gridDim.x;
            const int t0 = chunk * CH;
            // A warp whose wait gave up does no more work and no more waiting, but it still walks
            // the named barriers below (they have no time limit), so no other warp is left there.
            if (ok && !mbar_wait_bounded(&mma_bar[buf], (i >> 1) & 1u, abort_flag, p.status, WW_MMA)) ok = false;
            tc_fence_after();
            for (int qb = 0; qb < GW; qb += 32) {
                // two tiles taken in turn: a round's barrier also says that every warp is done
                // with the rows of the round before, so the tile of the round before that is free
                float *tile = lt + (rounds & 1) * 32 * kWlLT;
                ++rounds;
                if (ok) {
                    // lanes = positions 32 (warp % 4) .. of the chunk; warp w takes the query rows
                    // qb + CW (w / 4) .. of the block
                    constexpr int CW = 128 / NW;  // columns per warp: 16 or 8
                    uint32_t v[CW];
                    const int c0 = (warp >> 2) * CW;
                    if constexpr (CW == 16)
                        tmem_ld16(lane_base + buf * GW + qb + c0, v);
                    else
                        tmem_ld8(lane_base + buf * GW + qb + c0, v);
                    tc_fence_before();
#pragma unroll
                    for (int c = 0; c < CW; ++c)
                        tile[(c0 + c) * kWlLT + (warp & 3) * 32 + lane] = __uint_as_float(v[c]) * p.scale;
                }
                named_bar_sync(1, NW * 32);
                // The accumulator goes back only now, behind a barrier of all write-out warps: every
                // warp has then passed its wait for this chunk's product.  Handed back by the
                // loading warps as they finish, the barrier of that wait could complete twice more
                // -- the next product but one needs nothing else -- before a late warp has looked
                // at it, and that warp would wait for a phase that can no longer come.
                if (qb + 32 >= GW && warp < 4 && lane == 0) mbar_arrive(&acc_free[buf]);
                // warp w: query rows RW w .. of the block (RW = 4 or 2); lane: positions lane + 32 i
                constexpr int RW = 32 / NW;
#pragma unroll
                for (int jr = 0; jr < RW && ok; ++jr) {
                    const int gw = qb + warp * RW + jr;
                    const int tau = T_len - W + (gw % W);  // the query's own position: keys 0..tau
                    float m = -INFINITY;
                    float lg[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int t = t0 + lane + 32 * k;
                        lg[k] = (t < T_len && t <= tau) ? tile[(warp * RW + jr) * kWlLT + lane + 32 * k] : -INFINITY;
                        if (t < T_len) logits[(size_t)gw * T_len + t] = lg[k];
                        m = fmaxf(m, lg[k]);
                    }
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                    float sum = 0.f;
                    if (m > -INFINITY) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) sum += expf(lg[k] - m);
                    }
#pragma unroll
                    for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                    if (lane == 0) partial[(size_t)gw * n_chunks + chunk] = make_float2(m, sum);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                     : "memory");
}

// cuTensorMapEncodeTiled, looked up through the runtime so that the library does not link
// against the driver library directly.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// [heads][T][D] row-major, 16-bit elements, seen as (d, position, head); boxes of 64 x 128 x 1 with
// the 128-byte swizzle; positions past T read as zero.
bool make_map(CUtensorMap *map, const void *base, int heads, int T, int D, bool bf16) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)heads};
    const cuuint64_t gstride[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kTcKBlock, (cuuint32_t)kTcRows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
              const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows][D] row-major, 16-bit elements, seen as (d, row, 1): boxes of 64 x box_rows with the
// 128-byte swizzle.
bool make_map_rows(CUtensorMap *map, const void *base, size_t rows, int D, int box_rows, bool bf16) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)rows, 1};
    const cuuint64_t gstride[2] = {(cuuint64_t)D * 2, (cuuint64_t)rows * D * 2};
    const cuuint32_t box[3] = {(cuuint32_t)kTcKBlock, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
              const_cast<void *>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int D>
int launch_window_one(const WindowLogitsParams &p, int grid_x, cudaStream_t stream) {
    const int GW = p.G * p.W;
    CUtensorMap map_k, map_q;
    if (!make_map(&map_k, p.K, p.units, p.T, D, Elem<T>::kIsBf16) ||
        !make_map_rows(&map_q, p.Qw, (size_t)p.units * GW, D, GW, Elem<T>::kIsBf16))
        return static_cast<int>(cudaErrorInvalidValue);
    if (GW <= 64)
        window_logits_tc_kernel<T, D, 8><<<dim3(grid_x, p.units), 8 * 32 + 32, WlSmem<D>::total(GW), stream>>>(p, map_k, map_q);
    else
        window_logits_tc_kernel<T, D, 16><<<dim3(grid_x, p.units), 16 * 32 + 32, WlSmem<D>::total(GW), stream>>>(p, map_k, map_q);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D>
int prepare_window_one() {
    cudaError_t e = cudaFuncSetAttribute(window_logits_tc_kernel<T, D, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         WlSmem<D>::total(64));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(window_logits_tc_kernel<T, D, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 WlSmem<D>::total(128));
    return static_cast<int>(e);
}

template <typename T, int D>
int launch_full_one(const FullScoreParams &p, cudaStream_t stream) {
    constexpr int SMEM = TcSmem<D>::total;
    CUtensorMap map_k, map_q;
    if (!make_map(&map_k, p.K, p.batch * p.n_kv_heads, p.T, D, Elem<T>::kIsBf16) ||
        !make_map(&map_q, p.Q, p.batch * p.n_kv_heads * p.G, p.T, D, Elem<T>::kIsBf16))
        return static_cast<int>(cudaErrorInvalidValue);
    const int nres = (p.T + kTcRows - 1) / kTcRows;
    FullScoreParams q = p;
    if (!p.lse) {
        const dim3 grid(nres, p.batch * p.n_kv_heads * p.G);
        full_pass_tc_kernel<T, D, false><<<grid, kTcThreads, SMEM, stream>>>(q, map_k, map_q);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return static_cast<int>(e);
        q.lse = p.lse_out;
    }
    const dim3 grid(nres, p.batch * p.n_kv_heads);
    full_pass_tc_kernel<T, D, true><<<grid, kTcThreads, SMEM, stream>>>(q, map_k, map_q);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D>
int prepare_full_one() {
    cudaError_t e = cudaFuncSetAttribute(full_pass_tc_kernel<T, D, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, TcSmem<D>::total);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(full_pass_tc_kernel<T, D, true>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, TcSmem<D>::total);
    return static_cast<int>(e);
}

// Pass 1 alone: every query row's log-sum-exp into p.lse_out.
template <typename T, int D>
int launch_rows_one(const FullScoreParams &p, cudaStream_t stream) {
    CUtensorMap map_k, map_q;
    if (!make_map(&map_k, p.K, p.batch * p.n_kv_heads, p.T, D, Elem<T>::kIsBf16) ||
        !make_map(&map_q, p.Q, p.batch * p.n_kv_heads * p.G, p.T, D, Elem<T>::kIsBf16))
        return static_cast<int>(cudaErrorInvalidValue);
    const int nres = (p.T + kTcRows - 1) / kTcRows;
    const dim3 grid(nres, p.batch * p.n_kv_heads * p.G);
    full_pass_tc_kernel<T, D, false><<<grid, kTcThreads, TcSmem<D>::total, stream>>>(p, map_k, map_q);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D>
int launch_attn_one(const FullScoreParams &p, const void *V, void *out, cudaStream_t stream) {
    CUtensorMap map_k, map_v, map_q;
    if (!make_map(&map_k, p.K, p.batch * p.n_kv_heads, p.T, D, Elem<T>::kIsBf16) ||
        !make_map(&map_v, V, p.batch * p.n_kv_heads, p.T, D, Elem<T>::kIsBf16) ||
        !make_map(&map_q, p.Q, p.batch * p.n_kv_heads * p.G, p.T, D, Elem<T>::kIsBf16))
        return static_cast<int>(cudaErrorInvalidValue);
    const int nres = (p.T + kTcRows - 1) / kTcRows;
    const dim3 grid((nres + 1) / 2, p.batch * p.n_kv_heads * p.G);  // two query blocks per CTA
    attn_out_tc_kernel<T, D><<<grid, kAoThreads, AoSmem<D>::total, stream>>>(p, out, map_k, map_v, map_q);
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D>
int prepare_attn_one() {
    return static_cast<int>(cudaFuncSetAttribute(attn_out_tc_kernel<T, D>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, AoSmem<D>::total));
}

}  // namespace

int launch_attention_output(int dtype, int D, const FullScoreParams &p, const void *V, void *out,
                            cudaStream_t stream) {
    if (dtype == 1 && D == 64) return launch_attn_one<__half, 64>(p, V, out, stream);
    if (dtype == 1 && D == 128) return launch_attn_one<__half, 128>(p, V, out, stream);
    if (dtype == 2 && D == 64) return launch_attn_one<__nv_bfloat16, 64>(p, V, out, stream);
    if (dtype == 2 && D == 128) return launch_attn_one<__nv_bfloat16, 128>(p, V, out, stream);
    return -1;
}

int launch_row_statistics(int dtype, int D, const FullScoreParams &p, cudaStream_t stream) {
    if (dtype == 1 && D == 64) return launch_rows_one<__half, 64>(p, stream);
    if (dtype == 1 && D == 128) return launch_rows_one<__half, 128>(p, stream);
    if (dtype == 2 && D == 64) return launch_rows_one<__nv_bfloat16, 64>(p, stream);
    if (dtype == 2 && D == 128) return launch_rows_one<__nv_bfloat16, 128>(p, stream);
    return -1;
}

int launch_full_scores(int dtype, int D, const FullScoreParams &p, cudaStream_t stream) {
    if (dtype == 1 && D == 64) return launch_full_one<__half, 64>(p, stream);
    if (dtype == 1 && D == 128) return launch_full_one<__half, 128>(p, stream);
    if (dtype == 2 && D == 64) return launch_full_one<__nv_bfloat16, 64>(p, stream);
    if (dtype == 2 && D == 128) return launch_full_one<__nv_bfloat16, 128>(p, stream);
    return -1;
}

bool window_logits_tc_supported(int GW) { return GW >= 32 && GW <= 128 && GW % 32 == 0; }

int launch_window_logits_tc(int dtype, int D, const WindowLogitsParams &p, int grid_x, cudaStream_t stream) {
    if (!window_logits_tc_supported(p.G * p.W)) return -1;
    if (dtype == 1 && D == 64) return launch_window_one<__half, 64>(p, grid_x, stream);
    if (dtype == 1 && D == 128) return launch_window_one<__half, 128>(p, grid_x, stream);
    if (dtype == 2 && D == 64) return launch_window_one<__nv_bfloat16, 64>(p, grid_x, stream);
    if (dtype == 2 && D == 128) return launch_window_one<__nv_bfloat16, 128>(p, grid_x, stream);
    return -1;
}

int prepare_full_scores(int dtype, int D) {
    int rc = -1;
    if (dtype == 1 && D == 64)
        rc = prepare_full_one<__half, 64>() | prepare_attn_one<__half, 64>() | prepare_window_one<__half, 64>();
    if (dtype == 1 && D == 128)
        rc = prepare_full_one<__half, 128>() | prepare_attn_one<__half, 128>() | prepare_window_one<__half, 128>();
    if (dtype == 2 && D == 64)
        rc = prepare_full_one<__nv_bfloat16, 64>() | prepare_attn_one<__nv_bfloat16, 64>() |
             prepare_window_one<__nv_bfloat16, 64>();
    if (dtype == 2 && D == 128)
        rc = prepare_full_one<__nv_bfloat16, 128>() | prepare_attn_one<__nv_bfloat16, 128>() |
             prepare_window_one<__nv_bfloat16, 128>();
    return rc;
}

}  // namespace zsm
