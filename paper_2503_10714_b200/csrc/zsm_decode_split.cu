// Split form of the fused decode step (Algorithm 1 + Eq. (att_score2)): one thread-block cluster
// per unit.  Rank c of the cluster streams token rows [lo_c, hi_c) of the unit through its own
// ring (K, scores and positions, V: each row still crosses HBM once); rank 0 also takes the
// merged slots and the new token.  Three exchanges through distributed shared memory tie the
// slices together:
//   softmax   every rank posts (max, sum exp) of its slice to every rank           (D2)
//   victim    every rank posts its lowest (score, position) key to rank 0          (D5)
//   output    every rank posts its normalised partial output to rank 0             (D3)
// Every rank's tail warp folds its consumer warps' victim candidates and posts the result, so
// the consumer warps go from the score tiles straight on to the V tiles; rank 0's tail warp then
// does the residual fill / merge and the insertion (D6, D7) once every rank has read its last
// tile.  By the time the output pass starts its tiles are already in the ring (they were
// requested while the softmax exchange ran), so small groups of warps take different tiles at
// the same time instead of all warps sharing one.  All cross-CTA waits are on mbarriers with a
// time limit; the cluster barrier at the end keeps a CTA's shared memory alive until its peers
// are done with it.
//
// The launch is a programmatic dependent launch: barrier set-up, the cluster barrier and (when
// the caller's stream order allows it, SplitParams::early) the unit's counters and a ring-full of
// K tiles are taken care of while the preceding kernel of the stream is still running; only then
// does the kernel wait for that kernel (griddepcontrol.wait) and fetch what depends on it -- q,
// k_new, v_new and the fusion counts, into a header buffer of their own.  It lets its own
// successor start (griddepcontrol.launch_dependents) right after that wait, never before, so at
// most two kernels of a stream overlap.  A CTA is sized so that two fit on an SM: the next
// layer's CTAs settle in beside this layer's.
#include "zsm_decode_split.cuh"

#include <type_traits>

namespace zsm {

namespace {

constexpr int kSplitThreads = (kMaxConsumerWarps + kExtraWarps) * 32;
constexpr int kSplitPairThreads = (kPairConsumerWarps + kExtraWarps) * 32;
constexpr int kSplitMaxDynamicSmem = 232448;  // 227 KiB, the opt-in limit per CTA on sm_100
constexpr int kSplitVGroup = 2;

enum : int32_t {
    WS_PRODUCER = 21, WS_HEADER = 22, WS_K = 23, WS_KR = 24, WS_META = 25, WS_V = 26, WS_VR = 27,
    WS_SOFTMAX = 28, WS_VICTIM = 29, WS_DONE_OUT = 30, WS_DONE_TAIL = 31, WS_VICTIM_LOCAL = 32,
    WS_HEADER_TAIL = 33
};

struct __align__(16) VictimPost {
    uint64_t key;   // (score bits << 32) | position; all ones: no candidate
    int32_t slot;   // unit-wide token slot; -2: the new token itself (B_p = 0)
    int32_t pad;
};

// ---- cluster primitives ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(const void *p, uint32_t rank) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(p)), "r"(rank));
    return ra;
}
__device__ __forceinline__ void st_remote_f32(uint32_t ra, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}
__device__ __forceinline__ void st_remote_b64(uint32_t ra, uint64_t v) {
    asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(ra), "l"(v) : "memory");
}
__device__ __forceinline__ void st_remote_b32(uint32_t ra, uint32_t v) {
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(ra), "r"(v) : "memory");
}
// Arrival on a peer's mbarrier; orders this thread's earlier writes before it for the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t ra) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(ra) : "memory");
}
__device__ __forceinline__ void fence_cluster() {
    asm volatile("fence.acq_rel.cluster;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    cluster_arrive();
    cluster_wait();
}
// Programmatic dependent launch: wait until the kernels this launch depends on have completed
// and their writes are visible (returns at once for an ordinary launch) ...
__device__ __forceinline__ void griddep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// ... and let the next kernel of the stream begin its own prologue.
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that peers of the cluster arrive on; same contract as
// mbar_wait_bounded.
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint64_t *bar, uint32_t parity,
                                                          volatile int32_t *abort_flag,
                                                          int32_t *status, int32_t where) {
    const uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity, kSuspendHintNs)) return true;
        ++polls;
        if ((polls & 7u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                dev_set_status(status, DEV_ERR_TIMEOUT, where, static_cast<int32_t>(blockIdx.x));
                *abort_flag = 1;
                __threadfence_block();
                return false;
            }
        }
    }
}

// Lowest (score bits, position) key over the warp and the slot that carries it, in every lane.
// Scores are non-negative, so their bit patterns order like the values; keys are distinct
// (positions are) unless they are the all-ones "no candidate".
__device__ __forceinline__ void warp_min_key(uint64_t &key, int &slot) {
    const uint32_t hi = static_cast<uint32_t>(key >> 32), lo = static_cast<uint32_t>(key);
    const uint32_t mh = __reduce_min_sync(0xffffffffu, hi);
    const uint32_t ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
    const unsigned who = __ballot_sync(0xffffffffu, hi == mh && lo == ml);
    slot = __shfl_sync(0xffffffffu, slot, __ffs(who) - 1);
    key = (static_cast<uint64_t>(mh) << 32) | ml;
}

// Consumer warps of a CTA that post a share of its partial output (one output element per thread).
__device__ __forceinline__ int split_post_warps(int consumer_warps, int outputs) {
    const int w = (outputs + 31) / 32;
    return w < consumer_warps ? w : consumer_warps;
}

// Four consecutive elements of a row in the storage dtype, widened.
template <typename T>
__device__ __forceinline__ void load4s(const T *p, float (&f)[4]) {
    if constexpr (sizeof(T) == 4) {
        const float4 t = *reinterpret_cast<const float4 *>(p);
        f[0] = t.x;
        f[1] = t.y;
        f[2] = t.z;
        f[3] = t.w;
    } else {
        const uint2 t = *reinterpret_cast<const uint2 *>(p);
        const T *e = reinterpret_cast<const T *>(&t);
#pragma unroll
        for (int i = 0; i < 4; ++i) f[i] = Elem<T>::to_float(e[i]);
    }
}

// Everything between the two cluster barriers of the kernel.  A thread leaves this function
// when its role is done or a bounded wait gave up; it never leaves the kernel from here.
template <typename T, int D, int G>
__device__ __forceinline__ void split_body(const SplitParams &sp, uint8_t *smem, const SplitSmem &L,
                                           const UnitDesc &d, const int rank, const int C) {
    using E = Elem<T>;
    const DecodeParams &p = sp.d;
    constexpr int EPL = E::EPL;
    constexpr int EP2 = EPL / 2;
    constexpr int ROWB = D * (int)sizeof(T);
    constexpr int LPR = D / EPL;
    constexpr int RPW = 32 / LPR;
    constexpr int R = kTileBytes / ROWB;
    constexpr int ROWB32 = D * 4;
    constexpr int LPR32 = D / 4;
    constexpr int RPW32 = 32 / LPR32;
    constexpr int R32 = kTileBytes / ROWB32;
    constexpr int HDR_K = G * ROWB;  // header tile: q (G rows), k_new, v_new, fusion counts
    constexpr int HDR_V = HDR_K + ROWB;
    constexpr int HDR_W = HDR_V + ROWB;
    constexpr int UBV = G <= 4 ? 4 : 2;
    constexpr bool kMma = sizeof(T) == 2;
    constexpr int SEG = ROWB / 64;
    constexpr int RB = R / 16;

    const int NW = (blockDim.x >> 5) - kExtraWarps;
    const int NT = NW * 32;
    const int S = p.stages;

    uint8_t *ring = smem + L.ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *empty_bar = full_bar + S;
    uint64_t *x_soft = empty_bar + S;  // every rank arrives: softmax partials are in
    uint64_t *x_vict = x_soft + 1;     // rank 0's: every rank's victim candidate is in
    uint64_t *x_done = x_vict + 1;     // rank 0's: partial outputs in, last tiles read
    uint64_t *p_ready = x_done + 1;    // consumer warps -> tail warp: the slice's exponentials are written
    uint64_t *hdr_bar = p_ready + 1;   // the header (q, k_new, v_new, fusion counts) has landed
    uint64_t *meta_bar = hdr_bar + 1;  // the slice's scores and positions have landed
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(smem + L.flags);
    float *probs = reinterpret_cast<float *>(smem + L.probs);  // [local slot][G]
    float *qf = reinterpret_cast<float *>(smem + L.qf);
    const uint8_t *hdr = smem + L.hdr;
    float *meta_s = reinterpret_cast<float *>(smem + L.meta);                 // [l_stride] scores
    int32_t *meta_p = reinterpret_cast<int32_t *>(smem + L.meta) + p.l_stride;  // [l_stride] positions
    const uint4 *kn_raw = reinterpret_cast<const uint4 *>(hdr + HDR_K);
    const uint4 *vn_raw = reinterpret_cast<const uint4 *>(hdr + HDR_V);
    const uint32_t *w_s = reinterpret_cast<const uint32_t *>(hdr + HDR_W);
    float *krs = reinterpret_cast<float *>(smem + L.krs);
    float *opart = reinterpret_cast<float *>(smem + L.opart);
    float *redf = reinterpret_cast<float *>(smem + L.redf);
    float *redf2 = redf + kMaxConsumerWarps * 8;
    float *xs = reinterpret_cast<float *>(smem + L.xs);  // [rank][16]: max[8], sum[8]
    VictimPost *xv = reinterpret_cast<VictimPost *>(smem + L.xv);
    float *xo = reinterpret_cast<float *>(smem + L.xo);  // [rank][G][D]

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const bool is_producer = warp == NW && lane == 0;

    // Every peer's barriers exist once the cluster barrier of the prologue completes; the
    // producer thread needs only this CTA's own and passes it after its first copies are out.
    if (!is_producer) cluster_wait();
    // The unit's counters were written by this unit's previous step.  With `early` the caller's
    // stream order guarantees that step finished long ago; otherwise wait for the predecessor.
    if (!sp.early) griddep_wait();
    const int4 cnt = *reinterpret_cast<const int4 *>(p.counters + d.unit);
    const int cap = d.Bp + d.Bc;
    const int n_live = min(max(cnt.x, 0), cap);
    const int n_res = min(max(cnt.y, 0), d.Br);
    const int Tpos = cnt.z;
    const int ul = d.unit - p.unit_base;
    const int br_pad = (d.Br + 3) & ~3;
    int row_lo, row_hi;
    split_slice(n_live, n_res, (int)sizeof(T), C, rank, row_lo, row_hi);
    const int n_loc = row_hi - row_lo;
    const int nr_loc = rank == 0 ? n_res : 0;                   // merged slots live on rank 0
    const int n_ent = n_loc + nr_loc + (rank == 0 ? 1 : 0);     // + the new token

    // =====================================================================
    // Producer: one thread issues every bulk copy of this CTA.
    // =====================================================================
    if (warp == NW) {
        if (lane != 0) return;
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        // The header depends on the preceding kernel (q, k_new, v_new are its results; the
        // fusion counts may be): it is requested after the dependency wait.  With `early` up to a
        // ring-full of tiles is requested before that wait.
        bool header_out = false;
        int issued = 0;
        auto header = [&]() {
            if (sp.early) {
                cluster_wait();
                griddep_wait();
            }
            griddep_launch_dependents();
            mbar_arrive_expect_tx(hdr_bar, HDR_W + br_pad * 4u);
            uint8_t *dst = smem + L.hdr;
            bulk_g2s(dst, static_cast<const uint8_t *>(p.q) + (size_t)ul * G * ROWB, G * ROWB, hdr_bar);
            bulk_g2s(dst + HDR_K, static_cast<const uint8_t *>(p.k_new) + (size_t)ul * ROWB, ROWB, hdr_bar);
            bulk_g2s(dst + HDR_V, static_cast<const uint8_t *>(p.v_new) + (size_t)ul * ROWB, ROWB, hdr_bar);
            if (br_pad > 0) bulk_g2s(dst + HDR_W, p.base + d.w_off, br_pad * 4u, hdr_bar);
            header_out = true;
        };
        // scores and positions of the slice: a buffer of their own (the tail warp works on them
        // while the consumer warps are in the output pass); cache state, like the K tiles
        auto load_meta = [&]() {
            const uint32_t n4 = static_cast<uint32_t>((n_loc + 3) & ~3);
            mbar_arrive_expect_tx(meta_bar, n4 * 8u);
            if (n4 > 0) {
                bulk_g2s(meta_s, p.base + d.score_off + (size_t)row_lo * 4, n4 * 4u, meta_bar);
                bulk_g2s(meta_p, p.base + d.pos_off + (size_t)row_lo * 4, n4 * 4u, meta_bar);
            }
        };
        if (sp.early) {
            load_meta();
        } else {
            cluster_wait();
            header();
            load_meta();
        }
        auto acquire = [&](uint32_t bytes, uint64_t *&bar) -> uint8_t * {
            // the consumers free no stage before they have the header: once the ring is full
            // the header has to go out first
            if (!header_out && issued == S) header();
            if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, p.status, WS_PRODUCER)) {
                ok = false;
                return nullptr;
            }
            bar = &full_bar[s];
            mbar_arrive_expect_tx(bar, bytes);
            uint8_t *dst = ring + static_cast<size_t>(s) * kTileBytes;
            if (++s == S) {
                s = 0;
                ph ^= 1u;
            }
            ++issued;
            return dst;
        };
        uint64_t *bar = nullptr;
        uint8_t *dst;
        // merged keys first: they are few, and their logits need a logarithm each
        for (int r0 = 0; r0 < nr_loc && ok; r0 += R32) {
            const uint32_t bytes = static_cast<uint32_t>(min(R32, nr_loc - r0)) * ROWB32;
            dst = acquire(bytes, bar);
            if (ok) bulk_g2s(dst, p.base + d.kr_off + (size_t)r0 * ROWB32, bytes, bar);
        }
        for (int r0 = row_lo; r0 < row_hi && ok; r0 += R) {
            const uint32_t bytes = static_cast<uint32_t>(min(R, row_hi - r0)) * ROWB;
            dst = acquire(bytes, bar);
            if (ok) bulk_g2s(dst, p.base + d.k_off + (size_t)r0 * ROWB, bytes, bar);
        }
        for (int r0 = row_lo; r0 < row_hi && ok; r0 += R) {
            const uint32_t bytes = static_cast<uint32_t>(min(R, row_hi - r0)) * ROWB;
            dst = acquire(bytes, bar);
            if (ok) bulk_g2s(dst, p.base + d.v_off + (size_t)r0 * ROWB, bytes, bar);
        }
        for (int r0 = 0; r0 < nr_loc && ok; r0 += R32) {
            const uint32_t bytes = static_cast<uint32_t>(min(R32, nr_loc - r0)) * ROWB32;
            dst = acquire(bytes, bar);
            if (ok) bulk_g2s(dst, p.base + d.vr_off + (size_t)r0 * ROWB32, bytes, bar);
        }
        if (!header_out) header();  // a unit shorter than the ring
        if (!ok) {
            // give copies already in flight time to land before the CTA's memory goes away
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        return;
    }
    // every other thread: nothing below may run before the preceding kernel is complete, except
    // the tail warp's prefetch of the merged keys when `early` allows it
    const bool is_tail = warp == NW + 1;
    if (sp.early && !is_tail) griddep_wait();

    const int l32 = lane % LPR32;  // 16-byte column of an fp32 residual row
    const int sub32 = lane / LPR32;

    // =====================================================================
    // Tail warp (rank 0): residual fill / merge, insertion, counters.
    // =====================================================================
    if (warp == NW + 1) {
        float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
        float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
        // the merged keys of a full residual pool are fetched while the slices stream
        const bool resident = rank == 0 && n_res == d.Br && n_res > 0 && n_res <= sp.kr_rows;
        if (resident) {
            const int chunks = n_res * (ROWB32 / 16);
            for (int i = lane; i < chunks; i += 32)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(
                                 smem_u32(reinterpret_cast<uint8_t *>(krs) + (size_t)i * 16)),
                             "l"(reinterpret_cast<const uint8_t *>(Kr_g) + (size_t)i * 16)
                             : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (sp.early) griddep_wait();
        // D4 + D5 for this rank's slice, while the consumer warps are in the output pass: needs
        // the slice's exponentials, the cluster's normaliser, and the scores and positions
        if (!mbar_wait_bounded(p_ready, 0, abort_flag, p.status, WS_VICTIM_LOCAL) ||
            !mbar_wait_bounded_cluster(x_soft, 0, abort_flag, p.status, WS_SOFTMAX) ||
            !mbar_wait_bounded(meta_bar, 0, abort_flag, p.status, WS_META)) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            return;
        }
        float s_tok = 0.f;  // first score of the new token: its own attention weight (rank 0)
        {
            float fac[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float M = -INFINITY;
                for (int r = 0; r < C; ++r) M = fmaxf(M, xs[r * 16 + g]);
                float Z = 0.f;
                for (int r = 0; r < C; ++r) Z = fmaf(xs[r * 16 + 8 + g], expf(xs[r * 16 + g] - M), Z);
                fac[g] = expf(xs[rank * 16 + g] - M) / Z;
            }
            const bool evict_l = (n_live == cap);  // the new token does not fit: Alg. 1, overflow branch
            const int cut = Tpos - d.Bp;           // positions <= cut have left the proximity window
            float *score_g = reinterpret_cast<float *>(p.base + d.score_off) + row_lo;
            uint64_t key = ~0ull;
            int slot = -1;
            for (int k = lane; k < n_loc; k += 32) {
                float pv[G];
                load_group<G>(probs + k * G, pv);
                float a = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) a += pv[g] * fac[g];
                a *= (1.0f / G);
                const float s_new = fmaf(p.lambda, meta_s[k], a);  // Eq. (score)
                score_g[k] = s_new;
                const int32_t pj = meta_p[k];
                if (evict_l && pj <= cut) {
                    const uint64_t kk = (static_cast<uint64_t>(score_order_bits(s_new)) << 32) | (uint32_t)pj;
                    if (kk < key) {
                        key = kk;
                        slot = row_lo + k;
                    }
                }
            }
            if (rank == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g) s_tok += probs[(n_ent - 1) * G + g] * fac[g];
                s_tok *= (1.0f / G);
                if (evict_l && d.Bp == 0 && lane == 0) {
                    const uint64_t kk = (static_cast<uint64_t>(score_order_bits(s_tok)) << 32) | (uint32_t)Tpos;
                    if (kk < key) {
                        key = kk;
                        slot = -2;
                    }
                }
            }
            warp_min_key(key, slot);
            // the new scores are in global memory before rank 0 learns of the candidate (it
            // overwrites the victim's)
            fence_cluster();
            __syncwarp();
            if (lane == 0) {
                const uint32_t ra = map_to_rank(xv + rank, 0u);
                st_remote_b64(ra, key);
                st_remote_b32(ra + 8, static_cast<uint32_t>(slot));
                mbar_arrive_remote(map_to_rank(x_vict, 0u));
            }
        }
        if (rank != 0) return;
        if (!mbar_wait_bounded_cluster(x_vict, 0, abort_flag, p.status, WS_VICTIM) ||
            !mbar_wait_bounded(hdr_bar, 0, abort_flag, p.status, WS_HEADER_TAIL)) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            return;
        }
        const bool evict = (n_live == cap);
        int victim_slot = -1, victim_pos = -1;
        if (evict) {
            uint64_t best = ~0ull;
            for (int r = 0; r < C; ++r) {
                const uint64_t k = xv[r].key;
                if (k < best) {
                    best = k;
                    victim_slot = xv[r].slot;
                }
            }
            if (best == ~0ull) {
                if (lane == 0) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 2);
                victim_slot = -1;
            } else {
                victim_pos = static_cast<int>(static_cast<uint32_t>(best & 0xffffffffull));
            }
        }
        const bool have_victim = evict && victim_slot != -1;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        const float *Kr_src = resident ? krs : Kr_g;

        int merge_slot = -1;  // report: slot merged into, -2 fill, -1 none
        int res_target = -1;  // residual row to write
        uint32_t res_w = 0;
        float mk[4] = {0.f, 0.f, 0.f, 0.f}, mv[4] = {0.f, 0.f, 0.f, 0.f};
        if (have_victim && d.Br > 0) {
            float kc[4], vc[4];
            if (victim_slot >= 0) {
                load4s<T>(reinterpret_cast<const T *>(p.base + d.k_off + (size_t)victim_slot * ROWB) + l32 * 4, kc);
                load4s<T>(reinterpret_cast<const T *>(p.base + d.v_off + (size_t)victim_slot * ROWB) + l32 * 4, vc);
            } else {
                load4s<T>(reinterpret_cast<const T *>(kn_raw) + l32 * 4, kc);
                load4s<T>(reinterpret_cast<const T *>(vn_raw) + l32 * 4, vc);
            }
            if (n_res < d.Br) {
                // Alg. 1: a free residual slot takes the token as it is
                res_target = n_res;
                res_w = 1;
                merge_slot = -2;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    mk[e] = kc[e];
                    mv[e] = vc[e];
                }
            } else {
                // Eq. (hatr): raw dot product with every merged key (or its cosine form);
                // ties to the lowest slot
                float nt2 = 0.f;
                if (p.cosine) {
                    nt2 = kc[0] * kc[0];
                    nt2 = fmaf(kc[1], kc[1], nt2);
                    nt2 = fmaf(kc[2], kc[2], nt2);
                    nt2 = fmaf(kc[3], kc[3], nt2);
                    nt2 = group_sum<LPR32>(nt2);
                }
                float bd = -INFINITY;
                int br = 0x7fffffff;
                for (int r0 = 0; r0 < n_res; r0 += 4 * RPW32) {
                    float4 kr[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int r = r0 + u * RPW32 + sub32;
                        kr[u] = r < n_res ? *reinterpret_cast<const float4 *>(Kr_src + (size_t)r * D + l32 * 4)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int r = r0 + u * RPW32 + sub32;
                        float acc = 0.f;
                        acc = fmaf(kr[u].x, kc[0], acc);
                        acc = fmaf(kr[u].y, kc[1], acc);
                        acc = fmaf(kr[u].z, kc[2], acc);
                        acc = fmaf(kr[u].w, kc[3], acc);
                        acc = group_sum<LPR32>(acc);
                        if (p.cosine) {
                            float nr2 = kr[u].x * kr[u].x;
                            nr2 = fmaf(kr[u].y, kr[u].y, nr2);
                            nr2 = fmaf(kr[u].z, kr[u].z, nr2);
                            nr2 = fmaf(kr[u].w, kr[u].w, nr2);
                            nr2 = group_sum<LPR32>(nr2);
                            const float nn = sqrtf(nr2) * sqrtf(nt2);
                            acc = nn > 0.f ? acc / nn : 0.f;
                        }
                        if (r < n_res && (br == 0x7fffffff || acc > bd)) {
                            bd = acc;
                            br = r;
                        }
                    }
                }
#pragma unroll
                for (int off = LPR32; off < 32; off <<= 1) {
                    const float od = __shfl_xor_sync(0xffffffffu, bd, off);
                    const int orr = __shfl_xor_sync(0xffffffffu, br, off);
                    if (orr != 0x7fffffff && (br == 0x7fffffff || od > bd || (od == bd && orr < br))) {
                        bd = od;
                        br = orr;
                    }
                }
                res_target = br;
                merge_slot = br;
                const uint32_t wr_u = w_s[br];
                res_w = wr_u + 1u;
                const float wr = static_cast<float>(wr_u);
                // Eq. (kvr): incremental mean of key and value
                const float4 ko = *reinterpret_cast<const float4 *>(Kr_src + (size_t)br * D + l32 * 4);
                const float4 vo = *reinterpret_cast<const float4 *>(Vr_g + (size_t)br * D + l32 * 4);
                const float kof[4] = {ko.x, ko.y, ko.z, ko.w}, vof[4] = {vo.x, vo.y, vo.z, vo.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    mk[e] = fmaf(wr, kof[e], kc[e]) / (wr + 1.0f);
                    mv[e] = fmaf(wr, vof[e], vc[e]) / (wr + 1.0f);
                }
            }
        }

        // every rank has read its last tile: the unit's rows may now be overwritten
        if (!mbar_wait_bounded_cluster(x_done, 0, abort_flag, p.status, WS_DONE_TAIL)) return;
        const bool insert = evict ? (have_victim && victim_slot >= 0) : true;
        const int ins_slot = evict ? victim_slot : n_live;
        if (insert) {
            uint4 *kd = reinterpret_cast<uint4 *>(p.base + d.k_off + (size_t)ins_slot * ROWB);
            uint4 *vd = reinterpret_cast<uint4 *>(p.base + d.v_off + (size_t)ins_slot * ROWB);
            for (int c = lane; c < ROWB / 16; c += 32) {
                kd[c] = kn_raw[c];
                vd[c] = vn_raw[c];
            }
        }
        if (res_target >= 0 && sub32 == 0) {
            *reinterpret_cast<float4 *>(Kr_g + (size_t)res_target * D + l32 * 4) =
                make_float4(mk[0], mk[1], mk[2], mk[3]);
            *reinterpret_cast<float4 *>(Vr_g + (size_t)res_target * D + l32 * 4) =
                make_float4(mv[0], mv[1], mv[2], mv[3]);
        }
        if (lane == 0) {
            if (insert) {
                reinterpret_cast<float *>(p.base + d.score_off)[ins_slot] = s_tok;
                reinterpret_cast<int32_t *>(p.base + d.pos_off)[ins_slot] = Tpos;
            }
            if (res_target >= 0) reinterpret_cast<uint32_t *>(p.base + d.w_off)[res_target] = res_w;
            UnitCounters c;
            c.n_live = n_live + ((!evict) ? 1 : 0);
            c.n_res = n_res + ((merge_slot == -2) ? 1 : 0);
            c.T = Tpos + 1;
            c.pad = 0;
            *reinterpret_cast<int4 *>(p.counters + d.unit) = *reinterpret_cast<int4 *>(&c);
            if (p.victim_pos) p.victim_pos[ul] = victim_pos;
            if (p.merge_slot) p.merge_slot[ul] = merge_slot;
        }
        return;
    }

    // =====================================================================
    // Consumers
    // =====================================================================
    const int l = lane % LPR;    // 16-byte column of a token row
    const int sub = lane / LPR;  // which of the RPW rows of a warp-wide load

    int cs = 0;
    uint32_t cph = 0;
    auto wait_full = [&](int where) -> const uint8_t * {
        if (!mbar_wait_bounded(&full_bar[cs], cph, abort_flag, p.status, where)) return nullptr;
        return ring + static_cast<size_t>(cs) * kTileBytes;
    };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[cs]);
        if (++cs == S) {
            cs = 0;
            cph ^= 1u;
        }
    };
    auto csync = [&]() { named_bar_sync(1, NT); };

    // warps that share one V tile: few, so that several tiles are worked on at once
    const int vg = max(1, min(NW, min(kSplitVGroup, R / (RPW * UBV))));
    const int n_vgroups = NW / vg;
    const bool full_v = (R % (vg * RPW * UBV)) == 0;
    const int rb_step = RB % NW;

    if (tid == 0 && rank == 0 && (cnt.x < 0 || cnt.x > cap || cnt.y < 0 || cnt.y > d.Br))
        dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 1);

    // ---------------- header ----------------
    if (!mbar_wait_bounded(hdr_bar, 0, abort_flag, p.status, WS_HEADER)) return;
    const uint8_t *h = hdr;
    uint32_t qb[kMma ? SEG : 1][4];  // B fragments of q: head n = lane / 4; heads >= G are zero
    if constexpr (kMma) {
        const int gq = lane >> 2, tig = lane & 3;
#pragma unroll
        for (int j = 0; j < SEG; ++j) {
            uint4 t = make_uint4(0, 0, 0, 0);
            if (gq < G) t = *reinterpret_cast<const uint4 *>(h + gq * ROWB + j * 64 + tig * 16);
            qb[j][0] = t.x;
            qb[j][1] = t.y;
            qb[j][2] = t.z;
            qb[j][3] = t.w;
        }
    }
    {
        const T *qs = reinterpret_cast<const T *>(h);
        for (int k = tid; k < G * D; k += NT) qf[k] = E::to_float(qs[k]);
    }
    csync();  // qf is in place

    // ---------------- D1: logits of the merged slots, + alpha ln w (rank 0) ----------------
    for (int r0 = 0; r0 < nr_loc; r0 += R32) {
        const uint8_t *tile = wait_full(WS_KR);
        if (!tile) return;
        const int rows = min(R32, nr_loc - r0);
        for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
            const int row = base + sub32;
            float4 kr = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < rows) kr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float4 qv = *reinterpret_cast<const float4 *>(qf + g * D + l32 * 4);
                float acc = qv.x * kr.x;
                acc = fmaf(qv.y, kr.y, acc);
                acc = fmaf(qv.z, kr.z, acc);
                acc = fmaf(qv.w, kr.w, acc);
                acc = group_sum<LPR32>(acc);
                if (l32 == 0 && row < rows)
                    probs[(n_loc + r0 + row) * G + g] =
                        fmaf(p.alpha, logf(static_cast<float>(w_s[r0 + row])), acc * p.scale);
            }
        }
        release();
    }
    // ---------------- D1: logits of this rank's token slots ----------------
    int kturn = 0;
    for (int r0 = 0; r0 < n_loc; r0 += R) {
        const uint8_t *tile = wait_full(WS_K);
        if (!tile) return;
        const int rows = min(R, n_loc - r0);
        if constexpr (kMma) {
            // Blocks of 16 rows go round the warps; a thread reads 16 bytes of rows gq and
            // gq + 8 per 64-byte segment, with the contraction index permuted the same way on
            // both operands so that each 16-byte read feeds two tensor-core steps.
            const int gq = lane >> 2, tig = lane & 3;
            int rb_first = warp - kturn;
            if (rb_first < 0) rb_first += NW;
            for (int rb = rb_first; rb < RB && rb * 16 < rows; rb += NW) {
                const uint8_t *pa = tile + (rb * 16 + gq) * ROWB + tig * 16;
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < SEG; ++j) {
                    const uint4 ra = *reinterpret_cast<const uint4 *>(pa + j * 64);
                    const uint4 rc = *reinterpret_cast<const uint4 *>(pa + 8 * ROWB + j * 64);
                    mma_16x8x16<T>(c0, ra.x, rc.x, ra.y, rc.y, qb[j][0], qb[j][1]);
                    mma_16x8x16<T>(c1, ra.z, rc.z, ra.w, rc.w, qb[j][2], qb[j][3]);
                }
                const int n0 = tig * 2;
                if (n0 < G) {
                    const int ra_ = rb * 16 + gq, rc_ = ra_ + 8;
                    float *pr = probs + (r0 + ra_) * G + n0;
                    if (ra_ < rows) {
                        pr[0] = (c0[0] + c1[0]) * p.scale;
                        if (G > 1) pr[1] = (c0[1] + c1[1]) * p.scale;
                    }
                    if (rc_ < rows) {
                        pr[8 * G] = (c0[2] + c1[2]) * p.scale;
                        if (G > 1) pr[8 * G + 1] = (c0[3] + c1[3]) * p.scale;
                    }
                }
            }
            kturn += rb_step;
            if (kturn >= NW) kturn -= NW;
        } else {
            for (int base = warp * RPW; base < rows; base += NW * RPW) {
                const int row = base + sub;
                float f[EPL];
                E::widen(row < rows ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                    : make_uint4(0, 0, 0, 0), f);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float *qg = qf + g * D + l * EPL;
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc = fmaf(qg[e], f[e], acc);
                    acc = group_sum<LPR>(acc);
                    if (l == 0 && row < rows) probs[(r0 + row) * G + g] = acc * p.scale;
                }
            }
        }
        release();
    }

    // logit of the new token itself (rank 0)
    if (rank == 0 && warp == NW - 1) {
        float f[EPL];
        E::widen(sub == 0 ? kn_raw[l] : make_uint4(0, 0, 0, 0), f);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float *qg = qf + g * D + l * EPL;
            float acc = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc = fmaf(qg[e], f[e], acc);
            acc = group_sum<32>(acc);
            if (lane == 0) probs[(n_ent - 1) * G + g] = acc * p.scale;
        }
    }
    csync();

    // ---------------- D2: softmax, first over the slice, then over the cluster ----------------
    float mx[G], fac[G];
#pragma unroll
    for (int g = 0; g < G; ++g) mx[g] = -INFINITY;
    for (int j = tid; j < n_ent; j += NT) {
        float pv[G];
        load_group<G>(probs + j * G, pv);
#pragma unroll
        for (int g = 0; g < G; ++g) mx[g] = fmaxf(mx[g], pv[g]);
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1)
            mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], off));
        if (lane == 0) redf[warp * G + g] = mx[g];
    }
    csync();
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float m = redf[g];
        for (int wv = 1; wv < NW; ++wv) m = fmaxf(m, redf[wv * G + g]);
        mx[g] = m;
    }
    {
        float sm[G];
#pragma unroll
        for (int g = 0; g < G; ++g) sm[g] = 0.f;
        for (int j = tid; j < n_ent; j += NT) {
            float pv[G];
            load_group<G>(probs + j * G, pv);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                pv[g] = expf(pv[g] - mx[g]);
                sm[g] += pv[g];
            }
            store_group<G>(probs + j * G, pv);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            sm[g] = group_sum<32>(sm[g]);
            if (lane == 0) redf2[warp * G + g] = sm[g];
        }
    }
    csync();
    if (tid < C) {
        // thread t posts this rank's (max, sum) to rank t and arrives on its barrier
        const uint32_t ra = map_to_rank(xs + rank * 16, static_cast<uint32_t>(tid));
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float z = redf2[g];
            for (int wv = 1; wv < NW; ++wv) z += redf2[wv * G + g];
            st_remote_f32(ra + g * 4, mx[g]);
            st_remote_f32(ra + (8 + g) * 4, z);
        }
        mbar_arrive_remote(map_to_rank(x_soft, static_cast<uint32_t>(tid)));
    }
    // the slice's exponentials are final (un-normalised): the tail warp takes the score update
    // and the victim search from here (it waits for the cluster's normaliser), the consumer
    // warps go straight on to the V tiles, which need it only at the very end
    if (tid == 0) mbar_arrive(p_ready);

    // ---------------- D3: output ----------------
    float2 acc2[G][EP2];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < EP2; ++e) acc2[g][e] = make_float2(0.f, 0.f);
    int vturn = 0;
    for (int r0 = 0; r0 < n_loc; r0 += R) {
        const uint8_t *tile = wait_full(WS_V);
        if (!tile) return;
        const int rows = min(R, n_loc - r0);
        const int wv_ = warp - vturn * vg;  // this warp's place in the tile's group
        auto v_rows = [&](auto full) {
            constexpr bool FULL = decltype(full)::value;
            for (int base = wv_ * RPW; base < rows; base += vg * RPW * UBV) {
                uint4 raw[UBV];
#pragma unroll
                for (int u = 0; u < UBV; ++u) {
                    const int row = base + u * vg * RPW + sub;
                    raw[u] = (FULL || row < rows)
                                 ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                 : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int u = 0; u < UBV; ++u) {
                    const int row = base + u * vg * RPW + sub;
                    float f[EPL];
                    E::widen(raw[u], f);
                    float pv[G];
                    if (FULL || row < rows) {
                        load_group<G>(probs + (r0 + row) * G, pv);
                    } else {
#pragma unroll
                        for (int g = 0; g < G; ++g) pv[g] = 0.f;
                    }
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float2 pp = make_float2(pv[g], pv[g]);
#pragma unroll
                        for (int e = 0; e < EP2; ++e)
                            acc2[g][e] = __ffma2_rn(pp, make_float2(f[2 * e], f[2 * e + 1]), acc2[g][e]);
                    }
                }
            }
        };
        if (wv_ >= 0 && wv_ < vg) {
            if (rows == R && full_v) v_rows(std::true_type{}); else v_rows(std::false_type{});
        }
        if (++vturn == n_vgroups) vturn = 0;
        release();
    }
    float acc32[G][4];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc32[g][e] = 0.f;
    for (int r0 = 0; r0 < nr_loc; r0 += R32) {
        const uint8_t *tile = wait_full(WS_VR);
        if (!tile) return;
        const int rows = min(R32, nr_loc - r0);
        for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
            const int row = base + sub32;
            if (row < rows) {
                const float4 vr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
                float pv[G];
                load_group<G>(probs + (n_loc + r0 + row) * G, pv);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    acc32[g][0] = fmaf(pv[g], vr.x, acc32[g][0]);
                    acc32[g][1] = fmaf(pv[g], vr.y, acc32[g][1]);
                    acc32[g][2] = fmaf(pv[g], vr.z, acc32[g][2]);
                    acc32[g][3] = fmaf(pv[g], vr.w, acc32[g][3]);
                }
            }
        }
        release();
    }
    // fold the RPW row groups of a warp, then the warps
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            float v = (e & 1) ? acc2[g][e / 2].y : acc2[g][e / 2].x;
#pragma unroll
            for (int off = LPR; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (sub == 0) opart[(warp * G + g) * D + l * EPL + e] = v;
        }
    }
    __syncwarp();
    if (nr_loc > 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = acc32[g][e];
#pragma unroll
                for (int off = LPR32; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (sub32 == 0) opart[(warp * G + g) * D + l32 * 4 + e] += v;
            }
        }
    }
    csync();
    if (!mbar_wait_bounded_cluster(x_soft, 0, abort_flag, p.status, WS_SOFTMAX)) return;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float M = -INFINITY;
        for (int r = 0; r < C; ++r) M = fmaxf(M, xs[r * 16 + g]);
        float Z = 0.f;
        for (int r = 0; r < C; ++r) Z = fmaf(xs[r * 16 + 8 + g], expf(xs[r * 16 + g] - M), Z);
        fac[g] = expf(mx[g] - M) / Z;  // turns this slice's exponentials into attention weights
    }
    {
        // this rank's share of the output, already normalised, to rank 0
        const T *vn = reinterpret_cast<const T *>(vn_raw);
        const uint32_t ra = map_to_rank(xo + rank * G * D, 0u);
        for (int k = tid; k < G * D; k += NT) {
            const int g = k / D, dim = k % D;
            float sum = 0.f;
            for (int wv = 0; wv < NW; ++wv) sum += opart[(wv * G + g) * D + dim];
            if (rank == 0) sum = fmaf(probs[(n_ent - 1) * G + g], E::to_float(vn[dim]), sum);
            st_remote_f32(ra + k * 4, sum * fac[g]);
        }
        // Orders, for the cluster, everything this CTA wrote before the barrier above (its score
        // updates too: rank 0 may overwrite the victim's) before the arrival below.
        fence_cluster();
        __syncwarp();
        if (lane == 0 && warp < split_post_warps(NW, G * D)) mbar_arrive_remote(map_to_rank(x_done, 0u));
    }
    if (rank != 0) return;
    if (!mbar_wait_bounded_cluster(x_done, 0, abort_flag, p.status, WS_DONE_OUT)) return;
    {
        T *out = static_cast<T *>(p.out) + (size_t)ul * G * D;
        for (int k = tid; k < G * D; k += NT) {
            float sum = 0.f;
            for (int r = 0; r < C; ++r) sum += xo[r * G * D + k];
            out[k] = E::from_float(sum);
        }
    }
}

// TWO: launch bounds for two CTAs of ten warps per SM (the default shape); otherwise one CTA of up
// to eighteen warps.
template <typename T, int D, int G, bool TWO>
__global__ void __launch_bounds__(TWO ? kSplitPairThreads : kSplitThreads, TWO ? 2 : 1)
    decode_split_kernel(const SplitParams sp) {
    extern __shared__ __align__(128) uint8_t smem[];
    const DecodeParams &p = sp.d;
    const int NW = (blockDim.x >> 5) - kExtraWarps;
    const int C = static_cast<int>(cluster_nctarank());
    const int rank = static_cast<int>(cluster_ctarank());
    const int ci = blockIdx.x / C;  // the cluster's unit, in the launch's plain order
    const SplitSmem L = split_smem_layout(p.stages, G, D, D * (int)sizeof(T), p.l_stride,
                                          p.br_max_pad, sp.kr_rows, NW, C);
    // the descriptor table is written once, when the cache is created: safe to read at any time
    UnitDesc d;
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.sched_desc + ci);
        uint4 *dst = reinterpret_cast<uint4 *>(&d);
#pragma unroll
        for (int k = 0; k < 5; ++k) dst[k] = __ldg(src + k);
    }

    if (threadIdx.x == 0) {
        uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L.bars);
        const int S = p.stages;
        for (int s = 0; s < S; ++s) {
            mbar_init(&bars[s], 1);
            mbar_init(&bars[S + s], NW);
        }
        mbar_init(&bars[2 * S], C);      // softmax partials of every rank
        mbar_init(&bars[2 * S + 1], C);  // victim candidates (used on rank 0)
        // partial outputs, last tiles read (used on rank 0): every posting warp of every rank
        mbar_init(&bars[2 * S + 2], C * split_post_warps(NW, G * D));
        mbar_init(&bars[2 * S + 3], 1);   // the slice's exponentials are written
        mbar_init(&bars[2 * S + 4], 1);   // header
        mbar_init(&bars[2 * S + 5], 1);   // scores and positions
        *reinterpret_cast<volatile int32_t *>(smem + L.flags) = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // First cluster barrier: every peer's barriers exist before anything is posted to them.
    // Each thread completes it (cluster_wait) where its role first needs it, in split_body.
    cluster_arrive();
    if (d.unit == p.unit_base + ci) {
        split_body<T, D, G>(sp, smem, L, d, rank, C);
    } else {
        cluster_wait();
        if (threadIdx.x == 0) {
            griddep_wait();
            griddep_launch_dependents();
            if (rank == 0) dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 3);
        }
    }
    cluster_sync_all();  // no CTA leaves while a peer may still write to its shared memory
}

template <typename T, int D, int G>
int launch_split_one(const SplitParams &sp, int cluster, int consumer_warps, cudaStream_t stream) {
    const DecodeParams &p = sp.d;
    const int threads = (consumer_warps + kExtraWarps) * 32;
    const SplitSmem L = split_smem_layout(p.stages, G, D, D * (int)sizeof(T), p.l_stride,
                                          p.br_max_pad, sp.kr_rows, consumer_warps, cluster);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sp.n_units * cluster), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(threads), 1, 1);
    cfg.dynamicSmemBytes = L.total;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // the kernel orders itself after its predecessor with griddepcontrol.wait
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (threads <= kSplitPairThreads)
        return static_cast<int>(cudaLaunchKernelEx(&cfg, decode_split_kernel<T, D, G, true>, sp));
    return static_cast<int>(cudaLaunchKernelEx(&cfg, decode_split_kernel<T, D, G, false>, sp));
}

template <typename T, int D, int G, bool TWO>
int prepare_split_form(int cluster, int smem_bytes, int threads, int *max_clusters) {
    cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<T, D, G, TWO>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kSplitMaxDynamicSmem);
    if (e != cudaSuccess) return static_cast<int>(e);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(cluster), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(threads), 1, 1);
    cfg.dynamicSmemBytes = static_cast<size_t>(smem_bytes);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, decode_split_kernel<T, D, G, TWO>, &cfg);
    if (max_clusters) *max_clusters = n;
    return static_cast<int>(e);
}

template <typename T, int D, int G>
int prepare_split_one(int cluster, int smem_bytes, int threads, int *max_clusters) {
    if (threads <= kSplitPairThreads)
        return prepare_split_form<T, D, G, true>(cluster, smem_bytes, threads, max_clusters);
    return prepare_split_form<T, D, G, false>(cluster, smem_bytes, threads, max_clusters);
}

#define ZSM_SPLIT_DISPATCH(FN, ...)                                                   \
    do {                                                                              \
        if (dtype == 0) {                                                             \
            if (D == 64) ZSM_SPLIT_DISPATCH_G(FN, float, 64, __VA_ARGS__);            \
            if (D == 128) ZSM_SPLIT_DISPATCH_G(FN, float, 128, __VA_ARGS__);          \
        } else if (dtype == 1) {                                                      \
            if (D == 64) ZSM_SPLIT_DISPATCH_G(FN, __half, 64, __VA_ARGS__);           \
            if (D == 128) ZSM_SPLIT_DISPATCH_G(FN, __half, 128, __VA_ARGS__);         \
        } else if (dtype == 2) {                                                      \
            if (D == 64) ZSM_SPLIT_DISPATCH_G(FN, __nv_bfloat16, 64, __VA_ARGS__);    \
            if (D == 128) ZSM_SPLIT_DISPATCH_G(FN, __nv_bfloat16, 128, __VA_ARGS__);  \
        }                                                                             \
    } while (0)

#define ZSM_SPLIT_DISPATCH_G(FN, TT, DD, ...)                \
    do {                                                     \
        if (G == 1) return FN<TT, DD, 1>(__VA_ARGS__);       \
        if (G == 2) return FN<TT, DD, 2>(__VA_ARGS__);       \
        if (G == 4) return FN<TT, DD, 4>(__VA_ARGS__);       \
        if (G == 8) return FN<TT, DD, 8>(__VA_ARGS__);       \
    } while (0)

}  // namespace

int launch_decode_split(int dtype, int D, int G, const SplitParams &p, int cluster,
                        int consumer_warps, cudaStream_t stream) {
    ZSM_SPLIT_DISPATCH(launch_split_one, p, cluster, consumer_warps, stream);
    return -1;
}

int prepare_decode_split(int dtype, int D, int G, int cluster, int smem_bytes, int threads,
                         int *max_clusters) {
    ZSM_SPLIT_DISPATCH(prepare_split_one, cluster, smem_bytes, threads, max_clusters);
    return -1;
}

}  // namespace zsm
