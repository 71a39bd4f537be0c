// Fused decode step of the budgeted KV cache (Algorithm 1 + Eq. (att_score2)).
//
// Persistent CTAs (two per SM by default) each walk a static list of units.  Three roles:
//
// Producer warp: streams each unit's arrays through a ring of 16 KiB shared-memory stages
// with 1-D bulk copies (cp.async.bulk + mbarrier); it runs ahead across units, so a unit's
// serial phases (softmax reductions, victim search) overlap the next unit's loads.
//
// Consumer warps take the tiles in order:
//   header   counters, q (G heads), k_new, v_new, fusion counts w
//   K tiles  logits q.k/sqrt(d) of every live token slot          (D1)
//   Kr tiles logits of the merged slots, + alpha*ln w             (D1, Eq. (att_score2))
//   -- softmax over slots + new token                             (D2)
//   meta     score, pos: s <- lambda*s + mean_g a_hat; running argmin of
//            (s, pos) over slots that left the proximity window   (D4, D5)
//   -- the victim goes to the tail warp through a mailbox
//   V tiles, Vr tiles   o = sum a_hat v                            (D3)
//   -- write o
//
// Tail warp: off the streaming path, per unit: residual target (free slot, or argmax_r
// k_r.k_victim and the incremental mean; D6), then -- once the unit's last tile has been
// read -- the new token into the victim's slot, the merged rows, counts and counters (D6, D7).
//
// K and V rows cross HBM exactly once per step; grouped query heads share them.  Weights are
// kept interleaved, [slot][g], so one shared-memory load serves all heads of a group.
#include "zsm_decode.cuh"

namespace zsm {

namespace {

constexpr int kMaxThreads = (kMaxConsumerWarps + kExtraWarps) * 32;    // wide form, one CTA per SM
constexpr int kPairThreads = (kPairConsumerWarps + kExtraWarps) * 32;  // two CTAs per SM
constexpr int kMaxDynamicSmem = 232448;  // 227 KiB, the opt-in limit per CTA on sm_100

// "where" codes recorded with a timeout
enum : int32_t {
    W_PRODUCER = 1, W_HEADER = 2, W_K = 3, W_KR = 4, W_META = 5, W_V = 6, W_VR = 7,
    W_MAIL_FREE = 8, W_TAIL_POST = 9, W_TAIL_VDONE = 10
};

// Fixed part of a mailbox (kMailFixed bytes), followed by k_new, v_new (storage dtype) and w.
struct __align__(16) Mail {
    int4 cnt;
    UnitDesc d;
    int32_t victim_slot;  // >= 0 token slot; -2 the new token itself (B_p = 0); -1 none
    int32_t victim_pos;
    int32_t evict;
    float s_tok;
    int32_t pad[4];
};
static_assert(sizeof(Mail) == kMailFixed, "mailbox header size");

template <bool B>
struct BoolC {
    static constexpr bool value = B;
};

__host__ __device__ constexpr int ilog2(int x) { return x <= 1 ? 0 : 1 + ilog2(x / 2); }

// Sums each of the N values over the LG lanes of a group with a transposing butterfly: while
// more than one value is left, a step halves the values a lane carries instead of repeating
// the exchange for each.  Afterwards v[0 .. max(1, N/LG)) hold complete sums of the values
// treduce_index(l) + i.  N and LG are powers of two; l is the lane's index in its group.
template <int N, int LG>
__device__ __forceinline__ void treduce(float (&v)[N], int l) {
    constexpr int STEPS = ilog2(LG);
#pragma unroll
    for (int s = 0; s < STEPS; ++s) {
        const int off = LG >> (s + 1);
        const int n = (N >> s) > 1 ? (N >> s) : 1;
        if (n > 1) {
            const bool up = (l & off) != 0;
#pragma unroll
            for (int i = 0; i < n / 2; ++i) {
                const float keep = up ? v[i + n / 2] : v[i];
                const float send = up ? v[i] : v[i + n / 2];
                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], off);
        }
    }
}

template <int N, int LG>
__device__ __forceinline__ int treduce_index(int l) {
    constexpr int STEPS = ilog2(LG);
    int idx = 0;
#pragma unroll
    for (int s = 0; s < STEPS; ++s) {
        const int off = LG >> (s + 1);
        const int n = (N >> s) > 1 ? (N >> s) : 1;
        if (n > 1 && (l & off)) idx += n / 2;
    }
    return idx;
}

// Four consecutive elements of a row in the storage dtype, widened.
template <typename T>
__device__ __forceinline__ void load4(const T *p, float (&f)[4]) {
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

// WIDE: up to sixteen consumer warps in one CTA per SM, for launches with no more units than
// SMs, where a CTA has an SM to itself and its speed is what its warps can consume; otherwise
// up to eight consumer warps and two CTAs per SM.  Same code: the warp count is the launch's.
// COS: the cosine option of Eq. (hatr), compiled into its own instantiation (as a run-time branch
// it cost the default kernel registers: the G = 4 kernel began to spill).
template <typename T, int D, int G, bool WIDE, bool COS>
__global__ void __launch_bounds__(WIDE ? kMaxThreads : kPairThreads, WIDE ? 1 : 2)
    decode_fused_kernel(const DecodeParams p) {
    using E = Elem<T>;
    constexpr int EPL = E::EPL;               // elements per 16-byte lane load
    constexpr int EP2 = EPL / 2;
    constexpr int ROWB = D * (int)sizeof(T);  // bytes per token row
    constexpr int LPR = D / EPL;              // lanes per token row
    constexpr int RPW = 32 / LPR;             // token rows per warp-wide load
    constexpr int R = kTileBytes / ROWB;      // token rows per tile
    constexpr int ROWB32 = D * 4;             // residual rows are fp32
    constexpr int LPR32 = D / 4;
    constexpr int RPW32 = 32 / LPR32;
    constexpr int R32 = kTileBytes / ROWB32;
    constexpr int RM = kTileBytes / 8;        // (score, pos) entries per meta tile
    constexpr int HDR_D = 16;                 // unit descriptor
    constexpr int HDR_Q = HDR_D + (int)sizeof(UnitDesc);
    constexpr int HDR_K = HDR_Q + G * ROWB;
    constexpr int HDR_V = HDR_K + ROWB;
    constexpr int HDR_W = HDR_V + ROWB;
    constexpr int UBK = G <= 2 ? 4 : 2;       // row groups in flight per warp, logits pass
    constexpr int UBV = G <= 4 ? 4 : 2;       // same, output pass
    constexpr int NV = G * UBK;               // partial dot products a lane carries
    constexpr int NF = NV > LPR ? NV / LPR : 1;
    // 16-bit storage: the logits pass runs on the tensor cores, 16 slots x 8 query heads per step
    constexpr bool kMma = sizeof(T) == 2;
    constexpr int SEG = ROWB / 64;            // 64-byte column segments of a token row
    constexpr int RB = R / 16;                // 16-row blocks per tile

    extern __shared__ __align__(128) uint8_t smem[];
    const int NW = (blockDim.x >> 5) - kExtraWarps;  // consumer warps
    const int NT = NW * 32;
    const int S = p.stages;
    const int LS = p.l_stride;
    const DecodeSmem L = decode_smem_layout(S, G, D, ROWB, LS, p.br_max_pad, NW);

    uint8_t *ring = smem + L.ring;
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + L.bars);
    uint64_t *empty_bar = full_bar + S;
    uint64_t *post_bar = empty_bar + S;   // [2] consumers -> tail: the unit's victim is known
    uint64_t *vdone_bar = post_bar + 2;   // [2] consumers -> tail: the unit's last tile was read
    uint64_t *freed_bar = vdone_bar + 2;  // [2] tail -> consumers: the mailbox may be reused
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(smem + L.flags);
    float *probs = reinterpret_cast<float *>(smem + L.probs);  // [slot][G]
    float *qf = reinterpret_cast<float *>(smem + L.qf);
    float *opart = reinterpret_cast<float *>(smem + L.opart);
    float *redf = reinterpret_cast<float *>(smem + L.redf);
    float *redf2 = redf + kMaxConsumerWarps * 8;
    uint64_t *red64 = reinterpret_cast<uint64_t *>(smem + L.red64);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], NW);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&post_bar[b], 1);
            mbar_init(&vdone_bar[b], 1);
            mbar_init(&freed_bar[b], 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int first = p.sched_off[blockIdx.x];
    const int last = p.sched_off[blockIdx.x + 1];

    // =====================================================================
    // Producer: one thread issues every bulk copy of this CTA.
    // =====================================================================
    if (warp == NW) {
        if (lane != 0 || first >= last) return;
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        auto acquire = [&](uint32_t bytes, uint64_t *&bar) -> uint8_t * {
            if (!mbar_wait_bounded(&empty_bar[s], ph ^ 1u, abort_flag, p.status, W_PRODUCER)) {
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
            return dst;
        };
        auto load_desc = [&](int i) -> UnitDesc {
            UnitDesc d;
            const uint4 *src = reinterpret_cast<const uint4 *>(p.sched_desc + i);
            uint4 *dst = reinterpret_cast<uint4 *>(&d);
#pragma unroll
            for (int k = 0; k < 5; ++k) dst[k] = __ldg(src + k);
            return d;
        };
        auto load_cnt = [&](int unit) -> int4 {
            return *reinterpret_cast<const int4 *>(p.counters + unit);
        };

        // descriptors are fetched two units ahead, counters one unit ahead
        UnitDesc d_cur = load_desc(first);
        int4 c_cur = load_cnt(d_cur.unit);
        UnitDesc d_nxt = d_cur;
        if (first + 1 < last) d_nxt = load_desc(first + 1);

        for (int i = first; i < last && ok; ++i) {
            int4 c_nxt = c_cur;
            UnitDesc d_nx2 = d_nxt;
            if (i + 1 < last) c_nxt = load_cnt(d_nxt.unit);
            if (i + 2 < last) d_nx2 = load_desc(i + 2);

            const UnitDesc &d = d_cur;
            const int cap = d.Bp + d.Bc;
            const int n_live = min(max(c_cur.x, 0), cap);
            const int n_res = min(max(c_cur.y, 0), d.Br);
            const int ul = d.unit - p.unit_base;
            const int br_pad = (d.Br + 3) & ~3;
            uint64_t *bar = nullptr;
            uint8_t *dst;

            // header
            dst = acquire(HDR_W + br_pad * 4u, bar);
            if (!ok) break;
            bulk_g2s(dst, p.counters + d.unit, 16u, bar);
            bulk_g2s(dst + HDR_D, p.sched_desc + i, (uint32_t)sizeof(UnitDesc), bar);
            bulk_g2s(dst + HDR_Q, static_cast<const uint8_t *>(p.q) + (size_t)ul * G * ROWB,
                     G * ROWB, bar);
            bulk_g2s(dst + HDR_K, static_cast<const uint8_t *>(p.k_new) + (size_t)ul * ROWB, ROWB,
                     bar);
            bulk_g2s(dst + HDR_V, static_cast<const uint8_t *>(p.v_new) + (size_t)ul * ROWB, ROWB,
                     bar);
            if (br_pad > 0) bulk_g2s(dst + HDR_W, p.base + d.w_off, br_pad * 4u, bar);

            // K token rows, then residual K rows
            for (int r0 = 0; r0 < n_live && ok; r0 += R) {
                const uint32_t bytes = static_cast<uint32_t>(min(R, n_live - r0)) * ROWB;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.k_off + (size_t)r0 * ROWB, bytes, bar);
            }
            for (int r0 = 0; r0 < n_res && ok; r0 += R32) {
                const uint32_t bytes = static_cast<uint32_t>(min(R32, n_res - r0)) * ROWB32;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.kr_off + (size_t)r0 * ROWB32, bytes, bar);
            }
            // scores and positions
            for (int j0 = 0; j0 < n_live && ok; j0 += RM) {
                const uint32_t n4 = static_cast<uint32_t>((min(RM, n_live - j0) + 3) & ~3);
                dst = acquire(n4 * 8u, bar);
                if (ok) {
                    bulk_g2s(dst, p.base + d.score_off + (size_t)j0 * 4, n4 * 4u, bar);
                    bulk_g2s(dst + RM * 4, p.base + d.pos_off + (size_t)j0 * 4, n4 * 4u, bar);
                }
            }
            // V token rows, then residual V rows
            for (int r0 = 0; r0 < n_live && ok; r0 += R) {
                const uint32_t bytes = static_cast<uint32_t>(min(R, n_live - r0)) * ROWB;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.v_off + (size_t)r0 * ROWB, bytes, bar);
            }
            for (int r0 = 0; r0 < n_res && ok; r0 += R32) {
                const uint32_t bytes = static_cast<uint32_t>(min(R32, n_res - r0)) * ROWB32;
                dst = acquire(bytes, bar);
                if (ok) bulk_g2s(dst, p.base + d.vr_off + (size_t)r0 * ROWB32, bytes, bar);
            }
            d_cur = d_nxt;
            d_nxt = d_nx2;
            c_cur = c_nxt;
        }
        if (!ok) {
            // give copies already in flight time to land before the CTA's memory goes away
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
        return;
    }

    const int l32 = lane % LPR32;  // 16-byte column of an fp32 residual row
    const int sub32 = lane / LPR32;

    // =====================================================================
    // Tail warp: residual fill / merge and the write-back of each unit.
    // =====================================================================
    if (warp == NW + 1) {
        for (int n = 0; n < last - first; ++n) {
            const int mb = n & 1;
            const uint32_t mph = (n >> 1) & 1u;
            const uint8_t *mailp = smem + L.mail + mb * L.mail_stride;
            if (!mbar_wait_bounded(&post_bar[mb], mph, abort_flag, p.status, W_TAIL_POST)) return;
            const Mail *m = reinterpret_cast<const Mail *>(mailp);
            const uint4 *kn_raw = reinterpret_cast<const uint4 *>(mailp + kMailFixed);
            const uint4 *vn_raw = reinterpret_cast<const uint4 *>(mailp + kMailFixed + ROWB);
            const uint32_t *w_s = reinterpret_cast<const uint32_t *>(mailp + kMailFixed + 2 * ROWB);
            const int4 cnt = m->cnt;
            const UnitDesc d = m->d;
            const int cap = d.Bp + d.Bc;
            const int n_live = min(max(cnt.x, 0), cap);
            const int n_res = min(max(cnt.y, 0), d.Br);
            const int Tpos = cnt.z;
            const int ul = d.unit - p.unit_base;
            const int victim_slot = m->victim_slot;
            const int victim_pos = m->victim_pos;
            const bool evict = m->evict != 0;
            const float s_tok = m->s_tok;
            const bool have_victim = evict && victim_slot != -1;

            int merge_slot = -1;  // report: slot merged into, -2 fill, -1 none
            int res_target = -1;  // residual row to write
            uint32_t res_w = 0;
            float mk[4] = {0.f, 0.f, 0.f, 0.f}, mv[4] = {0.f, 0.f, 0.f, 0.f};
            float *Kr_g = reinterpret_cast<float *>(p.base + d.kr_off);
            float *Vr_g = reinterpret_cast<float *>(p.base + d.vr_off);
            if (have_victim && d.Br > 0) {
                float kc[4], vc[4];
                if (victim_slot >= 0) {
                    load4<T>(reinterpret_cast<const T *>(p.base + d.k_off + (size_t)victim_slot * ROWB) + l32 * 4, kc);
                    load4<T>(reinterpret_cast<const T *>(p.base + d.v_off + (size_t)victim_slot * ROWB) + l32 * 4, vc);
                } else {
                    load4<T>(reinterpret_cast<const T *>(kn_raw) + l32 * 4, kc);
                    load4<T>(reinterpret_cast<const T *>(vn_raw) + l32 * 4, vc);
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
                    if constexpr (COS) {
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
                            kr[u] = r < n_res ? *reinterpret_cast<const float4 *>(Kr_g + (size_t)r * D + l32 * 4)
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
                            if constexpr (COS) {
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
                    const float4 ko = *reinterpret_cast<const float4 *>(Kr_g + (size_t)br * D + l32 * 4);
                    const float4 vo = *reinterpret_cast<const float4 *>(Vr_g + (size_t)br * D + l32 * 4);
                    const float kof[4] = {ko.x, ko.y, ko.z, ko.w}, vof[4] = {vo.x, vo.y, vo.z, vo.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        mk[e] = fmaf(wr, kof[e], kc[e]) / (wr + 1.0f);
                        mv[e] = fmaf(wr, vof[e], vc[e]) / (wr + 1.0f);
                    }
                }
            }

            // every tile of this unit has been read: its rows may now be overwritten
            if (!mbar_wait_bounded(&vdone_bar[mb], mph, abort_flag, p.status, W_TAIL_VDONE)) return;
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
                if (res_target >= 0)
                    reinterpret_cast<uint32_t *>(p.base + d.w_off)[res_target] = res_w;
                UnitCounters c;
                c.n_live = n_live + ((!evict) ? 1 : 0);
                c.n_res = n_res + ((merge_slot == -2) ? 1 : 0);
                c.T = Tpos + 1;
                c.pad = 0;
                *reinterpret_cast<int4 *>(p.counters + d.unit) = *reinterpret_cast<int4 *>(&c);
                if (p.victim_pos) p.victim_pos[ul] = victim_pos;
                if (p.merge_slot) p.merge_slot[ul] = merge_slot;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&freed_bar[mb]);
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

    // A tile's rows are shared by a group of warps, kg (logits, FMA form) or vg (output) of
    // them; when there are more consumer warps than that, the groups take tiles in turn.
    const int kg = max(1, min(NW, R / (RPW * UBK)));
    const int vg = max(1, min(NW, R / (RPW * UBV)));
    const int n_kgroups = NW / kg, n_vgroups = NW / vg;
    // a full tile needs no row checks when the group's row sets tile it exactly
    const bool full_k = (R % (kg * RPW * UBK)) == 0;
    const bool full_v = (R % (vg * RPW * UBV)) == 0;
    const int rb_step = RB % NW;  // how far a tile's 16-row blocks advance the round-robin
    // where this lane's sums land after the transposing reduction of the logits pass
    const int tr_idx = treduce_index<NV, LPR>(l);
    const bool tr_writer = (NV >= LPR) || ((l & (LPR / (NV < LPR ? NV : LPR) - 1)) == 0);

    for (int i = first; i < last; ++i) {
        const int n = i - first;
        const int mb = n & 1;
        const uint32_t mph = (n >> 1) & 1u;
        uint8_t *mailp = smem + L.mail + mb * L.mail_stride;
        Mail *mail = reinterpret_cast<Mail *>(mailp);
        uint4 *kn_raw = reinterpret_cast<uint4 *>(mailp + kMailFixed);
        uint4 *vn_raw = reinterpret_cast<uint4 *>(mailp + kMailFixed + ROWB);
        uint32_t *w_s = reinterpret_cast<uint32_t *>(mailp + kMailFixed + 2 * ROWB);

        // ---------------- header ----------------
        const uint8_t *h = wait_full(W_HEADER);
        if (!h) return;
        // the tail warp is done with this mailbox's previous unit (two units back)
        if (!mbar_wait_bounded(&freed_bar[mb], mph ^ 1u, abort_flag, p.status, W_MAIL_FREE)) return;
        const int4 cnt = *reinterpret_cast<const int4 *>(h);
        const UnitDesc d = *reinterpret_cast<const UnitDesc *>(h + HDR_D);
        const int cap = d.Bp + d.Bc;
        const int ul = d.unit - p.unit_base;
        const int br_pad = (d.Br + 3) & ~3;
        if (tid == 0 && (cnt.x < 0 || cnt.x > cap || cnt.y < 0 || cnt.y > d.Br))
            dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 1);
        const int n_live = min(max(cnt.x, 0), cap);
        const int n_res = min(max(cnt.y, 0), d.Br);
        const int Tpos = cnt.z;
        const int n_ent = n_live + n_res + 1;

        // query operands of the logits pass: packed fp32 pairs for the FMA form, or the B
        // fragments (head n = lane / 4; heads >= G are zero) for the tensor-core form
        float2 q2[kMma ? 1 : G][kMma ? 1 : EP2];
        uint32_t qb[kMma ? SEG : 1][4];
        if constexpr (kMma) {
            const int gq = lane >> 2, tig = lane & 3;
#pragma unroll
            for (int j = 0; j < SEG; ++j) {
                uint4 t = make_uint4(0, 0, 0, 0);
                if (gq < G) t = *reinterpret_cast<const uint4 *>(h + HDR_Q + gq * ROWB + j * 64 + tig * 16);
                qb[j][0] = t.x;
                qb[j][1] = t.y;
                qb[j][2] = t.z;
                qb[j][3] = t.w;
            }
        } else {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint4 raw = *reinterpret_cast<const uint4 *>(h + HDR_Q + g * ROWB + l * 16);
                float f[EPL];
                E::widen(raw, f);
#pragma unroll
                for (int e = 0; e < EP2; ++e) q2[g][e] = make_float2(f[2 * e], f[2 * e + 1]);
            }
        }
        {
            const T *qs = reinterpret_cast<const T *>(h + HDR_Q);
            for (int k = tid; k < G * D; k += NT) qf[k] = E::to_float(qs[k]);
            const uint4 *ks = reinterpret_cast<const uint4 *>(h + HDR_K);
            const uint4 *vs = reinterpret_cast<const uint4 *>(h + HDR_V);
            for (int k = tid; k < ROWB / 16; k += NT) {
                kn_raw[k] = ks[k];
                vn_raw[k] = vs[k];
            }
            const uint32_t *ws = reinterpret_cast<const uint32_t *>(h + HDR_W);
            for (int k = tid; k < br_pad; k += NT) w_s[k] = ws[k];
            if (tid == 0) {
                mail->cnt = cnt;
                mail->d = d;
            }
        }
        release();

        // ---------------- D1: logits of the token slots ----------------
        int kturn = 0, gturn = 0;
        for (int r0 = 0; r0 < n_live; r0 += R) {
            const uint8_t *tile = wait_full(W_K);
            if (!tile) return;
            const int rows = min(R, n_live - r0);
            if constexpr (kMma) {
                // Blocks of 16 rows go round the warps.  A thread reads 16 bytes of rows
                // gq and gq + 8 per 64-byte segment; the contraction index is permuted the
                // same way on both operands, so each 16-byte read feeds two steps.
                const int gq = lane >> 2, tig = lane & 3;
                int rb_first = warp - kturn;  // kturn: this tile's first block, modulo NW
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
                    const int n0 = tig * 2;  // query heads n0, n0 + 1 of rows gq and gq + 8
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
                const int wk = warp - gturn * kg;  // this warp's place in the tile's group
                auto k_rows = [&](auto full) {
                    constexpr bool FULL = decltype(full)::value;  // every row of the pass exists
                    for (int base = wk * RPW; base < rows; base += kg * RPW * UBK) {
                        uint4 raw[UBK];
    #pragma unroll
                        for (int u = 0; u < UBK; ++u) {
                            const int row = base + u * kg * RPW + sub;
                            raw[u] = (FULL || row < rows)
                                         ? *reinterpret_cast<const uint4 *>(tile + row * ROWB + l * 16)
                                         : make_uint4(0, 0, 0, 0);
                        }
                        float v[NV];
    #pragma unroll
                        for (int u = 0; u < UBK; ++u) {
                            float f[EPL];
                            E::widen(raw[u], f);
    #pragma unroll
                            for (int g = 0; g < G; ++g) {
                                float2 a = make_float2(0.f, 0.f);
    #pragma unroll
                                for (int e = 0; e < EP2; ++e)
                                    a = __ffma2_rn(q2[g][e], make_float2(f[2 * e], f[2 * e + 1]), a);
                                v[u * G + g] = a.x + a.y;
                            }
                        }
                        treduce<NV, LPR>(v, l);
                        if (tr_writer) {
    #pragma unroll
                            for (int k = 0; k < NF; ++k) {
                                const int id = tr_idx + k;
                                const int u = id / G, g = id % G;
                                const int row = base + u * kg * RPW + sub;
                                if (FULL || row < rows) probs[(r0 + row) * G + g] = v[k] * p.scale;
                            }
                        }
                    }
                };
                if (wk >= 0 && wk < kg) {
                    if (rows == R && full_k) k_rows(BoolC<true>{}); else k_rows(BoolC<false>{});
                }
                if (++gturn == n_kgroups) gturn = 0;
            }
            release();
        }
        csync();  // qf and the mailbox arrays of this unit are in place

        // ---------------- D1: logits of the merged slots, + alpha ln w ----------------
        for (int r0 = 0; r0 < n_res; r0 += R32) {
            const uint8_t *tile = wait_full(W_KR);
            if (!tile) return;
            const int rows = min(R32, n_res - r0);
            for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
                const int row = base + sub32;
                float4 kr = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < rows)
                    kr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float4 qv = *reinterpret_cast<const float4 *>(qf + g * D + l32 * 4);
                    float acc = qv.x * kr.x;
                    acc = fmaf(qv.y, kr.y, acc);
                    acc = fmaf(qv.z, kr.z, acc);
                    acc = fmaf(qv.w, kr.w, acc);
                    acc = group_sum<LPR32>(acc);
                    if (l32 == 0 && row < rows)
                        probs[(n_live + r0 + row) * G + g] =
                            fmaf(p.alpha, logf(static_cast<float>(w_s[r0 + row])), acc * p.scale);
                }
            }
            release();
        }
        // logit of the new token itself
        if (warp == NW - 1) {
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

        // ---------------- D2: softmax over slots + new token ----------------
        float mx[G], inv[G];
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
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float z = redf2[g];
            for (int wv = 1; wv < NW; ++wv) z += redf2[wv * G + g];
            inv[g] = 1.0f / z;
        }

        // ---------------- D4 + D5: score update and victim search ----------------
        const bool evict = (n_live == cap);  // the new token does not fit: Alg. 1, overflow branch
        const int cut = Tpos - d.Bp;         // positions <= cut have left the proximity window
        float *score_g = reinterpret_cast<float *>(p.base + d.score_off);
        uint64_t best = ~0ull;
        int best_slot = -1;
        for (int j0 = 0; j0 < n_live; j0 += RM) {
            const uint8_t *tile = wait_full(W_META);
            if (!tile) return;
            const int nn = min(RM, n_live - j0);
            const float *ts = reinterpret_cast<const float *>(tile);
            const int32_t *tp = reinterpret_cast<const int32_t *>(tile + RM * 4);
            for (int k = tid; k < nn; k += NT) {
                float pv[G];
                load_group<G>(probs + (j0 + k) * G, pv);
                float a = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) a += pv[g] * inv[g];
                a *= (1.0f / G);
                const float s_new = fmaf(p.lambda, ts[k], a);  // Eq. (score)
                score_g[j0 + k] = s_new;
                const int32_t pj = tp[k];
                if (evict && pj <= cut) {
                    const uint64_t key =
                        (static_cast<uint64_t>(score_order_bits(s_new)) << 32) | (uint32_t)pj;
                    if (key < best) {
                        best = key;
                        best_slot = j0 + k;
                    }
                }
            }
            release();
        }
        float s_tok = 0.f;  // first score of the new token: its own attention weight
#pragma unroll
        for (int g = 0; g < G; ++g) s_tok += probs[(n_ent - 1) * G + g] * inv[g];
        s_tok *= (1.0f / G);

        if (evict) {
            if (tid == 0 && d.Bp == 0) {
                const uint64_t key =
                    (static_cast<uint64_t>(score_order_bits(s_tok)) << 32) | (uint32_t)Tpos;
                if (key < best) {
                    best = key;
                    best_slot = -2;
                }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                const uint64_t ob = __shfl_xor_sync(0xffffffffu, best, off);
                const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
                if (ob < best) {
                    best = ob;
                    best_slot = os;
                }
            }
            if (lane == 0) {
                red64[warp * 2] = best;
                red64[warp * 2 + 1] = static_cast<uint64_t>(static_cast<uint32_t>(best_slot));
            }
            csync();
        }
        // Thread 0 settles the victim and hands the unit's update to the tail warp.  Every
        // store the consumer warps made for this unit so far (mailbox arrays, updated scores)
        // is ordered before the hand-over by the barriers above.
        if (tid == 0) {
            int victim_slot = -1;  // >= 0: token slot; -2: the new token itself (B_p = 0)
            int victim_pos = -1;
            if (evict) {
                best = red64[0];
                best_slot = static_cast<int>(static_cast<uint32_t>(red64[1]));
                for (int wv = 1; wv < NW; ++wv) {
                    const uint64_t ob = red64[wv * 2];
                    if (ob < best) {
                        best = ob;
                        best_slot = static_cast<int>(static_cast<uint32_t>(red64[wv * 2 + 1]));
                    }
                }
                if (best == ~0ull) {
                    dev_set_status(p.status, DEV_ERR_CHECK, d.unit, 2);
                } else {
                    victim_slot = best_slot;
                    victim_pos = static_cast<int>(static_cast<uint32_t>(best & 0xffffffffull));
                }
            }
            mail->victim_slot = victim_slot;
            mail->victim_pos = victim_pos;
            mail->evict = evict ? 1 : 0;
            mail->s_tok = s_tok;
            mbar_arrive(&post_bar[mb]);
        }

        // ---------------- D3: output ----------------
        float2 acc2[G][EP2];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < EP2; ++e) acc2[g][e] = make_float2(0.f, 0.f);
        int vturn = 0;
        for (int r0 = 0; r0 < n_live; r0 += R) {
            const uint8_t *tile = wait_full(W_V);
            if (!tile) return;
            const int rows = min(R, n_live - r0);
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
                if (rows == R && full_v) v_rows(BoolC<true>{}); else v_rows(BoolC<false>{});
            }
            if (++vturn == n_vgroups) vturn = 0;
            release();
        }
        float acc32[G][4];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc32[g][e] = 0.f;
        for (int r0 = 0; r0 < n_res; r0 += R32) {
            const uint8_t *tile = wait_full(W_VR);
            if (!tile) return;
            const int rows = min(R32, n_res - r0);
            for (int base = warp * RPW32; base < rows; base += NW * RPW32) {
                const int row = base + sub32;
                if (row < rows) {
                    const float4 vr = *reinterpret_cast<const float4 *>(tile + row * ROWB32 + l32 * 16);
                    float pv[G];
                    load_group<G>(probs + (n_live + r0 + row) * G, pv);
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
        // The partial outputs are folded through the memory the weights occupy: keep the new
        // token's weights (the last entries) in registers, and let every warp finish reading
        // weights before the first partial is written.
        float pnew[G];
#pragma unroll
        for (int g = 0; g < G; ++g) pnew[g] = probs[(n_ent - 1) * G + g];
        csync();
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
        if (n_res > 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = acc32[g][e];
#pragma unroll
                    for (int off = LPR32; off < 32; off <<= 1)
                        v += __shfl_xor_sync(0xffffffffu, v, off);
                    if (sub32 == 0) opart[(warp * G + g) * D + l32 * 4 + e] += v;
                }
            }
        }
        csync();
        if (tid == 0) mbar_arrive(&vdone_bar[mb]);  // the unit's rows may be overwritten now
        {
            const T *vn = reinterpret_cast<const T *>(vn_raw);
            T *out = static_cast<T *>(p.out) + (size_t)ul * G * D;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                for (int dim = tid; dim < D; dim += NT) {
                    float sum = 0.f;
                    for (int wv = 0; wv < NW; ++wv) sum += opart[(wv * G + g) * D + dim];
                    sum = fmaf(pnew[g], E::to_float(vn[dim]), sum);
                    out[g * D + dim] = E::from_float(sum * inv[g]);
                }
            }
        }
        csync();  // shared scratch is free for the next unit
    }
}

template <typename T, int D, int G>
int launch_one(const DecodeParams &p, int grid, int consumer_warps, bool wide, cudaStream_t stream) {
    const int threads = (consumer_warps + kExtraWarps) * 32;
    const DecodeSmem L = decode_smem_layout(p.stages, G, D, D * (int)sizeof(T), p.l_stride,
                                            p.br_max_pad, consumer_warps);
    if (wide) {
        if (p.cosine)
            decode_fused_kernel<T, D, G, true, true><<<grid, threads, L.total, stream>>>(p);
        else
            decode_fused_kernel<T, D, G, true, false><<<grid, threads, L.total, stream>>>(p);
    } else {
        if (p.cosine)
            decode_fused_kernel<T, D, G, false, true><<<grid, threads, L.total, stream>>>(p);
        else
            decode_fused_kernel<T, D, G, false, false><<<grid, threads, L.total, stream>>>(p);
    }
    return static_cast<int>(cudaGetLastError());
}

template <typename T, int D, int G>
int prepare_one(int smem_bytes, int threads, int *max_ctas) {
    cudaError_t ew = cudaFuncSetAttribute(decode_fused_kernel<T, D, G, true, false>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          kMaxDynamicSmem);
    if (ew == cudaSuccess)
        ew = cudaFuncSetAttribute(decode_fused_kernel<T, D, G, true, true>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
    if (ew == cudaSuccess)
        ew = cudaFuncSetAttribute(decode_fused_kernel<T, D, G, false, true>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
    if (ew != cudaSuccess) return static_cast<int>(ew);
    // The limit belongs to the kernel, not to a cache: caches of one shape but different budgets
    // ask for different amounts, so it is raised to the most any of them can ask for.
    cudaError_t e = cudaFuncSetAttribute(decode_fused_kernel<T, D, G, false, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxDynamicSmem);
    if (e != cudaSuccess) return static_cast<int>(e);
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_fused_kernel<T, D, G, false, false>, threads,
                                                      smem_bytes);
    if (max_ctas) *max_ctas = n;
    return static_cast<int>(e);
}

#define ZSM_DISPATCH(FN, ...)                                                         \
    do {                                                                              \
        if (dtype == 0) {                                                             \
            if (D == 64) ZSM_DISPATCH_G(FN, float, 64, __VA_ARGS__);                  \
            if (D == 128) ZSM_DISPATCH_G(FN, float, 128, __VA_ARGS__);                \
        } else if (dtype == 1) {                                                      \
            if (D == 64) ZSM_DISPATCH_G(FN, __half, 64, __VA_ARGS__);                 \
            if (D == 128) ZSM_DISPATCH_G(FN, __half, 128, __VA_ARGS__);               \
        } else if (dtype == 2) {                                                      \
            if (D == 64) ZSM_DISPATCH_G(FN, __nv_bfloat16, 64, __VA_ARGS__);          \
            if (D == 128) ZSM_DISPATCH_G(FN, __nv_bfloat16, 128, __VA_ARGS__);        \
        }                                                                             \
    } while (0)

#define ZSM_DISPATCH_G(FN, TT, DD, ...)                      \
    do {                                                     \
        if (G == 1) return FN<TT, DD, 1>(__VA_ARGS__);       \
        if (G == 2) return FN<TT, DD, 2>(__VA_ARGS__);       \
        if (G == 4) return FN<TT, DD, 4>(__VA_ARGS__);       \
        if (G == 8) return FN<TT, DD, 8>(__VA_ARGS__);       \
    } while (0)

}  // namespace

int launch_decode_fused(int dtype, int D, int G, const DecodeParams &p, int grid,
                        int consumer_warps, bool wide, cudaStream_t stream) {
    ZSM_DISPATCH(launch_one, p, grid, consumer_warps, wide, stream);
    return -1;
}

int prepare_decode_fused(int dtype, int D, int G, int smem_bytes, int threads,
                         int *max_ctas_per_sm) {
    ZSM_DISPATCH(prepare_one, smem_bytes, threads, max_ctas_per_sm);
    return -1;
}

namespace {
constexpr int32_t W_SELFTEST = 99;

// The failure detector's own test: the wait below can only end by its time limit.
__global__ void __launch_bounds__(32) wait_selftest_kernel(int32_t *status, uint32_t limit_us) {
    __shared__ uint64_t bar;
    __shared__ int32_t abort_flag;
    if (threadIdx.x != 0) return;
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // phase 0 of a barrier with one expected arrival never completes here
    (void)mbar_wait_bounded(&bar, 0u, &abort_flag, status, W_SELFTEST,
                            static_cast<uint64_t>(limit_us) * 1000ull);
}
}  // namespace

int launch_wait_selftest(int32_t *status, uint32_t limit_us, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_us);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace zsm
