// Full-history prompt scores: s_t = (1/G) sum_g sum_{tau >= t} lambda^(T-1-tau) a^(tau)_{g,t},
// a^(tau) the causal softmax row of prompt query tau (App. B with the window taken as the whole
// prompt; Eq. (score) unrolled).  A dense T x T x d contraction done twice on the tensor cores:
//   pass 1  row statistics: log-sum-exp of every query's causal row (skipped when the caller
//           hands in the values its own prefill attention produced);
//   pass 2  column sums: for a block of 128 keys, over every later query tile and every query
//           head of the group, exp(logit - lse) weighted by the decay.
// Both passes are one kernel: a 128-row block of one operand stays in registers as A fragments
// (queries in pass 1, keys in pass 2), 64-row tiles of the other stream through a padded,
// double-buffered shared-memory stage (cp.async) and are read as B fragments with ldmatrix,
// each fragment feeding the warp's two 16-row tiles; each of the four warps owns 32 resident
// rows and reduces along the streamed index in registers, so nothing but the final per-row
// value leaves a thread.
#include "zsm_prefill_full.cuh"

namespace zsm {

namespace {

constexpr int kFullThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void *smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(smem_u32(smem_row)));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T, int D, bool COLSUM>
__global__ void __launch_bounds__(kFullThreads) full_pass_kernel(const FullScoreParams p) {
    constexpr int STRIDE = D * 2 + 16;  // staged row pitch in bytes: an odd number of 16-byte words
    constexpr int TILE = kFullBlock * STRIDE;
    constexpr int KS = D / 16;          // tensor-core steps along the head dimension
    constexpr int CPR = D * 2 / 16;     // 16-byte chunks per row
    constexpr int MT = kFullResident / 64;  // 16-row tiles of the resident block per warp
    extern __shared__ __align__(128) uint8_t smem[];
    float *off_s = reinterpret_cast<float *>(smem + 2 * TILE);  // [2][64]: pass 2, per query

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tig = lane & 3;
    const int Tn = p.T, G = p.G;
    const int nb = (Tn + kFullBlock - 1) / kFullBlock;  // streamed tiles that hold a position
    const int rb = blockIdx.x;                           // the resident block
    constexpr int RPS = kFullResident / kFullBlock;      // streamed tiles per resident block
    int b, hk, hq = 0;
    if (COLSUM) {
        b = blockIdx.y / p.n_kv_heads;
        hk = blockIdx.y % p.n_kv_heads;
    } else {
        b = blockIdx.y / (p.n_kv_heads * G);
        hq = blockIdx.y % (p.n_kv_heads * G);
        hk = hq / G;
    }
    const T *Kh = static_cast<const T *>(p.K) + ((size_t)b * p.n_kv_heads + hk) * Tn * D;
    const T *Qb = static_cast<const T *>(p.Q) + (size_t)b * p.n_kv_heads * G * Tn * D;
    const T *res = COLSUM ? Kh : Qb + (size_t)hq * Tn * D;

    // resident rows of this thread: gq and gq + 8 of each of the warp's MT 16-row tiles
    const int rbase = rb * kFullResident + warp * (16 * MT) + gq;
    uint32_t a[MT][KS][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const T *r0p = res + (size_t)min(rbase + 16 * mt, Tn - 1) * D;
        const T *r1p = res + (size_t)min(rbase + 16 * mt + 8, Tn - 1) * D;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            a[mt][ks][0] = *reinterpret_cast<const uint32_t *>(r0p + 16 * ks + 2 * tig);
            a[mt][ks][1] = *reinterpret_cast<const uint32_t *>(r1p + 16 * ks + 2 * tig);
            a[mt][ks][2] = *reinterpret_cast<const uint32_t *>(r0p + 16 * ks + 8 + 2 * tig);
            a[mt][ks][3] = *reinterpret_cast<const uint32_t *>(r1p + 16 * ks + 8 + 2 * tig);
        }
    }

    // streamed tiles: pass 1 key tiles 0 .. the resident block's last row; pass 2 query tiles
    // from the resident block's first row to the end, for each head of the group
    const int first = COLSUM ? rb * RPS : 0;
    const int per = COLSUM ? nb - first : min(rb * RPS + RPS, nb);
    const int items = COLSUM ? per * G : per;
    const float scale2 = p.scale * kLog2e;
    const float l2lam = log2f(p.lambda);

    auto stage_item = [&](int i, int s) {
        const int g = COLSUM ? i / per : 0;
        const int jb = first + (COLSUM ? i % per : i);
        const T *src = COLSUM ? Qb + (size_t)(hk * G + g) * Tn * D : Kh;
        uint8_t *dst = smem + s * TILE;
        for (int c = tid; c < kFullBlock * CPR; c += kFullThreads) {
            const int r = c / CPR, cc = c % CPR;
            const int grow = min(jb * kFullBlock + r, Tn - 1);
            cp_async16(dst + r * STRIDE + cc * 16, reinterpret_cast<const uint8_t *>(src + (size_t)grow * D) + cc * 16);
        }
        if (COLSUM && tid < kFullBlock) {
            // exponent offset of query q: decay lambda^(T-1-q) and the row's normaliser
            const int q = jb * kFullBlock + tid;
            float o = -INFINITY;
            if (q < Tn) {
                const float l = p.lse[((size_t)b * p.n_kv_heads * G + hk * G + g) * Tn + q];
                const float dec = (q == Tn - 1) ? 0.f : static_cast<float>(Tn - 1 - q) * l2lam;
                o = dec - l * kLog2e;
            }
            off_s[s * kFullBlock + tid] = o;
        }
        cp_async_commit();
    };

    float m[MT][2], z[MT][2], colsum[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            m[mt][h] = -INFINITY;  // pass 1: running max / sum (log2 domain)
            z[mt][h] = 0.f;
            colsum[mt][h] = 0.f;   // pass 2
        }
    stage_item(0, 0);
    for (int i = 0; i < items; ++i) {
        const int s = i & 1;
        if (i + 1 < items) {
            stage_item(i + 1, s ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const int jb = first + (COLSUM ? i % per : i);
        const uint8_t *tile = smem + s * TILE;
        // tiles that overlap the resident block's own positions need the causal test
        const bool diag = jb >= rb * RPS && jb < rb * RPS + RPS;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {  // half a tile (4 column tiles of 8) at a time
            float c[MT][4][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int n4 = 0; n4 < 4; ++n4) c[mt][n4][0] = c[mt][n4][1] = c[mt][n4][2] = c[mt][n4][3] = 0.f;
#pragma unroll
            for (int n4 = 0; n4 < 4; ++n4) {
                const int nt = hf * 4 + n4;
#pragma unroll
                for (int kq = 0; kq < D / 32; ++kq) {
                    uint32_t r[4];
                    ldmatrix_x4(r, tile + (nt * 8 + (lane & 7)) * STRIDE + (kq * 4 + (lane >> 3)) * 16);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        mma_16x8x16<T>(c[mt][n4], a[mt][2 * kq][0], a[mt][2 * kq][1], a[mt][2 * kq][2],
                                       a[mt][2 * kq][3], r[0], r[1]);
                        mma_16x8x16<T>(c[mt][n4], a[mt][2 * kq + 1][0], a[mt][2 * kq + 1][1],
                                       a[mt][2 * kq + 1][2], a[mt][2 * kq + 1][3], r[2], r[3]);
                    }
                }
            }
            if (!COLSUM) {
                // streamed index = key; resident rows = queries; keep key <= query
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    float bm[2] = {-INFINITY, -INFINITY};
#pragma unroll
                    for (int n4 = 0; n4 < 4; ++n4) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v = c[mt][n4][e] * scale2;
                            if (diag) {
                                const int key = jb * kFullBlock + (hf * 4 + n4) * 8 + 2 * tig + (e & 1);
                                if (key > rbase + 16 * mt + 8 * (e >> 1)) v = -INFINITY;
                            }
                            c[mt][n4][e] = v;
                            bm[e >> 1] = fmaxf(bm[e >> 1], v);
                        }
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float mn = fmaxf(m[mt][h], bm[h]);
                        const float mu = mn == -INFINITY ? 0.f : mn;
                        float sum = z[mt][h] * ex2(m[mt][h] - mu);
#pragma unroll
                        for (int n4 = 0; n4 < 4; ++n4)
                            sum += ex2(c[mt][n4][2 * h] - mu) + ex2(c[mt][n4][2 * h + 1] - mu);
                        z[mt][h] = sum;
                        m[mt][h] = mn;
                    }
                }
            } else {
                // streamed index = query; resident rows = keys; keep query >= key
                const float *off = off_s + s * kFullBlock;
#pragma unroll
                for (int n4 = 0; n4 < 4; ++n4) {
                    const float2 o = *reinterpret_cast<const float2 *>(off + (hf * 4 + n4) * 8 + 2 * tig);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v = ex2(fmaf(c[mt][n4][e], scale2, (e & 1) ? o.y : o.x));
                            if (diag) {
                                const int q = jb * kFullBlock + (hf * 4 + n4) * 8 + 2 * tig + (e & 1);
                                if (q < rbase + 16 * mt + 8 * (e >> 1)) v = 0.f;
                            }
                            colsum[mt][e >> 1] += v;
                        }
                    }
                }
            }
        }
        __syncthreads();  // the stage is refilled two items from now
    }

#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = rbase + 16 * mt + 8 * h;
            if (!COLSUM) {
                float mm = m[mt][h], zz = z[mt][h];
#pragma unroll
                for (int x = 1; x <= 2; x <<= 1) {
                    const float mo = __shfl_xor_sync(0xffffffffu, mm, x);
                    const float zo = __shfl_xor_sync(0xffffffffu, zz, x);
                    const float mn = fmaxf(mm, mo);
                    const float mu = mn == -INFINITY ? 0.f : mn;
                    zz = zz * ex2(mm - mu) + zo * ex2(mo - mu);
                    mm = mn;
                }
                if (tig == 0 && row < Tn)
                    p.lse_out[((size_t)b * p.n_kv_heads * G + hq) * Tn + row] = (mm + log2f(zz)) * kLn2;
            } else {
                float v = colsum[mt][h];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                if (tig == 0 && row < Tn)
                    p.scores[((size_t)b * p.n_kv_heads + hk) * Tn + row] = v * (1.0f / static_cast<float>(G));
            }
        }
    }
}

template <typename T, int D>
int launch_full_one(const FullScoreParams &p, cudaStream_t stream) {
    constexpr int SMEM = 2 * kFullBlock * (D * 2 + 16) + 2 * kFullBlock * 4;
    const int nres = (p.T + kFullResident - 1) / kFullResident;
    FullScoreParams q = p;
    if (!p.lse) {
        const dim3 grid(nres, p.batch * p.n_kv_heads * p.G);
        full_pass_kernel<T, D, false><<<grid, kFullThreads, SMEM, stream>>>(q);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return static_cast<int>(e);
        q.lse = p.lse_out;
    }
    const dim3 grid(nres, p.batch * p.n_kv_heads);
    full_pass_kernel<T, D, true><<<grid, kFullThreads, SMEM, stream>>>(q);
    return static_cast<int>(cudaGetLastError());
}

}  // namespace

int launch_full_scores(int dtype, int D, const FullScoreParams &p, cudaStream_t stream) {
    if (dtype == 1 && D == 64) return launch_full_one<__half, 64>(p, stream);
    if (dtype == 1 && D == 128) return launch_full_one<__half, 128>(p, stream);
    if (dtype == 2 && D == 64) return launch_full_one<__nv_bfloat16, 64>(p, stream);
    if (dtype == 2 && D == 128) return launch_full_one<__nv_bfloat16, 128>(p, stream);
    return -1;
}

}  // namespace zsm
